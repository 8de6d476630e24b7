// Forward shifted-window attention on the tcgen05 tensor cores (head dim 32, windows of <= 256 tokens).
//
// One persistent CTA per SM walks over (batch, window, head) items.  Roles:
//   warps 0-3 / 4-7  softmax warpgroups: one thread per query row of the first / second 128-row tile;
//                    S is read from TMEM, P = exp2(S*scale + bias - m) is written back to TMEM as bf16,
//                    O is read from TMEM, normalised and stored straight to the token's grid position
//   warp 8           issues tcgen05.mma (the whole warp runs the loop and waits, one elected lane issues):
//                    S = Q K^T (operands in shared memory), O = P [V | 1] (P from TMEM; 16 columns of ones behind
//                    V make the accumulator carry the row sums of P in its columns 32..47)
//   warps 9-11       loaders: undo the roll, gather the window's Q / K / V rows with cp.async into the
//                    64-byte-swizzled operand layout, stage the head's bias table and the slot metadata
// TMEM: columns [256 t, 256 t + 256) belong to query tile t: S (fp32) first; as pass 2 consumes it, bf16 P of
// keys 0..127 goes to columns 0..63, the O accumulator to 64..111 and bf16 P of keys 128..255 to 128..191, so
// that O += P V over the first 128 keys runs while the softmax of the second 128 keys is still going on.
// Row maximum: windows without mask labels use the upper bound max_j(raw score) * scale + max(bias) over the key
// slots that hold a token (softmax is shift invariant, so the result is the same; only the exponent range
// matters: the bound exceeds the true maximum by at most the spread of the head's bias table, and a head whose
// table spreads over more than 64 octaves takes the exact path); windows that mix shift-mask labels take the
// exact maximum over the keys the row may see.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, all roles leave their loops,
// TMEM is released and the host reads the device status word.
#include <cuda.h>
#include <cstdlib>
#include <cstring>

#include "swin_common.cuh"
#include "swin_kernels.h"
#include "tc_common.cuh"
#include "tma_rows.cuh"

// fp16 build of this file (through attn_fwd_tc_f16.cu): the kernel, its launcher and its status word get names of
// their own; the element-independent helpers below are compiled in the bf16 build only
#ifdef TERRA_ELEM_F16
#define g_tc_timeout g_tc_timeout_f16
#define launch_fwd_tc launch_fwd_tc_f16
#define read_tc_status read_tc_status_f16
#endif

namespace terra {

__device__ int g_tc_timeout = 0;   // set when a bounded wait expired in any CTA

namespace {

using namespace tc;

constexpr int kMmaWarp = 8;
constexpr int kLoaderWarp0 = 9;
constexpr int kLoaderWarps = 3;
constexpr int kLoaderThreads = kLoaderWarps * 32;
constexpr int kThreads = (kLoaderWarp0 + kLoaderWarps) * 32;   // 384 = three warpgroups
// Registers move between warpgroups at run time: the softmax warpgroups (0, 1) grow, the MMA + loader
// warpgroup (2) shrinks.  The kernel launches with kRegsLaunch per thread (the cap of 384 threads on a
// 64K-register SM); what the two growing warpgroups take must not exceed what the shrinking one gives
// back, or the register request would wait forever.
constexpr int kRegsLaunch = 168;
constexpr int kRegsSoftmax = 216;
constexpr int kRegsOther = 64;
static_assert(2 * (kRegsSoftmax - kRegsLaunch) <= (kRegsLaunch - kRegsOther), "register hand-over does not balance");
static_assert(kRegsLaunch * 384 <= 65536 && kRegsSoftmax % 8 == 0 && kRegsOther % 8 == 0, "register counts");
constexpr int kStages = 3;
constexpr int kMaxSlots = 256;
constexpr int kD = 32;
constexpr int kRowBytes = kD * 2;                              // 64

// shared-memory stage layout (bytes)
constexpr int kOffQ = 0;
constexpr int kOffK = kMaxSlots * kRowBytes;                   // 16384
constexpr int kOffV = 2 * kMaxSlots * kRowBytes;               // 32768
constexpr int kOffBias = 3 * kMaxSlots * kRowBytes;            // 49152: the head's prepared bias table
constexpr int kOffKc = kOffBias + kFwdBiasFloats * 4;          // per key slot: byte offset 4 * (c0 - code)
constexpr int kOffKlab = kOffKc + kMaxSlots * 4;               // per key slot: shift-mask label
constexpr int kOffRowMeta = kOffKlab + kMaxSlots * 4;          // per query slot: code | label << 16
constexpr int kOffRowTok = kOffRowMeta + kMaxSlots * 4;        // grid token of the slot, -1 if none
constexpr int kStageBytes = ((kOffRowTok + kMaxSlots * 4 + 1023) / 1024) * 1024;
// After the stages and barriers: a constant block that extends V by 16 columns of ones (256 key rows x 64 bytes
// in the operand layout, the first 16 bf16 of a row = 1).  O = P V then carries the row sums of the bf16 P in
// its columns 32..47, and the softmax threads need not add them up.
constexpr int kOffOnes = kStages * kStageBytes + 1024;
constexpr int kSmemBytes = kOffOnes + kMaxSlots * kRowBytes;
constexpr int kNO = kD + 16;                                   // columns of the O accumulator

// TMEM columns inside a query tile's 256-column region once S is being consumed: bf16 P of keys 0..127 in
// [0, 64), the O accumulator (with the row sums) in [64, 112) (S columns that the first half of pass 2 has already read), bf16
// P of keys 128..255 in [128, 192).  The PV product of the first 128 keys is issued while the softmax
// warpgroup is still working on the second 128 keys.
constexpr int kColO = 64;
constexpr int kColP1 = 128;
__device__ __forceinline__ int p_col(int chunk32) { return chunk32 < 4 ? 16 * chunk32 : kColP1 + 16 * (chunk32 - 4); }

// Bias codes use a row stride of w + 32 instead of 2w - 1: the 32 rows of a warp (consecutive slots of a
// full-width window) then read 32 different shared-memory banks.
// (In the layout of 16 slots per window row the stride is that of side 16, 48: a warp's 32 consecutive slots are two
// window rows, 48 = 16 mod 32 codes apart, and again read 32 different banks.)
__device__ __forceinline__ int code_stride(int w, bool pad16 = false) { return pad16 ? 48 : w + 32; }

struct Item {
    int b, win, head;
    WindowRef r;
    int npad;      // key slots rounded up to 16
    int ntiles;    // 128-row query tiles in use
    bool masked;   // the window mixes shift-mask labels
};

// pad16: the window's slots are laid out 16 to a window row (slot = 16 a + b; the slots with b >= the window's width
// hold no token), so that every group of 16 key columns is one window row whatever the window side
__device__ __forceinline__ Item make_item(const Geo& g, const ItemCursor& c, bool pad16 = false) {
    Item x;
    x.head = c.head;
    x.win = c.wr * g.Mw + c.wc;
    x.b = c.b;
    x.r = window_ref_rc(g, c.wr, c.wc);
    if (pad16) x.r.n = x.r.eh * 16;
    x.npad = (x.r.n + 15) & ~15;
    x.ntiles = (x.r.n + 127) >> 7;
    // rolled rows >= H - sh (columns >= W - sw) hold the tokens that wrapped across a non-periodic edge
    const int r0 = x.r.wr * g.w, c0 = x.r.wc * g.w;
    const bool mh = !g.ph && g.sh > 0 && r0 < g.H - g.sh && r0 + x.r.eh > g.H - g.sh;
    const bool mw = !g.pw && g.sw > 0 && c0 < g.W - g.sw && c0 + x.r.ew > g.W - g.sw;
    x.masked = mh || mw;
    return x;
}

// window offset (a, b) -> grid token, bias code a * (w + 32) + b and shift-mask label
__device__ __forceinline__ int offset_token_tc(const Geo& g, const WindowRef& r, int a, int b, int cs, int& code, int& label) {
    int u = r.wr * g.w + a + g.sh;
    if (u >= g.H) u -= g.H;
    int v = r.wc * g.w + b + g.sw;
    if (v >= g.W) v -= g.W;
    label = ((!g.ph && u < g.sh) ? 2 : 0) + ((!g.pw && v < g.sw) ? 1 : 0);
    code = a * cs + b;
    return u * g.W + v;
}

__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ int4 lds_i4(uint32_t addr) {
    int4 v;
    asm volatile("ld.shared.v4.s32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ int lds_i32(uint32_t addr) {
    int v;
    asm volatile("ld.shared.s32 %0, [%1];\n" : "=r"(v) : "r"(addr));
    return v;
}

// P for `N` consecutive key columns starting at `c`: exp2(raw * scale + bias - m), packed to bf16 pairs.
// bias_i / a_kc / a_klab are shared-memory byte addresses.  Returns the sum of the N values.
template <int N, bool MASKED>
__device__ __forceinline__ float softmax_cols(const uint32_t (&r)[N], uint32_t (&pk)[N / 2], int c, uint32_t bias_i,
                                              uint32_t a_kc, uint32_t a_klab, int label_i, float scale, float neg_m) {
#pragma unroll
    for (int e4 = 0; e4 < N / 4; ++e4) {
        const int4 kc4 = lds_i4(a_kc + 4 * (c + e4 * 4));
        const int kc[4] = {kc4.x, kc4.y, kc4.z, kc4.w};
        int kl[4] = {0, 0, 0, 0};
        if (MASKED) {
            const int4 kl4 = lds_i4(a_klab + 4 * (c + e4 * 4));
            kl[0] = kl4.x; kl[1] = kl4.y; kl[2] = kl4.z; kl[3] = kl4.w;
        }
        float p[4];
        if (MASKED) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float bv = lds_f32(bias_i + kc[e]);
                float xv = fmaf(__uint_as_float(r[e4 * 4 + e]), scale, bv) + neg_m;
                if (kl[e] != label_i) xv = -INFINITY;
                p[e] = fast_exp2(xv);
            }
        } else {
            float bv[4], xv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) bv[e] = lds_f32(bias_i + kc[e]);
#pragma unroll
            for (int e = 0; e < 4; e += 2) {
                fma2(xv[e], xv[e + 1], __uint_as_float(r[e4 * 4 + e]), __uint_as_float(r[e4 * 4 + e + 1]), scale, bv[e], bv[e + 1]);
                add2(xv[e], xv[e + 1], xv[e], xv[e + 1], neg_m);
                p[e] = fast_exp2(xv[e]);
                p[e + 1] = fast_exp2(xv[e + 1]);
            }
        }
        pk[e4 * 2] = pack_elem(p[0], p[1]);
        pk[e4 * 2 + 1] = pack_elem(p[2], p[3]);
    }
    return 0.f;       // the row sum comes from the ones columns of the P V product
}

// exact maximum of scale * raw + bias (log2 domain) over the keys of N columns that the row may see: a key of another
// mask group, or a slot without a token (its label matches no query's), gives -inf
template <int N>
__device__ __forceinline__ float score_max_cols(const uint32_t (&r)[N], int c, uint32_t bias_i, uint32_t a_kc, uint32_t a_klab,
                                                int label_i, float scale, float mx) {
#pragma unroll
    for (int e4 = 0; e4 < N / 4; ++e4) {
        const int4 kc4 = lds_i4(a_kc + 4 * (c + e4 * 4));
        const int4 kl4 = lds_i4(a_klab + 4 * (c + e4 * 4));
        const int kc[4] = {kc4.x, kc4.y, kc4.z, kc4.w};
        const int kl[4] = {kl4.x, kl4.y, kl4.z, kl4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float xv = fmaf(__uint_as_float(r[e4 * 4 + e]), scale, lds_f32(bias_i + kc[e]));
            mx = fmaxf(mx, kl[e] == label_i ? xv : -INFINITY);
        }
    }
    return mx;
}

template <int OFF>
__device__ __forceinline__ float lds_f32_at(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];\n" : "=f"(v) : "r"(addr), "n"(OFF));
    return v;
}
// 16 key columns that are one window row of a full 16 x 16 window without mask labels: their bias entries are
// consecutive (descending with the key), so each address is one base plus an immediate offset.  `top` = shared
// address of the entry of the row's first key.
// BW < 16: only the row's first BW keys hold a token; the others get P = 0 and cost nothing.
template <int BW = 16>
__device__ __forceinline__ void softmax_cols16_row(const uint32_t* r, uint32_t* pk, uint32_t top, float scale, float neg_m) {
    const uint32_t bb = top - 60;
    float bv[16];
    bv[0] = lds_f32_at<60>(bb);  bv[1] = lds_f32_at<56>(bb);  bv[2] = lds_f32_at<52>(bb);  bv[3] = lds_f32_at<48>(bb);
    bv[4] = lds_f32_at<44>(bb);  bv[5] = lds_f32_at<40>(bb);  bv[6] = lds_f32_at<36>(bb);  bv[7] = lds_f32_at<32>(bb);
    if (BW > 8) bv[8] = lds_f32_at<28>(bb);
    if (BW > 9) bv[9] = lds_f32_at<24>(bb);
    if (BW > 10) bv[10] = lds_f32_at<20>(bb);
    if (BW > 11) bv[11] = lds_f32_at<16>(bb);
    if (BW > 12) bv[12] = lds_f32_at<12>(bb);
    if (BW > 13) bv[13] = lds_f32_at<8>(bb);
    if (BW > 14) bv[14] = lds_f32_at<4>(bb);
    if (BW > 15) bv[15] = lds_f32_at<0>(bb);
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) {
        if (2 * e2 + 1 < BW) {
            float x0, x1;
            fma2(x0, x1, __uint_as_float(r[2 * e2]), __uint_as_float(r[2 * e2 + 1]), scale, bv[2 * e2], bv[2 * e2 + 1]);
            add2(x0, x1, x0, x1, neg_m);
            pk[e2] = pack_elem(fast_exp2(x0), fast_exp2(x1));
        } else if (2 * e2 < BW) {
            pk[e2] = pack_elem(fast_exp2(fmaf(__uint_as_float(r[2 * e2]), scale, bv[2 * e2]) + neg_m), 0.f);
        } else {
            pk[e2] = 0u;
        }
    }
}

template <int N>
__device__ __forceinline__ void max_cols(const uint32_t (&r)[N], float (&mx)[4]) {
#pragma unroll
    for (int e = 0; e < N; e += 8) {
#pragma unroll
        for (int a = 0; a < 4; ++a)
            mx[a] = max3(mx[a], __uint_as_float(r[e + 2 * a]), __uint_as_float(r[e + 2 * a + 1]));
    }
}
// the same over the first BW of every 16 columns only (the others are key slots without a token)
template <int N, int BW>
__device__ __forceinline__ void max_cols_width(const uint32_t (&r)[N], float (&mx)[4]) {
#pragma unroll
    for (int e = 0; e < N; e += 2) {
        if ((e & 15) + 1 < BW) mx[(e >> 1) & 3] = max3(mx[(e >> 1) & 3], __uint_as_float(r[e]), __uint_as_float(r[e + 1]));
        else if ((e & 15) < BW) mx[(e >> 1) & 3] = fmaxf(mx[(e >> 1) & 3], __uint_as_float(r[e]));
    }
}
// the same over the first `nv` of N columns only (the others are key slots without a token: zero rows, raw score 0)
template <int N>
__device__ __forceinline__ void max_cols_limit(const uint32_t (&r)[N], int nv, float (&mx)[4]) {
#pragma unroll
    for (int e = 0; e < N; ++e) mx[e & 3] = fmaxf(mx[e & 3], e < nv ? __uint_as_float(r[e]) : -INFINITY);
}

// One softmax row: two passes over the row's S columns in TMEM, 32 columns per load, the next load in
// flight while the current one is processed.  Returns m (log2 domain); the row sum goes to sum_out.
// ROW16: full 16 x 16 window without mask labels (npad = 256); `top0` = shared address of the bias entry of key 0
// for this query, `row_step` = bytes between the entries of keys one window row apart.
// BW < 16 (with ROW16): of every 16 columns only the first BW are keys with a token; the others are left out of the
// maximum and get P = 0.
template <bool MASKED, bool ROW16 = false, int BW = 16>
__device__ __forceinline__ float softmax_row(uint32_t t_s, int npad, int nvalid, uint32_t bias_i, uint32_t a_kc, uint32_t a_klab,
                                             int label_i, float scale, float bmax, float& sum_out, uint32_t bar_half,
                                             uint32_t top0 = 0, uint32_t row_step = 0) {
    constexpr bool COLMASK = BW < 16;
    const int nfull = npad >> 5;
    const bool tail = (npad & 16) != 0;
    uint32_t ra[32], rb[32];
    float m;
    if (MASKED) {
        // exact maximum over the keys this row may see (bias included)
        float mx = -INFINITY;
        for (int i = 0; i < nfull; ++i) {
            tmem_ld32(t_s + 32 * i, ra);
            tmem_ld_wait();
            mx = score_max_cols<32>(ra, 32 * i, bias_i, a_kc, a_klab, label_i, scale, mx);
        }
        if (tail) {
            uint32_t rt[16];
            tmem_ld16(t_s + 32 * nfull, rt);
            tmem_ld_wait();
            mx = score_max_cols<16>(rt, 32 * nfull, bias_i, a_kc, a_klab, label_i, scale, mx);
        }
        m = (mx == -INFINITY) ? 0.f : mx;     // a row without a token sees no key: its P is formed against 0 and is exactly 0
    } else {
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        // key slots without a token (zero rows, raw score 0) sit in the row's last 16 columns only and are left out
        const bool limit = nvalid < npad;
        const int nplain = (limit && !tail) ? nfull - 1 : nfull;
        int i = 0;
        for (; i + 4 <= nplain; i += 4) {      // 128 columns per round trip to TMEM
            uint32_t rc[32], rd[32];
            tmem_ld32(t_s + 32 * i, ra);
            tmem_ld32(t_s + 32 * (i + 1), rb);
            tmem_ld32(t_s + 32 * (i + 2), rc);
            tmem_ld32(t_s + 32 * (i + 3), rd);
            tmem_ld_wait();
            if (COLMASK) {
                max_cols_width<32, BW>(ra, mx4);
                max_cols_width<32, BW>(rb, mx4);
                max_cols_width<32, BW>(rc, mx4);
                max_cols_width<32, BW>(rd, mx4);
            } else {
                max_cols<32>(ra, mx4);
                max_cols<32>(rb, mx4);
                max_cols<32>(rc, mx4);
                max_cols<32>(rd, mx4);
            }
        }
        for (; i < nplain; ++i) {
            tmem_ld32(t_s + 32 * i, ra);
            tmem_ld_wait();
            if (COLMASK) max_cols_width<32, BW>(ra, mx4);
            else max_cols<32>(ra, mx4);
        }
        if (i < nfull) {                       // last full group, with a ragged end
            tmem_ld32(t_s + 32 * i, ra);
            tmem_ld_wait();
            max_cols_limit<32>(ra, nvalid - 32 * i, mx4);
        }
        if (tail) {
            uint32_t rt[16];
            tmem_ld16(t_s + 32 * nfull, rt);
            tmem_ld_wait();
            if (limit) max_cols_limit<16>(rt, nvalid - 32 * nfull, mx4);
            else if (COLMASK) max_cols_width<16, BW>(rt, mx4);
            else max_cols<16>(rt, mx4);
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        m = mx * scale + bmax;   // scale > 0: max of the scaled scores plus the largest bias
    }
    const float neg_m = -m;

    float sum = 0.f;
    if (nfull > 0) tmem_ld32(t_s, ra);
    for (int i = 0; i < nfull; i += 2) {
        uint32_t pk[16];
        tmem_ld_wait();
        if (i + 1 < nfull) tmem_ld32(t_s + 32 * (i + 1), rb);
        if (ROW16) {
            softmax_cols16_row<BW>(&ra[0], &pk[0], top0 - (2 * i) * row_step, scale, neg_m);
            softmax_cols16_row<BW>(&ra[16], &pk[8], top0 - (2 * i + 1) * row_step, scale, neg_m);
        } else {
            sum += softmax_cols<32, MASKED>(ra, pk, 32 * i, bias_i, a_kc, a_klab, label_i, scale, neg_m);
        }
        tmem_st16(t_s + p_col(i), pk);
        if (i + 1 < nfull) {
            tmem_ld_wait();
            if (i + 2 < nfull) tmem_ld32(t_s + 32 * (i + 2), ra);
            if (ROW16) {
                softmax_cols16_row<BW>(&rb[0], &pk[0], top0 - (2 * i + 2) * row_step, scale, neg_m);
                softmax_cols16_row<BW>(&rb[16], &pk[8], top0 - (2 * i + 3) * row_step, scale, neg_m);
            } else {
                sum += softmax_cols<32, MASKED>(rb, pk, 32 * (i + 1), bias_i, a_kc, a_klab, label_i, scale, neg_m);
            }
            tmem_st16(t_s + p_col(i + 1), pk);
        }
        if (i == 2 && npad > 128) {
            // P of keys 0..127 is complete: let the MMA lane start O += P V on it while this row goes on
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(bar_half);
        }
    }
    if (tail) {
        uint32_t rt[16], pk[8];
        tmem_ld16(t_s + 32 * nfull, rt);
        tmem_ld_wait();
        sum += softmax_cols<16, MASKED>(rt, pk, 32 * nfull, bias_i, a_kc, a_klab, label_i, scale, neg_m);
        tmem_st8(t_s + p_col(nfull), pk);
    }
    sum_out = sum;
    return m;
}

// W16 = the window side is 16: full unmasked windows take the immediate-offset table addressing, every other
// window of that grid (shift-mask labels, truncated at the grid's edge) the label-compare path, which also
// covers key slots without a token (their label never matches).  Two softmax paths per kernel either way.
// Tensor maps of the TMA variant: q, k, v as 2-D tensors [tokens][channels of the tensor] with a box of one head's 32
// channels x one window row of tokens (16, or 8 in the grid's last window column), 64-byte swizzle.
struct FwdMaps {
    CUtensorMap q16, k16, v16, q8, k8, v8;
};

// TMA = the window rows are fetched by tiled tensor copies (one per window row and tensor, issued by the lanes of
// ONE producer warp, the head's bias table by one bulk copy) instead of 16-byte cp.async copies from three loader
// warps.  For grids of 16-wide windows whose every window row is one run of consecutive tokens in memory.
// PADW = the window side, 9 .. 15, of a launch that lays the slots out 16 to a window row (see make_item): full-width
// windows without mask labels then take the immediate-offset addressing of the 16-wide case, with the columns beyond the
// window's width (a compile-time number) left out at no cost; 0 otherwise.  Never together with W16 or TMA.
template <bool W16, bool TMA, int PADW = 0>
__global__ void __launch_bounds__(kThreads, 1)
swin_fwd_tc_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                   const __nv_bfloat16* __restrict__ v, const float* __restrict__ bias_prep,
                   __nv_bfloat16* __restrict__ o, float* __restrict__ lse, long long n_items,
                   const __grid_constant__ FwdMaps maps) {
    constexpr bool PAD = PADW != 0;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bar0 = smem0 + kStages * kStageBytes;
    // barrier slots (8 bytes each)
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kStages + s); };
    auto bar_sready = [&](int t) { return bar0 + 8u * (2 * kStages + t); };
    auto bar_pready = [&](int t) { return bar0 + 8u * (2 * kStages + 2 + t); };
    auto bar_oready = [&](int t) { return bar0 + 8u * (2 * kStages + 4 + t); };
    auto bar_sfree = [&](int t) { return bar0 + 8u * (2 * kStages + 6 + t); };
    auto bar_phalf = [&](int t) { return bar0 + 8u * (2 * kStages + 8 + t); };   // P of the first 128 keys is in TMEM
    unsigned char* tail = smem + kStages * kStageBytes + 8 * (2 * kStages + 10);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail);
    volatile int* cta_abort = reinterpret_cast<volatile int*>(tail + 8);

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = tid >> 5;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full(s), TMA ? 32 : kLoaderThreads);
            mbar_init(bar_empty(s), 1 + 128);      // the issuer's commit + the second softmax warpgroup (see its loop)
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar_sready(t), 1);
            mbar_init(bar_pready(t), 128);
            mbar_init(bar_oready(t), 1);
            mbar_init(bar_sfree(t), 128);
            mbar_init(bar_phalf(t), 128);
        }
        *cta_abort = 0;
        fence_barrier_init();
    }
    for (int i = tid; i < kMaxSlots * 4; i += kThreads) {          // (row, 16-byte chunk): chunks 0, 1 = ones, 2, 3 = zeros
        const int row = i >> 2, chunk = i & 3;
        const uint32_t val = chunk < 2 ? kElemOnesPair : 0u;
        *reinterpret_cast<uint4*>(smem + kOffOnes + tile_off<kD>(row, chunk)) = make_uint4(val, val, val, val);
    }
    fence_proxy_async();
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int cs = code_stride(g.w, PAD);
    const int c0 = (g.w - 1) * (cs + 1);     // code of the last in-window offset; bias index = code_q - code_k + c0
    const size_t HW = (size_t)g.H * g.W;

    if (warp >= kMmaWarp) {
    // warpgroup 2 (MMA issuer + loaders) gives registers back: one instruction for the whole warpgroup
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsOther));
    if (TMA && warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ producer warp (TMA)
        if (warp == kLoaderWarp0) {
            int kuse = 0;
            ItemCursor cur_it = cursor_init(blockIdx.x, gridDim.x, g.heads, g.Mw, g.Mh);
            for (long long it = blockIdx.x; it < n_items; it += gridDim.x, ++kuse, cursor_advance(cur_it, g.heads, g.Mw, g.Mh)) {
                const int s = kuse % kStages;
                if (!mbar_wait_all(bar_empty(s), ((kuse / kStages) & 1) ^ 1, cta_abort)) break;
                const Item x = make_item(g, cur_it, PAD);
                unsigned char* st = smem + s * kStageBytes;
                const uint32_t st_a = smem0 + s * kStageBytes;
                const int ew = x.r.ew;                       // 16, or 8 in the last window column
                // lane a < eh: the three tensors' copies of window row a (ew consecutive tokens, this head's 64 bytes each)
                if (lane < x.r.eh) {
                    int u = x.r.wr * g.w + lane + g.sh;
                    if (u >= g.H) u -= g.H;
                    int v0 = x.r.wc * g.w + g.sw;
                    if (v0 >= g.W) v0 -= g.W;
                    const int y = (int)((size_t)x.b * HW + (size_t)u * g.W + v0), xc = x.head * kD;
                    const uint32_t dst = st_a + (uint32_t)(lane * ew * kRowBytes);
                    if (ew == 16) {
                        tma_load_2d(dst + kOffQ, &maps.q16, xc, y, bar_full(s));
                        tma_load_2d(dst + kOffK, &maps.k16, xc, y, bar_full(s));
                        tma_load_2d(dst + kOffV, &maps.v16, xc, y, bar_full(s));
                    } else {
                        tma_load_2d(dst + kOffQ, &maps.q8, xc, y, bar_full(s));
                        tma_load_2d(dst + kOffK, &maps.k8, xc, y, bar_full(s));
                        tma_load_2d(dst + kOffV, &maps.v8, xc, y, bar_full(s));
                    }
                }
                if (lane == 31) bulk_load(st_a + kOffBias, bias_prep + (size_t)x.head * kFwdBiasFloats, kFwdBiasFloats * 4, bar_full(s));
                // slot tables: 8 consecutive slots per lane
                {
                    int a_s = (8 * lane) / ew, b_s = 8 * lane - a_s * ew;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int slot = 8 * lane + i;
                        int code = 0, label = 0xff, tok = -1, kc = 4 * (2 * c0 + 1);
                        if (slot < x.r.n) {
                            tok = offset_token_tc(g, x.r, a_s, b_s, cs, code, label);
                            kc = 4 * (c0 - code);
                        }
                        reinterpret_cast<int*>(st + kOffKc)[slot] = kc;
                        reinterpret_cast<int*>(st + kOffKlab)[slot] = label;
                        reinterpret_cast<int*>(st + kOffRowMeta)[slot] = code | (label << 16);
                        reinterpret_cast<int*>(st + kOffRowTok)[slot] = tok;
                        if (++b_s == ew) { b_s = 0; ++a_s; }
                    }
                }
                // operand rows between the window's end and the next multiple of 16 must read as zeros
                for (int i = lane; i < (x.npad - x.r.n) * 12; i += 32) {
                    const int row = x.r.n + i / 12, piece = i % 12;
                    *reinterpret_cast<uint4*>(st + (piece >> 2) * (kMaxSlots * kRowBytes) + tile_off<kD>(row, piece & 3)) = make_uint4(0u, 0u, 0u, 0u);
                }
                fence_proxy_async();
                // 32 arrivals complete the phase once the copies' bytes have landed as well
                if (lane == 0) mbar_arrive_expect_tx(bar_full(s), (uint32_t)(3 * x.r.n * kRowBytes + kFwdBiasFloats * 4));
                else mbar_arrive(bar_full(s));
            }
        }
    } else if (warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loaders
        const int lt = (warp - kLoaderWarp0) * 32 + lane;
        int kuse = 0, pending_s = -1;
        ItemCursor cur_it = cursor_init(blockIdx.x, gridDim.x, g.heads, g.Mw, g.Mh);
        for (long long it = blockIdx.x; it < n_items; it += gridDim.x, ++kuse, cursor_advance(cur_it, g.heads, g.Mw, g.Mh)) {
            const int s = kuse % kStages;
            // if the next stage is not free yet, publish the copies already issued instead of holding them back
            if (pending_s >= 0 && !__all_sync(0xffffffffu, mbar_test_wait(bar_empty(s), ((kuse / kStages) & 1) ^ 1))) {
                cp_async_wait<0>();
                fence_proxy_async();
                mbar_arrive(bar_full(pending_s));
                pending_s = -1;
            }
            if (!mbar_wait_all_relaxed(bar_empty(s), ((kuse / kStages) & 1) ^ 1, cta_abort)) break;
            const Item x = make_item(g, cur_it, PAD);
            unsigned char* st = smem + s * kStageBytes;
            const uint32_t st_a = smem0 + s * kStageBytes;
            int* s_kc = reinterpret_cast<int*>(st + kOffKc);
            int* s_klab = reinterpret_cast<int*>(st + kOffKlab);
            int* s_rowmeta = reinterpret_cast<int*>(st + kOffRowMeta);
            int* s_rowtok = reinterpret_cast<int*>(st + kOffRowTok);
            const size_t sample_off = (size_t)x.b * HW;

            // Slots advance by a fixed step, so their window offsets (a, b) = (slot / width, slot mod width) are
            // carried along instead of divided out each time (a division is a long chain through the reciprocal unit).
            const int ew = PAD ? 16 : x.r.ew;               // slots per window row
            const int bw = x.r.ew;                          // PAD: offsets b >= bw hold no token
            const int q_s = kLoaderThreads / ew, r_s = kLoaderThreads - q_s * ew;              // slot loop: step of kLoaderThreads
            const int q_r = (kLoaderThreads / 4) / ew, r_r = (kLoaderThreads / 4) - q_r * ew;  // row loop: step of kLoaderThreads / 4
            int a_s = lt / ew, b_s = lt - a_s * ew;
            for (int slot = lt; slot < kMaxSlots; slot += kLoaderThreads) {
                // a slot without a token: as a key its bias index lands in the table's -inf zone
                int code = 0, label = 0xff, tok = -1, kc = 4 * (2 * c0 + 1);
                if (slot < x.r.n && (!PAD || b_s < bw)) {
                    tok = offset_token_tc(g, x.r, a_s, b_s, cs, code, label);
                    kc = 4 * (c0 - code);
                }
                s_kc[slot] = kc;
                s_klab[slot] = label;
                s_rowmeta[slot] = code | (label << 16);
                s_rowtok[slot] = tok;
                a_s += q_s; b_s += r_s;
                if (b_s >= ew) { b_s -= ew; ++a_s; }
            }
            // rows: this thread owns 16-byte chunk (lt & 3) of rows (lt >> 2) + (kLoaderThreads / 4) i
            const int chunk = lt & 3;
            int a_r = (lt >> 2) / ew, b_r = (lt >> 2) - a_r * ew;
            for (int row = lt >> 2; row < x.npad; row += kLoaderThreads / 4) {
                const __nv_bfloat16 *sq = q, *sk = k, *sv = v;
                int bytes = 0;   // rows past the window's end are written as zeros
                if (row < x.r.n && (!PAD || b_r < bw)) {
                    int code, label;
                    const int tok = offset_token_tc(g, x.r, a_r, b_r, cs, code, label);
                    const size_t off = (sample_off + (size_t)tok) * g.ts + x.head * kD + chunk * 8;
                    sq = q + off; sk = k + off; sv = v + off;
                    bytes = 16;
                }
                const uint32_t so = st_a + tile_off<kD>(row, chunk);
                cp_async16(so + kOffQ, sq, bytes);
                cp_async16(so + kOffK, sk, bytes);
                cp_async16(so + kOffV, sv, bytes);
                a_r += q_r; b_r += r_r;
                if (b_r >= ew) { b_r -= ew; ++a_r; }
            }
            const float* bsrc = bias_prep + (size_t)x.head * kFwdBiasFloats;
            for (int c = lt; c < kFwdBiasFloats / 4; c += kLoaderThreads)
                cp_async16(st_a + kOffBias + c * 16, bsrc + c * 4, 16);
            cp_async_commit();
            if (pending_s >= 0) {           // the previous item's copies have landed: publish it
                cp_async_wait<1>();
                fence_proxy_async();
                mbar_arrive(bar_full(pending_s));
            }
            pending_s = s;
        }
        if (pending_s >= 0) {
            cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(bar_full(pending_s));
        }
    } else {
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp runs the loop and waits (a warp whose 32 lanes wait together is parked and woken as a
        // whole); one elected lane issues the MMAs and commits.
        {
            const uint32_t idesc_pv = make_idesc_elem(128, kNO, 0, 1);   // B = [V | ones]: 32 + 16 columns
            int kuse = 0, use_t[2] = {0, 0}, freed_t[2] = {0, 0};   // uses begun / s_free phases consumed
            bool ok = true;
            auto issue_qk = [&](const Item& x, int s, int t) {
                const uint32_t qa = smem0 + s * kStageBytes + kOffQ + t * 128 * kRowBytes;
                const uint32_t ka = smem0 + s * kStageBytes + kOffK;
                const uint32_t idesc = make_idesc_elem(128, x.npad, 0, 0);
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks)
                        mma_ss(tmem_base + t * 256, make_sdesc_sw64(qa + ks * 32, 512), make_sdesc_sw64(ka + ks * 32, 512),
                               idesc, ks > 0 ? 1u : 0u);
                    mma_commit(bar_sready(t));
                }
                __syncwarp();
            };
            // O += P V over key steps [ks0, ks1) of 16 keys; P of step ks sits at TMEM column p_col(ks / 2) + 8 (ks & 1)
            const uint32_t d_hi = sdesc_hi(make_sdesc_sw64(smem0, 512));
            auto issue_pv = [&](const Item& x, int s, int t, int ks0, int ks1) {
                // descriptor low word = start address in 16-byte units; one key step = 16 rows of 64 bytes
                // the second 32-column group of B (the ones block) lies one leading-dimension stride behind V
                const uint32_t v_lo = sdesc_lo(make_sdesc_sw64_mn(smem0 + s * kStageBytes + kOffV, kOffOnes - (s * kStageBytes + kOffV), 512));
                const uint32_t t_o = tmem_base + t * 256 + kColO, t_p = tmem_base + t * 256;
                if (elect_one()) {
                    int ks = ks0;
                    if (ks == 0 && ks < ks1) {
                        mma_ts_h<false>(t_o, t_p + p_col(0), v_lo, d_hi, idesc_pv);
                        ks = 1;
                    }
                    for (; ks < ks1; ++ks)
                        mma_ts_h<true>(t_o, t_p + p_col(ks >> 1) + 8 * (ks & 1), v_lo + 64 * ks, d_hi, idesc_pv);
                }
                __syncwarp();
            };
            long long it = blockIdx.x;
            ItemCursor nx_it = cursor_init(blockIdx.x, gridDim.x, g.heads, g.Mw, g.Mh);     // runs one item ahead
            Item cur;
            if (it < n_items) {
                cur = make_item(g, nx_it, PAD);
                cursor_advance(nx_it, g.heads, g.Mw, g.Mh);
                ok = mbar_wait_all(bar_full(0), 0, cta_abort);
                if (ok) {
                    fence_proxy_async();
                    tc_fence_after();
                    for (int t = 0; t < cur.ntiles; ++t) issue_qk(cur, 0, t);   // TMEM regions start out free
                }
            }
            for (; ok && it < n_items; it += gridDim.x, ++kuse) {
                const int s = kuse % kStages;
                const long long nxt = it + gridDim.x;
                const bool has_next = nxt < n_items;
                Item nx;
                const int sn = (kuse + 1) % kStages;
                if (has_next) {
                    nx = make_item(g, nx_it, PAD);
                    cursor_advance(nx_it, g.heads, g.Mw, g.Mh);
                }
                bool next_ready = false;
                const int nks = cur.npad >> 4;
                // first 128 keys of each tile, as soon as their P is there
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (!ok || t >= cur.ntiles) continue;
                    ok = mbar_wait_all(bar_phalf(t), use_t[t] & 1, cta_abort);
                    if (!ok) continue;
                    tc_fence_after();
                    issue_pv(cur, s, t, 0, min(8, nks));
                }
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    if (!ok) break;
                    if (t < cur.ntiles) {
                        ok = mbar_wait_all(bar_pready(t), use_t[t] & 1, cta_abort);   // use_t[t] still counts earlier uses only
                        if (!ok) break;
                        tc_fence_after();
                        issue_pv(cur, s, t, 8, nks);
                        if (elect_one()) {
                            mma_commit(bar_oready(t));
                            if (t == cur.ntiles - 1) mma_commit(bar_empty(s));   // all operands of this stage consumed
                        }
                        __syncwarp();
                    }
                    if (has_next && t < nx.ntiles) {
                        if (!next_ready) {
                            ok = mbar_wait_all(bar_full(sn), ((kuse + 1) / kStages) & 1, cta_abort);
                            if (!ok) break;
                            fence_proxy_async();
                            next_ready = true;
                        }
                        if (t < cur.ntiles) ++use_t[t];
                        // region t is free once its softmax warpgroup has read O of the last item that used it
                        while (ok && freed_t[t] < use_t[t]) {
                            ok = mbar_wait_all(bar_sfree(t), freed_t[t] & 1, cta_abort);
                            ++freed_t[t];
                        }
                        if (!ok) break;
                        tc_fence_after();
                        issue_qk(nx, sn, t);
                    } else if (t < cur.ntiles) {
                        ++use_t[t];
                    }
                }
                cur = nx;
            }
        }
    }
    } else {
        // ------------------------------------------------------------------ softmax warpgroups
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsSoftmax));
        const int wg = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const int slot = wg * 128 + row;
        const uint32_t lane_addr = ((uint32_t)(32 * (warp & 3))) << 16;
        const uint32_t t_s = tmem_base + lane_addr + wg * 256;
        const float scale = g.scale_log2e;
        int kuse = 0, use = 0;
        ItemCursor cur_it = cursor_init(blockIdx.x, gridDim.x, g.heads, g.Mw, g.Mh);
        for (long long it = blockIdx.x; it < n_items; it += gridDim.x, ++kuse, cursor_advance(cur_it, g.heads, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur_it, PAD);
            const int s = kuse % kStages;
            const uint32_t st_a = smem0 + s * kStageBytes;
            // Every warpgroup follows the stage ring item by item, also the second one through items that have no
            // second query tile: a wait names its barrier phase by parity only, so a warpgroup that skipped ahead
            // by a whole turn of the ring would take an older phase for the one it wants.  Its arrival on the
            // stage's release barrier keeps the loaders from lapping it the other way round.
            if (!__all_sync(0xffffffffu, mbar_wait(bar_full(s), (kuse / kStages) & 1, cta_abort))) break;
            if (wg >= x.ntiles) {
                mbar_arrive(bar_empty(s));
                continue;
            }
            const int rmeta = lds_i32(st_a + kOffRowMeta + 4 * slot);
            const int tok = lds_i32(st_a + kOffRowTok + 4 * slot);
            const uint32_t bias_i = st_a + kOffBias + 4 * meta_code(rmeta);
            const int label_i = meta_label(rmeta);
            const float bmax = lds_f32(st_a + kOffBias + 4 * (kFwdBiasFloats - 1));

            if (!__all_sync(0xffffffffu, mbar_wait(bar_sready(wg), use & 1, cta_abort))) break;
            tc_fence_after();
            float m, sum;
            const bool wide = bmax == INFINITY;      // the head's bias table spreads too far for the bound on the row maximum
            if (PAD) {
                // full-width windows without mask labels: the row path, compiled for this width; the others: by the tables
                if (x.masked || wide || x.r.ew != PADW)
                    m = softmax_row<true>(t_s, x.npad, x.r.n, bias_i, st_a + kOffKc, st_a + kOffKlab, label_i, scale, bmax, sum, bar_phalf(wg));
                else
                    m = softmax_row<false, true, PAD ? PADW : 16>(t_s, x.npad, x.r.n, bias_i, st_a + kOffKc, st_a + kOffKlab, label_i, scale, bmax,
                                                                  sum, bar_phalf(wg), bias_i + 4 * c0, 4 * cs);
            } else if (W16) {
                if (x.masked || x.r.n != 256 || wide)
                    m = softmax_row<true>(t_s, x.npad, x.r.n, bias_i, st_a + kOffKc, st_a + kOffKlab, label_i, scale, bmax, sum, bar_phalf(wg));
                else
                    m = softmax_row<false, true>(t_s, x.npad, x.r.n, bias_i, st_a + kOffKc, st_a + kOffKlab, label_i, scale, bmax, sum, bar_phalf(wg),
                                                 bias_i + 4 * c0, 4 * cs);
            } else {
                if (x.masked || wide) m = softmax_row<true>(t_s, x.npad, x.r.n, bias_i, st_a + kOffKc, st_a + kOffKlab, label_i, scale, bmax, sum, bar_phalf(wg));
                else m = softmax_row<false>(t_s, x.npad, x.r.n, bias_i, st_a + kOffKc, st_a + kOffKlab, label_i, scale, bmax, sum, bar_phalf(wg));
            }
            tmem_st_wait();
            tc_fence_before();
            if (x.npad <= 128) mbar_arrive(bar_phalf(wg));      // short rows: both halves at once
            mbar_arrive(bar_pready(wg));
            if (wg == 1) mbar_arrive(bar_empty(s));            // this warpgroup has read all it needs from the stage

            const size_t row_off = ((size_t)x.b * HW + (size_t)(tok < 0 ? 0 : tok)) * g.heads + x.head;

            if (!__all_sync(0xffffffffu, mbar_wait(bar_oready(wg), use & 1, cta_abort))) break;
            tc_fence_after();
            uint32_t ro[32], rsum;
            tmem_ld32(t_s + kColO, ro);
            tmem_ld1(t_s + kColO + kD, rsum);       // row sum of P (as rounded to bf16), from the ones columns
            tmem_ld_wait();
            sum = __uint_as_float(rsum);
            if (tok >= 0) lse[row_off] = (m + log2f(sum)) * kLn2;
            const float inv = 1.f / sum;
            tc_fence_before();
            mbar_arrive(bar_sfree(wg));
            ++use;
            if (tok >= 0) {
                uint4* dst = reinterpret_cast<uint4*>(o + row_off * kD);
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint4 val;
                    val.x = pack_elem(__uint_as_float(ro[c4 * 8 + 0]) * inv, __uint_as_float(ro[c4 * 8 + 1]) * inv);
                    val.y = pack_elem(__uint_as_float(ro[c4 * 8 + 2]) * inv, __uint_as_float(ro[c4 * 8 + 3]) * inv);
                    val.z = pack_elem(__uint_as_float(ro[c4 * 8 + 4]) * inv, __uint_as_float(ro[c4 * 8 + 5]) * inv);
                    val.w = pack_elem(__uint_as_float(ro[c4 * 8 + 6]) * inv, __uint_as_float(ro[c4 * 8 + 7]) * inv);
                    dst[c4] = val;
                }
            }
        }
    }

    // teardown: every role ends up here, also after an expired wait
    cp_async_wait<0>();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
    if (tid == 0 && *cta_abort) atomicExch(&g_tc_timeout, 1);
}

// Per head, with code stride cs = w + 32 and c0 = (w - 1) * (cs + 1):
//   table[(da + w - 1) * cs + (db + w - 1)] = T[(da + w - 1) * (2w - 1) + (db + w - 1), head] * log2(e)
//   for |da|, |db| < w (unused gaps 0), table[2 c0 + 1 .. 3 c0 + 1] = -inf (where key slots without a
//   token point), and the head's largest entry in the last float (+inf instead if the head's entries spread over
//   more than 64 octaves: the forward kernel then takes exact row maxima).
__global__ void __launch_bounds__(256)
swin_fwd_bias_prep_kernel(const float* __restrict__ bias, float* __restrict__ prep, int w, int heads, int cs) {
    const int head = blockIdx.x;
    const int nw = 2 * w - 1;
    const int c0 = (w - 1) * (cs + 1);
    float* dst = prep + (size_t)head * kFwdBiasFloats;
    float mx = -INFINITY, mn = INFINITY;
    for (int e = threadIdx.x; e < kFwdBiasFloats - 1; e += blockDim.x) {
        float val = 0.f;
        if (e > 2 * c0) {
            val = -INFINITY;
        } else {
            const int ra = e / cs, rb = e - ra * cs;
            if (rb < nw) {
                val = bias[(size_t)(ra * nw + rb) * heads + head] * kLog2e;
                mx = fmaxf(mx, val);
                mn = fminf(mn, val);
            }
        }
        dst[e] = val;
    }
    __shared__ float red[8], red_mn[8];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, off));
    }
    if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = mx; red_mn[threadIdx.x >> 5] = mn; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) { mx = fmaxf(mx, red[i]); mn = fminf(mn, red_mn[i]); }
        dst[kFwdBiasFloats - 1] = (mx - mn <= 64.f) ? mx : INFINITY;
    }
}

}  // namespace

#ifndef TERRA_ELEM_F16
// window sides 9 .. 15 run in the layout of 16 slots per window row (TERRA_NO_PAD16=1: a debugging switch that keeps
// the packed layout)
bool pad16_layout(const Geo& g) {
    static const bool pad_off = [] { const char* e_ = std::getenv("TERRA_NO_PAD16"); return e_ && e_[0] == '1'; }();
    return g.d == 32 && g.w > 8 && g.w < 16 && !pad_off;
}

bool fwd_tc_supported(const Geo& g) { return g.d == 32 && g.nmax <= kMaxSlots && g.w <= 16; }

// The TMA variants fetch a window row with one tiled copy: every window row must be one run of consecutive tokens
// (the longitude roll may not cut through a window) of 16 tokens, or 8 in the last window column.
bool tma_row_shape(const Geo& g) {
    if (g.w != 16 || g.d != 32 || g.W < 16 || (g.W % 16 != 0 && g.W % 16 != 8)) return false;
    if ((long long)g.B * g.H * g.W >= 0x7fffffffLL) return false;       // token coordinate of the tensor map is int32
    for (int wc = 0; wc < g.Mw; ++wc) {
        const int ew = g.W - wc * 16 < 16 ? g.W - wc * 16 : 16;
        const int v0 = (wc * 16 + g.sw) % g.W;
        if (v0 + ew > g.W) return false;
    }
    return true;
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's encoder, looked up through the runtime (the library does not link against the driver library).
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess || qres != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

// [tokens][channels] bf16 with a token stride of `token_stride` elements; box = 32 channels x `box_tokens` tokens,
// 64-byte swizzle.  `map` points to a CUtensorMap.
bool make_row_map(void* map, const Geo& g, const void* base, int token_stride, int box_tokens) {
    CUtensorMap* m = reinterpret_cast<CUtensorMap*>(map);
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)g.heads * g.d, (cuuint64_t)g.B * g.H * g.W};
    const cuuint64_t strides[1] = {(cuuint64_t)token_stride * 2};
    const cuuint32_t box[2] = {32u, (cuuint32_t)box_tokens};
    const cuuint32_t estr[2] = {1u, 1u};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_col_map(CUtensorMap* map, const Geo& g, const void* base, int token_stride) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)g.heads * g.d, (cuuint64_t)g.W, (cuuint64_t)g.B * g.H};
    const cuuint64_t strides[2] = {(cuuint64_t)token_stride * 2, (cuuint64_t)g.W * token_stride * 2};
    const cuuint32_t box[3] = {32u, 1u, 16u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_col_map4(CUtensorMap* map, const Geo& g, const void* base, int token_stride) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc || g.W < 4 || g.H < 16) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)g.heads * g.d, (cuuint64_t)g.B * g.H, (cuuint64_t)g.W};
    const cuuint64_t strides[2] = {(cuuint64_t)g.W * token_stride * 2, (cuuint64_t)token_stride * 2};
    const cuuint32_t box[3] = {32u, 16u, 4u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_row_maps3(RowMaps3* maps, const Geo& g, const void* base, int token_stride) {
    for (int i = 0; i < 3; ++i)
        if (!make_row_map(&maps->m[i], g, base, token_stride, 32 >> i)) return false;
    // window sides 64 and 128: boxes of 64 and 128 tokens (a box may not be longer than the token axis); window side 32
    // on grids of complete windows: boxes of 2 and 4 token rows x 32 token columns of the tensor as a 3-D array
    for (int i = 3; i < 5; ++i) {
        const long long tokens = (long long)g.B * g.H * g.W;
        if (g.w == 32 && g.H % 32 == 0 && g.W % 32 == 0) {
            EncodeTiledFn enc = encode_tiled_fn();
            if (!enc) return false;
            const cuuint64_t dims[3] = {(cuuint64_t)g.heads * g.d, (cuuint64_t)g.W, (cuuint64_t)g.B * g.H};
            const cuuint64_t strides[2] = {(cuuint64_t)token_stride * 2, (cuuint64_t)g.W * token_stride * 2};
            const cuuint32_t box[3] = {32u, 32u, i == 3 ? 2u : 4u};
            const cuuint32_t estr[3] = {1u, 1u, 1u};
            if (enc(&maps->m[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
                return false;
            continue;
        }
        const int box = (g.w >= 64 && tokens >= (8 << i)) ? (8 << i) : 32;           // m[3]: 64 tokens, m[4]: 128 tokens
        if (!make_row_map(&maps->m[i], g, base, token_stride, box)) return false;
    }
    return true;
}

size_t fwd_tc_workspace_bytes(const Geo& g) { return (size_t)g.heads * kFwdBiasFloats * sizeof(float); }
#endif  // !TERRA_ELEM_F16

cudaError_t launch_fwd_tc(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                          void* o, float* lse, void* workspace, int sm_count, cudaStream_t stream) {
    const long long items = (long long)g.B * g.Mh * g.Mw * g.heads;
    float* prep = reinterpret_cast<float*>(workspace);
    const bool pad = pad16_layout(g);
    swin_fwd_bias_prep_kernel<<<g.heads, 256, 0, stream>>>(bias, prep, g.w, g.heads, pad ? 48 : g.w + 32);
    count_launch(stream);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    FwdMaps maps;
    std::memset(&maps, 0, sizeof maps);
    static const bool tma_off = [] { const char* e_ = std::getenv("TERRA_NO_TMA"); return e_ && e_[0] == '1'; }();
    const bool tma = !tma_off && tma_row_shape(g) && make_row_map(&maps.q16, g, q, g.ts, 16) && make_row_map(&maps.k16, g, k, g.ts, 16) &&
                     make_row_map(&maps.v16, g, v, g.ts, 16) && make_row_map(&maps.q8, g, q, g.ts, 8) && make_row_map(&maps.k8, g, k, g.ts, 8) &&
                     make_row_map(&maps.v8, g, v, g.ts, 8);
    auto kern = tma ? swin_fwd_tc_kernel<true, true> : (g.w == 16 ? swin_fwd_tc_kernel<true, false> : swin_fwd_tc_kernel<false, false>);
    if (pad) {
        switch (g.w) {
            case 9: kern = swin_fwd_tc_kernel<false, false, 9>; break;
            case 10: kern = swin_fwd_tc_kernel<false, false, 10>; break;
            case 11: kern = swin_fwd_tc_kernel<false, false, 11>; break;
            case 12: kern = swin_fwd_tc_kernel<false, false, 12>; break;
            case 13: kern = swin_fwd_tc_kernel<false, false, 13>; break;
            case 14: kern = swin_fwd_tc_kernel<false, false, 14>; break;
            default: kern = swin_fwd_tc_kernel<false, false, 15>; break;
        }
    }
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)(items < sm_count ? items : sm_count);
    prof_begin("swin_fwd_tc_kernel", stream);
    kern<<<grid, kThreads, kSmemBytes, stream>>>(g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, prep,
                                                 (__nv_bfloat16*)o, lse, items, maps);
    count_launch(stream);
    return cudaGetLastError();
}

#ifndef TERRA_ELEM_F16
// Self-test of the failure report: one CTA waits, with a short cycle limit, on a barrier that nothing ever
// arrives on; the wait gives up, the kernel raises the device status word and returns normally.
__global__ void bounded_wait_selftest_kernel(long long limit_cycles) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        tc::fence_barrier_init();
    }
    __syncthreads();
    const bool ok = tc::mbar_wait(smem_u32(&bar), 0, &abort_flag, limit_cycles);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_flag)) atomicExch(&g_tc_timeout, 1);
}

cudaError_t launch_bounded_wait_selftest(long long limit_cycles, cudaStream_t stream) {
    bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(limit_cycles);
    count_launch(stream);
    return cudaGetLastError();
}

// prepared bias tables for every head (also used by the backward kernels)
cudaError_t launch_bias_prep(const Geo& g, const float* bias, float* prep, cudaStream_t stream) {
    swin_fwd_bias_prep_kernel<<<g.heads, 256, 0, stream>>>(bias, prep, g.w, g.heads, pad16_layout(g) ? 48 : g.w + 32);
    count_launch(stream);
    return cudaGetLastError();
}

#endif  // !TERRA_ELEM_F16

cudaError_t read_tc_status(int* timed_out, cudaStream_t stream) {
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return e;
    int zero = 0;
    e = cudaMemcpyFromSymbol(timed_out, g_tc_timeout, sizeof(int));
    if (e != cudaSuccess) return e;
    if (*timed_out) e = cudaMemcpyToSymbol(g_tc_timeout, &zero, sizeof(int));
    return e;
}

}  // namespace terra
