// Backward shifted-window attention on the tcgen05 tensor cores (head dim 32, windows of <= 256 tokens).
//
// One kernel template, launched twice per call:
//   query side (KV = false): rows = queries.  S = Q K^T and dP = dO V^T per key block, dS = P (dP - delta)
//                            written to TMEM as bf16, dQ += dS K (dS read from TMEM); the bias gradient is
//                            summed in a per-CTA shared-memory table and flushed once with global atomics.
//   key side   (KV = true):  rows = keys.  S^T = K Q^T and dP^T = V dO^T per query block, P^T and dS^T
//                            written to TMEM as bf16, dV += P^T dO and dK += dS^T Q.
// P is recomputed from the saved log-sum-exp, so the column blocks of a row are independent (no running
// maximum).  Structure as in the forward kernel: persistent CTAs, two 128-row tiles (one per elementwise
// warpgroup, one thread per row), one MMA-issuing lane per tile (so one tile's elementwise work never delays the other tile's
// MMAs), two loader warps gathering the window's rows with
// cp.async into the 64-byte-swizzled operand layout.  CTAs are bound to one head (grid = heads x CTAs per
// head), so the head's bias table is staged once per CTA and the bias-gradient table belongs to one head.
// TMEM, per 128-row tile (256 columns): two buffers [S 48 | dP 48] for column blocks in flight (the MMAs
// run up to two blocks ahead of the elementwise warpgroup), then the accumulators: query side dQ (32
// columns), key side dV and dK (32 each).  The bf16 P / dS overwrite the fp32 S / dP they came from.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag and all roles leave their loops.
#include "swin_common.cuh"
#include "swin_kernels.h"
#include "tc_common.cuh"

namespace terra {

__device__ int g_bwd_tc_timeout = 0;   // set when a bounded wait expired in any CTA of the kernels below

namespace {

using namespace tc;

constexpr int kMmaWarp = 8;         // warps 8 and 9: one MMA-issuing lane per 128-row tile
constexpr int kLoaderWarp0 = 10;
constexpr int kLoaderWarps = 2;
constexpr int kLoaderThreads = kLoaderWarps * 32;
constexpr int kThreads = (kLoaderWarp0 + kLoaderWarps) * 32;   // 384 = three warpgroups
constexpr int kRegsLaunch = 168;
constexpr int kRegsWork = 216;      // elementwise warpgroups after setmaxnreg.inc
constexpr int kRegsOther = 64;      // MMA + loader warpgroup after setmaxnreg.dec
static_assert(2 * (kRegsWork - kRegsLaunch) <= (kRegsLaunch - kRegsOther), "register hand-over does not balance");

constexpr int kStages = 2;
constexpr int kMaxSlots = 256;
constexpr int kD = 32;
constexpr int kRowBytes = kD * 2;
constexpr int kTileBytes = kMaxSlots * kRowBytes;              // 16384

// stage layout (bytes)
constexpr int kOffQ = 0;
constexpr int kOffK = kTileBytes;
constexpr int kOffV = 2 * kTileBytes;
constexpr int kOffDO = 3 * kTileBytes;
constexpr int kOffColOff = 4 * kTileBytes;                     // per slot as a column: byte offset into the bias table
constexpr int kOffLab = kOffColOff + kMaxSlots * 4;            // per slot: shift-mask label (0xff: no token)
constexpr int kOffCode = kOffLab + kMaxSlots * 4;              // per slot: bias code a * (w + 32) + b
constexpr int kOffTok = kOffCode + kMaxSlots * 4;              // per slot: grid token, -1 if none
constexpr int kOffLse = kOffTok + kMaxSlots * 4;               // per slot: lse * log2(e), +inf if none
constexpr int kOffDelta = kOffLse + kMaxSlots * 4;             // per slot: delta
constexpr int kStageBytes = ((kOffDelta + kMaxSlots * 4 + 1023) / 1024) * 1024;   // 71680
// after the stages
constexpr int kOffBias = kStages * kStageBytes;                // the head's prepared bias table (kFwdBiasFloats floats)
constexpr int kOffDBias = kOffBias + kFwdBiasFloats * 4;       // query side: one bias-gradient table per elementwise warp
constexpr int kDBiasFloats = 1536;                             // >= 2 c0 + 1 for w <= 16
constexpr int kOffBars = kOffDBias + 8 * kDBiasFloats * 4;
constexpr int kOffOutStage = kOffBars + 256;                   // per elementwise warp: 32 output rows on their way out (query side)
constexpr int kSmemBytes = kOffOutStage + 8 * 32 * kRowBytes;

__device__ __forceinline__ int code_stride(int w) { return w + 32; }

struct Item {
    int b, win;
    WindowRef r;
    int npad;      // slots rounded up to 16
    int ntiles;    // 128-row tiles in use
    bool masked;   // the window mixes shift-mask labels
    bool ragged;   // some row of a 128-row tile, or some column below npad, has no token
};

__device__ __forceinline__ Item make_item(const Geo& g, long long it) {
    Item x;
    const int M = g.Mh * g.Mw;
    x.win = (int)(it % M);
    x.b = (int)(it / M);
    x.r = window_ref(g, x.win);
    x.npad = (x.r.n + 15) & ~15;
    x.ntiles = (x.r.n + 127) >> 7;
    const int r0 = x.r.wr * g.w, c0 = x.r.wc * g.w;
    const bool mh = !g.ph && g.sh > 0 && r0 < g.H - g.sh && r0 + x.r.eh > g.H - g.sh;
    const bool mw = !g.pw && g.sw > 0 && c0 < g.W - g.sw && c0 + x.r.ew > g.W - g.sw;
    x.masked = mh || mw;
    x.ragged = x.npad != x.r.n || x.r.n != x.ntiles * 128;   // some row of a tile or some column has no token
    return x;
}

__device__ __forceinline__ int slot_token_tc(const Geo& g, const WindowRef& r, int slot, int& code, int& label) {
    const int a = slot / r.ew;
    const int b = slot - a * r.ew;
    int u = r.wr * g.w + a + g.sh;
    if (u >= g.H) u -= g.H;
    int v = r.wc * g.w + b + g.sw;
    if (v >= g.W) v -= g.W;
    label = ((!g.ph && u < g.sh) ? 2 : 0) + ((!g.pw && v < g.sw) ? 1 : 0);
    code = a * code_stride(g.w) + b;
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
__device__ __forceinline__ float4 lds_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ int lds_i32(uint32_t addr) {
    int v;
    asm volatile("ld.shared.s32 %0, [%1];\n" : "=r"(v) : "r"(addr));
    return v;
}
// table[addr] += v in the warp's own table.  Not atomic: within one warp instruction the 32 lanes (32
// different rows, same column) touch 32 different entries, and successive instructions of a warp reach
// shared memory in program order, so nothing is lost.
__device__ __forceinline__ void rmw_shared_f32(uint32_t addr, float v) {
    asm volatile(
        "{\n\t.reg .f32 t;\n\t"
        "ld.shared.f32 t, [%0];\n\t"
        "add.f32 t, t, %1;\n\t"
        "st.shared.f32 [%0], t;\n\t}\n" ::"r"(addr), "f"(v) : "memory");
}

// What one elementwise thread knows about its row.
struct RowCtx {
    uint32_t bias_row;   // shared address: bias table + the row's part of the index
    uint32_t dbias_row;  // shared address: this warp's bias-gradient table + the row's part of the index (query side)
    int label;
    float lse2, delta;   // query side: of this row
    bool valid;
};

// 16 columns of one row: P = exp2(S * scale + bias - lse), dS = P * (dP - delta); packs dS (and P) to bf16.
//   KV = false: rows are queries (lse, delta per row); adds dS into the bias-gradient table.
//   KV = true : rows are keys    (lse, delta per column).
// Two table updates whose entries cannot coincide (see bwd_block), issued together so that their
// load-add-store latencies overlap.
__device__ __forceinline__ void rmw2_shared_f32(uint32_t addr0, float v0, uint32_t addr1, float v1) {
    asm volatile(
        "{\n\t.reg .f32 t0, t1;\n\t"
        "ld.shared.f32 t0, [%0];\n\t"
        "ld.shared.f32 t1, [%2];\n\t"
        "add.f32 t0, t0, %1;\n\t"
        "add.f32 t1, t1, %3;\n\t"
        "st.shared.f32 [%0], t0;\n\t"
        "st.shared.f32 [%2], t1;\n\t}\n" ::"r"(addr0), "f"(v0), "r"(addr1), "f"(v1) : "memory");
}

// HOLD = 0: add dS into the bias-gradient table now; 1: only hand the 16 (address, dS) pairs back in
// held_addr / held_ds; 2: add them together with this step's pairs, two entries at a time.
template <bool KV, bool MASKED, bool RAGGED, int HOLD = 0>
__device__ __forceinline__ void bwd_cols16(const uint32_t (&rs)[16], const uint32_t (&rp)[16], uint32_t (&pk_p)[8], uint32_t (&pk_ds)[8],
                                           int c, const RowCtx& rc, uint32_t st_a, float scale, int dbias_limit,
                                           uint32_t (&held_addr)[16], float (&held_ds)[16]) {
    // all shared-memory loads first (the explicit loads keep their order), then the arithmetic
    int co[16], kl[16];
    float l2[16], dl[16], bv[16];
#pragma unroll
    for (int e4 = 0; e4 < 4; ++e4) {
        const int4 co4 = lds_i4(st_a + kOffColOff + 4 * (c + e4 * 4));
        co[e4 * 4] = co4.x; co[e4 * 4 + 1] = co4.y; co[e4 * 4 + 2] = co4.z; co[e4 * 4 + 3] = co4.w;
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) bv[e] = lds_f32(rc.bias_row + co[e]);
    if (MASKED) {
#pragma unroll
        for (int e4 = 0; e4 < 4; ++e4) {
            const int4 kl4 = lds_i4(st_a + kOffLab + 4 * (c + e4 * 4));
            kl[e4 * 4] = kl4.x; kl[e4 * 4 + 1] = kl4.y; kl[e4 * 4 + 2] = kl4.z; kl[e4 * 4 + 3] = kl4.w;
        }
    }
    if (KV) {
#pragma unroll
        for (int e4 = 0; e4 < 4; ++e4) {
            const float4 a = lds_f4(st_a + kOffLse + 4 * (c + e4 * 4));
            const float4 b = lds_f4(st_a + kOffDelta + 4 * (c + e4 * 4));
            l2[e4 * 4] = a.x; l2[e4 * 4 + 1] = a.y; l2[e4 * 4 + 2] = a.z; l2[e4 * 4 + 3] = a.w;
            dl[e4 * 4] = b.x; dl[e4 * 4 + 1] = b.y; dl[e4 * 4 + 2] = b.z; dl[e4 * 4 + 3] = b.w;
        }
    }
    float p[16], ds[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        const float lse_e = KV ? l2[e] : rc.lse2;
        const float del_e = KV ? dl[e] : rc.delta;
        float xv = fmaf(__uint_as_float(rs[e]), scale, bv[e]) - lse_e;
        if (MASKED && kl[e] != rc.label) xv = -INFINITY;
        p[e] = fast_exp2(xv);
        ds[e] = p[e] * (__uint_as_float(rp[e]) - del_e);
    }
    if (!KV && HOLD == 1) {
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            held_addr[e] = rc.dbias_row + co[e];
            held_ds[e] = ds[e];
        }
    } else if (!KV && HOLD == 2) {
#pragma unroll
        for (int e = 0; e < 16; ++e) rmw2_shared_f32(held_addr[e], held_ds[e], rc.dbias_row + co[e], ds[e]);
    } else if (!KV) {
        // one warp instruction touches 32 different table entries (32 different rows, one column)
#pragma unroll
        for (int e = 0; e < 16; ++e) {
            if (RAGGED) {
                if (rc.valid && co[e] < dbias_limit) rmw_shared_f32(rc.dbias_row + co[e], ds[e]);
            } else {
                rmw_shared_f32(rc.dbias_row + co[e], ds[e]);
            }
        }
    }
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) {
        if (KV) pk_p[e2] = pack_bf16(p[2 * e2], p[2 * e2 + 1]);
        pk_ds[e2] = pack_bf16(ds[2 * e2], ds[2 * e2 + 1]);
    }
}

// All columns [0, ncols) of one column block for one row; S at t_s, dP at t_dp (fp32), overwritten in place
// by bf16 P (key side) and dS.  16 columns per step, the next step's loads in flight.
template <bool KV, bool MASKED, bool RAGGED>
__device__ __forceinline__ void bwd_block(uint32_t t_s, uint32_t t_dp, int c_first, int ncols, const RowCtx& rc, uint32_t st_a,
                                          float scale, int dbias_limit) {
    uint32_t sa[16], pa[16], sb[16], pb[16];
    uint32_t held_addr[16];
    float held_ds[16];
    const int nsteps = ncols >> 4;
    tmem_ld16(t_s, sa);
    tmem_ld16(t_dp, pa);
    if (!KV && !RAGGED && nsteps == 3) {
        // Query side, full block of three 16-column steps.  Table updates of one step must stay in program
        // order with those of the next step (lane l at column j and lane l + 1 at column j + 1 share an
        // entry), but columns 32 apart never share one inside a warp: bias codes grow with the slot and
        // determine the slot distance, and a warp spans only 32 slots.  So steps 0 and 2 are updated
        // together, two independent entries per instruction group, and the serial chain is a third shorter.
        uint32_t pk_p[8], pk_ds[8];
        tmem_ld_wait();
        tmem_ld16(t_s + 16, sb);
        tmem_ld16(t_dp + 16, pb);
        bwd_cols16<KV, MASKED, RAGGED, 1>(sa, pa, pk_p, pk_ds, c_first, rc, st_a, scale, dbias_limit, held_addr, held_ds);
        tmem_st8(t_dp, pk_ds);
        tmem_ld_wait();
        tmem_ld16(t_s + 32, sa);
        tmem_ld16(t_dp + 32, pa);
        {
            uint32_t na[16];
            float nd[16];
            bwd_cols16<KV, MASKED, RAGGED, 0>(sb, pb, pk_p, pk_ds, c_first + 16, rc, st_a, scale, dbias_limit, na, nd);
        }
        tmem_st8(t_dp + 8, pk_ds);
        tmem_ld_wait();
        bwd_cols16<KV, MASKED, RAGGED, 2>(sa, pa, pk_p, pk_ds, c_first + 32, rc, st_a, scale, dbias_limit, held_addr, held_ds);
        tmem_st8(t_dp + 16, pk_ds);
        return;
    }
    for (int i = 0; i < nsteps; i += 2) {
        uint32_t pk_p[8], pk_ds[8];
        tmem_ld_wait();
        if (i + 1 < nsteps) {
            tmem_ld16(t_s + 16 * (i + 1), sb);
            tmem_ld16(t_dp + 16 * (i + 1), pb);
        }
        bwd_cols16<KV, MASKED, RAGGED, 0>(sa, pa, pk_p, pk_ds, c_first + 16 * i, rc, st_a, scale, dbias_limit, held_addr, held_ds);
        if (KV) tmem_st8(t_s + 8 * i, pk_p);
        tmem_st8(t_dp + 8 * i, pk_ds);
        if (i + 1 < nsteps) {
            tmem_ld_wait();
            if (i + 2 < nsteps) {
                tmem_ld16(t_s + 16 * (i + 2), sa);
                tmem_ld16(t_dp + 16 * (i + 2), pa);
            }
            bwd_cols16<KV, MASKED, RAGGED, 0>(sb, pb, pk_p, pk_ds, c_first + 16 * (i + 1), rc, st_a, scale, dbias_limit, held_addr, held_ds);
            if (KV) tmem_st8(t_s + 8 * (i + 1), pk_p);
            tmem_st8(t_dp + 8 * (i + 1), pk_ds);
        }
    }
}

template <bool KV>
__global__ void __launch_bounds__(kThreads, 1)
swin_bwd_tc_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                   const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o,
                   const float* __restrict__ bias_prep, const float* __restrict__ lse, const float* __restrict__ delta,
                   __nv_bfloat16* __restrict__ out1, __nv_bfloat16* __restrict__ out2, float* __restrict__ dbias,
                   long long n_items, int ctas_per_head) {
    constexpr int CB = 48;                      // columns per block; two blocks (buffers) in flight per tile
    constexpr int kBufCols = 2 * CB;            // one buffer = [S 48 | dP 48]
    constexpr int kColAcc1 = 2 * kBufCols;      // key side: dV at 192; query side: dQ at 192
    constexpr int kColAcc2 = 2 * kBufCols + 32; // key side: dK at 224
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bar0 = smem0 + kOffBars;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };
    auto bar_empty = [&](int s) { return bar0 + 8u * (kStages + s); };
    auto bar_sdp = [&](int t, int b) { return bar0 + 8u * (2 * kStages + 2 * t + b); };      // S and dP of a block are in buffer b
    auto bar_ds = [&](int t, int b) { return bar0 + 8u * (2 * kStages + 4 + 2 * t + b); };   // bf16 P / dS of a block are in buffer b
    auto bar_acc = [&](int t) { return bar0 + 8u * (2 * kStages + 8 + t); };    // the item's accumulators are final
    auto bar_free = [&](int t) { return bar0 + 8u * (2 * kStages + 10 + t); };  // the accumulators have been read back
    unsigned char* tail = smem + kOffBars + 8 * (2 * kStages + 12);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail);
    volatile int* cta_abort = reinterpret_cast<volatile int*>(tail + 8);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.x % g.heads;
    const int cta_in_head = blockIdx.x / g.heads;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full(s), kLoaderThreads);
            mbar_init(bar_empty(s), 2);      // one arrival per MMA issuer
        }
        for (int t = 0; t < 2; ++t) {
            for (int b = 0; b < 2; ++b) {
                mbar_init(bar_sdp(t, b), 1);
                mbar_init(bar_ds(t, b), 128);
            }
            mbar_init(bar_acc(t), 1);
            mbar_init(bar_free(t), 128);
        }
        *cta_abort = 0;
        fence_barrier_init();
    }
    // the head's prepared bias table, and a zeroed bias-gradient table
    for (int i = tid; i < kFwdBiasFloats; i += kThreads)
        reinterpret_cast<float*>(smem + kOffBias)[i] = bias_prep[(size_t)head * kFwdBiasFloats + i];
    if (!KV)
        for (int i = tid; i < 8 * kDBiasFloats; i += kThreads) reinterpret_cast<float*>(smem + kOffDBias)[i] = 0.f;
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int cs = code_stride(g.w);
    const int c0 = (g.w - 1) * (cs + 1);
    const size_t HW = (size_t)g.H * g.W;

    if (warp >= kMmaWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsOther));
    if (warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loaders
        const int lt = tid - kLoaderWarp0 * 32;
        int kuse = 0, pending_s = -1;
        for (long long it = cta_in_head; it < n_items; it += ctas_per_head, ++kuse) {
            const int s = kuse % kStages;
            // if the next stage is not free yet, publish the copies already issued instead of holding them back
            if (pending_s >= 0 && !__all_sync(0xffffffffu, mbar_test_wait(bar_empty(s), ((kuse / kStages) & 1) ^ 1))) {
                cp_async_wait<0>();
                fence_proxy_async();
                mbar_arrive(bar_full(pending_s));
                pending_s = -1;
            }
            if (!__all_sync(0xffffffffu, mbar_wait(bar_empty(s), ((kuse / kStages) & 1) ^ 1, cta_abort))) break;
            const Item x = make_item(g, it);
            unsigned char* st = smem + s * kStageBytes;
            const uint32_t st_a = smem0 + s * kStageBytes;
            const size_t sample_off = (size_t)x.b * HW;
            // slot metadata; the lse / delta gathers stay in flight while the row copies are issued below
            constexpr int kSlotIters = (kMaxSlots + kLoaderThreads - 1) / kLoaderThreads;
            float l2v[kSlotIters], dlv[kSlotIters];
#pragma unroll
            for (int i = 0; i < kSlotIters; ++i) {
                const int slot = lt + i * kLoaderThreads;
                l2v[i] = INFINITY;                       // no token: P = exp2(.. - inf) = 0
                dlv[i] = 0.f;
                if (slot >= kMaxSlots) continue;
                int code = 0, label = 0xff, tok = -1;
                // as a column of the query side a slot without a token points into the table's -inf zone
                int coloff = KV ? 0 : 4 * (2 * c0 + 1);
                if (slot < x.r.n) {
                    tok = slot_token_tc(g, x.r, slot, code, label);
                    const size_t li = (sample_off + (size_t)tok) * g.heads + head;
                    l2v[i] = __ldg(lse + li);
                    dlv[i] = __ldg(delta + li);
                    coloff = KV ? 4 * code : 4 * (c0 - code);
                }
                reinterpret_cast<int*>(st + kOffColOff)[slot] = coloff;
                reinterpret_cast<int*>(st + kOffLab)[slot] = label;
                reinterpret_cast<int*>(st + kOffCode)[slot] = code;
                reinterpret_cast<int*>(st + kOffTok)[slot] = tok;
            }
            const int chunk = lt & 3;
            for (int row = lt >> 2; row < x.npad; row += kLoaderThreads / 4) {
                const __nv_bfloat16 *sq = q, *sk = k, *sv = v, *sg = d_o;
                int bytes = 0;   // rows past the window's end are written as zeros
                if (row < x.r.n) {
                    int code, label;
                    const int tok = slot_token_tc(g, x.r, row, code, label);
                    const size_t off = ((sample_off + (size_t)tok) * g.heads + head) * kD + chunk * 8;
                    sq = q + off; sk = k + off; sv = v + off; sg = d_o + off;
                    bytes = 16;
                }
                const uint32_t so = st_a + tile_off<kD>(row, chunk);
                cp_async16(so + kOffQ, sq, bytes);
                cp_async16(so + kOffK, sk, bytes);
                cp_async16(so + kOffV, sv, bytes);
                cp_async16(so + kOffDO, sg, bytes);
            }
            cp_async_commit();
#pragma unroll
            for (int i = 0; i < kSlotIters; ++i) {
                const int slot = lt + i * kLoaderThreads;
                if (slot < kMaxSlots) {
                    reinterpret_cast<float*>(st + kOffLse)[slot] = l2v[i] * kLog2e;
                    reinterpret_cast<float*>(st + kOffDelta)[slot] = dlv[i];
                }
            }
            if (pending_s >= 0) {
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
        // ------------------------------------------------------------------ MMA issuers (one lane of warp 8 / 9)
        if (lane == 0) {
            const uint32_t idesc_acc = make_idesc_bf16(128, kD, 0, 1);   // A from TMEM, B = 16 rows x 32 (MN-major)
            // row operands (A of the S-type products) and column operands (their B, and B of the accumulations)
            const uint32_t off_r1 = KV ? kOffK : kOffQ, off_r2 = KV ? kOffV : kOffDO;
            const uint32_t off_c1 = KV ? kOffQ : kOffK, off_c2 = KV ? kOffDO : kOffV;
            const uint64_t d_r1 = make_sdesc_sw64(smem0 + off_r1, 512), d_r2 = make_sdesc_sw64(smem0 + off_r2, 512);
            const uint64_t d_c1 = make_sdesc_sw64(smem0 + off_c1, 512), d_c2 = make_sdesc_sw64(smem0 + off_c2, 512);
            bool ok = true;
            // S = R1 C1^T and dP = R2 C2^T for column block cb of tile t
            auto issue_sdp = [&](int s, int t, int cb, int ncols) {
                const uint64_t so = (uint64_t)((s * kStageBytes) >> 4);
                const uint64_t ro = so + (uint64_t)((t * 128 * kRowBytes) >> 4), co = so + (uint64_t)((cb * CB * kRowBytes) >> 4);
                const uint32_t idesc = make_idesc_bf16(128, ncols, 0, 0);
                const uint32_t t_s = tmem_base + t * 256 + (cb & 1) * kBufCols, t_dp = t_s + CB;
                mma_ss(t_s, d_r1 + ro, d_c1 + co, idesc, 0u);
                mma_ss(t_s, d_r1 + ro + 2, d_c1 + co + 2, idesc, 1u);
                mma_ss(t_dp, d_r2 + ro, d_c2 + co, idesc, 0u);
                mma_ss(t_dp, d_r2 + ro + 2, d_c2 + co + 2, idesc, 1u);
                mma_commit(bar_sdp(t, cb & 1));
            };
            // accumulations of column block cb: query side dQ += dS C1; key side dV += P C2, dK += dS C1
            auto issue_acc = [&](int s, int t, int cb, int ncols) {
                const uint64_t co = (uint64_t)((s * kStageBytes + cb * CB * kRowBytes) >> 4);
                const uint32_t t_p = tmem_base + t * 256 + (cb & 1) * kBufCols, t_ds = t_p + CB;
                const uint32_t first = cb == 0 ? 0u : 1u;
                for (int ks = 0; ks < (ncols >> 4); ++ks) {
                    const uint32_t acc = (ks > 0) ? 1u : first;
                    if (KV) {
                        mma_ts(tmem_base + t * 256 + kColAcc1, t_p + ks * 8, d_c2 + co + (uint64_t)(ks * 64), idesc_acc, acc);
                        mma_ts(tmem_base + t * 256 + kColAcc2, t_ds + ks * 8, d_c1 + co + (uint64_t)(ks * 64), idesc_acc, acc);
                    } else {
                        mma_ts(tmem_base + t * 256 + kColAcc1, t_ds + ks * 8, d_c1 + co + (uint64_t)(ks * 64), idesc_acc, acc);
                    }
                }
            };
            const int t = warp - kMmaWarp;      // this issuer's tile
            int kuse = 0, n_ds[2] = {0, 0}, n_free = 0, n_acc_used = 0;
            for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, ++kuse) {
                const int s = kuse % kStages;
                const Item x = make_item(g, it);
                const int ncb = (x.npad + CB - 1) / CB;
                ok = mbar_wait(bar_full(s), (kuse / kStages) & 1, cta_abort);
                if (!ok) break;
                if (t >= x.ntiles) {            // nothing to issue for this tile: just release the stage
                    mma_commit(bar_empty(s));
                    continue;
                }
                fence_proxy_async();
                tc_fence_after();
                // Both buffers are free here: the previous item's elementwise work is over (its ds barriers
                // were waited for) and the accumulation MMAs that read the buffers were issued earlier by this
                // lane, so they execute first.  Run two blocks ahead of the elementwise warpgroup.
                issue_sdp(s, t, 0, min(CB, x.npad));
                if (ncb > 1) issue_sdp(s, t, 1, min(CB, x.npad - CB));
                for (int cb = 0; cb < ncb && ok; ++cb) {
                    const int buf = cb & 1;
                    ok = mbar_wait(bar_ds(t, buf), n_ds[buf] & 1, cta_abort);
                    ++n_ds[buf];
                    if (ok && cb == 0 && n_acc_used > n_free) {
                        // the first accumulation overwrites the accumulators: the previous item's must have been read
                        ok = mbar_wait(bar_free(t), n_free & 1, cta_abort);
                        ++n_free;
                    }
                    if (!ok) break;
                    tc_fence_after();
                    issue_acc(s, t, cb, min(CB, x.npad - cb * CB));
                    if (cb + 2 < ncb) issue_sdp(s, t, cb + 2, min(CB, x.npad - (cb + 2) * CB));
                }
                if (!ok) break;
                mma_commit(bar_acc(t));
                ++n_acc_used;
                mma_commit(bar_empty(s));
            }
        }
    }
    } else {
        // ------------------------------------------------------------------ elementwise warpgroups
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsWork));
        const int wg = warp >> 2;
        const int row = tid & 127;
        const int slot = wg * 128 + row;
        const uint32_t lane_addr = ((uint32_t)(32 * (warp & 3))) << 16;
        const uint32_t t_reg = tmem_base + lane_addr + wg * 256;
        const float scale = g.scale_log2e;
        const float out_scale = g.scale_log2e * kLn2;          // dQ and dK carry the score scale
        const int dbias_limit = 4 * (2 * c0 + 1);
        int kuse = 0, n_sdp[2] = {0, 0}, n_acc = 0;
        for (long long it = cta_in_head; it < n_items; it += ctas_per_head, ++kuse) {
            const Item x = make_item(g, it);
            if (wg >= x.ntiles) continue;
            const int s = kuse % kStages;
            const uint32_t st_a = smem0 + s * kStageBytes;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_full(s), (kuse / kStages) & 1, cta_abort))) break;
            const int code_i = lds_i32(st_a + kOffCode + 4 * slot);
            const int tok = lds_i32(st_a + kOffTok + 4 * slot);
            RowCtx rc;
            rc.label = lds_i32(st_a + kOffLab + 4 * slot);
            rc.valid = tok >= 0;
            rc.lse2 = lds_f32(st_a + kOffLse + 4 * slot);
            rc.delta = lds_f32(st_a + kOffDelta + 4 * slot);
            // bias index = code_query - code_key + c0
            rc.bias_row = smem0 + kOffBias + (KV ? 4 * (c0 - code_i) : 4 * code_i);
            rc.dbias_row = smem0 + kOffDBias + 4 * (warp * kDBiasFloats + code_i);
            const int ncb = (x.npad + CB - 1) / CB;
            bool ok = true;
            for (int cb = 0; cb < ncb; ++cb) {
                const int ncols = min(CB, x.npad - cb * CB);
                const int buf = cb & 1;
                const uint32_t t_buf = t_reg + buf * kBufCols;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_sdp(wg, buf), n_sdp[buf] & 1, cta_abort));
                if (!ok) break;
                ++n_sdp[buf];
                tc_fence_after();
                if (x.masked)
                    bwd_block<KV, true, true>(t_buf, t_buf + CB, cb * CB, ncols, rc, st_a, scale, dbias_limit);
                else if (x.ragged)
                    bwd_block<KV, false, true>(t_buf, t_buf + CB, cb * CB, ncols, rc, st_a, scale, dbias_limit);
                else
                    bwd_block<KV, false, false>(t_buf, t_buf + CB, cb * CB, ncols, rc, st_a, scale, dbias_limit);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_ds(wg, buf));
            }
            if (!ok) break;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_acc(wg), n_acc & 1, cta_abort))) break;
            ++n_acc;
            tc_fence_after();
            uint32_t r1[32], r2[32];
            if (KV) {
                tmem_ld32(t_reg + kColAcc1, r1);      // dV
                tmem_ld32(t_reg + kColAcc2, r2);      // dK
            } else {
                tmem_ld32(t_reg + kColAcc1, r2);      // dQ
            }
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(bar_free(wg));
            if (KV) {
                // Each thread holds one 64-byte row of dV and of dK.  Rows go through a per-warp shared-memory
                // tile (the bias-gradient area is unused on the key side) so that one store instruction
                // writes 8 whole rows (4 lanes x 16 bytes each) instead of 32 scattered 16-byte pieces.
                unsigned char* stg = smem + kOffDBias + warp * 2 * 32 * kRowBytes;
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint4 a, b;
                    a.x = pack_bf16(__uint_as_float(r1[c4 * 8 + 0]), __uint_as_float(r1[c4 * 8 + 1]));
                    a.y = pack_bf16(__uint_as_float(r1[c4 * 8 + 2]), __uint_as_float(r1[c4 * 8 + 3]));
                    a.z = pack_bf16(__uint_as_float(r1[c4 * 8 + 4]), __uint_as_float(r1[c4 * 8 + 5]));
                    a.w = pack_bf16(__uint_as_float(r1[c4 * 8 + 6]), __uint_as_float(r1[c4 * 8 + 7]));
                    b.x = pack_bf16(__uint_as_float(r2[c4 * 8 + 0]) * out_scale, __uint_as_float(r2[c4 * 8 + 1]) * out_scale);
                    b.y = pack_bf16(__uint_as_float(r2[c4 * 8 + 2]) * out_scale, __uint_as_float(r2[c4 * 8 + 3]) * out_scale);
                    b.z = pack_bf16(__uint_as_float(r2[c4 * 8 + 4]) * out_scale, __uint_as_float(r2[c4 * 8 + 5]) * out_scale);
                    b.w = pack_bf16(__uint_as_float(r2[c4 * 8 + 6]) * out_scale, __uint_as_float(r2[c4 * 8 + 7]) * out_scale);
                    *reinterpret_cast<uint4*>(stg + tile_off<kD>(lane, c4)) = a;                       // dV
                    *reinterpret_cast<uint4*>(stg + 32 * kRowBytes + tile_off<kD>(lane, c4)) = b;      // dK
                }
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int rr = 8 * j + (lane >> 2), c4 = lane & 3;
                    const int tok_r = __shfl_sync(0xffffffffu, tok, rr);
                    const uint4 a = *reinterpret_cast<const uint4*>(stg + tile_off<kD>(rr, c4));
                    const uint4 b = *reinterpret_cast<const uint4*>(stg + 32 * kRowBytes + tile_off<kD>(rr, c4));
                    if (tok_r >= 0) {
                        const size_t off = (((size_t)x.b * HW + (size_t)tok_r) * g.heads + head) * kD + c4 * 8;
                        *reinterpret_cast<uint4*>(out2 + off) = a;
                        *reinterpret_cast<uint4*>(out1 + off) = b;
                    }
                }
                __syncwarp();
            }
            if (!KV) {
                unsigned char* stg = smem + kOffOutStage + warp * 32 * kRowBytes;
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint4 b;
                    b.x = pack_bf16(__uint_as_float(r2[c4 * 8 + 0]) * out_scale, __uint_as_float(r2[c4 * 8 + 1]) * out_scale);
                    b.y = pack_bf16(__uint_as_float(r2[c4 * 8 + 2]) * out_scale, __uint_as_float(r2[c4 * 8 + 3]) * out_scale);
                    b.z = pack_bf16(__uint_as_float(r2[c4 * 8 + 4]) * out_scale, __uint_as_float(r2[c4 * 8 + 5]) * out_scale);
                    b.w = pack_bf16(__uint_as_float(r2[c4 * 8 + 6]) * out_scale, __uint_as_float(r2[c4 * 8 + 7]) * out_scale);
                    *reinterpret_cast<uint4*>(stg + tile_off<kD>(lane, c4)) = b;                       // dQ
                }
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int rr = 8 * j + (lane >> 2), c4 = lane & 3;
                    const int tok_r = __shfl_sync(0xffffffffu, tok, rr);
                    const uint4 b = *reinterpret_cast<const uint4*>(stg + tile_off<kD>(rr, c4));
                    if (tok_r >= 0)
                        *reinterpret_cast<uint4*>(out1 + (((size_t)x.b * HW + (size_t)tok_r) * g.heads + head) * kD + c4 * 8) = b;
                }
                __syncwarp();
            }
        }
    }

    // teardown: every role ends up here, also after an expired wait
    cp_async_wait<0>();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
    if (!KV) {
        // this CTA's table = sum of its warps' tables (fixed order), written to the CTA's slot of the workspace
        const float* tbl = reinterpret_cast<const float*>(smem + kOffDBias);
        for (int e = tid; e < kDBiasFloats; e += kThreads) {
            float acc = 0.f;
#pragma unroll
            for (int wq = 0; wq < 8; ++wq) acc += tbl[wq * kDBiasFloats + e];
            dbias[(size_t)blockIdx.x * kDBiasFloats + e] = acc;
        }
    }
    if (tid == 0 && *cta_abort) atomicExch(&g_bwd_tc_timeout, 1);
}

// dbias[(da, db), head] = sum over the head's CTAs of their tables (entry (da + w - 1) * cs + (db + w - 1)).
// Fixed summation order over warps and CTAs: the bias gradient is reproducible run to run.
__global__ void __launch_bounds__(256)
swin_bwd_tc_dbias_finalize_kernel(const float* __restrict__ parts, float* __restrict__ dbias, int w, int heads, int ctas_per_head) {
    const int nw = 2 * w - 1, cs = w + 32;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;       // (table row, head)
    if (i >= nw * nw * heads) return;
    const int head = i % heads, r = i / heads;
    const int e = (r / nw) * cs + (r % nw);
    float acc = 0.f;
    for (int c = 0; c < ctas_per_head; ++c) acc += parts[(size_t)(c * heads + head) * kDBiasFloats + e];
    dbias[i] = acc;
}

}  // namespace

cudaError_t read_bwd_tc_status(int* timed_out) {
    int zero = 0;
    cudaError_t e = cudaMemcpyFromSymbol(timed_out, g_bwd_tc_timeout, sizeof(int));
    if (e != cudaSuccess) return e;
    if (*timed_out) e = cudaMemcpyToSymbol(g_bwd_tc_timeout, &zero, sizeof(int));
    return e;
}

constexpr int kMaxGrid = 160;   // CTAs whose bias-gradient tables fit the workspace

bool bwd_tc_supported(const Geo& g) { return g.d == 32 && g.nmax <= kMaxSlots && g.w <= 16 && g.heads <= 148; }

// workspace: delta [B*H*W*heads] fp32, then the prepared bias tables [heads * kFwdBiasFloats] fp32
size_t bwd_tc_workspace_bytes(const Geo& g) {
    const size_t delta = (((size_t)g.B * g.H * g.W * g.heads * sizeof(float)) + 255) / 256 * 256;
    return delta + (size_t)g.heads * kFwdBiasFloats * sizeof(float) + (size_t)kMaxGrid * kDBiasFloats * sizeof(float);
}

cudaError_t launch_bwd_tc(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                          const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, float* dbias,
                          void* workspace, int sm_count, cudaStream_t stream) {
    float* delta = reinterpret_cast<float*>(workspace);
    const size_t delta_bytes = (((size_t)g.B * g.H * g.W * g.heads * sizeof(float)) + 255) / 256 * 256;
    float* prep = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + delta_bytes);
    cudaError_t e = launch_bwd_delta(g, o, d_o, delta, stream);
    if (e != cudaSuccess) return e;
    e = launch_bias_prep(g, bias, prep, stream);
    if (e != cudaSuccess) return e;
    float* parts = prep + (size_t)g.heads * kFwdBiasFloats;
    e = cudaMemsetAsync(parts, 0, sizeof(float) * (size_t)kMaxGrid * kDBiasFloats, stream);
    if (e != cudaSuccess) return e;
    const long long items = (long long)g.B * g.Mh * g.Mw;
    long long cph = (sm_count < kMaxGrid ? sm_count : kMaxGrid) / g.heads;
    if (cph < 1) cph = 1;
    if (cph > items) cph = items;
    const unsigned grid = (unsigned)(cph * g.heads);
    e = cudaFuncSetAttribute(swin_bwd_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(swin_bwd_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    prof_begin("swin_bwd_tc_kernel<key side>", stream);
    swin_bwd_tc_kernel<true><<<grid, kThreads, kSmemBytes, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, prep, lse, delta,
        (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, nullptr, items, (int)cph);
    count_launch(stream);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    prof_begin("swin_bwd_tc_kernel<query side>", stream);
    swin_bwd_tc_kernel<false><<<grid, kThreads, kSmemBytes, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, prep, lse, delta,
        (__nv_bfloat16*)dq, nullptr, parts, items, (int)cph);
    count_launch(stream);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int nrows = (2 * g.w - 1) * (2 * g.w - 1) * g.heads;
    swin_bwd_tc_dbias_finalize_kernel<<<(nrows + 255) / 256, 256, 0, stream>>>(parts, dbias, g.w, g.heads, (int)cph);
    count_launch(stream);
    return cudaGetLastError();
}

}  // namespace terra
