// Forward shifted-window attention on the tcgen05 tensor cores for head dims 64 and 128 in the large-window regime,
// where a score row no longer fits tensor memory: windows of up to 1024 tokens (window side <= 32) on any grid, and
// complete windows of side 64 and 128 (4096 and 16 384 tokens) whose rows the bulk-copy loader can fetch.
//
// One persistent CTA per SM, bound to one head, walks over (batch, window, pair of 128-row query tiles) items.
// The window's keys are streamed once, in chunks of 128, through a ring of shared-memory slots.  Per chunk:
//   S = Q K_c^T                                                        (SS MMAs into the tile's columns)
//   online softmax: the softmax threads take the chunk's maximum (for complete windows without mask labels the bound
//   max_j(raw) * scale + max(bias); for windows that mix mask labels or hold slots without a token, and for heads
//   whose bias table spreads over more than 64 octaves, the exact maximum over the keys the row may see), raise the
//   row's reference m when the chunk exceeds it by more than 8 octaves (then O and the row sum are scaled down in
//   tensor memory), and write P = exp2(S * scale + bias - m) back over S as bf16;
//   O += P [V_c | 1]                                                   (A from TMEM; at head dim 64, 16 columns of
//   ones behind V make the accumulator's columns 64..79 carry the row sums; at head dim 128 tensor memory has no
//   columns left for them and the softmax threads add the row sums themselves).
// Roles: warps 0-3 / 4-7 softmax warpgroups (one thread per query row of the pair's first / second tile),
// warp 8 issues every tcgen05.mma (whole warp runs the loop, one elected lane issues), warps 9-11 load rows, undoing
// the roll: on grids of complete windows warp 9 fetches Q and K rows with tiled bulk copies, and the V rows come from
// warp 10 by bulk copies of large boxes (window sides 32, 64, 128: four window rows, or one, per copy) or are gathered
// by warps 10-11 with cp.async (window side 16); otherwise all three gather with cp.async.  A row is kept as head dim / 32 parts of 32 columns in
// the 64-byte-swizzled operand layout of the small-window kernels, so that the same descriptors serve.
// TMEM: columns [256 t, 256 t + 256) belong to query tile t of the pair: S chunk (fp32, 128 columns), overwritten
// in place by bf16 P (64 columns); the O accumulator at +128.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, all roles leave their loops, TMEM is
// released and the host reads the device status word.  Every role follows every ring item by item.
#include <cstdlib>
#include <cstring>

#include "swin_common.cuh"
#include "swin_kernels.h"
#include "tc_common.cuh"
#include "tma_rows.cuh"

// fp16 build of this file (through the _f16 wrapper file): the kernel, its launcher and its status word get names of
// their own; the element-independent helpers are compiled in the bf16 build only
#ifdef TERRA_ELEM_F16
#define g_fwd_tc64_timeout g_fwd_tc64_timeout_f16
#define launch_fwd_tc64 launch_fwd_tc64_f16
#define read_fwd_tc64_status read_fwd_tc64_status_f16
#endif

namespace terra {

__device__ int g_fwd_tc64_timeout = 0;   // set when a bounded wait expired in any CTA of the kernel below

namespace {

using namespace tc;

constexpr int kMmaWarp = 8;
constexpr int kLoaderWarp0 = 9;
constexpr int kLoaderThreads = 96;
constexpr int kThreads = 384;
constexpr int kRegsLaunch = 168, kRegsSoftmax = 216, kRegsOther = 72;
static_assert(2 * (kRegsSoftmax - kRegsLaunch) <= (kRegsLaunch - kRegsOther), "register hand-over does not balance");

constexpr int kPartBytes = 64;                        // one 32-column part of a row
constexpr int kQRows = 256, kChunk = 128;
constexpr int kQPart = kQRows * kPartBytes;           // 16384: the region of one 32-column part of the Q rows
constexpr int kKPart = kChunk * kPartBytes;           // 8192:  ... of a key chunk
constexpr int kBiasFloats = 6048;                     // 3 c0 + 3 with c0 = 31 * 65 (window side 32)
constexpr int kColO = 128;

// Shared-memory plan per head dim D (64 or 128): a row is kept as D / 32 parts of 32 columns, each part a region in the
// 64-byte-swizzled operand layout.  Head dim 64: two Q stages, three ring slots of K | V | ones.  Head dim 128: rows
// are twice as long, so one Q stage and two ring slots of K | V, and no ones block: tensor memory has no columns
// left for the row sums next to a 128-column accumulator, the softmax threads add them up themselves.
template <int D>
struct Lay {
    static constexpr int kParts = D / 32;
    static constexpr bool kOnes = D == 64;
    static constexpr int kQStages = D == 64 ? 2 : 1, kSlots = D == 64 ? 3 : 2;
    static constexpr int kQStageBytes = kParts * kQPart;
    static constexpr int kOffK = 0, kOffV = kParts * kKPart, kOffOnes = 2 * kParts * kKPart;
    static constexpr int kSlotBytes = (2 * kParts + (kOnes ? 1 : 0)) * kKPart;
    static constexpr int kOffSlots = kQStages * kQStageBytes;
    static constexpr int kOffKeyMeta = kOffSlots + kSlots * kSlotBytes;            // per chunk number % 4: kc[128], klab[128]
    static constexpr int kOffRowMeta = kOffKeyMeta + 4 * 1024;                     // per Q stage: rowmeta[256], rowtok[256]
    static constexpr int kOffBias = kOffRowMeta + kQStages * 2048;
    static constexpr int kOffBars = ((kOffBias + kBiasFloats * 4 + 1023) / 1024) * 1024;
    static constexpr int kSmemBytes = kOffBars + 1024;
    static constexpr int kNO = kOnes ? D + 16 : D;    // columns of the PV product
    static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
    static_assert(kColO + kNO <= 256, "tensor memory columns of one query tile");
};

__device__ __forceinline__ int code_stride(int w) { return w + 32; }

struct Item {
    int b, pair;
    WindowRef r;
    int npad;      // key slots rounded up to 16
    int nch;       // 128-key chunks
    int ntiles;    // query tiles of this pair that exist (0, 1 or 2)
    bool masked;
};

__device__ __forceinline__ Item make_item(const Geo& g, const ItemCursor& c) {
    Item x;
    x.pair = c.head;                                  // the cursor's fastest digit counts tile pairs here
    x.b = c.b;
    x.r = window_ref_rc(g, c.wr, c.wc);
    x.npad = (x.r.n + 15) & ~15;
    x.nch = (x.npad + kChunk - 1) / kChunk;
    const int tiles = (x.r.n + 127) >> 7;
    x.ntiles = min(2, max(0, tiles - 2 * x.pair));
    const int r0 = x.r.wr * g.w, c0 = x.r.wc * g.w;
    const bool mh = !g.ph && g.sh > 0 && r0 < g.H - g.sh && r0 + x.r.eh > g.H - g.sh;
    const bool mw = !g.pw && g.sw > 0 && c0 < g.W - g.sw && c0 + x.r.ew > g.W - g.sw;
    x.masked = mh || mw;
    return x;
}

__device__ __forceinline__ int offset_token(const Geo& g, const WindowRef& r, int a, int b, int& code, int& label) {
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
__device__ __forceinline__ int lds_i32(uint32_t addr) {
    int v;
    asm volatile("ld.shared.s32 %0, [%1];\n" : "=r"(v) : "r"(addr));
    return v;
}

// P for N consecutive key columns of the chunk starting at local column c: exp2(raw * scale + bias - m), packed
// (SUM: also adds the values, before rounding, onto `sum`)
template <int N, bool MASKED, bool SUM>
__device__ __forceinline__ void softmax_cols(const uint32_t (&r)[N], uint32_t (&pk)[N / 2], int c, uint32_t bias_i,
                                             uint32_t a_kc, uint32_t a_klab, int label_i, float scale, float neg_m,
                                             float (&sum)[2]) {
#pragma unroll
    for (int e4 = 0; e4 < N / 4; ++e4) {
        const int4 kc4 = lds_i4(a_kc + 4 * (c + e4 * 4));
        const int kc[4] = {kc4.x, kc4.y, kc4.z, kc4.w};
        int kl[4] = {0, 0, 0, 0};
        if (MASKED) {
            const int4 kl4 = lds_i4(a_klab + 4 * (c + e4 * 4));
            kl[0] = kl4.x; kl[1] = kl4.y; kl[2] = kl4.z; kl[3] = kl4.w;
        }
        float p[4], bv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) bv[e] = lds_f32(bias_i + kc[e]);
#pragma unroll
        for (int e = 0; e < 4; e += 2) {
            float x0, x1;
            fma2(x0, x1, __uint_as_float(r[e4 * 4 + e]), __uint_as_float(r[e4 * 4 + e + 1]), scale, bv[e], bv[e + 1]);
            add2(x0, x1, x0, x1, neg_m);
            if (MASKED && kl[e] != label_i) x0 = -INFINITY;
            if (MASKED && kl[e + 1] != label_i) x1 = -INFINITY;
            p[e] = fast_exp2(x0);
            p[e + 1] = fast_exp2(x1);
        }
        pk[e4 * 2] = pack_elem(p[0], p[1]);
        pk[e4 * 2 + 1] = pack_elem(p[2], p[3]);
        if (SUM) {
            sum[0] += p[0] + p[2];
            sum[1] += p[1] + p[3];
        }
    }
}

template <int OFF>
__device__ __forceinline__ float lds_f32_at(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];\n" : "=f"(v) : "r"(addr), "n"(OFF));
    return v;
}
// 32 key columns that are one window row of a full-width 32-wide window without mask labels: their bias entries are
// consecutive (descending with the key), so each address is one base plus an immediate offset: no per-key offsets to
// load, no address arithmetic.  `top` = shared address of the entry of the row's first key.
__device__ __forceinline__ void load_bias_row32(float (&bv)[32], uint32_t top) {
    const uint32_t bb = top - 124;
    bv[0] = lds_f32_at<124>(bb);
    bv[1] = lds_f32_at<120>(bb);
    bv[2] = lds_f32_at<116>(bb);
    bv[3] = lds_f32_at<112>(bb);
    bv[4] = lds_f32_at<108>(bb);
    bv[5] = lds_f32_at<104>(bb);
    bv[6] = lds_f32_at<100>(bb);
    bv[7] = lds_f32_at<96>(bb);
    bv[8] = lds_f32_at<92>(bb);
    bv[9] = lds_f32_at<88>(bb);
    bv[10] = lds_f32_at<84>(bb);
    bv[11] = lds_f32_at<80>(bb);
    bv[12] = lds_f32_at<76>(bb);
    bv[13] = lds_f32_at<72>(bb);
    bv[14] = lds_f32_at<68>(bb);
    bv[15] = lds_f32_at<64>(bb);
    bv[16] = lds_f32_at<60>(bb);
    bv[17] = lds_f32_at<56>(bb);
    bv[18] = lds_f32_at<52>(bb);
    bv[19] = lds_f32_at<48>(bb);
    bv[20] = lds_f32_at<44>(bb);
    bv[21] = lds_f32_at<40>(bb);
    bv[22] = lds_f32_at<36>(bb);
    bv[23] = lds_f32_at<32>(bb);
    bv[24] = lds_f32_at<28>(bb);
    bv[25] = lds_f32_at<24>(bb);
    bv[26] = lds_f32_at<20>(bb);
    bv[27] = lds_f32_at<16>(bb);
    bv[28] = lds_f32_at<12>(bb);
    bv[29] = lds_f32_at<8>(bb);
    bv[30] = lds_f32_at<4>(bb);
    bv[31] = lds_f32_at<0>(bb);
}
// MASKED: keys whose mask label (32 ints at shared address `a_klab`) differs from the row's give P = 0
template <bool SUM, bool MASKED = false>
__device__ __forceinline__ void softmax_cols32_row(const uint32_t (&r)[32], uint32_t (&pk)[16], uint32_t top, float scale, float neg_m,
                                                   float (&sum)[2], uint32_t a_klab = 0, int label_i = 0) {
    float bv[32];
    load_bias_row32(bv, top);
#pragma unroll
    for (int e2 = 0; e2 < 16; ++e2) {
        // two-wide fp32 operations: one instruction per pair of columns
        float x0, x1;
        fma2(x0, x1, __uint_as_float(r[2 * e2]), __uint_as_float(r[2 * e2 + 1]), scale, bv[2 * e2], bv[2 * e2 + 1]);
        add2(x0, x1, x0, x1, neg_m);
        if (MASKED) {
            int kl0, kl1;
            asm volatile("ld.shared.v2.s32 {%0,%1}, [%2];\n" : "=r"(kl0), "=r"(kl1) : "r"(a_klab + 8 * e2));
            if (kl0 != label_i) x0 = -INFINITY;
            if (kl1 != label_i) x1 = -INFINITY;
        }
        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
        pk[e2] = pack_elem(p0, p1);
        if (SUM) add2vv(sum[0], sum[1], sum[0], sum[1], p0, p1);
    }
}

// exact maximum of scale * raw + bias over the keys of N columns that the row may see (others, and slots without a
// token, give -inf)
template <int N>
__device__ __forceinline__ float score_max_cols(const uint32_t* r, int c, uint32_t bias_i, uint32_t a_kc, uint32_t a_klab,
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

// the same for 32 key columns whose bias entries are consecutive (see softmax_cols32_row)
__device__ __forceinline__ float score_max_cols32_row(const uint32_t (&r)[32], uint32_t top, uint32_t a_klab, int label_i, float scale,
                                                      float mx) {
    float bv[32];
    load_bias_row32(bv, top);
#pragma unroll
    for (int e4 = 0; e4 < 8; ++e4) {
        const int4 kl4 = lds_i4(a_klab + 16 * e4);
        const int kl[4] = {kl4.x, kl4.y, kl4.z, kl4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float xv = fmaf(__uint_as_float(r[e4 * 4 + e]), scale, bv[e4 * 4 + e]);
            mx = fmaxf(mx, kl[e] == label_i ? xv : -INFINITY);
        }
    }
    return mx;
}

// 32 accumulator columns of one row, scaled by 1 / row sum, as 64 bytes of bf16
__device__ __forceinline__ void store_o32(uint4* dst, const uint32_t (&ro)[32], float inv) {
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

template <int N>
__device__ __forceinline__ void max_cols(const uint32_t (&r)[N], float (&mx)[4]) {
#pragma unroll
    for (int e = 0; e < N; e += 8) {
#pragma unroll
        for (int a = 0; a < 4; ++a)
            mx[a] = fmaxf(mx[a], fmaxf(__uint_as_float(r[e + 2 * a]), __uint_as_float(r[e + 2 * a + 1])));
    }
}

struct FwdMaps64 {
    RowMaps3 q, k, v;
};

// TMA: the grid consists of complete windows of side 16 or 32 and the longitude shift is a multiple of 8: a window row
// is then one run of tokens (two where it wraps around the longitude seam), and one loader warp fetches every row with
// tiled bulk copies; otherwise three loader warps gather the rows with 16-byte cp.async copies.
//
// MODE 0: gathered rows.  MODE 1: bulk-copied Q and K rows, window side 16 or 32, the head's whole bias table in
// shared memory.  MODE 2: bulk-copied rows, window side 64 or 128 (complete windows of 4096 or 16384 tokens): the bias
// table no longer fits, and the bulk-copy warp stages, per chunk and query tile, the table rows the tile's rows need.
// A chunk's 128 keys are kr = 128 / w window rows and a tile's 128 queries qr = kr window rows, so the row offsets
// between them span 2 kr - 1 table rows; in the prepared layout (2 w floats per table row) those are one contiguous
// block, and within a 32-key group the entries a query row needs are consecutive, as in the 32-wide case.
template <int D, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
swin_fwd_tc64_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                     const __nv_bfloat16* __restrict__ v, const float* __restrict__ bias_prep,
                     __nv_bfloat16* __restrict__ o, float* __restrict__ lse, long long n_items, int ctas_per_head,
                     int max_pairs, const __grid_constant__ FwdMaps64 maps) {
    using L = Lay<D>;
    constexpr bool TMA = MODE >= 1, ROWS = MODE == 2;
    constexpr int kStageBytes = 4096, kStageTile = 1536;      // MODE 2: ring of four bias stages, two tiles each
    static_assert(4 * kStageBytes <= (kBiasFloats - 1) * 4, "bias stages lie below the table's last float");
    constexpr int kParts = L::kParts, kQStages = L::kQStages, kSlots = L::kSlots, kQStageBytes = L::kQStageBytes;
    constexpr int kOffK = L::kOffK, kOffV = L::kOffV, kSlotBytes = L::kSlotBytes, kOffSlots = L::kOffSlots;
    constexpr int kOffKeyMeta = L::kOffKeyMeta, kOffRowMeta = L::kOffRowMeta, kOffBias = L::kOffBias, kOffBars = L::kOffBars;
    constexpr int kNO = L::kNO;
    constexpr bool kSum = !L::kOnes;                    // row sums of P are added up by the softmax threads
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bar0 = smem0 + kOffBars;
    auto bar_qfull = [&](int s) { return bar0 + 8u * s; };               // Q rows and row tables of an item are there
    auto bar_qempty = [&](int s) { return bar0 + 8u * (2 + s); };        // ... and no longer needed
    // a ring slot's K rows and V rows are handed over separately: the K rows go back when the chunk's QK products are
    // complete, long before its PV products, so that the K rows of the chunk after next are on their way early
    auto bar_kfull = [&](int s) { return bar0 + 8u * (4 + s); };         // the K rows (and key tables) of a chunk are in slot s
    auto bar_kempty = [&](int s) { return bar0 + 8u * (7 + s); };        // ... and every MMA that reads them is complete
    auto bar_vfull = [&](int s) { return bar0 + 8u * (20 + s); };        // the same for the V rows
    auto bar_vempty = [&](int s) { return bar0 + 8u * (23 + s); };
    auto bar_sready = [&](int t) { return bar0 + 8u * (10 + t); };       // S of a chunk is in tile t's columns
    auto bar_pready = [&](int t) { return bar0 + 8u * (14 + t); };       // pass B: P of the chunk is in TMEM
    auto bar_oready = [&](int t) { return bar0 + 8u * (16 + t); };       // O of the item is final
    auto bar_ofree = [&](int t) { return bar0 + 8u * (18 + t); };        // ... and has been read
    unsigned char* tail = smem + kOffBars + 8 * 26;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail);
    volatile int* cta_abort = reinterpret_cast<volatile int*>(tail + 8);

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = tid >> 5;
    const int head = blockIdx.x % g.heads;
    const int cta_in_head = blockIdx.x / g.heads;

    if (tid == 0) {
        for (int s = 0; s < kQStages; ++s) {
            mbar_init(bar_qfull(s), TMA ? 32 : kLoaderThreads);
            mbar_init(bar_qempty(s), 1 + 256);        // the issuer's commit + every softmax thread
        }
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(bar_kfull(s), TMA ? 32 : kLoaderThreads);       // TMA: the bulk-copy warp's lanes
            // TMA: the 64 threads that gather V rows; MODE 2 and 32-wide windows: the lanes of the warp that bulk-copies them
            mbar_init(bar_vfull(s), (ROWS || (TMA && g.w == 32)) ? 32 : TMA ? 64 : kLoaderThreads);
            mbar_init(bar_kempty(s), 1);
            mbar_init(bar_vempty(s), 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(bar_sready(t), 1);
            mbar_init(bar_pready(t), 128);
            mbar_init(bar_oready(t), 1);
            mbar_init(bar_ofree(t), 128);
        }
        *cta_abort = 0;
        fence_barrier_init();
    }
    // the head's prepared bias table; the ones block of every ring slot (first 16 bf16 of a row = 1)
    const int lw = 31 - __clz(g.w);                         // MODE 2: w = 1 << lw
    const int rows_floats = (2 * g.w - 1) * 2 * g.w + 4;    // MODE 2: floats of one head's prepared table
    if (ROWS) {
        if (tid == 0) reinterpret_cast<float*>(smem + kOffBias)[kBiasFloats - 1] = bias_prep[(size_t)(head + 1) * rows_floats - 1];
    } else {
        for (int i = tid; i < kBiasFloats; i += kThreads)
            reinterpret_cast<float*>(smem + kOffBias)[i] = bias_prep[(size_t)head * kBiasFloats + i];
    }
    if (L::kOnes) {
        for (int i = tid; i < kSlots * kChunk * 4; i += kThreads) {
            const int s = i / (kChunk * 4), rem = i - s * (kChunk * 4), row = rem >> 2, chunk = rem & 3;
            const uint32_t val = chunk < 2 ? kElemOnesPair : 0u;
            *reinterpret_cast<uint4*>(smem + kOffSlots + s * kSlotBytes + L::kOffOnes + tile_off<32>(row, chunk)) = make_uint4(val, val, val, val);
        }
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

    const int cs = code_stride(g.w);
    const int c0 = (g.w - 1) * (cs + 1);
    const size_t HW = (size_t)g.H * g.W;
    // the table's last float: the head's largest entry, or +inf if the table spreads too far for the bound on the row maximum
    const bool wide = reinterpret_cast<const float*>(smem + kOffBias)[kBiasFloats - 1] == INFINITY;
    // windows whose row maxima are taken exactly (every role derives this the same way)
    auto exact_max = [&](const Item& x) { return x.masked || x.npad != x.r.n || wide; };

    if (warp >= kMmaWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsOther));
    if (TMA && warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loader warp (TMA); the other two have no work
        if (warp == kLoaderWarp0) {
            const int wrows = kChunk / g.w;                   // window rows per 128 slots
            int v0 = 0;                                       // first token column of the current window's rows
            int xb = 0, xwr = 0;
            // the copies of window row `a`, part `part` of a row: w consecutive slots from `dst` on
            auto copy_row = [&](const RowMaps3& m3, uint32_t dst, int a, int part, uint32_t bar) {
                bulk_copy_window_row(m3, dst, g, xb, xwr, v0, a, head * D + part * 32, bar);
            };
            int kuse = 0;
            long long ru = 0;
            bool ok = true;
            ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_pairs, g.Mw, g.Mh);
            for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_pairs, g.Mw, g.Mh)) {
                const Item x = make_item(g, cur);
                if (x.ntiles == 0) continue;
                const int qs = kuse % kQStages;
                ok = mbar_wait_all(bar_qempty(qs), ((kuse / kQStages) & 1) ^ 1, cta_abort);
                if (!ok) break;
                xb = x.b;
                xwr = x.r.wr;
                v0 = x.r.wc * g.w + g.sw;
                if (v0 >= g.W) v0 -= g.W;
                const int ew = x.r.ew;                        // = w: the windows are complete
                // ---- Q rows of the pair and the row tables
                {
                    int* rowmeta = reinterpret_cast<int*>(smem + kOffRowMeta + qs * 2048);
                    int* rowtok = rowmeta + 256;
                    const int slot0 = x.pair * kQRows;
                    for (int row = lane; row < kQRows; row += 32) {
                        const int slot = slot0 + row;
                        int code = 0, label = 0xff, tok = -1;
                        if (slot < x.r.n) {
                            const int a = slot / ew;
                            tok = offset_token(g, x.r, a, slot - a * ew, code, label);
                        }
                        rowmeta[row] = code | (label << 16);
                        rowtok[row] = tok;
                    }
                    const uint32_t qb = smem0 + qs * kQStageBytes;
                    const int a0 = slot0 / g.w, combos = x.ntiles * wrows * kParts;
                    for (int i = lane; i < combos; i += 32) {
                        const int ar = i / kParts, part = i - ar * kParts;
                        copy_row(maps.q, qb + part * kQPart + ar * g.w * kPartBytes, a0 + ar, part, bar_qfull(qs));
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive_expect_tx(bar_qfull(qs), (uint32_t)(x.ntiles * 128 * D * 2));
                    else mbar_arrive(bar_qfull(qs));
                }
                // ---- the key chunks (K rows and the key tables)
                {
                    for (int c = 0; c < x.nch; ++c, ++ru) {
                        const int s = (int)(ru % kSlots);
                        ok = mbar_wait_all(bar_kempty(s), (uint32_t)((ru / kSlots) & 1) ^ 1u, cta_abort);
                        if (!ok) break;
                        {
                            int* kcs = reinterpret_cast<int*>(smem + kOffKeyMeta + (int)(ru & 3) * 1024);
                            int* klab = kcs + 128;
                            for (int row = lane; row < kChunk; row += 32) {
                                const int slot = c * kChunk + row;
                                int code = 0, label = 0xff, kc = 4 * (2 * c0 + 1);
                                if (slot < x.r.n) {
                                    const int a = slot / ew;
                                    offset_token(g, x.r, a, slot - a * ew, code, label);
                                    kc = 4 * (c0 - code);
                                }
                                kcs[row] = kc;
                                klab[row] = label;
                            }
                        }
                        if (ROWS && lane < x.ntiles) {
                            // the 2 kr - 1 table rows that tile `lane` of the pair needs against this chunk
                            const int kr = kChunk >> lw;
                            const int r0 = (((x.pair * kQRows + lane * 128) >> lw) - c * kr - (kr - 1)) + g.w - 1;
                            bulk_load(smem0 + kOffBias + (int)(ru & 3) * kStageBytes + lane * kStageTile,
                                      bias_prep + (size_t)head * rows_floats + (size_t)r0 * 2 * g.w, (uint32_t)((2 * kr - 1) * 8 * g.w),
                                      bar_kfull(s));
                        }
                        // K rows (the V rows are gathered by the other two loader warps: the bulk-copy
                        // engine takes a fixed time per 64-byte row, and the two ways of loading run side by side)
                        const uint32_t sb = smem0 + kOffSlots + s * kSlotBytes;
                        for (int i = lane; i < wrows * kParts; i += 32) {
                            const int ar = i / kParts, part = i - ar * kParts;
                            copy_row(maps.k, sb + kOffK + part * kKPart + ar * g.w * kPartBytes, c * wrows + ar, part, bar_kfull(s));
                        }
                        __syncwarp();
                        if (lane == 0)
                            mbar_arrive_expect_tx(bar_kfull(s), (uint32_t)(kChunk * D * 2 + (ROWS ? x.ntiles * (2 * (kChunk >> lw) - 1) * 8 * g.w : 0)));
                        else mbar_arrive(bar_kfull(s));
                    }
                }
                ++kuse;
            }
        } else if (ROWS || g.w == 32) {
            // ---- MODE 2 and 32-wide windows, warp 10: the V rows by bulk copies as well (a window row is one or two boxes of 64 or 128 tokens,
            // which the copy engine moves at several times the rate of 32-token boxes); warp 11 has no work
            if (warp == kLoaderWarp0 + 1) {
                const int wrows = kChunk / g.w;
                long long ru = 0;
                bool ok = true;
                ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_pairs, g.Mw, g.Mh);
                for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_pairs, g.Mw, g.Mh)) {
                    const Item x = make_item(g, cur);
                    if (x.ntiles == 0) continue;
                    int v0 = x.r.wc * g.w + g.sw;
                    if (v0 >= g.W) v0 -= g.W;
                    for (int c = 0; c < x.nch; ++c, ++ru) {
                        const int s = (int)(ru % kSlots);
                        ok = mbar_wait_all(bar_vempty(s), (uint32_t)((ru / kSlots) & 1) ^ 1u, cta_abort);
                        if (!ok) break;
                        const uint32_t sb = smem0 + kOffSlots + s * kSlotBytes;
                        // (one lane per part: the chunk's window rows, in groups of 4 where a 32-wide window allows it)
                        if (lane < kParts)
                            bulk_copy_window_rows(maps.v, sb + kOffV + lane * kKPart, g, x.b, x.r.wr, v0, c * wrows, wrows, head * D + lane * 32,
                                                  bar_vfull(s));
                        __syncwarp();
                        if (lane == 0) mbar_arrive_expect_tx(bar_vfull(s), (uint32_t)(kChunk * D * 2));
                        else mbar_arrive(bar_vfull(s));
                    }
                }
            }
        } else {
            // ---- warps 10, 11: the V rows with 16-byte cp.async copies; a thread's arrival on the chunk's
            // barrier is tied to the completion of its copies, so it never waits for data
            const int vt = (warp - kLoaderWarp0 - 1) * 32 + lane;      // 0 .. 63
            const int part = vt % kParts, row0 = vt / kParts;
            constexpr int kRowStep = 64 / kParts;
            long long ru = 0;
            bool ok = true;
            ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_pairs, g.Mw, g.Mh);
            for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_pairs, g.Mw, g.Mh)) {
                const Item x = make_item(g, cur);
                if (x.ntiles == 0) continue;
                const size_t sample_off = (size_t)x.b * HW;
                const int ew = x.r.ew;
                {
                    for (int c = 0; c < x.nch; ++c, ++ru) {
                        const int s = (int)(ru % kSlots);
                        ok = mbar_wait_all(bar_vempty(s), (uint32_t)((ru / kSlots) & 1) ^ 1u, cta_abort);
                        if (!ok) break;
                        const uint32_t vb = smem0 + kOffSlots + s * kSlotBytes + kOffV + part * kKPart;
                        for (int row = row0; row < kChunk; row += kRowStep) {
                            const int slot = c * kChunk + row, a = slot / ew;
                            int code, label;
                            const int tok = offset_token(g, x.r, a, slot - a * ew, code, label);
                            const __nv_bfloat16* src = v + (sample_off + (size_t)tok) * g.ts + head * D + part * 32;
#pragma unroll
                            for (int c4 = 0; c4 < 4; ++c4) cp_async16(vb + tile_off<32>(row, c4), src + c4 * 8, 16);
                        }
                        cp_async_mbar_arrive_noinc(bar_vfull(s));
                    }
                }
            }
        }
    } else if (warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loaders
        // D / 32 lanes per row: each takes one 32-column part of the row and issues its four 16-byte copies with one
        // address computation.  A thread never waits for data: its arrival on a stage's or slot's barrier is tied to
        // the completion of the copies it has issued, so as many chunks are in flight as the ring has free slots.
        const int lt = (warp - kLoaderWarp0) * 32 + lane;
        const int hf = lt % kParts;                       // which 32-column part of the row this thread copies
        const int lrow = lt / kParts;
        constexpr int kRowsPerIter = kLoaderThreads / kParts;
        int kuse = 0;
        long long ru = 0;                                 // ring uses so far
        bool ok = true;
        auto acquire = [&](uint32_t bar, uint32_t parity) -> bool { return mbar_wait_all(bar, parity, cta_abort); };
        // the thread's table entries are visible to the CTA before its arrival, which follows its copies
        auto issued = [&](uint32_t bar) {
            __threadfence_block();
            cp_async_mbar_arrive_noinc(bar);
        };
        ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_pairs, g.Mw, g.Mh);
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_pairs, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur);
            if (x.ntiles == 0) continue;
            const int qs = kuse % kQStages;
            ok = acquire(bar_qempty(qs), ((kuse / kQStages) & 1) ^ 1);
            if (!ok) break;
            const size_t sample_off = (size_t)x.b * HW;
            const int ew = x.r.ew;
            const int q_r = kRowsPerIter / ew, r_r = kRowsPerIter - q_r * ew;       // window-offset step of 48 slots
            // ---- Q rows of the pair (rows without a token as zeros) and the row tables
            {
                const uint32_t qb = smem0 + qs * kQStageBytes + hf * kQPart;
                int* rowmeta = reinterpret_cast<int*>(smem + kOffRowMeta + qs * 2048);
                int* rowtok = rowmeta + 256;
                const int slot0 = x.pair * kQRows;
                for (int row = lt; row < kQRows; row += kLoaderThreads) {
                    const int slot = slot0 + row;
                    int code = 0, label = 0xff, tok = -1;
                    if (slot < x.r.n) {
                        const int a = slot / ew;
                        tok = offset_token(g, x.r, a, slot - a * ew, code, label);
                    }
                    rowmeta[row] = code | (label << 16);
                    rowtok[row] = tok;
                }
                const int nrows = x.ntiles * 128;
                int a_r = (slot0 + lrow) / ew, b_r = (slot0 + lrow) - a_r * ew;
                for (int row = lrow; row < nrows; row += kRowsPerIter, a_r += q_r, b_r += r_r) {
                    if (b_r >= ew) { b_r -= ew; ++a_r; }
                    const __nv_bfloat16* src = q;
                    int bytes = 0;
                    if (slot0 + row < x.r.n) {
                        int code, label;
                        const int tok = offset_token(g, x.r, a_r, b_r, code, label);
                        src = q + (sample_off + (size_t)tok) * g.ts + head * D + hf * 32;
                        bytes = 16;
                    }
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4) cp_async16(qb + tile_off<32>(row, c4), bytes ? src + c4 * 8 : src, bytes);
                }
                issued(bar_qfull(qs));
            }
            // ---- the key chunks: K and V rows and the key tables
            {
                for (int c = 0; c < x.nch; ++c, ++ru) {
                    const int s = (int)(ru % kSlots);
                    ok = acquire(bar_kempty(s), (uint32_t)((ru / kSlots) & 1) ^ 1u) && acquire(bar_vempty(s), (uint32_t)((ru / kSlots) & 1) ^ 1u);
                    if (!ok) break;
                    const uint32_t sb = smem0 + kOffSlots + s * kSlotBytes + hf * kKPart;
                    const int ncols = min(kChunk, x.npad - c * kChunk);
                    {
                        int* kcs = reinterpret_cast<int*>(smem + kOffKeyMeta + (int)(ru & 3) * 1024);
                        int* klab = kcs + 128;
                        for (int row = lt; row < kChunk; row += kLoaderThreads) {
                            const int slot = c * kChunk + row;
                            int code = 0, label = 0xff, kc = 4 * (2 * c0 + 1);
                            if (slot < x.r.n) {
                                const int a = slot / ew;
                                offset_token(g, x.r, a, slot - a * ew, code, label);
                                kc = 4 * (c0 - code);
                            }
                            kcs[row] = kc;
                            klab[row] = label;
                        }
                    }
                    const int slot_first = c * kChunk + lrow;
                    int a_r = slot_first / ew, b_r = slot_first - a_r * ew;
                    for (int row = lrow; row < ncols; row += kRowsPerIter, a_r += q_r, b_r += r_r) {
                        if (b_r >= ew) { b_r -= ew; ++a_r; }
                        const __nv_bfloat16 *sk = k, *sv = v;
                        int bytes = 0;
                        if (c * kChunk + row < x.r.n) {
                            int code, label;
                            const int tok = offset_token(g, x.r, a_r, b_r, code, label);
                            const size_t off = (sample_off + (size_t)tok) * g.ts + head * D + hf * 32;
                            sk = k + off; sv = v + off;
                            bytes = 16;
                        }
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) {
                            const uint32_t so = tile_off<32>(row, c4);
                            cp_async16(sb + kOffK + so, bytes ? sk + c4 * 8 : sk, bytes);
                            cp_async16(sb + kOffV + so, bytes ? sv + c4 * 8 : sv, bytes);
                        }
                    }
                    issued(bar_kfull(s));
                    cp_async_mbar_arrive_noinc(bar_vfull(s));
                }
            }
            ++kuse;
        }
    } else {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc_pv = make_idesc_elem(128, kNO, 0, 1);
        int kuse = 0;
        long long ru = 0;
        int n_p[2] = {0, 0}, n_items_t[2] = {0, 0};
        bool ok = true;
        ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_pairs, g.Mw, g.Mh);
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_pairs, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur);
            if (x.ntiles == 0) continue;
            const int qs = kuse % kQStages;
            ok = mbar_wait_all(bar_qfull(qs), (kuse / kQStages) & 1, cta_abort);
            if (!ok) break;
            fence_proxy_async();
            tc_fence_after();
            const uint32_t qb = smem0 + qs * kQStageBytes;
            // S = Q_t K_c^T into tile t's columns
            // (descriptor low words = start address in 16-byte units: + 2 per 32-byte K step, + region / 16 per 32-column part)
            const uint32_t sd_hi = sdesc_hi(make_sdesc_sw64(smem0, 512));
            const uint32_t q_lo0 = sdesc_lo(make_sdesc_sw64(qb, 512));
            auto issue_qk = [&](int t, uint32_t sb, int ncols) {
                const uint32_t idesc = make_idesc_elem(128, ncols, 0, 0);
                const uint32_t q_lo = q_lo0 + ((t * 128 * kPartBytes) >> 4), k_lo = sdesc_lo(make_sdesc_sw64(sb, 512));
                const uint32_t t_d = tmem_base + t * 256;
                if (elect_one()) {
                    mma_ss_h<false>(t_d, q_lo, k_lo, sd_hi, idesc);
                    mma_ss_h<true>(t_d, q_lo + 2, k_lo + 2, sd_hi, idesc);
#pragma unroll
                    for (int pt = 1; pt < kParts; ++pt) {
                        mma_ss_h<true>(t_d, q_lo + pt * (kQPart >> 4), k_lo + pt * (kKPart >> 4), sd_hi, idesc);
                        mma_ss_h<true>(t_d, q_lo + pt * (kQPart >> 4) + 2, k_lo + pt * (kKPart >> 4) + 2, sd_hi, idesc);
                    }
                    mma_commit(bar_sready(t));
                }
                __syncwarp();
            };
            // tile t's S columns are free for the next chunk's QK product by the order of the MMAs: the P that replaced S
            // was consumed by its PV product, issued earlier from this thread
            auto k_ready = [&](long long use) -> bool {
                if (!mbar_wait_all(bar_kfull((int)(use % kSlots)), (uint32_t)((use / kSlots) & 1), cta_abort)) return false;
                fence_proxy_async();
                return true;
            };
            auto v_ready = [&](long long use) -> bool {
                if (!mbar_wait_all(bar_vfull((int)(use % kSlots)), (uint32_t)((use / kSlots) & 1), cta_abort)) return false;
                fence_proxy_async();
                return true;
            };
            // after the QK products of the item's last chunk have been issued: the commit frees the Q stage when they
            // are complete, so that the next item's query rows load while this item's last chunk is worked on
            auto last_qk_issued = [&]() {
                if (elect_one()) mma_commit(bar_qempty(qs));
                __syncwarp();
            };
            // ---- per tile, PV of chunk c is followed at once by QK of chunk c + 1, so that a tile's softmax threads wait
            // for one PV and one QK product only, whatever the other tile is doing
            ok = k_ready(ru);
            for (int t = 0; t < x.ntiles && ok; ++t)
                issue_qk(t, smem0 + kOffSlots + (int)(ru % kSlots) * kSlotBytes, min(kChunk, x.npad));
            if (ok) {
                if (elect_one()) mma_commit(bar_kempty((int)(ru % kSlots)));
                __syncwarp();
                if (x.nch == 1) last_qk_issued();
            }
            for (int c = 0; c < x.nch && ok; ++c, ++ru) {
                const int s = (int)(ru % kSlots);
                const uint32_t sb = smem0 + kOffSlots + s * kSlotBytes;
                const int ncols = min(kChunk, x.npad - c * kChunk);
                const bool has_next = c + 1 < x.nch;
                if (has_next) {
                    ok = k_ready(ru + 1);
                    if (!ok) break;
                }
                ok = v_ready(ru);
                if (!ok) break;
                const uint32_t sb_n = smem0 + kOffSlots + (int)((ru + 1) % kSlots) * kSlotBytes;
                const int ncols_n = min(kChunk, x.npad - (c + 1) * kChunk);
                for (int t = 0; t < x.ntiles && ok; ++t) {
                    ok = mbar_wait_all(bar_pready(t), n_p[t] & 1, cta_abort);
                    ++n_p[t];
                    if (ok && c == 0 && n_items_t[t] > 0)      // the accumulator still holds the tile's previous O
                        ok = mbar_wait_all(bar_ofree(t), (n_items_t[t] - 1) & 1, cta_abort);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t vd = make_sdesc_sw64_mn(sb + kOffV, kKPart, 512);
                    const uint32_t v_lo = sdesc_lo(vd), d_hi = sdesc_hi(vd);
                    const uint32_t t_o = tmem_base + t * 256 + kColO, t_p = tmem_base + t * 256;
                    const int nks = ncols >> 4;
                    if (elect_one()) {
                        int ks = 0;
                        if (c == 0) {
                            mma_ts_h<false>(t_o, t_p, v_lo, d_hi, idesc_pv);
                            ks = 1;
                        }
                        for (; ks < nks; ++ks) mma_ts_h<true>(t_o, t_p + 8 * ks, v_lo + 64 * ks, d_hi, idesc_pv);
                        if (!has_next) mma_commit(bar_oready(t));
                    }
                    __syncwarp();
                    if (!has_next) ++n_items_t[t];
                    else issue_qk(t, sb_n, ncols_n);
                }
                if (!ok) break;
                if (elect_one()) {
                    mma_commit(bar_vempty(s));
                    if (has_next) mma_commit(bar_kempty((int)((ru + 1) % kSlots)));
                }
                __syncwarp();
                if (has_next && c + 2 == x.nch) last_qk_issued();
            }
            if (!ok) break;
            ++kuse;
        }
    }
    } else {
        // ------------------------------------------------------------------ softmax warpgroups
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsSoftmax));
        const int wg = warp >> 2;
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = ((uint32_t)(32 * (warp & 3))) << 16;
        const uint32_t t_s = tmem_base + lane_addr + wg * 256;
        const float scale = g.scale_log2e;
        int kuse = 0, n_s = 0, n_o = 0;
        long long ru = 0;
        ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_pairs, g.Mw, g.Mh);
        for (long long it = cta_in_head; it < n_items; it += ctas_per_head, cursor_advance(cur, max_pairs, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur);
            if (x.ntiles == 0) continue;
            const int qs = kuse % kQStages;
            if (!mbar_wait_all(bar_qfull(qs), (kuse / kQStages) & 1, cta_abort)) break;
            const int rmeta = lds_i32(smem0 + kOffRowMeta + qs * 2048 + 4 * (wg * 128 + row));
            const int tok = lds_i32(smem0 + kOffRowMeta + qs * 2048 + 1024 + 4 * (wg * 128 + row));
            mbar_arrive(bar_qempty(qs));                  // this thread has what it needs from the stage
            ++kuse;
            const long long ru0 = ru;
            ru += x.nch;
            if (wg >= x.ntiles) continue;                 // the pair's second tile does not exist in this window
            const uint32_t bias_i = smem0 + kOffBias + 4 * meta_code(rmeta);
            const int label_i = meta_label(rmeta);
            const float bmax = lds_f32(smem0 + kOffBias + 4 * (kBiasFloats - 1));
            const bool row32 = g.w == 32 && x.r.ew == 32 && !x.masked;       // then every key slot holds a token, too
            const bool exact = exact_max(x);
            bool ok = true;
            // MODE 2: this row's window row within its tile, and the byte offset of its entry for key column 0 of a table row
            const int slot_q = x.pair * kQRows + wg * 128 + row;
            const int aq_l = (slot_q >> lw) - ((x.pair * kQRows + wg * 128) >> lw), kr = kChunk >> lw;
            const int colq = 4 * ((slot_q & (g.w - 1)) + g.w - 1);
            // shared address of the entry of this row for the first key of 32-column group i, in a stage at `stage`
            auto row_top = [&](uint32_t stage, int i) -> uint32_t {
                return stage + wg * kStageTile + (aq_l - ((32 * i) >> lw) + kr - 1) * 8 * g.w + colq - 4 * ((32 * i) & (g.w - 1));
            };
            // Online softmax, chunk by chunk: P is formed against a reference m that is at least the row's maximum so
            // far minus 8 octaves; only when a chunk's maximum exceeds the reference by more than that is the reference
            // raised and the accumulated O (with the row sum) scaled down by 2^(old - new).  Without mask labels the
            // chunk maximum is the bound max_j(raw) * scale + max(bias); for windows that mix mask labels or hold slots
            // without a token, and for heads whose bias table spreads over more than 64 octaves, it is the exact
            // maximum over the keys the row may see.  A row that has seen no key yet forms its P against 0: exactly 0.
            float m = -INFINITY;
            float psum[2] = {0.f, 0.f};
            for (int c = 0; c < x.nch; ++c) {
                const int ncols = min(kChunk, x.npad - c * kChunk);
                const uint32_t a_kc = smem0 + kOffKeyMeta + (int)((ru0 + c) & 3) * 1024, a_klab = a_kc + 512;
                const uint32_t stage = smem0 + kOffBias + (int)((ru0 + c) & 3) * kStageBytes;
                ok = mbar_wait_all(bar_sready(wg), n_s & 1, cta_abort);
                if (!ok) break;
                ++n_s;
                tc_fence_after();
                uint32_t ra[32], rb[32];
                // ---- the chunk's maximum
                float mc;
                {
                    int cc = 0;
                    if (exact) {
                        float mxe = -INFINITY;
                        for (; cc + 32 <= ncols; cc += 32) {
                            tmem_ld32(t_s + cc, ra);
                            tmem_ld_wait();
                            if (ROWS) mxe = score_max_cols32_row(ra, row_top(stage, cc >> 5), a_klab + 4 * cc, label_i, scale, mxe);
                            else mxe = score_max_cols<32>(ra, cc, bias_i, a_kc, a_klab, label_i, scale, mxe);
                        }
                        if (cc < ncols) {
                            uint32_t rt[16];
                            tmem_ld16(t_s + cc, rt);
                            tmem_ld_wait();
                            mxe = score_max_cols<16>(rt, cc, bias_i, a_kc, a_klab, label_i, scale, mxe);
                        }
                        mc = mxe;
                    } else {
                        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                        for (; cc + 64 <= ncols; cc += 64) {
                            tmem_ld32(t_s + cc, ra);
                            tmem_ld32(t_s + cc + 32, rb);
                            tmem_ld_wait();
                            max_cols<32>(ra, mx4);
                            max_cols<32>(rb, mx4);
                        }
                        if (cc + 32 <= ncols) {
                            tmem_ld32(t_s + cc, ra);
                            tmem_ld_wait();
                            max_cols<32>(ra, mx4);
                            cc += 32;
                        }
                        if (cc < ncols) {
                            uint32_t rt[16];
                            tmem_ld16(t_s + cc, rt);
                            tmem_ld_wait();
                            max_cols<16>(rt, mx4);
                        }
                        mc = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale + bmax;
                    }
                }
                // ---- raise the reference if the chunk exceeds it by more than 8 octaves (always from -inf)
                const bool raise = mc > m + 8.f || (m == -INFINITY && mc > -INFINITY);
                const bool rescale = raise && m > -INFINITY;          // O holds contributions formed against the old reference
                if (c > 0 && __any_sync(0xffffffffu, rescale)) {
                    // the PV products issued so far are complete (this chunk's S was committed after them) and the next
                    // one waits for this thread's arrival below: O is this thread's to modify
                    const float f = rescale ? fast_exp2(m - mc) : 1.f;
#pragma unroll 1
                    for (int oc = 0; oc < kNO; oc += 16) {
                        uint32_t ro[16];
                        tmem_ld16(t_s + kColO + oc, ro);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 16; ++e) ro[e] = __float_as_uint(__uint_as_float(ro[e]) * f);
                        tmem_st16(t_s + kColO + oc, ro);
                    }
                    psum[0] *= f;
                    psum[1] *= f;
                }
                if (raise) m = mc;
                const float neg_m = m == -INFINITY ? 0.f : -m;
                // ---- P
                const int nfull = ncols >> 5;
                if (nfull > 0) tmem_ld32(t_s, ra);
                // full-width 32-wide window without mask labels: 32-column group i of chunk c is key row 4 c + i
                const uint32_t top_c = bias_i + 4 * (c0 - 4 * c * cs);
                for (int i = 0; i < nfull; i += 2) {
                    uint32_t pk[16];
                    tmem_ld_wait();
                    if (i + 1 < nfull) tmem_ld32(t_s + 32 * (i + 1), rb);
                    if (ROWS) {
                        if (x.masked) softmax_cols32_row<kSum, true>(ra, pk, row_top(stage, i), scale, neg_m, psum, a_klab + 128 * i, label_i);
                        else softmax_cols32_row<kSum>(ra, pk, row_top(stage, i), scale, neg_m, psum);
                    } else if (row32) softmax_cols32_row<kSum>(ra, pk, top_c - 4 * i * cs, scale, neg_m, psum);
                    else if (x.masked) softmax_cols<32, true, kSum>(ra, pk, 32 * i, bias_i, a_kc, a_klab, label_i, scale, neg_m, psum);
                    else softmax_cols<32, false, kSum>(ra, pk, 32 * i, bias_i, a_kc, a_klab, label_i, scale, neg_m, psum);
                    tmem_st16(t_s + 16 * i, pk);
                    if (i + 1 < nfull) {
                        tmem_ld_wait();
                        if (i + 2 < nfull) tmem_ld32(t_s + 32 * (i + 2), ra);
                        if (ROWS) {
                            if (x.masked) softmax_cols32_row<kSum, true>(rb, pk, row_top(stage, i + 1), scale, neg_m, psum, a_klab + 128 * (i + 1), label_i);
                            else softmax_cols32_row<kSum>(rb, pk, row_top(stage, i + 1), scale, neg_m, psum);
                        } else if (row32) softmax_cols32_row<kSum>(rb, pk, top_c - 4 * (i + 1) * cs, scale, neg_m, psum);
                        else if (x.masked) softmax_cols<32, true, kSum>(rb, pk, 32 * (i + 1), bias_i, a_kc, a_klab, label_i, scale, neg_m, psum);
                        else softmax_cols<32, false, kSum>(rb, pk, 32 * (i + 1), bias_i, a_kc, a_klab, label_i, scale, neg_m, psum);
                        tmem_st16(t_s + 16 * (i + 1), pk);
                    }
                }
                if (ncols & 16) {
                    uint32_t rt[16], pk[8];
                    tmem_ld16(t_s + 32 * nfull, rt);
                    tmem_ld_wait();
                    if (x.masked) softmax_cols<16, true, kSum>(rt, pk, 32 * nfull, bias_i, a_kc, a_klab, label_i, scale, neg_m, psum);
                    else softmax_cols<16, false, kSum>(rt, pk, 32 * nfull, bias_i, a_kc, a_klab, label_i, scale, neg_m, psum);
                    tmem_st8(t_s + 16 * nfull, pk);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_pready(wg));
            }
            if (!ok) break;
            // ---- O and the row sum
            if (!mbar_wait_all(bar_oready(wg), n_o & 1, cta_abort)) break;
            ++n_o;
            tc_fence_after();
            if (!kSum) {
                uint32_t ro[32], ro2[32], rsum;
                tmem_ld32(t_s + kColO, ro);
                tmem_ld32(t_s + kColO + 32, ro2);
                tmem_ld1(t_s + kColO + D, rsum);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(bar_ofree(wg));
                if (tok >= 0) {
                    const float sum = __uint_as_float(rsum);
                    const size_t row_off = ((size_t)x.b * HW + (size_t)tok) * g.heads + head;
                    lse[row_off] = (m + log2f(sum)) * kLn2;
                    const float inv = 1.f / sum;
                    uint4* dst = reinterpret_cast<uint4*>(o + row_off * D);
                    store_o32(dst, ro, inv);
                    store_o32(dst + 4, ro2, inv);
                }
            } else {
                // the accumulator's 128 columns in two rounds of 64, to keep the registers in hand
                const float sum = psum[0] + psum[1];
                const float inv = 1.f / sum;
                const size_t row_off = ((size_t)x.b * HW + (size_t)(tok >= 0 ? tok : 0)) * g.heads + head;
                uint4* dst = reinterpret_cast<uint4*>(o + row_off * D);
                if (tok >= 0) lse[row_off] = (m + log2f(sum)) * kLn2;
#pragma unroll
                for (int hq = 0; hq < D / 64; ++hq) {
                    uint32_t ro[32], ro2[32];
                    tmem_ld32(t_s + kColO + 64 * hq, ro);
                    tmem_ld32(t_s + kColO + 64 * hq + 32, ro2);
                    tmem_ld_wait();
                    if (hq == D / 64 - 1) {
                        tc_fence_before();
                        mbar_arrive(bar_ofree(wg));
                    }
                    if (tok >= 0) {
                        store_o32(dst + 8 * hq, ro, inv);
                        store_o32(dst + 8 * hq + 4, ro2, inv);
                    }
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
    if (tid == 0 && *cta_abort) atomicExch(&g_fwd_tc64_timeout, 1);
}

// The prepared bias table of the small-window kernel, sized for window sides up to 32: per head
//   table[(da + w - 1) * cs + (db + w - 1)] = T[(da + w - 1) * (2w - 1) + (db + w - 1), head] * log2(e)   (cs = w + 32),
//   table[2 c0 + 1 .. 3 c0 + 1] = -inf (where key slots without a token point), the head's largest entry in the last float
//   (+inf instead if the head's entries spread over more than 64 octaves).
// Window sides 64 and 128 (`rows`): per head (2w - 1) table rows of 2w floats (the last one padding) and four more
// floats, the last of which is the head's largest entry as above; `rows` = 2: the table reflected through its centre
// (entry (r, c) holds T[2w - 2 - r][2w - 2 - c]), for the query-side use of the key-major backward kernel.
__global__ void __launch_bounds__(256)
swin_fwd_bias_prep64_kernel(const float* __restrict__ bias, float* __restrict__ prep, int w, int heads, int rows) {
    const int head = blockIdx.x;
    const int cs = rows ? 2 * w : w + 32, nw = 2 * w - 1;
    const int c0 = (w - 1) * (cs + 1);
    const int total = rows ? nw * cs + 4 : kBiasFloats;
    float* dst = prep + (size_t)head * total;
    float mx = -INFINITY, mn = INFINITY;
    for (int e = threadIdx.x; e < total - 1; e += blockDim.x) {
        float val = 0.f;
        if (!rows && e > 2 * c0) {
            val = -INFINITY;
        } else {
            const int ra = e / cs, rb = e - ra * cs;
            if (rb < nw && ra < nw) {
                const int sa = rows == 2 ? nw - 1 - ra : ra, sb = rows == 2 ? nw - 1 - rb : rb;
                val = bias[(size_t)(sa * nw + sb) * heads + head] * kLog2e;
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
        // a table that spreads over more than 64 octaves makes the bound max(raw) * scale + max(bias) on the row
        // maximum too loose for the exponent range: +inf here tells the forward kernel to take exact row maxima
        dst[total - 1] = (mx - mn <= 64.f) ? mx : INFINITY;
    }
}

}  // namespace

cudaError_t read_fwd_tc64_status(int* timed_out) {
    int zero = 0;
    cudaError_t e = cudaMemcpyFromSymbol(timed_out, g_fwd_tc64_timeout, sizeof(int));
    if (e != cudaSuccess) return e;
    if (*timed_out) e = cudaMemcpyToSymbol(g_fwd_tc64_timeout, &zero, sizeof(int));
    return e;
}

#ifndef TERRA_ELEM_F16
// prepared bias tables for the kernels of the large-window regime: kBiasFloats = 6048 floats per head for window
// sides up to 32, whole table rows for sides 64 and 128 (see the kernel above)
cudaError_t launch_bias_prep64(const Geo& g, const float* bias, float* prep, cudaStream_t stream, bool reflect) {
    if (reflect && g.w <= 32) return cudaErrorNotSupported;
    swin_fwd_bias_prep64_kernel<<<g.heads, 256, 0, stream>>>(bias, prep, g.w, g.heads, g.w > 32 ? (reflect ? 2 : 1) : 0);
    count_launch(stream);
    return cudaGetLastError();
}

// window sides up to 32 on any grid; sides 64 and 128 on grids of complete windows that the bulk-copy loaders serve
bool fwd_tc64_supported(const Geo& g) {
    if (!(g.d == 64 || g.d == 128) || g.heads > 148) return false;
    if (g.w <= 32) return g.nmax <= 1024;
    return (g.w == 64 || g.w == 128) && bulk_rows_shape(g);
}

size_t fwd_tc64_workspace_bytes(const Geo& g) {
    const size_t per_head = g.w <= 32 ? (size_t)kBiasFloats : (size_t)(2 * g.w - 1) * 2 * g.w + 4;
    return (size_t)g.heads * per_head * sizeof(float);
}
#endif  // !TERRA_ELEM_F16

cudaError_t launch_fwd_tc64(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                            void* o, float* lse, void* workspace, int sm_count, cudaStream_t stream) {
    float* prep = reinterpret_cast<float*>(workspace);
    const bool rows = g.w > 32;
    swin_fwd_bias_prep64_kernel<<<g.heads, 256, 0, stream>>>(bias, prep, g.w, g.heads, rows ? 1 : 0);
    count_launch(stream);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int max_pairs = (((g.nmax + 127) >> 7) + 1) / 2;
    const long long items = (long long)g.B * g.Mh * g.Mw * max_pairs;
    long long cph = sm_count / g.heads;
    if (cph < 1) cph = 1;
    if (cph > items) cph = items;
    const unsigned grid = (unsigned)(cph * g.heads);
    FwdMaps64 maps;
    std::memset(&maps, 0, sizeof maps);
    static const bool tma_off = [] { const char* e_ = std::getenv("TERRA_NO_TMA"); return e_ && e_[0] == '1'; }();
    const bool tma = (!tma_off || rows) && bulk_rows_shape(g) && make_row_maps3(&maps.q, g, q, g.ts) && make_row_maps3(&maps.k, g, k, g.ts) &&
                     make_row_maps3(&maps.v, g, v, g.ts);
    if (rows && !tma) return cudaErrorNotSupported;       // windows of side 64 and 128 have no gathering loader
    auto kern = g.d == 64 ? (rows ? swin_fwd_tc64_kernel<64, 2> : tma ? swin_fwd_tc64_kernel<64, 1> : swin_fwd_tc64_kernel<64, 0>)
                          : (rows ? swin_fwd_tc64_kernel<128, 2> : tma ? swin_fwd_tc64_kernel<128, 1> : swin_fwd_tc64_kernel<128, 0>);
    const int smem_bytes = g.d == 64 ? Lay<64>::kSmemBytes : Lay<128>::kSmemBytes;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    prof_begin("swin_fwd_tc64_kernel", stream);
    kern<<<grid, kThreads, smem_bytes, stream>>>(g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, prep,
                                                 (__nv_bfloat16*)o, lse, items, (int)cph, max_pairs, maps);
    count_launch(stream);
    return cudaGetLastError();
}

}  // namespace terra
