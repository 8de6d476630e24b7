// Key side of the backward pass (dK, dV) on the tcgen05 tensor cores for head dims 64 and 128 and windows of up to
// 1024 tokens (window side <= 32).  The query side (dQ, dBias) of this regime runs its own tcgen05 kernel on grids of
// complete 32 x 32 windows and the register-tile kernel otherwise.
//
// One persistent CTA per SM, bound to one head, walks over (batch, window, 128-key tile) items.  The tile's K and V
// rows stay in shared memory; the window's queries stream through a ring of slots in chunks of 128 (Q, dO rows and
// per-query lse, delta, bias code, mask label).  Orientation as in the small-window backward kernel: TMEM lanes =
// keys, columns = queries.  Per half chunk of 64 queries:
//   S^T = K Q_c^T, dP^T = V dO_c^T                                   (SS MMAs, N = the half chunk's queries)
//   P^T = exp2(S^T scale + bias - lse_q), dS^T = P^T (dP^T - delta_q)   (elementwise warps, one key row per thread,
//                                                                      written back over S^T / dP^T as bf16)
//   dV += P^T dO_c, dK += dS^T Q_c                                   (A from TMEM, B = the chunk's rows, MN-major)
// P is recomputed from the saved log-sum-exp, so the chunks are independent.
// Roles: warps 0-7 elementwise (warps w and w + 4 share TMEM lane quarter w & 3 and take the chunk's first / second
// 64 query columns), warp 8 issues every MMA, warps 9-11 load rows (bulk copies from warp 9 on grids of complete
// windows, else cp.async gathers from all three).  A row is kept as head dim / 32 parts of 32 columns in the
// 64-byte-swizzled operand layout, as in the forward kernel of this regime.
// Half chunks rotate through TMEM buffers (S^T 64 columns | dP^T 64 columns): three at head dim 64, so that the scores of
// a group's next half chunk are issued while it still works on the current one, two at head dim 128, where the
// accumulators dV and dK (head dim columns each, behind the buffers) take the rest of the 512 columns.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, all roles leave their loops, TMEM is
// released and the host reads the device status word.  Every role follows every ring item by item.
#include "swin_common.cuh"
#include "swin_kernels.h"
#include "tc_common.cuh"
#include "tma_rows.cuh"

#include <cstdlib>
#include <cstring>

// fp16 build of this file (through the _f16 wrapper file): the kernel, its launcher and its status word get names of
// their own; the element-independent helpers are compiled in the bf16 build only
#ifdef TERRA_ELEM_F16
#define g_bwd_kv64_timeout g_bwd_kv64_timeout_f16
#define launch_bwd_kv64 launch_bwd_kv64_f16
#define launch_bwd_kv64_qside launch_bwd_kv64_qside_f16
#define read_bwd_kv64_status read_bwd_kv64_status_f16
#endif

namespace terra {

__device__ int g_bwd_kv64_timeout = 0;   // set when a bounded wait expired in any CTA of the kernel below

namespace {

using namespace tc;

constexpr int kMmaWarp = 8;
constexpr int kLoaderWarp0 = 9;
constexpr int kLoaderThreads = 96;
constexpr int kThreads = 384;
constexpr int kWorkThreads = 256;
constexpr int kRegsLaunch = 168, kRegsWork = 208, kRegsOther = 80;
static_assert(2 * (kRegsWork - kRegsLaunch) <= (kRegsLaunch - kRegsOther), "register hand-over does not balance");

constexpr int kPartBytes = 64;                        // one 32-column part of a row
constexpr int kTile = 128;                            // keys per item, queries per chunk
constexpr int kPart = kTile * kPartBytes;             // 8192: the region of one 32-column part of 128 rows
constexpr int kHalf = 64;                             // queries per half chunk
constexpr int kBiasFloats = 6048;
constexpr int kBufCols = 128;                         // TMEM buffer b: S^T of a half chunk at 128 b, dP^T at 128 b + 64

// Shared-memory plan per head dim D (64 or 128): a row is kept as D / 32 parts of 32 columns, each part a region in
// the 64-byte-swizzled operand layout.  The queries stream through a ring of slots.  Head dim 64: two key stages, three
// slots of a whole chunk (128 rows, 32 KB); head dim 128: one key stage and four slots of a half chunk (64 rows, 32 KB:
// with two 64 KB slots one copy was in flight at a time and the issuing warp waited for rows more than half of the
// time; several smaller copies in flight hide the copy latency better.  At head dim 64 the same split was slower).
template <int D>
struct Lay {
    static constexpr int kParts = D / 32;
    static constexpr int kKvStages = D == 64 ? 2 : 1, kSlots = D == 64 ? 3 : 4;
    static constexpr int kHPS = D == 64 ? 2 : 1;      // half chunks per ring slot
    static constexpr int kSlotQ = kHalf * kHPS;       // query rows per ring slot
    static constexpr int kSPart = kSlotQ * kPartBytes;            // the region of one 32-column part of a slot's rows
    static constexpr int kRows = 2 * kParts * kPart;  // two tensors' rows
    // key stage: K parts | V parts, then per key row: 4 * bias code, label, token
    static constexpr int kOffK = 0, kOffV = kParts * kPart;
    static constexpr int kOffKCode = kRows, kOffKLab = kRows + 512, kOffKTok = kRows + 1024;
    static constexpr int kKvStageBytes = kRows + 2048;
    // query slot: Q parts | dO parts, then per query column: 4 * bias code, label, lse, delta
    static constexpr int kSlotRows = 2 * kParts * kSPart;
    static constexpr int kTab = 4 * kSlotQ;           // bytes of one per-query table
    static constexpr int kOffQ = 0, kOffG = kParts * kSPart;
    static constexpr int kOffQCode = kSlotRows, kOffQLab = kSlotRows + kTab, kOffQLse = kSlotRows + 2 * kTab, kOffQDelta = kSlotRows + 3 * kTab;
    static constexpr int kSlotBytes = kSlotRows + 4 * kTab;
    static constexpr int kOffSlots = kKvStages * kKvStageBytes;
    static constexpr int kOffBias = kOffSlots + kSlots * kSlotBytes;
    static constexpr int kOffBars = ((kOffBias + kBiasFloats * 4 + 1023) / 1024) * 1024;
    static constexpr int kSmemBytes = kOffBars + 1024;
    // Half chunks (64 queries) rotate through kBufs TMEM buffers; with three (head dim 64) the scores of a group's next
    // half chunk are issued while it still works on the current one.  At head dim 128 the accumulators leave room for two.
    static constexpr int kBufs = D == 64 ? 3 : 2;
    static constexpr int kColDV = kBufs * kBufCols, kColDK = kColDV + D;
    static_assert(kKvStageBytes % 1024 == 0 && kSlotBytes % 1024 == 0, "tiles keep the swizzle alignment");
    static_assert(kSlots * 1536 <= kBiasFloats * 4, "the staged table rows of every slot fit the bias table's place");
    static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
    static_assert(kColDK + D <= 512, "tensor memory columns");
};

__device__ __forceinline__ int code_stride(int w) { return w + 32; }

struct Item {
    int b, kt;
    WindowRef r;
    int npad;      // query slots rounded up to 16
    int nch;       // 128-query chunks
    bool has;      // the window has this key tile
    bool masked;
};

__device__ __forceinline__ Item make_item(const Geo& g, const ItemCursor& c) {
    Item x;
    x.kt = c.head;                                    // the cursor's fastest digit counts key tiles here
    x.b = c.b;
    x.r = window_ref_rc(g, c.wr, c.wc);
    x.npad = (x.r.n + 15) & ~15;
    x.nch = (x.npad + kTile - 1) / kTile;
    x.has = x.kt * kTile < x.r.n;
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

// 16 query columns [c, c + 16) of one key row: P = exp2(S scale + bias - lse), dS = P (dP - delta), packed to bf16.
// `bias_row` = shared address of the bias table + the key row's part of the index (the -inf zone if the row has no
// token); a query column without a token has lse = +inf, so its P is 0.
// ROW32: the window is 32 tokens wide, so the group's 16 queries sit in one window row and their bias codes are
// consecutive: `code4` = 4 * code of column c, no per-query code table is read.
// `sl_a` = shared address of the slot's per-query tables (code, label, lse, delta: TAB bytes each); c counts within the slot.
template <bool MASKED, bool ROW32, int TAB>
__device__ __forceinline__ void cols16(const uint32_t (&rs)[16], const uint32_t (&rp)[16], int c, uint32_t bias_row, int klabel,
                                       uint32_t sl_a, float scale, uint32_t (&pk_p)[8], uint32_t (&pk_ds)[8], int code4 = 0) {
    constexpr int kOffQCode = 0, kOffQLab = TAB, kOffQLse = 2 * TAB, kOffQDelta = 3 * TAB;
    // all table loads first (they are issued in program order), then the gathers that depend on them, then the math
    int co[16], ql[16];
    float l2[16], dl[16], bv[16];
    if (!ROW32) {
#pragma unroll
        for (int e4 = 0; e4 < 4; ++e4) {
            const int4 c4 = lds_i4(sl_a + kOffQCode + 4 * (c + e4 * 4));
            co[e4 * 4] = c4.x; co[e4 * 4 + 1] = c4.y; co[e4 * 4 + 2] = c4.z; co[e4 * 4 + 3] = c4.w;
        }
    }
#pragma unroll
    for (int e4 = 0; e4 < 4; ++e4) {
        const float4 a = lds_f4(sl_a + kOffQLse + 4 * (c + e4 * 4));
        const float4 b = lds_f4(sl_a + kOffQDelta + 4 * (c + e4 * 4));
        l2[e4 * 4] = a.x; l2[e4 * 4 + 1] = a.y; l2[e4 * 4 + 2] = a.z; l2[e4 * 4 + 3] = a.w;
        dl[e4 * 4] = b.x; dl[e4 * 4 + 1] = b.y; dl[e4 * 4 + 2] = b.z; dl[e4 * 4 + 3] = b.w;
    }
    if (MASKED) {
#pragma unroll
        for (int e4 = 0; e4 < 4; ++e4) {
            const int4 q4 = lds_i4(sl_a + kOffQLab + 4 * (c + e4 * 4));
            ql[e4 * 4] = q4.x; ql[e4 * 4 + 1] = q4.y; ql[e4 * 4 + 2] = q4.z; ql[e4 * 4 + 3] = q4.w;
        }
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) bv[e] = ROW32 ? lds_f32(bias_row + code4 + 4 * e) : lds_f32(bias_row + co[e]);
    // two-wide fp32 operations: one instruction per pair of columns
    float p[16], ds[16];
#pragma unroll
    for (int e = 0; e < 16; e += 2) {
        float x0, x1, t0, t1;
        fma2(x0, x1, __uint_as_float(rs[e]), __uint_as_float(rs[e + 1]), scale, bv[e], bv[e + 1]);
        fma2(x0, x1, l2[e], l2[e + 1], -kLog2e, x0, x1);
        if (MASKED && ql[e] != klabel) x0 = -INFINITY;
        if (MASKED && ql[e + 1] != klabel) x1 = -INFINITY;
        p[e] = fast_exp2(x0);
        p[e + 1] = fast_exp2(x1);
        sub2(t0, t1, __uint_as_float(rp[e]), __uint_as_float(rp[e + 1]), dl[e], dl[e + 1]);
        mul2(ds[e], ds[e + 1], p[e], p[e + 1], t0, t1);
    }
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) {
        pk_p[e2] = pack_elem(p[2 * e2], p[2 * e2 + 1]);
        pk_ds[e2] = pack_elem(ds[2 * e2], ds[2 * e2 + 1]);
    }
}

// Query-side use of the kernel (rows = queries, columns = keys): 16 key columns [c, c + 16) of one query row.
// `neg_l2` = -lse * log2(e) and `dl` = delta of the row; `bias_a` = shared address of the row's bias entry for column
// c (the following keys' entries follow); the key columns' mask labels are the slot's label table.  dS leaves as
// packed bf16 for the dQ product and in fp32 for the bias gradient.
template <bool MASKED, int TAB>
__device__ __forceinline__ void cols16_qside(const uint32_t (&rs)[16], const uint32_t (&rp)[16], int c, uint32_t bias_a, int rlabel,
                                             uint32_t sl_a, float scale, float neg_l2, float dl, uint32_t (&pk_ds)[8], float (&ds)[16]) {
    constexpr int kOffQLab = TAB;
    int cl[16];
    float bv[16];
    if (MASKED) {
#pragma unroll
        for (int e4 = 0; e4 < 4; ++e4) {
            const int4 q4 = lds_i4(sl_a + kOffQLab + 4 * (c + e4 * 4));
            cl[e4 * 4] = q4.x; cl[e4 * 4 + 1] = q4.y; cl[e4 * 4 + 2] = q4.z; cl[e4 * 4 + 3] = q4.w;
        }
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) bv[e] = lds_f32(bias_a + 4 * e);
#pragma unroll
    for (int e = 0; e < 16; e += 2) {
        float x0, x1, t0, t1;
        fma2(x0, x1, __uint_as_float(rs[e]), __uint_as_float(rs[e + 1]), scale, bv[e], bv[e + 1]);
        add2(x0, x1, x0, x1, neg_l2);
        if (MASKED && cl[e] != rlabel) x0 = -INFINITY;
        if (MASKED && cl[e + 1] != rlabel) x1 = -INFINITY;
        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
        add2(t0, t1, __uint_as_float(rp[e]), __uint_as_float(rp[e + 1]), -dl);
        mul2(ds[e], ds[e + 1], p0, p1, t0, t1);
    }
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) pk_ds[e2] = pack_elem(ds[2 * e2], ds[2 * e2 + 1]);
}

// 32 accumulator columns of one row, scaled, as 64 bytes of bf16
__device__ __forceinline__ void store_scaled32(uint4* dst, const uint32_t (&r)[32], float f) {
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
        uint4 a;
        a.x = pack_elem(__uint_as_float(r[c4 * 8 + 0]) * f, __uint_as_float(r[c4 * 8 + 1]) * f);
        a.y = pack_elem(__uint_as_float(r[c4 * 8 + 2]) * f, __uint_as_float(r[c4 * 8 + 3]) * f);
        a.z = pack_elem(__uint_as_float(r[c4 * 8 + 4]) * f, __uint_as_float(r[c4 * 8 + 5]) * f);
        a.w = pack_elem(__uint_as_float(r[c4 * 8 + 6]) * f, __uint_as_float(r[c4 * 8 + 7]) * f);
        dst[c4] = a;
    }
}

struct KvMaps64 {
    RowMaps3 q, k, v, g;      // g: the output gradient dO
};

// TMA: complete windows of side 16 or 32 and a longitude shift that is a multiple of 8: one loader warp fetches every
// window row with tiled bulk copies (per-query lse and delta by 4-byte cp.async copies tied to the same barrier);
// otherwise three loader warps gather the rows with 16-byte cp.async copies.  (Gathering the dO rows with the two
// idle warps next to the bulk copies, as the forward kernel does with V, was measured and is slightly slower here.)
//
// MODE 0: gathered rows.  MODE 1: bulk-copied rows, window side 16 or 32, the head's whole bias table in shared memory.
// MODE 2: bulk-copied rows, complete windows of side 64 or 128: the table does not fit, and the loader warp stages,
// with every query chunk, the 2 kr - 1 table rows (kr = 128 / w window rows per 128 slots) that the chunk's queries
// need against the item's key tile; in the prepared layout (2 w floats per table row) they are one contiguous block,
// and the 16 queries of a column group read consecutive entries, as in the 32-wide case.
// MODE 3: MODE 2 put to use for the query side (dQ, dBias) of such windows.  The host hands over the tensors with the
// roles exchanged (Q and dO as the "key tile", K and V as the streamed "queries") and the bias table reflected through
// its centre, so that rows are queries and columns keys: S = Q K_c^T, dP = dO V_c^T, dS as above with the row's own
// lse and delta, and the accumulator that is dK in the key-side use is dQ = dS K_c; the other one is not computed.
// dBias: the 32 lanes of a warp are 32 consecutive queries of one window row and a half chunk's 64 columns are 64
// consecutive keys of one window row, so the entries (b_q - b_k) run along the diagonals of the warp's 32 x 64 block.
// The block has 95 diagonals; each is summed in one of three accumulators of one lane: a column's 32 values reach
// their diagonals' lanes with one rotation of the warp (one shuffle per element, no chain between columns), and after
// the half chunk the lanes add their accumulators to the global gradient: 95 float atomics per warp and half chunk.
template <int D, int MODE>
__global__ void __launch_bounds__(kThreads, 1)
swin_bwd_kv64_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                     const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o,
                     const float* __restrict__ bias_prep, const float* __restrict__ lse, const float* __restrict__ delta,
                     __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv, float* __restrict__ dbias, long long n_items,
                     int ctas_per_head, int max_tiles, const __grid_constant__ KvMaps64 maps) {
    using L = Lay<D>;
    constexpr bool TMA = MODE >= 1, ROWS = MODE >= 2, QS = MODE == 3;
    constexpr int kStageBytes = 1536;                 // MODE 2: the staged table rows of one query slot
    constexpr int kHPS = L::kHPS, kSlotQ = L::kSlotQ, kSPart = L::kSPart, kTab = L::kTab;
    constexpr int kParts = L::kParts, kKvStages = L::kKvStages, kSlots = L::kSlots;
    constexpr int kOffK = L::kOffK, kOffV = L::kOffV, kOffKCode = L::kOffKCode, kOffKLab = L::kOffKLab, kOffKTok = L::kOffKTok;
    constexpr int kKvStageBytes = L::kKvStageBytes, kOffQ = L::kOffQ, kOffG = L::kOffG, kOffQCode = L::kOffQCode;
    constexpr int kOffQLab = L::kOffQLab, kOffQLse = L::kOffQLse, kOffQDelta = L::kOffQDelta, kSlotBytes = L::kSlotBytes;
    constexpr int kOffSlots = L::kOffSlots, kOffBias = L::kOffBias, kOffBars = L::kOffBars, kColDV = L::kColDV, kColDK = L::kColDK;
    constexpr int kBufs = L::kBufs;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bar0 = smem0 + kOffBars;
    auto bar_kvfull = [&](int s) { return bar0 + 8u * s; };              // the tile's K, V rows and key tables are there
    auto bar_kvempty = [&](int s) { return bar0 + 8u * (2 + s); };       // ... and no longer needed
    auto bar_qfull = [&](int s) { return bar0 + 8u * (4 + s); };         // a half chunk of queries is in ring slot s
    auto bar_qempty = [&](int s) { return bar0 + 8u * (10 + s); };       // ... and every MMA that reads it is complete
    // A chunk's 64-query halves are separate units of work, numbered through the whole run (only halves that exist
    // count); half number p belongs to elementwise warps 4 h .. 4 h + 3 (h = which half of its chunk) and lives in TMEM
    // buffer p % kBufs, with the buffer's own hand-overs.
    auto bar_sdp = [&](int b) { return bar0 + 8u * (16 + b); };          // S^T and dP^T of a half chunk are in TMEM buffer b
    auto bar_ds = [&](int b) { return bar0 + 8u * (19 + b); };           // bf16 P^T and dS^T of the half chunk are in buffer b
    const uint32_t bar_acc = bar0 + 8u * 22;                              // dV, dK of the item are final
    const uint32_t bar_accfree = bar0 + 8u * 23;                          // ... and have been read
    unsigned char* tail = smem + kOffBars + 8 * 24;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail);
    volatile int* cta_abort = reinterpret_cast<volatile int*>(tail + 8);

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = tid >> 5;
    const int head = blockIdx.x % g.heads;
    const int cta_in_head = blockIdx.x / g.heads;

    if (tid == 0) {
        for (int s = 0; s < kKvStages; ++s) {
            mbar_init(bar_kvfull(s), TMA ? 32 : kLoaderThreads);
            mbar_init(bar_kvempty(s), 1 + kWorkThreads);   // the issuer's commit + every elementwise thread
        }
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(bar_qfull(s), TMA ? 32 : kLoaderThreads);
            mbar_init(bar_qempty(s), 1);
        }
        for (int b = 0; b < kBufs; ++b) {
            mbar_init(bar_sdp(b), 1);
            mbar_init(bar_ds(b), kWorkThreads / 2);
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_accfree, kWorkThreads);
        *cta_abort = 0;
        fence_barrier_init();
    }
    if (!ROWS) {
        for (int i = tid; i < kBiasFloats; i += kThreads)
            reinterpret_cast<float*>(smem + kOffBias)[i] = bias_prep[(size_t)head * kBiasFloats + i];
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

    if (warp >= kMmaWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsOther));
    if (TMA && warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loader warp (TMA); the other two have no work
        if (warp == kLoaderWarp0) {
            const int wrows = max(1, kTile / g.w);            // window rows per 128 slots
            int kuse = 0;
            unsigned ru = 0;                                  // half chunks so far (every role counts them the same way)
            bool ok = true;
            ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_tiles, g.Mw, g.Mh);
            for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_tiles, g.Mw, g.Mh)) {
                const Item x = make_item(g, cur);
                if (!x.has) continue;
                const int ks = kuse % kKvStages;
                ok = mbar_wait_all(bar_kvempty(ks), ((kuse / kKvStages) & 1) ^ 1, cta_abort);
                if (!ok) break;
                const size_t sample_off = (size_t)x.b * HW;
                const int ew = x.r.ew;                        // = w: the windows are complete
                int v0 = x.r.wc * g.w + g.sw;
                if (v0 >= g.W) v0 -= g.W;
                // ---- the key tile
                {
                    unsigned char* st = smem + ks * kKvStageBytes;
                    const int slot0 = x.kt * kTile;
                    for (int row = lane; row < kTile; row += 32) {
                        const int slot = slot0 + row;
                        int code, label;
                        const int a = slot / ew;
                        const int tok = offset_token(g, x.r, a, slot - a * ew, code, label);
                        reinterpret_cast<int*>(st + kOffKCode)[row] = 4 * code;
                        reinterpret_cast<int*>(st + kOffKLab)[row] = label;
                        reinterpret_cast<int*>(st + kOffKTok)[row] = tok;
                    }
                    const uint32_t sb = smem0 + ks * kKvStageBytes;
                    if (!ROWS && g.w == 32) {
                        // one lane per tensor and part: the tile's four window rows, in groups where the copies allow it
                        for (int i = lane; i < 2 * kParts; i += 32) {
                            const int tsr = i >= kParts ? 1 : 0, part = i - tsr * kParts;
                            bulk_copy_window_rows(tsr ? maps.v : maps.k, sb + (tsr ? kOffV : kOffK) + part * kPart, g, x.b, x.r.wr, v0,
                                                  x.kt * wrows, wrows, head * D + part * 32, bar_kvfull(ks));
                        }
                    } else {
                        const int per_tensor = wrows * kParts;
                        for (int i = lane; i < 2 * per_tensor; i += 32) {
                            const int tsr = i >= per_tensor ? 1 : 0, rem = i - tsr * per_tensor;
                            const int ar = rem / kParts, part = rem - ar * kParts;
                            bulk_copy_window_row(tsr ? maps.v : maps.k, sb + (tsr ? kOffV : kOffK) + part * kPart + ar * g.w * kPartBytes, g,
                                                 x.b, x.r.wr, v0, x.kt * wrows + ar, head * D + part * 32, bar_kvfull(ks));
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive_expect_tx(bar_kvfull(ks), (uint32_t)(kTile * D * 2 * 2));
                    else mbar_arrive(bar_kvfull(ks));
                }
                // ---- the window's queries, slot by slot (the windows are complete: every slot is full)
                const int nu = x.npad / kSlotQ;
                const int n_run = min(g.w, kSlotQ), runs = kSlotQ / n_run;        // runs of one window row per slot
                for (int i = 0; i < nu; ++i, ++ru) {
                    const int s = (int)(ru % kSlots);
                    ok = mbar_wait_all(bar_qempty(s), (uint32_t)((ru / kSlots) & 1) ^ 1u, cta_abort);
                    if (!ok) break;
                    unsigned char* sl = smem + kOffSlots + s * kSlotBytes;
                    const uint32_t sb = smem0 + kOffSlots + s * kSlotBytes;
                    const int slot0 = i * kSlotQ;
                    for (int row = lane; row < kSlotQ; row += 32) {
                        const int slot = slot0 + row;
                        int code, label;
                        const int a = slot / ew;
                        const int tok = offset_token(g, x.r, a, slot - a * ew, code, label);
                        const size_t li = (sample_off + (size_t)tok) * g.heads + head;
                        if (!QS) {
                            cp_async4(sb + kOffQLse + 4 * row, lse + li);
                            cp_async4(sb + kOffQDelta + 4 * row, delta + li);
                        }
                        reinterpret_cast<int*>(sl + kOffQCode)[row] = 4 * code;
                        reinterpret_cast<int*>(sl + kOffQLab)[row] = label;
                    }
                    if (!ROWS && g.w == 32) {
                        // whole window rows: one lane per tensor and part, groups of window rows where the copies allow it
                        for (int j = lane; j < 2 * kParts; j += 32) {
                            const int tsr = j >= kParts ? 1 : 0, part = j - tsr * kParts;
                            bulk_copy_window_rows(tsr ? maps.g : maps.q, sb + (tsr ? kOffG : kOffQ) + part * kSPart, g, x.b, x.r.wr, v0,
                                                  slot0 / 32, runs, head * D + part * 32, bar_qfull(s));
                        }
                    } else {
                        for (int j = lane; j < 2 * runs * kParts; j += 32) {
                            const int tsr = j >= runs * kParts ? 1 : 0, rem = j - tsr * runs * kParts;
                            const int rr = rem / kParts, part = rem - rr * kParts;
                            const int rslot = slot0 + rr * n_run, a = rslot / g.w;
                            bulk_copy_window_run(tsr ? maps.g : maps.q, sb + (tsr ? kOffG : kOffQ) + part * kSPart + rr * n_run * kPartBytes, g,
                                                 x.b, x.r.wr, v0, a, rslot - a * g.w, n_run, head * D + part * 32, bar_qfull(s));
                        }
                    }
                    if (ROWS && lane == 0) {
                        // the table rows that this slot's ur window rows need against the key tile's kr window rows
                        const int lw = 31 - __clz(g.w), kr = kTile >> lw, ur = max(1, kSlotQ >> lw);
                        const int r0 = (slot0 >> lw) - x.kt * kr - (kr - 1) + g.w - 1;
                        bulk_load(smem0 + kOffBias + s * kStageBytes,
                                  bias_prep + (size_t)head * ((2 * g.w - 1) * 2 * g.w + 4) + (size_t)r0 * 2 * g.w,
                                  (uint32_t)((ur + kr - 1) * 8 * g.w), bar_qfull(s));
                        mbar_expect_tx(bar_qfull(s), (uint32_t)((ur + kr - 1) * 8 * g.w));
                    }
                    if (lane == 0) mbar_expect_tx(bar_qfull(s), (uint32_t)(kSlotQ * D * 2 * 2));
                    // the lane's arrival: when its lse / delta copies have landed (its table entries were written before)
                    if (QS) mbar_arrive(bar_qfull(s));
                    else cp_async_mbar_arrive_noinc(bar_qfull(s));
                }
                ++kuse;
            }
        }
    } else if (warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loaders
        // D / 32 lanes per row (one 32-column part of the row each, four 16-byte copies).  A thread never waits for
        // data: its arrival on a stage's or slot's barrier is tied to the completion of the copies it has issued.
        const int lt = (warp - kLoaderWarp0) * 32 + lane;
        const int hf = lt % kParts;
        const int lrow = lt / kParts;
        constexpr int kRowsPerIter = kLoaderThreads / kParts;
        int kuse = 0;
        unsigned ru = 0;                                      // half chunks so far
        bool ok = true;
        auto acquire = [&](uint32_t bar, uint32_t parity) -> bool { return mbar_wait_all(bar, parity, cta_abort); };
        // the thread's table entries are visible to the CTA before its arrival, which follows its copies
        auto issued = [&](uint32_t bar) {
            __threadfence_block();
            cp_async_mbar_arrive_noinc(bar);
        };
        ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_tiles, g.Mw, g.Mh);
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_tiles, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur);
            if (!x.has) continue;
            const int ks = kuse % kKvStages;
            ok = acquire(bar_kvempty(ks), ((kuse / kKvStages) & 1) ^ 1);
            if (!ok) break;
            const size_t sample_off = (size_t)x.b * HW;
            const int ew = x.r.ew;
            const int q_r = kRowsPerIter / ew, r_r = kRowsPerIter - q_r * ew;
            // ---- the key tile: K, V rows (rows without a token as zeros) and the key tables
            {
                unsigned char* st = smem + ks * kKvStageBytes;
                const uint32_t sb = smem0 + ks * kKvStageBytes + hf * kPart;
                const int slot0 = x.kt * kTile;
                for (int row = lt; row < kTile; row += kLoaderThreads) {
                    const int slot = slot0 + row;
                    int code = 0, label = 0xff, tok = -1;
                    if (slot < x.r.n) {
                        const int a = slot / ew;
                        tok = offset_token(g, x.r, a, slot - a * ew, code, label);
                    }
                    reinterpret_cast<int*>(st + kOffKCode)[row] = 4 * code;
                    reinterpret_cast<int*>(st + kOffKLab)[row] = label;
                    reinterpret_cast<int*>(st + kOffKTok)[row] = tok;
                }
                int a_r = (slot0 + lrow) / ew, b_r = (slot0 + lrow) - a_r * ew;
                for (int row = lrow; row < kTile; row += kRowsPerIter, a_r += q_r, b_r += r_r) {
                    if (b_r >= ew) { b_r -= ew; ++a_r; }
                    const __nv_bfloat16 *sk = k, *sv = v;
                    int bytes = 0;
                    if (slot0 + row < x.r.n) {
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
                issued(bar_kvfull(ks));
            }
            // ---- the window's queries, slot by slot (the last one may be partly filled)
            const int nu = (x.npad + kSlotQ - 1) / kSlotQ;
            for (int i = 0; i < nu; ++i, ++ru) {
                const int s = (int)(ru % kSlots);
                ok = acquire(bar_qempty(s), (uint32_t)((ru / kSlots) & 1) ^ 1u);
                if (!ok) break;
                unsigned char* sl = smem + kOffSlots + s * kSlotBytes;
                const uint32_t sb = smem0 + kOffSlots + s * kSlotBytes + hf * kSPart;
                const int slot0 = i * kSlotQ;
                const int ncols = min(kSlotQ, x.npad - slot0);
                for (int row = lt; row < kSlotQ; row += kLoaderThreads) {
                    const int slot = slot0 + row;
                    int code = 0, label = 0xff;
                    if (slot < x.r.n) {
                        // lse and delta travel with the rows (no load the loader would have to wait for)
                        const int a = slot / ew;
                        const int tok = offset_token(g, x.r, a, slot - a * ew, code, label);
                        const size_t li = (sample_off + (size_t)tok) * g.heads + head;
                        cp_async4(smem0 + kOffSlots + s * kSlotBytes + kOffQLse + 4 * row, lse + li);
                        cp_async4(smem0 + kOffSlots + s * kSlotBytes + kOffQDelta + 4 * row, delta + li);
                    } else {
                        reinterpret_cast<float*>(sl + kOffQLse)[row] = INFINITY;   // no token: P = exp2(.. - inf) = 0
                        reinterpret_cast<float*>(sl + kOffQDelta)[row] = 0.f;
                    }
                    reinterpret_cast<int*>(sl + kOffQCode)[row] = 4 * code;
                    reinterpret_cast<int*>(sl + kOffQLab)[row] = label;
                }
                const int slot_first = slot0 + lrow;
                int a_r = slot_first / ew, b_r = slot_first - a_r * ew;
                for (int row = lrow; row < ncols; row += kRowsPerIter, a_r += q_r, b_r += r_r) {
                    if (b_r >= ew) { b_r -= ew; ++a_r; }
                    const __nv_bfloat16 *sq = q, *sg = d_o;
                    int bytes = 0;
                    if (slot0 + row < x.r.n) {
                        int code, label;
                        const int tok = offset_token(g, x.r, a_r, b_r, code, label);
                        sq = q + (sample_off + (size_t)tok) * g.ts + head * D + hf * 32;
                        sg = d_o + ((sample_off + (size_t)tok) * g.heads + head) * D + hf * 32;
                        bytes = 16;
                    }
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4) {
                        const uint32_t so = tile_off<32>(row, c4);
                        cp_async16(sb + kOffQ + so, bytes ? sq + c4 * 8 : sq, bytes);
                        cp_async16(sb + kOffG + so, bytes ? sg + c4 * 8 : sg, bytes);
                    }
                }
                issued(bar_qfull(s));
            }
            ++kuse;
        }
    } else {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc_acc = make_idesc_elem(128, D, 0, 1);        // A from TMEM, B = 16 rows x D (MN-major)
        const uint32_t sd_hi = sdesc_hi(make_sdesc_sw64(smem0, 512));    // common high word of the K-major descriptors
        int kuse = 0;
        unsigned p0 = 0;                                  // half chunks before the current item
        unsigned u0 = 0;                                  // ring slots used before the current item; use u is in slot u % kSlots
        bool ok = true;
        ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_tiles, g.Mw, g.Mh);
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_tiles, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur);
            if (!x.has) continue;
            const int ks = kuse % kKvStages;
            ok = mbar_wait_all(bar_kvfull(ks), (kuse / kKvStages) & 1, cta_abort);
            if (!ok) break;
            fence_proxy_async();
            const uint32_t kb = smem0 + ks * kKvStageBytes;
            // queries of half h of chunk c (a multiple of 16; 0: the half does not exist)
            auto half_cols = [&](int c, int h) { return max(0, min(64, x.npad - c * kTile - 64 * h)); };
            auto half_ready = [&](unsigned use) -> bool {
                if (!mbar_wait_all(bar_qfull((int)(use % kSlots)), (uint32_t)((use / kSlots) & 1), cta_abort)) return false;
                fence_proxy_async();
                return true;
            };
            // S^T = K Q^T, dP^T = V dO^T for the queries of the half chunk in ring slot `sb`
            // (descriptor low words = start address in 16-byte units: + 2 per 32-byte K step, + region / 16 per 32-column part)
            const uint32_t k_lo = sdesc_lo(make_sdesc_sw64(kb + kOffK, 512)), v_lo = sdesc_lo(make_sdesc_sw64(kb + kOffV, 512));
            // (`sb` = the address of the half chunk's first row in its slot)
            auto issue_sdp = [&](uint32_t sb, int nc, int buf) {
                const uint32_t idesc = make_idesc_elem(128, nc, 0, 0);
                const uint32_t q_lo = sdesc_lo(make_sdesc_sw64(sb + kOffQ, 512));
                const uint32_t g_lo = sdesc_lo(make_sdesc_sw64(sb + kOffG, 512));
                const uint32_t t_s = tmem_base + kBufCols * buf, t_dp = t_s + 64;
                constexpr uint32_t kNext = kPart >> 4, kNextH = kSPart >> 4;
                tc_fence_after();
                if (elect_one()) {
                    mma_ss_h<false>(t_s, k_lo, q_lo, sd_hi, idesc);
                    mma_ss_h<true>(t_s, k_lo + 2, q_lo + 2, sd_hi, idesc);
#pragma unroll
                    for (int pt = 1; pt < kParts; ++pt) {
                        mma_ss_h<true>(t_s, k_lo + pt * kNext, q_lo + pt * kNextH, sd_hi, idesc);
                        mma_ss_h<true>(t_s, k_lo + pt * kNext + 2, q_lo + pt * kNextH + 2, sd_hi, idesc);
                    }
                    mma_ss_h<false>(t_dp, v_lo, g_lo, sd_hi, idesc);
                    mma_ss_h<true>(t_dp, v_lo + 2, g_lo + 2, sd_hi, idesc);
#pragma unroll
                    for (int pt = 1; pt < kParts; ++pt) {
                        mma_ss_h<true>(t_dp, v_lo + pt * kNext, g_lo + pt * kNextH, sd_hi, idesc);
                        mma_ss_h<true>(t_dp, v_lo + pt * kNext + 2, g_lo + pt * kNextH + 2, sd_hi, idesc);
                    }
                    mma_commit(bar_sdp(buf));
                }
                __syncwarp();
            };
            // the item's half chunks in order: half i is half i % 2 of chunk i / 2 (only the last chunk can lack its second half)
            const int nh = 2 * x.nch - (half_cols(x.nch - 1, 1) > 0 ? 0 : 1);
            int ready_units = 0;                          // ring slots of the item known to be filled
            // the rows of half i are in their ring slot
            auto ensure_half = [&](int i) -> bool {
                while (ready_units <= i / kHPS) {
                    if (!half_ready(u0 + (unsigned)ready_units)) return false;
                    ++ready_units;
                }
                return true;
            };
            // the address of half i's first row in its slot
            auto half_rows = [&](int i) -> uint32_t {
                return smem0 + kOffSlots + (int)((u0 + (unsigned)(i / kHPS)) % kSlots) * kSlotBytes + (i % kHPS) * kHalf * kPartBytes;
            };
            // scores of half i into its buffer
            auto issue_half = [&](int i) { issue_sdp(half_rows(i), half_cols(i >> 1, i & 1), (int)((p0 + i) % kBufs)); };
            for (int i = 0; i < kBufs && i < nh && ok; ++i) {
                ok = ensure_half(i);
                if (ok) issue_half(i);
            }
            for (int i = 0; i < nh && ok; ++i) {
                const int c = i >> 1, h = i & 1;
                const unsigned p = p0 + i;
                const int buf = (int)(p % kBufs);
                const int s = (int)((u0 + (unsigned)(i / kHPS)) % kSlots);
                const uint32_t sb = half_rows(i);
                const int nc = half_cols(c, h);
                ok = mbar_wait_all(bar_ds(buf), (p / kBufs) & 1, cta_abort);
                if (ok && i == 0 && kuse > 0) ok = mbar_wait_all(bar_accfree, (kuse - 1) & 1, cta_abort);
                if (!ok) break;
                tc_fence_after();
                // dV += P^T dO, dK += dS^T Q over the half chunk's query columns
                const uint64_t gd = make_sdesc_sw64_mn(sb + kOffG, kSPart, 512);
                const uint64_t qd = make_sdesc_sw64_mn(sb + kOffQ, kSPart, 512);
                const uint32_t g_lo = sdesc_lo(gd), q_lo = sdesc_lo(qd), d_hi = sdesc_hi(gd);
                const uint32_t t_p = tmem_base + kBufCols * buf, t_ds = t_p + 64;
                const int nks = nc >> 4;
                if (elect_one()) {
                    int j = 0;
                    if (i == 0) {
                        if (!QS) mma_ts_h<false>(tmem_base + kColDV, t_p, g_lo, d_hi, idesc_acc);
                        mma_ts_h<false>(tmem_base + kColDK, t_ds, q_lo, d_hi, idesc_acc);
                        j = 1;
                    }
                    for (; j < nks; ++j) {
                        if (!QS) mma_ts_h<true>(tmem_base + kColDV, t_p + 16 * j, g_lo + 64 * j, d_hi, idesc_acc);
                        mma_ts_h<true>(tmem_base + kColDK, t_ds + 16 * j, q_lo + 64 * j, d_hi, idesc_acc);
                    }
                    // the slot's last readers were issued just above
                    if (kHPS == 1 || h == 1 || half_cols(c, 1) == 0) mma_commit(bar_qempty(s));
                    if (i + 1 == nh) {
                        mma_commit(bar_acc);
                        mma_commit(bar_kvempty(ks));
                    }
                }
                __syncwarp();
                // the buffer is free again (the products that read it were issued just above): the scores of the half
                // chunk kBufs further on follow at once
                // (its rows are waited for only now: where they are late, the current half should not wait for them)
                if (i + kBufs < nh) {
                    ok = ensure_half(i + kBufs);
                    if (ok) issue_half(i + kBufs);
                }
            }
            if (!ok) break;
            p0 += (unsigned)nh;
            u0 += (unsigned)((nh + kHPS - 1) / kHPS);
            ++kuse;
        }
    }
    } else {
        // ------------------------------------------------------------------ elementwise warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsWork));
        const int hcol = warp >> 2;                       // which 64 query columns of a chunk
        const int quarter = warp & 3;
        const int krow = 32 * quarter + lane;             // key row inside the tile
        const uint32_t lane_addr = ((uint32_t)(32 * quarter)) << 16;
        const float scale = g.scale_log2e;
        const float out_scale = g.scale_log2e * kLn2;     // dK carries the score scale
        int kuse = 0;
        unsigned p0 = 0;                                  // half chunks before the current item
        unsigned u0 = 0;                                  // ring slots used before the current item
        bool ok = true;
        ItemCursor cur = cursor_init(cta_in_head, ctas_per_head, max_tiles, g.Mw, g.Mh);
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, cursor_advance(cur, max_tiles, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur);
            if (!x.has) continue;
            const int ks = kuse % kKvStages;
            if (!mbar_wait_all(bar_kvfull(ks), (kuse / kKvStages) & 1, cta_abort)) break;
            const uint32_t st_a = smem0 + ks * kKvStageBytes;
            const int kcode4 = lds_i32(st_a + kOffKCode + 4 * krow);
            const int klabel = lds_i32(st_a + kOffKLab + 4 * krow);
            const int ktok = lds_i32(st_a + kOffKTok + 4 * krow);
            mbar_arrive(bar_kvempty(ks));                 // this thread has what it needs from the key stage
            // MODE 3: the row is a query; its lse and delta
            float neg_l2 = 0.f, row_dl = 0.f;
            if (QS) {
                const size_t li = ((size_t)x.b * HW + (size_t)ktok) * g.heads + head;
                neg_l2 = -lse[li] * kLog2e;
                row_dl = delta[li];
            }
            // bias index = code_query - code_key + c0; a key row without a token reads the table's -inf zone
            uint32_t bias_row = smem0 + kOffBias + (ktok >= 0 ? 4 * c0 - kcode4 : 4 * (2 * c0 + 1));
            const bool row32 = ROWS || x.r.ew == 32;
            const int lw = 31 - __clz(g.w);
            if (ROWS) {
                // relative to a slot's stage: this key's window row within the tile and its column
                const int kslot = x.kt * kTile + krow, kr = kTile >> lw;
                bias_row = smem0 + kOffBias + (kr - 1 - ((kslot >> lw) - ((x.kt * kTile) >> lw))) * 8 * g.w + 4 * (g.w - 1 - (kslot & (g.w - 1)));
            }
            for (int c = 0; c < x.nch && ok; ++c) {
                const int ncols = min(kTile, x.npad - c * kTile);
                if (ncols <= 64 * hcol) continue;          // this group's half of the chunk does not exist
                const unsigned p = p0 + 2 * c + hcol;      // the half chunk's number; its buffer holds S^T at column 0, dP^T at 64
                const int buf = (int)(p % kBufs);
                const int s = (int)((u0 + (unsigned)((2 * c + hcol) / kHPS)) % kSlots);     // ... and its rows and tables are in this ring slot
                const int sc0 = ((2 * c + hcol) % kHPS) * kHalf;                            // its first column within the slot
                const uint32_t sl_a = smem0 + kOffSlots + s * kSlotBytes + kOffQCode + 4 * sc0;      // the half chunk's part of the slot's per-query tables
                ok = mbar_wait_all(bar_sdp(buf), (p / kBufs) & 1, cta_abort);
                if (!ok) break;
                tc_fence_after();
                // (columns count within the half chunk)
                const uint32_t t_s = tmem_base + lane_addr + kBufCols * buf, t_dp = t_s + 64;
                const int col_end = min(ncols - 64 * hcol, 64);
                // 4 * bias code of query column `col` of this half chunk in a 32-wide window: slot = 128 c + 64 hcol + col = 32 a + b
                // (MODE 2: the offset into the slot's staged table rows; the half chunk lies in one window row)
                auto code4_of = [&](int col) {
                    return ROWS ? s * kStageBytes + (((sc0 + col) >> lw) * 2 * g.w + ((64 * hcol + col) & (g.w - 1))) * 4
                                : 4 * ((4 * c + 2 * hcol + (col >> 5)) * cs + (col & 31));
                };
                // groups of 16 columns; the next group's S^T / dP^T travel from TMEM while this one is worked on
                uint32_t rs[16], rp[16], rs2[16], rp2[16], pk_p[8], pk_ds[8];
                if (QS) {
                    // this warp's rows: 32 queries b_q = bq0 + lane of window row a_q; the half chunk's columns: 64 keys
                    // b_k = bk0 + j of window row a_k.  `dst`: the lane's entry of the gradient for the current column.
                    // Diagonal D = lane - j (j = column within the half chunk, -63 <= D <= 31) is kept by lane (D + 63) % 32
                    // in accumulator (D + 63) / 32: column j's values move up by r = 31 - j % 32 lanes (around the warp),
                    // the lanes below r receive values of the next higher accumulator.
                    const int nw = 2 * g.w - 1;
                    const int qslot0 = x.kt * kTile + 32 * quarter, kslot = c * kTile + 64 * hcol;
                    const int da = (qslot0 >> lw) - (kslot >> lw) + g.w - 1, db0 = (qslot0 & (g.w - 1)) - (kslot & (g.w - 1)) + g.w - 1;
                    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f;
                    float ds[16];
                    auto diag16 = [&](int j0, float& lo, float& hi) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const int r = 31 - ((j0 + e) & 31);
                            const float val = __shfl_sync(0xffffffffu, ds[e], (lane - r) & 31);
                            const bool up = lane < r;
                            hi += up ? val : 0.f;
                            lo += up ? 0.f : val;
                        }
                    };
                    tmem_ld16(t_s, rs);
                    tmem_ld16(t_dp, rp);
#pragma unroll
                    for (int gi = 0; gi < 4; ++gi) {
                        const int cc = 16 * gi;
                        tmem_ld_wait();
                        if (x.masked) cols16_qside<true, kTab>(rs, rp, cc, bias_row + code4_of(cc), klabel, sl_a, scale, neg_l2, row_dl, pk_ds, ds);
                        else cols16_qside<false, kTab>(rs, rp, cc, bias_row + code4_of(cc), klabel, sl_a, scale, neg_l2, row_dl, pk_ds, ds);
                        if (gi < 3) {
                            tmem_ld16(t_s + cc + 16, rs);
                            tmem_ld16(t_dp + cc + 16, rp);
                        }
                        tmem_st8(t_dp + cc, pk_ds);
                        if (gi < 2) diag16(16 * gi, acc1, acc2);          // columns 0..31: diagonals -31..31
                        else diag16(16 * gi, acc0, acc1);                 // columns 32..63: diagonals -63..-1
                    }
                    // accumulator a of this lane is diagonal 32 a + lane - 63: entry db0 + that of table row da
                    float* dst = dbias + ((size_t)da * nw + (db0 + lane - 63)) * g.heads + head;
                    atomicAdd(dst, acc0);
                    atomicAdd(dst + 32 * g.heads, acc1);
                    if (lane < 31) atomicAdd(dst + 64 * g.heads, acc2);
                } else {
                if (0 < col_end) {
                    tmem_ld16(t_s, rs);
                    tmem_ld16(t_dp, rp);
                }
                for (int cc = 0; cc < col_end; cc += 32) {
                    tmem_ld_wait();
                    if (cc + 16 < col_end) {
                        tmem_ld16(t_s + cc + 16, rs2);
                        tmem_ld16(t_dp + cc + 16, rp2);
                    }
                    if (ROWS && x.masked) cols16<true, true, kTab>(rs, rp, cc, bias_row, klabel, sl_a, scale, pk_p, pk_ds, code4_of(cc));
                    else if (x.masked) cols16<true, false, kTab>(rs, rp, cc, bias_row, klabel, sl_a, scale, pk_p, pk_ds);
                    else if (row32) cols16<false, true, kTab>(rs, rp, cc, bias_row, klabel, sl_a, scale, pk_p, pk_ds, code4_of(cc));
                    else cols16<false, false, kTab>(rs, rp, cc, bias_row, klabel, sl_a, scale, pk_p, pk_ds);
                    tmem_st8(t_s + cc, pk_p);              // 16 queries -> 8 packed columns at the group's own place
                    tmem_st8(t_dp + cc, pk_ds);
                    if (cc + 16 < col_end) {
                        tmem_ld_wait();
                        if (cc + 32 < col_end) {
                            tmem_ld16(t_s + cc + 32, rs);
                            tmem_ld16(t_dp + cc + 32, rp);
                        }
                        if (ROWS && x.masked) cols16<true, true, kTab>(rs2, rp2, cc + 16, bias_row, klabel, sl_a, scale, pk_p, pk_ds, code4_of(cc + 16));
                        else if (x.masked) cols16<true, false, kTab>(rs2, rp2, cc + 16, bias_row, klabel, sl_a, scale, pk_p, pk_ds);
                        else if (row32) cols16<false, true, kTab>(rs2, rp2, cc + 16, bias_row, klabel, sl_a, scale, pk_p, pk_ds, code4_of(cc + 16));
                        else cols16<false, false, kTab>(rs2, rp2, cc + 16, bias_row, klabel, sl_a, scale, pk_p, pk_ds);
                        tmem_st8(t_s + cc + 16, pk_p);
                        tmem_st8(t_dp + cc + 16, pk_ds);
                    }
                }
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_ds(buf));
            }
            if (!ok) break;
            {
                const int nh = 2 * x.nch - (min(kTile, x.npad - (x.nch - 1) * kTile) > 64 ? 0 : 1);
                p0 += (unsigned)nh;
                u0 += (unsigned)((nh + kHPS - 1) / kHPS);
            }
            // ---- read-out: dV rows by warps 0-3, dK rows by warps 4-7
            if (!mbar_wait_all(bar_acc, kuse & 1, cta_abort)) break;
            tc_fence_after();
            const float f = (QS || hcol != 0) ? out_scale : 1.f;
            __nv_bfloat16* out = (QS || hcol != 0) ? dk : dv;
            uint4* dst = reinterpret_cast<uint4*>(out + ((size_t)x.b * HW + (size_t)(ktok >= 0 ? ktok : 0)) * g.ts + head * D);
            if (QS) {
                // one accumulator (dQ): each group of warps reads half of its columns
#pragma unroll
                for (int hq = 0; hq < D / 64; ++hq) {
                    uint32_t r0[32];
                    const int col = hcol * (D / 2) + 32 * hq;
                    tmem_ld32(tmem_base + lane_addr + kColDK + col, r0);
                    tmem_ld_wait();
                    if (hq == D / 64 - 1) {
                        tc_fence_before();
                        mbar_arrive(bar_accfree);
                    }
                    store_scaled32(dst + col / 8, r0, f);
                }
            } else {
#pragma unroll
            for (int hq = 0; hq < D / 64; ++hq) {
                uint32_t r0[32], r1[32];
                tmem_ld32(tmem_base + lane_addr + (hcol == 0 ? kColDV : kColDK) + 64 * hq, r0);
                tmem_ld32(tmem_base + lane_addr + (hcol == 0 ? kColDV : kColDK) + 64 * hq + 32, r1);
                tmem_ld_wait();
                if (hq == D / 64 - 1) {
                    tc_fence_before();
                    mbar_arrive(bar_accfree);
                }
                if (ktok >= 0) {
                    store_scaled32(dst + 8 * hq, r0, f);
                    store_scaled32(dst + 8 * hq + 4, r1, f);
                }
            }
            }
            ++kuse;
        }
    }

    // teardown: every role ends up here, also after an expired wait
    cp_async_wait<0>();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
    if (tid == 0 && *cta_abort) atomicExch(&g_bwd_kv64_timeout, 1);
}

}  // namespace

cudaError_t read_bwd_kv64_status(int* timed_out) {
    int zero = 0;
    cudaError_t e = cudaMemcpyFromSymbol(timed_out, g_bwd_kv64_timeout, sizeof(int));
    if (e != cudaSuccess) return e;
    if (*timed_out) e = cudaMemcpyToSymbol(g_bwd_kv64_timeout, &zero, sizeof(int));
    return e;
}

namespace {
bool no_tma_env() {
    static const bool off = [] { const char* e_ = std::getenv("TERRA_NO_TMA"); return e_ && e_[0] == '1'; }();
    return off;
}
}  // namespace

#ifndef TERRA_ELEM_F16
// window sides up to 32 on any grid; sides 64 and 128 on grids of complete windows that the bulk-copy loader serves
bool bwd_kv64_supported(const Geo& g) {
    if (!(g.d == 64 || g.d == 128) || g.heads > 148) return false;
    if (g.w <= 32) return g.nmax <= 1024;
    return (g.w == 64 || g.w == 128) && bulk_rows_shape(g);
}
#endif  // !TERRA_ELEM_F16

// `prep` = the prepared bias tables of the head-dim-64 forward kernel (kBiasFloats per head; for window sides 64 and
// 128 its layout of whole table rows), filled by the caller
static cudaError_t launch_kv64(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                               const float* lse, const float* delta, void* dk, void* dv, float* dbias, bool qside, int sm_count,
                               cudaStream_t stream);

cudaError_t launch_bwd_kv64(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                            const float* lse, const float* delta, void* dk, void* dv, int sm_count, cudaStream_t stream) {
    return launch_kv64(g, q, k, v, d_o, prep, lse, delta, dk, dv, nullptr, false, sm_count, stream);
}

// The query side (dQ, dBias) of complete windows of side 64 and 128 with the same kernel: the tensors change roles and
// `prep_reflected` is the bias table reflected through its centre (launch_bias_prep64 with reflect = true); dbias is
// overwritten.
cudaError_t launch_bwd_kv64_qside(const Geo& g, const void* q, const void* k, const void* v, const void* d_o,
                                  const float* prep_reflected, const float* lse, const float* delta, void* dq, float* dbias,
                                  int sm_count, cudaStream_t stream) {
    if (g.w <= 32) return cudaErrorNotSupported;
    cudaError_t e = cudaMemsetAsync(dbias, 0, sizeof(float) * (size_t)(2 * g.w - 1) * (2 * g.w - 1) * g.heads, stream);
    if (e != cudaSuccess) return e;
    return launch_kv64(g, q, k, v, d_o, prep_reflected, lse, delta, dq, nullptr, dbias, true, sm_count, stream);
}

static cudaError_t launch_kv64(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                               const float* lse, const float* delta, void* dk, void* dv, float* dbias, bool qside, int sm_count,
                               cudaStream_t stream) {
    const int max_tiles = (g.nmax + 127) >> 7;
    const long long items = (long long)g.B * g.Mh * g.Mw * max_tiles;
    long long cph = sm_count / g.heads;
    if (cph < 1) cph = 1;
    if (cph > items) cph = items;
    KvMaps64 maps;
    std::memset(&maps, 0, sizeof maps);
    const bool rows = g.w > 32;
    // the kernel's tile rows ("k", "v") and streamed rows ("q", "g"); the query side exchanges the roles
    const bool tma = (!no_tma_env() || rows) && bulk_rows_shape(g) &&
                     (qside ? make_row_maps3(&maps.k, g, q, g.ts) && make_row_maps3(&maps.v, g, d_o, g.heads * g.d) &&
                                  make_row_maps3(&maps.q, g, k, g.ts) && make_row_maps3(&maps.g, g, v, g.ts)
                            : make_row_maps3(&maps.q, g, q, g.ts) && make_row_maps3(&maps.k, g, k, g.ts) &&
                                  make_row_maps3(&maps.v, g, v, g.ts) && make_row_maps3(&maps.g, g, d_o, g.heads * g.d));
    if ((rows || qside) && !tma) return cudaErrorNotSupported;       // windows of side 64 and 128 have no gathering loader
    auto kern = g.d == 64 ? (qside ? swin_bwd_kv64_kernel<64, 3> : rows ? swin_bwd_kv64_kernel<64, 2> : tma ? swin_bwd_kv64_kernel<64, 1> : swin_bwd_kv64_kernel<64, 0>)
                          : (qside ? swin_bwd_kv64_kernel<128, 3> : rows ? swin_bwd_kv64_kernel<128, 2> : tma ? swin_bwd_kv64_kernel<128, 1> : swin_bwd_kv64_kernel<128, 0>);
    const int smem_bytes = g.d == 64 ? Lay<64>::kSmemBytes : Lay<128>::kSmemBytes;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    prof_begin(qside ? "swin_bwd_kv64_kernel<query side>" : "swin_bwd_kv64_kernel", stream);
    kern<<<(unsigned)(cph * g.heads), kThreads, smem_bytes, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, prep, lse, delta,
        (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, dbias, items, (int)cph, max_tiles, maps);
    count_launch(stream);
    return cudaGetLastError();
}

}  // namespace terra
