// Query side of the backward pass (dQ, dBias) on the tcgen05 tensor cores for head dims 64 and 128 and complete
// 32 x 32 windows (window side 32, grid extents multiples of 32).  Other shapes of this regime run the register-tile kernel.
//
// One persistent CTA per SM, bound to one head, walks over a contiguous range of (128-query tile, batch, window)
// items, the tile index slowest.  The tile's Q and dO rows stay in shared memory; the window's keys stream through
// two rings of units of 64 rows, one for K and one for V (with per-key mask labels next to the K units).
// TMEM lanes = queries, columns = keys.  Per half chunk of 64 keys:
//   S = Q K_c^T, dP = dO V_c^T                                        (SS MMAs, N = 64 keys)
//   P = exp2(S scale + bias - lse_q), dS = P (dP - delta_q)           (elementwise warps, one query row per thread;
//                                                                      dS written back over dP as bf16)
//   dQ += dS K_c                                                      (A from TMEM, B = the unit's rows, MN-major)
// The V unit is free again when the dP product is complete, the K unit after the dQ product.
// dBias: a warp's 32 lanes are the 32 queries of one window row (a_q fixed, b_q = lane), so for one key column the
// lanes update 32 consecutive entries of the row a_q - a_k of the table.  Each TMEM lane quarter owns a private
// shared-memory table [a_k][b_q - b_k + 31] and updates it with plain load-add-store.  A key chunk is four columns
// of the window (b_k = 4 c .. 4 c + 3, all 32 rows a_k), ordered so that 16 consecutive TMEM columns are 16
// different key rows at one b_k: the 16 updates of a column group touch 16 different table rows and are independent
// loads, adds and stores.  The two warps of a quarter take key rows 0..15 and 16..31, so they never meet.  Because
// the tile index is the slowest digit of the item order, a_q = 4 tile + quarter changes at most once or twice per
// CTA; the tables are added to the global gradient (float atomics) at each change and at the end.
// Roles: warps 0-7 elementwise (warps w and w + 4 share lane quarter w & 3 and take the chunk's first / second 64 key
// columns), warp 8 issues every MMA, warps 9-11 gather rows with cp.async.  A row is kept as head dim / 32 parts of 32
// columns in the 64-byte-swizzled operand layout.
// Half chunks are the units of work (16 per item, numbered through the whole run); half chunk n belongs to
// elementwise warps 4 (n % 2) .. 4 (n % 2) + 3 and lives in TMEM buffer n % 3 (S in the buffer's first 64 columns, dP
// in the second).  With three buffers for two groups of warps the scores of a group's next half chunk are issued
// while it still works on the current one (as soon as the other group's previous half chunk has been consumed), so
// the MMA round trip is hidden behind the elementwise work.
// TMEM columns: buffers 0..127, 128..255, 256..383; dQ from 384 on (head dim columns).
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
#define g_bwd_q64_timeout g_bwd_q64_timeout_f16
#define launch_bwd_q64 launch_bwd_q64_f16
#define read_bwd_q64_status read_bwd_q64_status_f16
#endif

namespace terra {

__device__ int g_bwd_q64_timeout = 0;   // set when a bounded wait expired in any CTA of the kernel below

namespace {

using namespace tc;

constexpr int kMmaWarp = 8;
constexpr int kLoaderWarp0 = 9;
constexpr int kLoaderThreads = 96;
constexpr int kThreads = 384;
constexpr int kWorkThreads = 256;
// every SM sub-partition holds two elementwise warps and one of warps 8-11: 2 * 192 + 112 <= 512 registers per lane
constexpr int kRegsLaunch = 168, kRegsWork = 192, kRegsOther = 112;
static_assert(2 * (kRegsWork - kRegsLaunch) <= (kRegsLaunch - kRegsOther), "register hand-over does not balance");

constexpr int kW = 32;                                // window side
constexpr int kPartBytes = 64;                        // one 32-column part of a row
constexpr int kTile = 128;                            // queries per item, keys per chunk
constexpr int kPart = kTile * kPartBytes;             // 8192: the region of one 32-column part of the 128 query rows
constexpr int kUPart = 64 * kPartBytes;               // 4096: ... of the 64 key rows of a half chunk
constexpr int kTiles = kW * kW / kTile;               // 8 query tiles = 8 key chunks per window
constexpr int kBiasFloats = 6048;
constexpr int kTabFloats = kW * 64;                   // bias-gradient tables: per lane quarter [a_k 32][b_q - b_k + 31, padded to 64]
constexpr int kBufCols = 128, kColDQ = 384;           // buffer b: S at 128 b, dP at 128 b + 64
constexpr int kHalfChunks = 2 * kTiles;               // per item

// Shared-memory plan per head dim D (64 or 128): a row is kept as D / 32 parts of 32 columns, each part a region in
// the 64-byte-swizzled operand layout.  The keys of a half chunk arrive as two units, its 64 K rows and its 64 V rows,
// in rings of their own: a V unit is free again as soon as the half chunk's dP product is complete, a K unit only
// after its dQ product.  Head dim 64: two query stages, six K and six V units; head dim 128: one stage, four K and
// two V units.
template <int D>
struct Lay {
    static constexpr int kParts = D / 32;
    static constexpr int kQStages = D == 64 ? 2 : 1;
    static constexpr int kKUnits = D == 64 ? 6 : 4, kVUnits = D == 64 ? 6 : 2;
    // query stage: Q parts | dO parts, then per query row: 4 * bias code, label, token, lse, delta
    static constexpr int kOffQ = 0, kOffG = kParts * kPart;
    static constexpr int kRows = 2 * kParts * kPart;
    static constexpr int kOffQCode = kRows, kOffQLab = kRows + 512, kOffQTok = kRows + 1024, kOffQLse = kRows + 1536, kOffQDelta = kRows + 2048;
    static constexpr int kQStageBytes = kRows + 3072;
    static constexpr int kUnitBytes = kParts * kUPart;
    static constexpr int kOffKRing = kQStages * kQStageBytes;
    static constexpr int kOffVRing = kOffKRing + kKUnits * kUnitBytes;
    static constexpr int kOffKLab = kOffVRing + kVUnits * kUnitBytes;               // per K unit: the 64 keys' mask labels
    static constexpr int kOffBias = kOffKLab + ((kKUnits * 256 + 1023) / 1024) * 1024;
    static constexpr int kOffTab = kOffBias + kBiasFloats * 4;
    static constexpr int kOffBars = ((kOffTab + 4 * kTabFloats * 4 + 1023) / 1024) * 1024;
    static constexpr int kSmemBytes = kOffBars + 1024;
    // the loader fetches this many half chunks of the next item before its query rows (with one query stage those can
    // only follow when the item before is complete, and the keys should not wait for that)
    static constexpr int kKeysFirst = kQStages == 1 ? 2 : 0;
    static_assert(kQStageBytes % 1024 == 0 && kUnitBytes % 1024 == 0, "tiles keep the swizzle alignment");
    static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
    static_assert(kColDQ + D <= 512, "tensor memory columns");
    static_assert(kKeysFirst <= kVUnits && kKeysFirst < kKUnits, "the keys fetched first must fit their rings");
};

constexpr int kCodeStride = kW + 32;
constexpr int kC0 = (kW - 1) * (kCodeStride + 1);

struct Cursor {                                       // (tile, batch, window row, window column), the last fastest
    int wc, wr, b, qt;
};
__device__ __forceinline__ Cursor cursor_at(const Geo& g, long long i) {
    const long long nwin = (long long)g.B * g.Mh * g.Mw;
    Cursor c;
    c.qt = (int)(i / nwin);
    long long rem = i - (long long)c.qt * nwin;
    c.b = (int)(rem / ((long long)g.Mh * g.Mw));
    rem -= (long long)c.b * g.Mh * g.Mw;
    c.wr = (int)(rem / g.Mw);
    c.wc = (int)(rem - (long long)c.wr * g.Mw);
    return c;
}
__device__ __forceinline__ void cursor_next(const Geo& g, Cursor& c) {
    if (++c.wc == g.Mw) {
        c.wc = 0;
        if (++c.wr == g.Mh) {
            c.wr = 0;
            if (++c.b == g.B) { c.b = 0; ++c.qt; }
        }
    }
}

__device__ __forceinline__ bool window_masked(const Geo& g, const Cursor& c) {
    const int r0 = c.wr * kW, c0 = c.wc * kW;
    const bool mh = !g.ph && g.sh > 0 && r0 < g.H - g.sh && r0 + kW > g.H - g.sh;
    const bool mw = !g.pw && g.sw > 0 && c0 < g.W - g.sw && c0 + kW > g.W - g.sw;
    return mh || mw;
}

// window slot (= 32 a_k + b_k) of column j of key chunk c: a_k = 16 (j / 64) + j % 16, b_k = 4 c + (j / 16) % 4
__device__ __forceinline__ int chunk_slot(int c, int j) { return (16 * (j >> 6) + (j & 15)) * kW + 4 * c + ((j >> 4) & 3); }

// token of window slot `slot` (= 32 a + b) with its bias code and mask label
__device__ __forceinline__ int slot_token(const Geo& g, const Cursor& c, int slot, int& code, int& label) {
    const int a = slot >> 5, b = slot & 31;
    int u = c.wr * kW + a + g.sh;
    if (u >= g.H) u -= g.H;
    int v = c.wc * kW + b + g.sw;
    if (v >= g.W) v -= g.W;
    label = ((!g.ph && u < g.sh) ? 2 : 0) + ((!g.pw && v < g.sw) ? 1 : 0);
    code = a * kCodeStride + b;
    return u * g.W + v;
}

__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;\n" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ int4 lds_i4(uint32_t addr) {
    int4 v;
    asm volatile("ld.shared.v4.s32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ int lds_i32(uint32_t addr) {
    int v;
    asm volatile("ld.shared.s32 %0, [%1];\n" : "=r"(v) : "r"(addr) : "memory");
    return v;
}

// 16 key columns [c, c + 16) of one query row: P = exp2(S scale + bias - lse), dS = P (dP - delta); dS is packed to
// bf16 for the dQ product and added, in fp32, to the row's 16 entries of the bias-gradient table (`tab` = address of
// the entry of column c; the following columns are the following key rows, one table row further each).
// `bias_grp` = address of the bias entry of column c: the group's columns are 16 consecutive key rows at one b_k, so
// the following entries lie one code stride below each (no per-key table is read for them).
// `lab_a` = shared address of the mask label of the chunk's key column 0 (as if the table had all 128 columns).
template <bool MASKED>
__device__ __forceinline__ void cols16(const uint32_t (&rs)[16], const uint32_t (&rp)[16], int c, uint32_t bias_grp, int qlabel,
                                       float l2, float dl, uint32_t lab_a, float scale, uint32_t tab, uint32_t (&pk_ds)[8]) {
    int kl[16];
    float bv[16], tv[16];
    if (MASKED) {
#pragma unroll
        for (int e4 = 0; e4 < 4; ++e4) {
            const int4 k4 = lds_i4(lab_a + 4 * (c + e4 * 4));
            kl[e4 * 4] = k4.x; kl[e4 * 4 + 1] = k4.y; kl[e4 * 4 + 2] = k4.z; kl[e4 * 4 + 3] = k4.w;
        }
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) bv[e] = lds_f32(bias_grp - 4 * kCodeStride * e);
    // two-wide fp32 operations: one instruction per pair of columns
    float ds[16];
#pragma unroll
    for (int e = 0; e < 16; e += 2) {
        float x0, x1, t0, t1;
        fma2(x0, x1, __uint_as_float(rs[e]), __uint_as_float(rs[e + 1]), scale, bv[e], bv[e + 1]);
        add2(x0, x1, x0, x1, -l2);
        if (MASKED && kl[e] != qlabel) x0 = -INFINITY;
        if (MASKED && kl[e + 1] != qlabel) x1 = -INFINITY;
        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
        add2(t0, t1, __uint_as_float(rp[e]), __uint_as_float(rp[e + 1]), -dl);
        mul2(ds[e], ds[e + 1], p0, p1, t0, t1);
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) tv[e] = lds_f32(tab + 256 * e);
#pragma unroll
    for (int e = 0; e < 16; ++e) sts_f32(tab + 256 * e, tv[e] + ds[e]);
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) pk_ds[e2] = pack_elem(ds[2 * e2], ds[2 * e2 + 1]);
    __syncwarp();                                         // the next group's entries are this group's, one lane over
}

struct QMaps64 {
    RowMaps3 q, g;            // query rows and their output gradients, by window rows
    CUtensorMap k;            // K rows by runs of 16 vertically adjacent tokens
    CUtensorMap k4, v4;       // ... four such runs (4 adjacent token columns) of K / V in one copy, if the encoder took the axis order
    int k4_ok;
};

// TMA: both shifts are multiples of 16 (8 suffices for the longitude): one loader warp fetches the query rows (four
// window rows per copy where the grid allows it) and the K units with tiled bulk copies (per-query lse and delta by
// 4-byte cp.async copies tied to the same barrier), the other two fetch the V units.  A unit is four runs of 16
// vertically adjacent tokens: one 4 KB copy per 32-column part where its four token columns do not cross the longitude
// seam (a tensor map with the token-row axis before the token-column axis), else four 1 KB copies (K) or 16-byte
// cp.async copies (V).  Otherwise all three warps gather every row.
template <int D, bool TMA>
__global__ void __launch_bounds__(kThreads, 1)
swin_bwd_q64_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o,
                    const float* __restrict__ bias_prep, const float* __restrict__ lse, const float* __restrict__ delta,
                    __nv_bfloat16* __restrict__ dq, float* __restrict__ dbias, long long items_per_head, int ctas_per_head,
                    const __grid_constant__ QMaps64 maps) {
    using L = Lay<D>;
    constexpr int kParts = L::kParts, kQStages = L::kQStages, kKUnits = L::kKUnits, kVUnits = L::kVUnits;
    constexpr int kOffQ = L::kOffQ, kOffG = L::kOffG, kOffQCode = L::kOffQCode, kOffQLab = L::kOffQLab, kOffQTok = L::kOffQTok;
    constexpr int kOffQLse = L::kOffQLse, kOffQDelta = L::kOffQDelta, kQStageBytes = L::kQStageBytes, kUnitBytes = L::kUnitBytes;
    constexpr int kOffKRing = L::kOffKRing, kOffVRing = L::kOffVRing, kOffKLab = L::kOffKLab, kOffBias = L::kOffBias;
    constexpr int kOffTab = L::kOffTab, kOffBars = L::kOffBars;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bar0 = smem0 + kOffBars;
    auto bar_qfull = [&](int s) { return bar0 + 8u * s; };               // the tile's Q, dO rows and row tables are there
    auto bar_qempty = [&](int s) { return bar0 + 8u * (2 + s); };        // ... and no longer needed
    // half chunk number p has its K rows in unit p % kKUnits of the K ring and its V rows in unit p % kVUnits of the V ring
    auto bar_kfull = [&](int u) { return bar0 + 8u * (4 + u); };
    auto bar_kempty = [&](int u) { return bar0 + 8u * (10 + u); };       // every MMA that reads the unit is complete
    auto bar_vfull = [&](int u) { return bar0 + 8u * (25 + u); };
    auto bar_vempty = [&](int u) { return bar0 + 8u * (31 + u); };
    auto bar_sdp = [&](int b) { return bar0 + 8u * (16 + b); };          // S and dP of a half chunk are in TMEM buffer b
    auto bar_ds = [&](int b) { return bar0 + 8u * (19 + b); };           // bf16 dS of the half chunk is in TMEM buffer b
    const uint32_t bar_acc = bar0 + 8u * 22;                              // dQ of the item is final
    const uint32_t bar_accfree = bar0 + 8u * 23;                          // ... and has been read
    const uint32_t bar_flush = bar0 + 8u * 24;                            // the elementwise warps meet around a table flush
    unsigned char* tail = smem + kOffBars + 8 * 37;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail);
    volatile int* cta_abort = reinterpret_cast<volatile int*>(tail + 8);

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = tid >> 5;
    const int head = blockIdx.x % g.heads;
    const int cta_in_head = blockIdx.x / g.heads;
    const long long it_lo = items_per_head * cta_in_head / ctas_per_head;
    const long long it_hi = items_per_head * (cta_in_head + 1) / ctas_per_head;

    if (tid == 0) {
        for (int s = 0; s < kQStages; ++s) {
            mbar_init(bar_qfull(s), TMA ? 32 : kLoaderThreads);
            mbar_init(bar_qempty(s), 1 + kWorkThreads);    // the issuer's commit + every elementwise thread
        }
        for (int u = 0; u < kKUnits; ++u) {
            mbar_init(bar_kfull(u), TMA ? 32 : kLoaderThreads);
            mbar_init(bar_kempty(u), 1);
        }
        for (int u = 0; u < kVUnits; ++u) {
            mbar_init(bar_vfull(u), TMA ? 64 : kLoaderThreads);       // TMA: the 64 threads that gather V rows
            mbar_init(bar_vempty(u), 1);
        }
        for (int b = 0; b < 3; ++b) {
            mbar_init(bar_sdp(b), 1);
            mbar_init(bar_ds(b), kWorkThreads / 2);
        }
        mbar_init(bar_acc, 1);
        mbar_init(bar_accfree, kWorkThreads);
        mbar_init(bar_flush, kWorkThreads);
        *cta_abort = 0;
        fence_barrier_init();
    }
    for (int i = tid; i < kBiasFloats; i += kThreads)
        reinterpret_cast<float*>(smem + kOffBias)[i] = bias_prep[(size_t)head * kBiasFloats + i];
    for (int i = tid; i < 4 * kTabFloats; i += kThreads) reinterpret_cast<float*>(smem + kOffTab)[i] = 0.f;
    fence_proxy_async();
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const size_t HW = (size_t)g.H * g.W;

    if (warp >= kMmaWarp) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsOther));
    if (TMA && warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loader warp (TMA); the other two have no work
        if (warp == kLoaderWarp0) {
            int quse = 0;
            unsigned ru = 0;                              // half chunks so far
            bool ok = true;
            // the K unit of half chunk n of the window at `cw`: rows 16 i .. 16 i + 15 of a unit are the tokens of window
            // rows 16 (n % 2) .. + 15 in window column 4 (n / 2) + i.  (The V units are gathered by the other two loader
            // warps: the bulk-copy engine takes a fixed time per 64-byte row, and the two ways of loading run side by side.)
            auto load_half = [&](const Cursor& cw, int n) -> bool {
                const int c = n >> 1, h = n & 1;
                int u0 = cw.wr * kW + 16 * h + g.sh;
                if (u0 >= g.H) u0 -= g.H;
                const int z = cw.b * g.H + u0;
                const int i = lane / kParts, part = lane - i * kParts;      // this lane's run and part (lanes < 4 * kParts)
                int vcol = cw.wc * kW + 4 * c + i + g.sw;
                if (vcol >= g.W) vcol -= g.W;
                const uint32_t uoff = part * kUPart + i * 16 * kPartBytes;
                const int uk = (int)(ru % kKUnits);
                if (!mbar_wait_all(bar_kempty(uk), (uint32_t)((ru / kKUnits) & 1) ^ 1u, cta_abort)) return false;
                for (int r = lane; r < 64; r += 32) {
                    int code, label;
                    slot_token(g, cw, chunk_slot(c, 64 * h + r), code, label);
                    reinterpret_cast<int*>(smem + kOffKLab + uk * 256)[r] = label;
                }
                int vcol0 = cw.wc * kW + 4 * c + g.sw;
                if (vcol0 >= g.W) vcol0 -= g.W;
                if (maps.k4_ok && vcol0 + 4 <= g.W) {
                    // the unit's four token columns do not cross the longitude seam: one copy per part
                    if (lane < kParts)
                        tma_load_3d(smem0 + kOffKRing + uk * kUnitBytes + lane * kUPart, &maps.k4, head * D + lane * 32, z, vcol0, bar_kfull(uk));
                } else if (lane < 4 * kParts) {
                    tma_load_3d(smem0 + kOffKRing + uk * kUnitBytes + uoff, &maps.k, head * D + part * 32, vcol, z, bar_kfull(uk));
                }
                if (lane == 0) mbar_arrive_expect_tx(bar_kfull(uk), (uint32_t)(64 * D * 2));
                else mbar_arrive(bar_kfull(uk));
                ++ru;
                return true;
            };
            Cursor cur = cursor_at(g, it_lo);
            int fetched = 0;                              // half chunks of the current item already fetched
            for (long long it = it_lo; ok && it < it_hi; ++it, ++quse) {
                const int qs = quse % kQStages;
                ok = mbar_wait_all(bar_qempty(qs), ((quse / kQStages) & 1) ^ 1, cta_abort);
                if (!ok) break;
                const size_t sample_off = (size_t)cur.b * HW;
                // ---- the query tile: Q, dO rows and the row tables
                {
                    unsigned char* st = smem + qs * kQStageBytes;
                    const uint32_t sb = smem0 + qs * kQStageBytes;
                    const int slot0 = cur.qt * kTile;
                    for (int row = lane; row < kTile; row += 32) {
                        int code, label;
                        const int tok = slot_token(g, cur, slot0 + row, code, label);
                        const size_t li = (sample_off + (size_t)tok) * g.heads + head;
                        reinterpret_cast<int*>(st + kOffQCode)[row] = 4 * code;
                        reinterpret_cast<int*>(st + kOffQLab)[row] = label;
                        reinterpret_cast<int*>(st + kOffQTok)[row] = tok;
                        cp_async4(sb + kOffQLse + 4 * row, lse + li);
                        cp_async4(sb + kOffQDelta + 4 * row, delta + li);
                    }
                    int v0 = cur.wc * kW + g.sw;
                    if (v0 >= g.W) v0 -= g.W;
                    // (one lane per tensor and part: the tile's four window rows, as one copy where the grid allows it)
                    for (int i = lane; i < 2 * kParts; i += 32) {
                        const int tsr = i >= kParts ? 1 : 0, part = i - tsr * kParts;
                        bulk_copy_window_rows(tsr ? maps.g : maps.q, sb + (tsr ? kOffG : kOffQ) + part * kPart, g, cur.b, cur.wr, v0,
                                              cur.qt * (kTile / kW), kTile / kW, head * D + part * 32, bar_qfull(qs));
                    }
                    if (lane == 0) mbar_expect_tx(bar_qfull(qs), (uint32_t)(kTile * D * 2 * 2));
                    // the lane's arrival: when its lse / delta copies have landed (its table entries were written before)
                    cp_async_mbar_arrive_noinc(bar_qfull(qs));
                }
                // ---- the window's keys, half chunk by half chunk; then the first ones of the next item
                for (int n = fetched; n < kHalfChunks && ok; ++n) ok = load_half(cur, n);
                if (!ok) break;
                cursor_next(g, cur);
                fetched = 0;
                if (it + 1 < it_hi)
                    for (; fetched < L::kKeysFirst && ok; ++fetched) ok = load_half(cur, fetched);
            }
        } else {
            // ---- warps 10, 11: the V units, one row of 64 per thread, with 16-byte cp.async copies; a thread's arrival
            // on the unit's barrier is tied to the completion of its copies, so it never waits for data
            const int r = (warp - kLoaderWarp0 - 1) * 32 + lane;       // 0 .. 63
            unsigned ru = 0;
            bool ok = true;
            Cursor cur = cursor_at(g, it_lo);
            for (long long it = it_lo; ok && it < it_hi; ++it, cursor_next(g, cur)) {
                const size_t sample_off = (size_t)cur.b * HW;
                for (int n = 0; n < kHalfChunks; ++n, ++ru) {
                    const int uv = (int)(ru % kVUnits);
                    ok = mbar_wait_all(bar_vempty(uv), (uint32_t)((ru / kVUnits) & 1) ^ 1u, cta_abort);
                    if (!ok) break;
                    const uint32_t vb = smem0 + kOffVRing + uv * kUnitBytes;
                    int vcol0 = cur.wc * kW + 4 * (n >> 1) + g.sw;
                    if (vcol0 >= g.W) vcol0 -= g.W;
                    if (maps.k4_ok && vcol0 + 4 <= g.W) {
                        // the unit's four token columns do not cross the longitude seam: one bulk copy per part
                        int u0 = cur.wr * kW + 16 * (n & 1) + g.sh;
                        if (u0 >= g.H) u0 -= g.H;
                        if (r < kParts) tma_load_3d(vb + r * kUPart, &maps.v4, head * D + r * 32, cur.b * g.H + u0, vcol0, bar_vfull(uv));
                        if (r == 0) mbar_arrive_expect_tx(bar_vfull(uv), (uint32_t)(64 * D * 2));
                        else mbar_arrive(bar_vfull(uv));
                        continue;
                    }
                    int code, label;
                    const int tok = slot_token(g, cur, chunk_slot(n >> 1, 64 * (n & 1) + r), code, label);
                    const __nv_bfloat16* src = v + (sample_off + (size_t)tok) * g.ts + head * D;
#pragma unroll
                    for (int piece = 0; piece < D / 8; ++piece)
                        cp_async16(vb + (piece >> 2) * kUPart + tile_off<32>(r, piece & 3), src + piece * 8, 16);
                    cp_async_mbar_arrive_noinc(bar_vfull(uv));
                }
            }
        }
    } else if (warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loaders
        const int lt = (warp - kLoaderWarp0) * 32 + lane;
        // D / 8 lanes per row, one 16-byte piece of the row each (pieces 4 p .. 4 p + 3: the row's part p): a warp's
        // copy instruction reads whole rows.
        constexpr int kPieces = D / 8;
        const int piece = lt % kPieces, rsub = lt / kPieces;
        constexpr int kRowsPerStep = kLoaderThreads / kPieces;
        const uint32_t q_piece_off = (uint32_t)(piece >> 2) * kPart;      // the piece's part in a query stage
        const uint32_t u_piece_off = (uint32_t)(piece >> 2) * kUPart;     // ... in a key unit
        int quse = 0;
        unsigned ru = 0;                                  // half chunks so far (a CTA sees far fewer than 2^32)
        bool ok = true;
        // A thread never waits for data: its arrival on a barrier is tied to the completion of the copies it has issued.
        auto acquire = [&](uint32_t bar, uint32_t parity) -> bool { return mbar_wait_all(bar, parity, cta_abort); };
        // (the thread's table entries are visible to the CTA before its arrivals, which follow its copies)
        auto issued = [&](uint32_t bar, uint32_t bar2) {
            __threadfence_block();
            cp_async_mbar_arrive_noinc(bar);
            if (bar2) cp_async_mbar_arrive_noinc(bar2);
        };
        // the K and V rows of half chunk n of the window at `cw`, one group of copies
        auto load_half = [&](const Cursor& cw, int n) -> bool {
            const size_t sample_off = (size_t)cw.b * HW;
            const int c = n >> 1, row0 = 64 * (n & 1);
            const int uk = (int)(ru % kKUnits), uv = (int)(ru % kVUnits);
            if (!acquire(bar_kempty(uk), (uint32_t)((ru / kKUnits) & 1) ^ 1u)) return false;
            if (!acquire(bar_vempty(uv), (uint32_t)((ru / kVUnits) & 1) ^ 1u)) return false;
            const uint32_t kb = smem0 + kOffKRing + uk * kUnitBytes + u_piece_off;
            const uint32_t vb = smem0 + kOffVRing + uv * kUnitBytes + u_piece_off;
#pragma unroll
            for (int step = 0; step < (64 + kRowsPerStep - 1) / kRowsPerStep; ++step) {
                const int r = rsub + kRowsPerStep * step;
                if (r < 64) {
                    int code, label;
                    const int tok = slot_token(g, cw, chunk_slot(c, row0 + r), code, label);
                    if (piece == 0) reinterpret_cast<int*>(smem + kOffKLab + uk * 256)[r] = label;
                    const size_t off = (sample_off + (size_t)tok) * g.ts + head * D + piece * 8;
                    const uint32_t so = tile_off<32>(r, piece & 3);
                    cp_async16(kb + so, k + off, 16);
                    cp_async16(vb + so, v + off, 16);
                }
            }
            issued(bar_kfull(uk), bar_vfull(uv));
            ++ru;
            return true;
        };
        Cursor cur = cursor_at(g, it_lo);
        int fetched = 0;                                  // half chunks of the current item already fetched
        for (long long it = it_lo; ok && it < it_hi; ++it, ++quse) {
            const int qs = quse % kQStages;
            ok = acquire(bar_qempty(qs), ((quse / kQStages) & 1) ^ 1);
            if (!ok) break;
            const size_t sample_off = (size_t)cur.b * HW;
            // ---- the query tile: Q, dO rows and the row tables
            {
                unsigned char* st = smem + qs * kQStageBytes;
                const uint32_t sb = smem0 + qs * kQStageBytes + q_piece_off;
                const int slot0 = cur.qt * kTile;
#pragma unroll 1
                for (int step = 0; step < (kTile + kRowsPerStep - 1) / kRowsPerStep; ++step) {
                    const int row = rsub + kRowsPerStep * step;
                    if (row < kTile) {
                        int code, label;
                        const int tok = slot_token(g, cur, slot0 + row, code, label);
                        const size_t li = (sample_off + (size_t)tok) * g.heads + head;
                        if (piece == 0) {
                            reinterpret_cast<int*>(st + kOffQCode)[row] = 4 * code;
                            reinterpret_cast<int*>(st + kOffQLab)[row] = label;
                            reinterpret_cast<int*>(st + kOffQTok)[row] = tok;
                            // lse and delta travel with the rows (no load the loader would have to wait for)
                            cp_async4(smem0 + qs * kQStageBytes + kOffQLse + 4 * row, lse + li);
                            cp_async4(smem0 + qs * kQStageBytes + kOffQDelta + 4 * row, delta + li);
                        }
                        const uint32_t so = tile_off<32>(row, piece & 3);
                        cp_async16(sb + kOffQ + so, q + (sample_off + (size_t)tok) * g.ts + head * D + piece * 8, 16);
                        cp_async16(sb + kOffG + so, d_o + li * D + piece * 8, 16);
                    }
                }
                issued(bar_qfull(qs), 0);
            }
            // ---- the window's keys, half chunk by half chunk; then the first ones of the next item
            for (int n = fetched; n < kHalfChunks && ok; ++n) ok = load_half(cur, n);
            if (!ok) break;
            cursor_next(g, cur);
            fetched = 0;
            if (it + 1 < it_hi)
                for (; fetched < L::kKeysFirst && ok; ++fetched) ok = load_half(cur, fetched);
        }
    } else {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc_s = make_idesc_elem(128, 64, 0, 0);
        const uint32_t idesc_acc = make_idesc_elem(128, D, 0, 1);        // A from TMEM, B = 16 rows x D (MN-major)
        const uint32_t sd_hi = sdesc_hi(make_sdesc_sw64(smem0, 512));    // common high word of the K-major descriptors
        int quse = 0;
        bool ok = true;
        for (long long it = it_lo; ok && it < it_hi; ++it, ++quse) {
            const int qs = quse % kQStages;
            ok = mbar_wait_all(bar_qfull(qs), (quse / kQStages) & 1, cta_abort);
            if (!ok) break;
            fence_proxy_async();
            const uint32_t qb = smem0 + qs * kQStageBytes;
            const unsigned n0 = (unsigned)quse * kHalfChunks;     // number of the item's half chunk 0
            auto half_ready = [&](int n) -> bool {        // the K and V rows of the item's half chunk n are in their units
                const unsigned p = n0 + n;
                if (!mbar_wait_all(bar_kfull((int)(p % kKUnits)), (uint32_t)((p / kKUnits) & 1), cta_abort)) return false;
                if (!mbar_wait_all(bar_vfull((int)(p % kVUnits)), (uint32_t)((p / kVUnits) & 1), cta_abort)) return false;
                fence_proxy_async();
                return true;
            };
            // S = Q K^T, dP = dO V^T for half chunk n of the item into its buffer; the V unit goes back with them
            // (descriptor low words = start address in 16-byte units: + 2 per 32-byte K step, + region / 16 per 32-column part)
            const uint32_t q_lo = sdesc_lo(make_sdesc_sw64(qb + kOffQ, 512)), g_lo = sdesc_lo(make_sdesc_sw64(qb + kOffG, 512));
            auto issue_sdp = [&](int n) {
                const unsigned p = n0 + n;
                const int buf = (int)(p % 3), uv = (int)(p % kVUnits);
                const uint32_t k_lo = sdesc_lo(make_sdesc_sw64(smem0 + kOffKRing + (int)(p % kKUnits) * kUnitBytes, 512));
                const uint32_t v_lo = sdesc_lo(make_sdesc_sw64(smem0 + kOffVRing + uv * kUnitBytes, 512));
                const uint32_t t_s = tmem_base + kBufCols * buf, t_dp = t_s + 64;
                constexpr uint32_t kQNext = kPart >> 4, kUNext = kUPart >> 4;
                tc_fence_after();
                if (elect_one()) {
                    mma_ss_h<false>(t_s, q_lo, k_lo, sd_hi, idesc_s);
                    mma_ss_h<true>(t_s, q_lo + 2, k_lo + 2, sd_hi, idesc_s);
#pragma unroll
                    for (int pt = 1; pt < kParts; ++pt) {
                        mma_ss_h<true>(t_s, q_lo + pt * kQNext, k_lo + pt * kUNext, sd_hi, idesc_s);
                        mma_ss_h<true>(t_s, q_lo + pt * kQNext + 2, k_lo + pt * kUNext + 2, sd_hi, idesc_s);
                    }
                    mma_ss_h<false>(t_dp, g_lo, v_lo, sd_hi, idesc_s);
                    mma_ss_h<true>(t_dp, g_lo + 2, v_lo + 2, sd_hi, idesc_s);
#pragma unroll
                    for (int pt = 1; pt < kParts; ++pt) {
                        mma_ss_h<true>(t_dp, g_lo + pt * kQNext, v_lo + pt * kUNext, sd_hi, idesc_s);
                        mma_ss_h<true>(t_dp, g_lo + pt * kQNext + 2, v_lo + pt * kUNext + 2, sd_hi, idesc_s);
                    }
                    mma_commit(bar_sdp(buf));
                    mma_commit(bar_vempty(uv));
                }
                __syncwarp();
            };
            // the item's first three half chunks (every buffer is free: the previous item's were all consumed)
            for (int n = 0; n < 3 && ok; ++n) {
                ok = half_ready(n);
                if (ok) issue_sdp(n);
            }
            if (!ok) break;
            for (int n = 0; n < kHalfChunks && ok; ++n) {
                const unsigned ng = n0 + n;
                const int buf = (int)(ng % 3);
                ok = mbar_wait_all(bar_ds(buf), (uint32_t)((ng / 3) & 1), cta_abort);
                if (ok && n == 0 && quse > 0) ok = mbar_wait_all(bar_accfree, (quse - 1) & 1, cta_abort);
                if (!ok) break;
                tc_fence_after();
                // dQ += dS K over the half chunk's key columns
                const uint64_t kd = make_sdesc_sw64_mn(smem0 + kOffKRing + (int)(ng % kKUnits) * kUnitBytes, kUPart, 512);
                const uint32_t k_lo = sdesc_lo(kd), d_hi = sdesc_hi(kd);
                const uint32_t t_ds = tmem_base + kBufCols * buf + 64;
                if (elect_one()) {
                    int j = 0;
                    if (n == 0) {
                        mma_ts_h<false>(tmem_base + kColDQ, t_ds, k_lo, d_hi, idesc_acc);
                        j = 1;
                    }
                    for (; j < 4; ++j) mma_ts_h<true>(tmem_base + kColDQ, t_ds + 16 * j, k_lo + 64 * j, d_hi, idesc_acc);
                    mma_commit(bar_kempty((int)(ng % kKUnits)));    // the K unit's last reader: it goes back at once
                    if (n + 1 == kHalfChunks) {
                        mma_commit(bar_acc);
                        mma_commit(bar_qempty(qs));
                    }
                }
                __syncwarp();
                // the buffer is free again (the product that reads it was issued just above): the scores of the half
                // chunk three further on follow at once
                if (n + 3 < kHalfChunks) {
                    ok = half_ready(n + 3);
                    if (!ok) break;
                    issue_sdp(n + 3);
                }
            }
        }
    }
    } else {
        // ------------------------------------------------------------------ elementwise warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsWork));
        const int hcol = warp >> 2;                       // which 64 key columns of a chunk
        const int quarter = warp & 3;
        const int qrow = 32 * quarter + lane;             // query row inside the tile
        const uint32_t lane_addr = ((uint32_t)(32 * quarter)) << 16;
        const float scale = g.scale_log2e;
        const float out_scale = g.scale_log2e * kLn2;     // dQ carries the score scale
        const uint32_t tab0 = smem0 + kOffTab;
        // this lane's entry for key (a_k = 16 hcol, b_k = 0): [a_k][lane + 31]; b_k lies b_k floats below, a_k rows above
        const uint32_t tab_lane = tab0 + 4 * (quarter * kTabFloats + 16 * hcol * 64 + lane + 31);
        int quse = 0, n_flush = 0;
        int tab_qt = -1;                                  // the tile whose gradients the tables hold
        bool ok = true;
        // all elementwise threads meet (bounded), the tables go to the global gradient and are cleared, they meet again
        auto flush = [&](int qt) -> bool {
            mbar_arrive(bar_flush);
            if (!mbar_wait_all(bar_flush, n_flush & 1, cta_abort)) return false;
            ++n_flush;
            for (int i = tid; i < 4 * kTabFloats; i += kWorkThreads) {
                const int db = i & 63;
                if (db == 63) continue;
                const float val = lds_f32(tab0 + 4 * i);
                if (val != 0.f) {
                    const int da = 4 * qt + (i >> 11) - ((i >> 6) & 31) + kW - 1;
                    atomicAdd(dbias + (size_t)(da * (2 * kW - 1) + db) * g.heads + head, val);
                    sts_f32(tab0 + 4 * i, 0.f);
                }
            }
            mbar_arrive(bar_flush);
            if (!mbar_wait_all(bar_flush, n_flush & 1, cta_abort)) return false;
            ++n_flush;
            return true;
        };
        Cursor cur = cursor_at(g, it_lo);
        for (long long it = it_lo; ok && it < it_hi; ++it, cursor_next(g, cur), ++quse) {
            if (cur.qt != tab_qt) {
                if (tab_qt >= 0) ok = flush(tab_qt);
                if (!ok) break;
                tab_qt = cur.qt;
            }
            const bool masked = window_masked(g, cur);
            const int qs = quse % kQStages;
            if (!mbar_wait_all(bar_qfull(qs), (quse / kQStages) & 1, cta_abort)) { ok = false; break; }
            const uint32_t st_a = smem0 + qs * kQStageBytes;
            const int qcode4 = lds_i32(st_a + kOffQCode + 4 * qrow);
            const int qlabel = lds_i32(st_a + kOffQLab + 4 * qrow);
            const int qtok = lds_i32(st_a + kOffQTok + 4 * qrow);
            const float l2 = lds_f32(st_a + kOffQLse + 4 * qrow) * kLog2e;
            const float dl = lds_f32(st_a + kOffQDelta + 4 * qrow);
            mbar_arrive(bar_qempty(qs));                  // this thread has what it needs from the query stage
            const uint32_t bias_row = smem0 + kOffBias + qcode4;
            for (int c = 0; c < kTiles && ok; ++c) {
                const unsigned ng = (unsigned)quse * kHalfChunks + 2 * c + hcol;     // this group's half chunk
                // labels of the half chunk's 64 keys, addressed by the chunk's column number
                const uint32_t sl_a = smem0 + kOffKLab + (int)(ng % kKUnits) * 256 - 256 * hcol;
                const int buf = (int)(ng % 3);
                ok = mbar_wait_all(bar_sdp(buf), (uint32_t)((ng / 3) & 1), cta_abort);
                if (!ok) break;
                tc_fence_after();
                // buffer columns of key column cc of the chunk: S at cc - 64 hcol, dP 64 further
                const uint32_t t_s = tmem_base + lane_addr + kBufCols * buf - 64 * hcol, t_dp = t_s + 64;
                // a 16-column group is key rows 16 hcol .. 16 hcol + 15 at b_k = 4 c + (column / 16) % 4
                auto tab_of = [&](int col) { return tab_lane - 4 * (4 * c + ((col >> 4) & 3)); };
                // bias index = code_query - code_key + c0 with code_key = (16 hcol + e) * stride + b_k
                auto bias_of = [&](int col) { return bias_row + 4 * (kC0 - 16 * hcol * kCodeStride - 4 * c - ((col >> 4) & 3)); };
                // groups of 16 columns; the next group's S / dP travel from TMEM while this one is worked on
                uint32_t rs[16], rp[16], rs2[16], rp2[16], pk_ds[8];
                const int col0 = 64 * hcol;
                tmem_ld16(t_s + col0, rs);
                tmem_ld16(t_dp + col0, rp);
#pragma unroll
                for (int cc = col0; cc < col0 + 64; cc += 32) {
                    tmem_ld_wait();
                    tmem_ld16(t_s + cc + 16, rs2);
                    tmem_ld16(t_dp + cc + 16, rp2);
                    if (masked) cols16<true>(rs, rp, cc, bias_of(cc), qlabel, l2, dl, sl_a, scale, tab_of(cc), pk_ds);
                    else cols16<false>(rs, rp, cc, bias_of(cc), qlabel, l2, dl, sl_a, scale, tab_of(cc), pk_ds);
                    tmem_st8(t_dp + cc, pk_ds);            // 16 keys -> 8 packed columns at the group's own place
                    tmem_ld_wait();
                    if (cc + 32 < col0 + 64) {
                        tmem_ld16(t_s + cc + 32, rs);
                        tmem_ld16(t_dp + cc + 32, rp);
                    }
                    if (masked) cols16<true>(rs2, rp2, cc + 16, bias_of(cc + 16), qlabel, l2, dl, sl_a, scale, tab_of(cc + 16), pk_ds);
                    else cols16<false>(rs2, rp2, cc + 16, bias_of(cc + 16), qlabel, l2, dl, sl_a, scale, tab_of(cc + 16), pk_ds);
                    tmem_st8(t_dp + cc + 16, pk_ds);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_ds(buf));
            }
            if (!ok) break;
            // ---- read-out: dQ columns 0..31 by warps 0-3, 32..63 by warps 4-7
            if (!mbar_wait_all(bar_acc, quse & 1, cta_abort)) { ok = false; break; }
            tc_fence_after();
            // ---- read-out: the first half of dQ's columns by warps 0-3, the second by warps 4-7
            uint4* dst = reinterpret_cast<uint4*>(dq + ((size_t)cur.b * HW + (size_t)qtok) * g.ts + head * D + (D / 2) * hcol);
#pragma unroll
            for (int hq = 0; hq < D / 64; ++hq) {
                uint32_t r0[32];
                tmem_ld32(tmem_base + lane_addr + kColDQ + (D / 2) * hcol + 32 * hq, r0);
                tmem_ld_wait();
                if (hq == D / 64 - 1) {
                    tc_fence_before();
                    mbar_arrive(bar_accfree);
                }
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    uint4 a;
                    a.x = pack_elem(__uint_as_float(r0[c4 * 8 + 0]) * out_scale, __uint_as_float(r0[c4 * 8 + 1]) * out_scale);
                    a.y = pack_elem(__uint_as_float(r0[c4 * 8 + 2]) * out_scale, __uint_as_float(r0[c4 * 8 + 3]) * out_scale);
                    a.z = pack_elem(__uint_as_float(r0[c4 * 8 + 4]) * out_scale, __uint_as_float(r0[c4 * 8 + 5]) * out_scale);
                    a.w = pack_elem(__uint_as_float(r0[c4 * 8 + 6]) * out_scale, __uint_as_float(r0[c4 * 8 + 7]) * out_scale);
                    dst[4 * hq + c4] = a;
                }
            }
        }
        if (ok && tab_qt >= 0) flush(tab_qt);
    }

    // teardown: every role ends up here, also after an expired wait
    cp_async_wait<0>();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
    if (tid == 0 && *cta_abort) atomicExch(&g_bwd_q64_timeout, 1);
}

}  // namespace

cudaError_t read_bwd_q64_status(int* timed_out) {
    int zero = 0;
    cudaError_t e = cudaMemcpyFromSymbol(timed_out, g_bwd_q64_timeout, sizeof(int));
    if (e != cudaSuccess) return e;
    if (*timed_out) e = cudaMemcpyToSymbol(g_bwd_q64_timeout, &zero, sizeof(int));
    return e;
}

#ifndef TERRA_ELEM_F16
bool bwd_q64_supported(const Geo& g) {
    return (g.d == 64 || g.d == 128) && g.w == kW && g.H % kW == 0 && g.W % kW == 0 && g.heads <= 148;
}
#endif  // !TERRA_ELEM_F16

// `prep` = the prepared bias tables of the head-dim-64 forward kernel (kBiasFloats per head), filled by the caller;
// dbias is overwritten
cudaError_t launch_bwd_q64(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                           const float* lse, const float* delta, void* dq, float* dbias, int sm_count, cudaStream_t stream) {
    const long long items = (long long)kTiles * g.B * g.Mh * g.Mw;      // per head
    long long cph = sm_count / g.heads;
    if (cph < 1) cph = 1;
    if (cph > items) cph = items;
    cudaError_t e = cudaMemsetAsync(dbias, 0, sizeof(float) * (size_t)(2 * kW - 1) * (2 * kW - 1) * g.heads, stream);
    if (e != cudaSuccess) return e;
    QMaps64 maps;
    std::memset(&maps, 0, sizeof maps);
    static const bool tma_off = [] { const char* e_ = std::getenv("TERRA_NO_TMA"); return e_ && e_[0] == '1'; }();
    // (at head dim 64 the runs of 16 tokens are 1 KB copies, and the three gathering warps are faster)
    const bool tma = !tma_off && g.d == 128 && bulk_rows_shape(g) && g.sh % 16 == 0 && make_row_maps3(&maps.q, g, q, g.ts) &&
                     make_row_maps3(&maps.g, g, d_o, g.heads * g.d) && make_col_map(&maps.k, g, k, g.ts);
    static const bool k4_off = [] { const char* e_ = std::getenv("TERRA_NO_K4"); return e_ && e_[0] == '1'; }();
    maps.k4_ok = (tma && !k4_off && make_col_map4(&maps.k4, g, k, g.ts) && make_col_map4(&maps.v4, g, v, g.ts)) ? 1 : 0;
    auto kern = g.d == 64 ? swin_bwd_q64_kernel<64, false> : (tma ? swin_bwd_q64_kernel<128, true> : swin_bwd_q64_kernel<128, false>);
    const int smem_bytes = g.d == 64 ? Lay<64>::kSmemBytes : Lay<128>::kSmemBytes;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    if (e != cudaSuccess) return e;
    prof_begin("swin_bwd_q64_kernel", stream);
    kern<<<(unsigned)(cph * g.heads), kThreads, smem_bytes, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, prep, lse, delta,
        (__nv_bfloat16*)dq, dbias, items, (int)cph, maps);
    count_launch(stream);
    return cudaGetLastError();
}

}  // namespace terra
