// Query side of the backward pass (dQ, dBias) on the tcgen05 tensor cores for head dim 64 and complete 32 x 32
// windows (window side 32, grid extents multiples of 32).  Other shapes of this regime run the register-tile kernel.
//
// One persistent CTA per SM, bound to one head, walks over a contiguous range of (128-query tile, batch, window)
// items, the tile index slowest.  The tile's Q and dO rows stay in shared memory; the window's keys stream through a
// ring of slots in chunks of 128 (K, V rows and per-key bias code, mask label).  TMEM lanes = queries, columns = keys.
// Per chunk:
//   S = Q K_c^T, dP = dO V_c^T                                        (SS MMAs, N = 64 keys per half chunk)
//   P = exp2(S scale + bias - lse_q), dS = P (dP - delta_q)           (elementwise warps, one query row per thread;
//                                                                      dS written back over dP as bf16)
//   dQ += dS K_c                                                      (A from TMEM, B = the chunk's rows, MN-major)
// dBias: a warp's 32 lanes are the 32 queries of one window row (a_q fixed, b_q = lane), so for one key column the
// lanes update 32 consecutive entries of the row a_q - a_k of the table.  Each TMEM lane quarter owns a private
// shared-memory table [a_k][b_q - b_k + 31] and updates it with plain load-add-store.  A key chunk is four columns
// of the window (b_k = 4 c .. 4 c + 3, all 32 rows a_k), ordered so that 16 consecutive TMEM columns are 16
// different key rows at one b_k: the 16 updates of a column group touch 16 different table rows and are independent
// loads, adds and stores.  The two warps of a quarter take key rows 0..15 and 16..31, so they never meet.  Because
// the tile index is the slowest digit of the item order, a_q = 4 tile + quarter changes at most once or twice per
// CTA; the tables are added to the global gradient (float atomics) at each change and at the end.
// Roles: warps 0-7 elementwise (warps w and w + 4 share lane quarter w & 3 and take the chunk's first / second 64 key
// columns), warp 8 issues every MMA, warps 9-11 gather rows with cp.async.  Head dim 64 is kept as two 32-column
// halves in the 64-byte-swizzled operand layout (lo | hi regions).
// A chunk's two 64-key halves are separate units of work ("half chunks", 16 per item, numbered through the whole
// run); half chunk n belongs to elementwise warps 4 (n % 2) .. 4 (n % 2) + 3 and lives in TMEM buffer n % 3 (S in the
// buffer's first 64 columns, dP in the second).  With three buffers for two groups of warps the scores of a group's
// next half chunk are issued while it still works on the current one (as soon as the other group's previous half
// chunk has been consumed), so the MMA round trip is hidden behind the elementwise work.
// TMEM columns: buffers 0..127, 128..255, 256..383; dQ 384..447.
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, all roles leave their loops, TMEM is
// released and the host reads the device status word.  Every role follows every ring item by item.
#include "swin_common.cuh"
#include "swin_kernels.h"
#include "tc_common.cuh"

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

constexpr int kD = 64;
constexpr int kW = 32;                                // window side
constexpr int kHalfBytes = 64;
constexpr int kTile = 128;                            // queries per item, keys per chunk
constexpr int kHalf = kTile * kHalfBytes;             // 8192: one 32-column half of 128 rows
constexpr int kTiles = kW * kW / kTile;               // 8 query tiles = 8 key chunks per window
constexpr int kQStages = 2, kSlots = 3;
// query stage: Q lo | Q hi | dO lo | dO hi, then per query row: 4 * bias code, label, token, lse, delta
constexpr int kOffQlo = 0, kOffGlo = 2 * kHalf;     // hi halves follow at + kHalf
constexpr int kRows = 4 * kHalf;                      // 32768
constexpr int kOffQCode = kRows, kOffQLab = kRows + 512, kOffQTok = kRows + 1024, kOffQLse = kRows + 1536, kOffQDelta = kRows + 2048;
constexpr int kQStageBytes = kRows + 3072;
// key slot: K lo | K hi | V lo | V hi, then per key column: label
constexpr int kOffKlo = 0, kOffVlo = 2 * kHalf;     // hi halves follow at + kHalf
constexpr int kOffKLab = kRows;
constexpr int kSlotBytes = kRows + 1024;
constexpr int kOffSlots = kQStages * kQStageBytes;
constexpr int kBiasFloats = 6048;
constexpr int kOffBias = kOffSlots + kSlots * kSlotBytes;
// bias-gradient tables: per lane quarter [a_k 32][b_q - b_k + 31, padded to 64]
constexpr int kTabFloats = kW * 64;
constexpr int kOffTab = kOffBias + kBiasFloats * 4;
constexpr int kOffBars = ((kOffTab + 4 * kTabFloats * 4 + 1023) / 1024) * 1024;
constexpr int kSmemBytes = kOffBars + 1024;
static_assert(kQStageBytes % 1024 == 0 && kSlotBytes % 1024 == 0, "tiles keep the swizzle alignment");
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
constexpr int kBufCols = 128, kColDQ = 384;           // buffer b: S at 128 b, dP at 128 b + 64
constexpr int kHalfChunks = 2 * kTiles;               // per item

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

__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(dst), "l"(src));
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
template <bool MASKED>
__device__ __forceinline__ void cols16(const uint32_t (&rs)[16], const uint32_t (&rp)[16], int c, uint32_t bias_grp, int qlabel,
                                       float l2, float dl, uint32_t sl_a, float scale, uint32_t tab, uint32_t (&pk_ds)[8]) {
    int kl[16];
    float bv[16], tv[16];
    if (MASKED) {
#pragma unroll
        for (int e4 = 0; e4 < 4; ++e4) {
            const int4 k4 = lds_i4(sl_a + kOffKLab + 4 * (c + e4 * 4));
            kl[e4 * 4] = k4.x; kl[e4 * 4 + 1] = k4.y; kl[e4 * 4 + 2] = k4.z; kl[e4 * 4 + 3] = k4.w;
        }
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) bv[e] = lds_f32(bias_grp - 4 * kCodeStride * e);
    float ds[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        float xv = fmaf(__uint_as_float(rs[e]), scale, bv[e]) - l2;
        if (MASKED && kl[e] != qlabel) xv = -INFINITY;
        const float p = fast_exp2(xv);
        ds[e] = p * (__uint_as_float(rp[e]) - dl);
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) tv[e] = lds_f32(tab + 256 * e);
#pragma unroll
    for (int e = 0; e < 16; ++e) sts_f32(tab + 256 * e, tv[e] + ds[e]);
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) pk_ds[e2] = pack_bf16(ds[2 * e2], ds[2 * e2 + 1]);
    __syncwarp();                                         // the next group's entries are this group's, one lane over
}

__global__ void __launch_bounds__(kThreads, 1)
swin_bwd_q64_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o,
                    const float* __restrict__ bias_prep, const float* __restrict__ lse, const float* __restrict__ delta,
                    __nv_bfloat16* __restrict__ dq, float* __restrict__ dbias, long long items_per_head, int ctas_per_head) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bar0 = smem0 + kOffBars;
    auto bar_qfull = [&](int s) { return bar0 + 8u * s; };               // the tile's Q, dO rows and row tables are there
    auto bar_qempty = [&](int s) { return bar0 + 8u * (2 + s); };        // ... and no longer needed
    // the ring is handed over in half slots: half chunk number p sits in rows 64 (p % 2) .. of slot (p / 2) % 3
    auto bar_kfull = [&](int hs) { return bar0 + 8u * (4 + hs); };       // half slot hs = p % 6 holds its 64 keys
    auto bar_kempty = [&](int hs) { return bar0 + 8u * (10 + hs); };     // ... and every MMA that reads them is complete
    auto bar_sdp = [&](int b) { return bar0 + 8u * (16 + b); };          // S and dP of a half chunk are in TMEM buffer b
    auto bar_ds = [&](int b) { return bar0 + 8u * (19 + b); };           // bf16 dS of the half chunk is in TMEM buffer b
    const uint32_t bar_acc = bar0 + 8u * 22;                              // dQ of the item is final
    const uint32_t bar_accfree = bar0 + 8u * 23;                          // ... and has been read
    const uint32_t bar_flush = bar0 + 8u * 24;                            // the elementwise warps meet around a table flush
    unsigned char* tail = smem + kOffBars + 8 * 25;
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
            mbar_init(bar_qfull(s), kLoaderThreads);
            mbar_init(bar_qempty(s), 1 + kWorkThreads);    // the issuer's commit + every elementwise thread
        }
        for (int hs = 0; hs < 2 * kSlots; ++hs) {
            mbar_init(bar_kfull(hs), kLoaderThreads);
            mbar_init(bar_kempty(hs), 1);
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
    if (warp >= kLoaderWarp0) {
        // ------------------------------------------------------------------ loaders
        const int lt = (warp - kLoaderWarp0) * 32 + lane;
        // Eight lanes per row, one 16-byte piece of the row's 128 bytes each (pieces 0-3: the lo half, 4-7: the hi
        // half), twelve rows per step: a warp's copy instruction reads four whole rows.
        const int piece = lt & 7, rsub = lt >> 3;
        constexpr int kRowsPerStep = kLoaderThreads / 8;      // 12
        const uint32_t piece_off = (uint32_t)(piece >> 2) * kHalf;
        int quse = 0;
        long long ru = 0;                                 // half chunks so far
        uint32_t pending_bar = 0;                         // barrier of the group in flight
        bool ok = true;
        auto publish = [&]() {
            cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(pending_bar);
            pending_bar = 0;
        };
        // no free place yet: the group in flight is published first
        auto acquire = [&](uint32_t bar, uint32_t parity) -> bool {
            if (pending_bar && !__all_sync(0xffffffffu, mbar_test_wait(bar, parity))) publish();
            return mbar_wait_all(bar, parity, cta_abort);
        };
        // a group is published when the next one has been issued
        auto issued = [&](uint32_t bar) {
            cp_async_commit();
            if (pending_bar) {
                cp_async_wait<1>();
                fence_proxy_async();
                mbar_arrive(pending_bar);
            }
            pending_bar = bar;
        };
        Cursor cur = cursor_at(g, it_lo);
        for (long long it = it_lo; ok && it < it_hi; ++it, cursor_next(g, cur), ++quse) {
            const int qs = quse % kQStages;
            ok = acquire(bar_qempty(qs), ((quse / kQStages) & 1) ^ 1);
            if (!ok) break;
            const size_t sample_off = (size_t)cur.b * HW;
            // ---- the query tile: Q, dO rows and the row tables
            {
                unsigned char* st = smem + qs * kQStageBytes;
                const uint32_t sb = smem0 + qs * kQStageBytes + piece_off;
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
                        cp_async16(sb + kOffQlo + so, q + (sample_off + (size_t)tok) * g.ts + head * kD + piece * 8, 16);
                        cp_async16(sb + kOffGlo + so, d_o + li * kD + piece * 8, 16);
                    }
                }
                issued(bar_qfull(qs));
            }
            // ---- the window's keys, half chunk by half chunk
            for (int n = 0; n < kHalfChunks; ++n, ++ru) {
                const int hs = (int)(ru % (2 * kSlots));
                ok = acquire(bar_kempty(hs), (uint32_t)((ru / (2 * kSlots)) & 1) ^ 1u);
                if (!ok) break;
                unsigned char* sl = smem + kOffSlots + (hs >> 1) * kSlotBytes;
                const uint32_t sb = smem0 + kOffSlots + (hs >> 1) * kSlotBytes + piece_off;
                const int c = n >> 1, row0 = 64 * (n & 1);
#pragma unroll
                for (int step = 0; step < (64 + kRowsPerStep - 1) / kRowsPerStep; ++step) {
                    const int r = rsub + kRowsPerStep * step;
                    if (r < 64) {
                        const int row = row0 + r;
                        int code, label;
                        const int tok = slot_token(g, cur, chunk_slot(c, row), code, label);
                        if (piece == 0) reinterpret_cast<int*>(sl + kOffKLab)[row] = label;
                        const size_t off = (sample_off + (size_t)tok) * g.ts + head * kD + piece * 8;
                        const uint32_t so = tile_off<32>(row, piece & 3);
                        cp_async16(sb + kOffKlo + so, k + off, 16);
                        cp_async16(sb + kOffVlo + so, v + off, 16);
                    }
                }
                issued(bar_kfull(hs));
            }
        }
        if (pending_bar) publish();
    } else {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc_s = make_idesc_bf16(128, 64, 0, 0);
        const uint32_t idesc_acc = make_idesc_bf16(128, kD, 0, 1);       // A from TMEM, B = 16 rows x 64 (MN-major)
        const uint32_t sd_hi = sdesc_hi(make_sdesc_sw64(smem0, 512));    // common high word of the K-major descriptors
        int quse = 0;
        bool ok = true;
        for (long long it = it_lo; ok && it < it_hi; ++it, ++quse) {
            const int qs = quse % kQStages;
            ok = mbar_wait_all(bar_qfull(qs), (quse / kQStages) & 1, cta_abort);
            if (!ok) break;
            fence_proxy_async();
            const uint32_t qb = smem0 + qs * kQStageBytes;
            const long long n0 = (long long)quse * kHalfChunks;   // number of the item's half chunk 0
            auto half_ready = [&](int n) -> bool {        // the keys of the item's half chunk n are in their half slot
                const long long p = n0 + n;
                if (!mbar_wait_all(bar_kfull((int)(p % (2 * kSlots))), (uint32_t)((p / (2 * kSlots)) & 1), cta_abort)) return false;
                fence_proxy_async();
                return true;
            };
            // S = Q K^T, dP = dO V^T for half chunk n of the item (chunk n / 2, keys 64 (n % 2) ..), into its buffer
            // (descriptor low words = start address in 16-byte units: + 2 per 32-byte K step, + kHalf / 16 for the hi half)
            const uint32_t q_lo = sdesc_lo(make_sdesc_sw64(qb + kOffQlo, 512)), g_lo = sdesc_lo(make_sdesc_sw64(qb + kOffGlo, 512));
            auto issue_sdp = [&](int n) {
                const uint32_t sb = smem0 + kOffSlots + (int)(((n0 + n) >> 1) % kSlots) * kSlotBytes + (n & 1) * 64 * kHalfBytes;
                const int buf = (int)((n0 + n) % 3);
                const uint32_t k_lo = sdesc_lo(make_sdesc_sw64(sb + kOffKlo, 512));
                const uint32_t v_lo = sdesc_lo(make_sdesc_sw64(sb + kOffVlo, 512));
                const uint32_t t_s = tmem_base + kBufCols * buf, t_dp = t_s + 64;
                constexpr uint32_t kHi = kHalf >> 4;
                tc_fence_after();
                if (elect_one()) {
                    mma_ss_h<false>(t_s, q_lo, k_lo, sd_hi, idesc_s);
                    mma_ss_h<true>(t_s, q_lo + 2, k_lo + 2, sd_hi, idesc_s);
                    mma_ss_h<true>(t_s, q_lo + kHi, k_lo + kHi, sd_hi, idesc_s);
                    mma_ss_h<true>(t_s, q_lo + kHi + 2, k_lo + kHi + 2, sd_hi, idesc_s);
                    mma_ss_h<false>(t_dp, g_lo, v_lo, sd_hi, idesc_s);
                    mma_ss_h<true>(t_dp, g_lo + 2, v_lo + 2, sd_hi, idesc_s);
                    mma_ss_h<true>(t_dp, g_lo + kHi, v_lo + kHi, sd_hi, idesc_s);
                    mma_ss_h<true>(t_dp, g_lo + kHi + 2, v_lo + kHi + 2, sd_hi, idesc_s);
                    mma_commit(bar_sdp(buf));
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
                const long long ng = n0 + n;
                const int buf = (int)(ng % 3);
                ok = mbar_wait_all(bar_ds(buf), (uint32_t)((ng / 3) & 1), cta_abort);
                if (ok && n == 0 && quse > 0) ok = mbar_wait_all(bar_accfree, (quse - 1) & 1, cta_abort);
                if (!ok) break;
                tc_fence_after();
                // dQ += dS K over the half chunk's key columns
                const uint32_t sb = smem0 + kOffSlots + (int)((ng >> 1) % kSlots) * kSlotBytes + (n & 1) * 64 * kHalfBytes;
                const uint64_t kd = make_sdesc_sw64_mn(sb + kOffKlo, kHalf, 512);
                const uint32_t k_lo = sdesc_lo(kd), d_hi = sdesc_hi(kd);
                const uint32_t t_ds = tmem_base + kBufCols * buf + 64;
                if (elect_one()) {
                    int j = 0;
                    if (n == 0) {
                        mma_ts_h<false>(tmem_base + kColDQ, t_ds, k_lo, d_hi, idesc_acc);
                        j = 1;
                    }
                    for (; j < 4; ++j) mma_ts_h<true>(tmem_base + kColDQ, t_ds + 16 * j, k_lo + 64 * j, d_hi, idesc_acc);
                    mma_commit(bar_kempty((int)(ng % (2 * kSlots))));   // the half slot's last reader: it goes back at once
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
        long long ru = 0;
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
            for (int c = 0; c < kTiles && ok; ++c, ++ru) {
                const int s = (int)(ru % kSlots);         // the chunk's slot: half chunk p is in slot (p / 2) % 3
                const uint32_t sl_a = smem0 + kOffSlots + s * kSlotBytes;
                const long long ng = (long long)quse * kHalfChunks + 2 * c + hcol;   // this group's half chunk
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
            uint32_t r0[32];
            tmem_ld32(tmem_base + lane_addr + kColDQ + 32 * hcol, r0);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(bar_accfree);
            uint4* dst = reinterpret_cast<uint4*>(dq + ((size_t)cur.b * HW + (size_t)qtok) * g.ts + head * kD + 32 * hcol);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint4 a;
                a.x = pack_bf16(__uint_as_float(r0[c4 * 8 + 0]) * out_scale, __uint_as_float(r0[c4 * 8 + 1]) * out_scale);
                a.y = pack_bf16(__uint_as_float(r0[c4 * 8 + 2]) * out_scale, __uint_as_float(r0[c4 * 8 + 3]) * out_scale);
                a.z = pack_bf16(__uint_as_float(r0[c4 * 8 + 4]) * out_scale, __uint_as_float(r0[c4 * 8 + 5]) * out_scale);
                a.w = pack_bf16(__uint_as_float(r0[c4 * 8 + 6]) * out_scale, __uint_as_float(r0[c4 * 8 + 7]) * out_scale);
                dst[c4] = a;
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

bool bwd_q64_supported(const Geo& g) {
    return g.d == 64 && g.w == kW && g.H % kW == 0 && g.W % kW == 0 && g.heads <= 148;
}

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
    e = cudaFuncSetAttribute(swin_bwd_q64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    prof_begin("swin_bwd_q64_kernel", stream);
    swin_bwd_q64_kernel<<<(unsigned)(cph * g.heads), kThreads, kSmemBytes, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, prep, lse, delta,
        (__nv_bfloat16*)dq, dbias, items, (int)cph);
    count_launch(stream);
    return cudaGetLastError();
}

}  // namespace terra
