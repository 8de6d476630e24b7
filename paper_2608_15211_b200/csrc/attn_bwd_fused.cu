// Backward shifted-window attention on the tcgen05 tensor cores, one pass (head dim 32, windows of <= 256
// tokens): P and dS of a (window, head) item are computed once and feed all three gradients.
//
// Orientation: TMEM lanes (rows) = keys of a 128-key tile, columns = queries, 64 query columns per block.
//   S^T  = K Q^T, dP^T = V dO^T                      (SS MMAs, N = the block's columns)
//   P^T  = exp2(S^T scale + bias - lse_q), dS^T = P^T (dP^T - delta_q)       (elementwise warps, one key row per thread)
//   dV  += P^T dO, dK += dS^T Q                      (A = bf16 P^T / dS^T read from TMEM, per block)
//   dQ  += dS K                                      (A = dS^T from shared memory, read transposed (MN-major),
//                                                     per pair of blocks = 128 queries)
//   dBias: every elementwise warp adds its dS into a private shared-memory table (plain load-add-store: the
//          32 lanes of one instruction are 32 different keys at one query = 32 different entries; the keys of
//          a tile are interleaved over the warps so that 4 or 8 consecutive queries can be updated together).
// Roles: warps 0..7 elementwise, warp 8 issues every MMA (the whole warp runs the loop, one elected lane
// issues), warps 9..11 gather the window's rows with cp.async into the 64-byte-swizzled operand layout,
// warps 12..15 read the finished accumulators out of TMEM and store them.
// The eight elementwise warps work on ONE key tile at a time: warps w and w + 4 share the 32 key rows of TMEM
// lane quarter w & 3 and split each block's four 16-column steps (steps 0, 2 and steps 1, 3).
// The CTA's blocks form one sequence across tiles and items; S^T / dP^T of a block are issued two blocks ahead.
// TMEM columns: two [S 64 | dP 64] buffers, two (dV, dK) accumulator sets, two dQ accumulators (queries
// 0..127 and 128..255).  A tile's dV / dK and an item's dQ are read out by the read-out warps as soon as their
// last MMA has completed; the elementwise warps never wait for them.
// Outputs leave through the item's own operand tiles in shared memory (dK over the K rows, dV over V, dQ
// over Q, once the MMAs that read them are complete), so that whole 64-byte rows are stored.
// CTAs are bound to one head (grid = heads x CTAs per head): the head's bias table is staged once per CTA
// and the bias-gradient tables belong to one head; they are summed in a fixed order (reproducible dBias).
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag and all roles leave their loops.
#include <cstdlib>

#include "swin_common.cuh"
#include "swin_kernels.h"
#include "tc_common.cuh"

// fp16 build of this file (through the _f16 wrapper file): the kernel, its launcher and its status word get names of
// their own; the element-independent helpers are compiled in the bf16 build only
#ifdef TERRA_ELEM_F16
#define g_bwd_tc_timeout g_bwd_tc_timeout_f16
#define launch_bwd_tc launch_bwd_tc_f16
#define read_bwd_tc_status read_bwd_tc_status_f16
#endif

namespace terra {

__device__ int g_bwd_tc_timeout = 0;   // set when a bounded wait expired in any CTA of the kernel below

namespace {

using namespace tc;

constexpr int kIssuerWarp = 8;      // warp 8: MMA issuer (also owns the TMEM allocation)
constexpr int kLoaderWarp0 = 9;     // warps 9..11: loaders
constexpr int kLoaderWarps = 3;
constexpr int kLoaderThreads = kLoaderWarps * 32;
constexpr int kEpiWarp0 = 12;       // warps 12..15: read-out of the accumulators (one warp per TMEM lane quarter)
constexpr int kEpiThreads = 128;
constexpr int kThreads = 16 * 32;                               // 512 = four warpgroups
constexpr int kWorkThreads = 256;          // elementwise threads; each arrives once per barrier phase
constexpr int kRegsLaunch = 128;
constexpr int kRegsWork = 184;      // elementwise warpgroups after setmaxnreg.inc
constexpr int kRegsOther = 80;      // MMA + loader warpgroup after setmaxnreg.dec
constexpr int kRegsEpi = 64;        // read-out warpgroup after setmaxnreg.dec
static_assert(2 * (kRegsWork - kRegsLaunch) <= (kRegsLaunch - kRegsOther) + (kRegsLaunch - kRegsEpi), "register hand-over does not balance");

constexpr int kStages = 2;
constexpr int kMaxSlots = 256;
constexpr int kD = 32;
constexpr int kRowBytes = kD * 2;
constexpr int kTileBytes = kMaxSlots * kRowBytes;              // 16384
constexpr int CB = 64;                                         // query columns per block

// stage layout (bytes)
constexpr int kOffQ = 0;
constexpr int kOffK = kTileBytes;
constexpr int kOffV = 2 * kTileBytes;
constexpr int kOffDO = 3 * kTileBytes;
constexpr int kOffColOff = 4 * kTileBytes;                     // per slot: 4 * bias code, code = a * (w + 32) + b (0 if no token)
constexpr int kOffLab = kOffColOff + kMaxSlots * 4;            // per slot: shift-mask label (0xff: no token)
constexpr int kOffTok = kOffLab + kMaxSlots * 4;               // per slot: grid token, -1 if none
constexpr int kOffLse = kOffTok + kMaxSlots * 4;               // per slot: lse * log2(e), +inf if none
constexpr int kOffDelta = kOffLse + kMaxSlots * 4;             // per slot: delta
constexpr int kStageBytes = kOffDelta + kMaxSlots * 4;         // 70656
static_assert(kStageBytes % 1024 == 0, "stages keep the swizzle alignment");
// after the stages
constexpr int kOffBias = kStages * kStageBytes;                // the head's prepared bias table (kFwdBiasFloats floats)
constexpr int kDBiasEntries = 1472;                            // >= 2 c0 + 1 for w <= 16
constexpr int kDBiasFloats = kDBiasEntries + 32;               // + one scratch float per lane (where pairs without a token add their 0)
constexpr int kOffDBias = kOffBias + kFwdBiasFloats * 4;       // one bias-gradient table per elementwise warp
constexpr int kOffDS = kOffDBias + 8 * kDBiasFloats * 4;       // dS^T of one pair of blocks: [128 keys][128 queries] bf16
static_assert(kOffDS % 1024 == 0, "the dS tile keeps the swizzle alignment");
constexpr int kDSGroupBytes = 128 * kRowBytes;                 // 32 queries x 128 keys
constexpr int kOffBars = kOffDS + 4 * kDSGroupBytes;
constexpr int kSmemBytes = kOffBars + 256;
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

// TMEM columns
constexpr int kColBuf = 128;        // buffer b at b * 128: S at +0, dP at +64
constexpr int kColDV = 256;         // accumulator set s: dV at 256 + 64 s, dK at 288 + 64 s
constexpr int kColDK = 288;
constexpr int kColDQ = 384;         // dQ of query pair p at 384 + 32 p

// (48, the stride of side 16, in the layout of 16 slots per window row: code = slot + 32 a again, so a warp's 32 key
// rows update 32 different banks)
__device__ __forceinline__ int code_stride(int w, bool pad16 = false) { return pad16 ? 48 : w + 32; }
// floats in front of a warp's bias-gradient table in the 16-slots-per-row layout of window sides 9 .. 15
__host__ __device__ __forceinline__ int dbias_margin(int w) { return (16 - w) * 48 + 8; }

// Key rows of a tile are interleaved over the elementwise warps: lane l of warp W = 4 t + quarter holds slot
// 32 ((W + c l) mod M) + l, M = 4 * (tiles in use).  c = 1, except c = 5 for two-tile windows whose side does not
// divide 32 (see the bias-gradient updates in the kernel).
__device__ __forceinline__ int key_interleave(int w, int ntiles) { return (ntiles == 2 && (32 % w) != 0) ? 5 : 1; }

struct Item {
    int b, win;
    WindowRef r;
    int npad;      // slots rounded up to 16
    int ntiles;    // 128-key tiles in use
    int nblk;      // 64-query blocks in use
    bool masked;   // the window mixes shift-mask labels
    bool ragged;   // some row of a key tile, or some column below npad, has no token
};

// pad16: the window's slots are laid out 16 to a window row (slot = 16 a + b; the slots with b >= the window's width
// hold no token), so that every group of 16 query columns is one window row whatever the window side
__device__ __forceinline__ Item make_item(const Geo& g, const ItemCursor& c, bool pad16 = false) {
    Item x;
    x.win = c.wr * g.Mw + c.wc;
    x.b = c.b;
    x.r = window_ref_rc(g, c.wr, c.wc);
    if (pad16) x.r.n = x.r.eh * 16;
    x.npad = (x.r.n + 15) & ~15;
    x.ntiles = (x.r.n + 127) >> 7;
    x.nblk = (x.npad + CB - 1) / CB;
    const int r0 = x.r.wr * g.w, c0 = x.r.wc * g.w;
    const bool mh = !g.ph && g.sh > 0 && r0 < g.H - g.sh && r0 + x.r.eh > g.H - g.sh;
    const bool mw = !g.pw && g.sw > 0 && c0 < g.W - g.sw && c0 + x.r.ew > g.W - g.sw;
    x.masked = mh || mw;
    x.ragged = pad16 || x.npad != x.r.n || x.r.n != x.ntiles * 128;
    return x;
}

// window offset (a, b) -> grid token, bias code and shift-mask label
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
__device__ __forceinline__ void sts_u4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// table[addr] += v in the warp's own table.  Not atomic: within one warp instruction the 32 lanes (32
// different keys, same query) touch 32 different entries, and successive instructions of a warp reach
// shared memory in program order, so nothing is lost.
__device__ __forceinline__ void rmw_shared_f32(uint32_t addr, float v) {
    asm volatile(
        "{\n\t.reg .f32 t;\n\t"
        "ld.shared.f32 t, [%0];\n\t"
        "add.f32 t, t, %1;\n\t"
        "st.shared.f32 [%0], t;\n\t}\n" ::"r"(addr), "f"(v) : "memory");
}
// G table updates of one lane, issued together so that their load-add-store latencies overlap.  Allowed only
// where no two of the warp's 32 x G updates can meet in one entry (see the key-row order in the kernel).
__device__ __forceinline__ void rmw4_shared_f32(const uint32_t* a, const float* v) {
    asm volatile(
        "{\n\t.reg .f32 t0, t1, t2, t3;\n\t"
        "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%1];\n\tld.shared.f32 t2, [%2];\n\tld.shared.f32 t3, [%3];\n\t"
        "add.f32 t0, t0, %4;\n\tadd.f32 t1, t1, %5;\n\tadd.f32 t2, t2, %6;\n\tadd.f32 t3, t3, %7;\n\t"
        "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%1], t1;\n\tst.shared.f32 [%2], t2;\n\tst.shared.f32 [%3], t3;\n\t}\n"
        ::"r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
    __syncwarp();   // later groups stay behind these stores (see rmw8_consecutive_f32)
}
__device__ __forceinline__ void rmw8_shared_f32(const uint32_t* a, const float* v) {
    asm volatile(
        "{\n\t.reg .f32 t0, t1, t2, t3, t4, t5, t6, t7;\n\t"
        "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%1];\n\tld.shared.f32 t2, [%2];\n\tld.shared.f32 t3, [%3];\n\t"
        "ld.shared.f32 t4, [%4];\n\tld.shared.f32 t5, [%5];\n\tld.shared.f32 t6, [%6];\n\tld.shared.f32 t7, [%7];\n\t"
        "add.f32 t0, t0, %8;\n\tadd.f32 t1, t1, %9;\n\tadd.f32 t2, t2, %10;\n\tadd.f32 t3, t3, %11;\n\t"
        "add.f32 t4, t4, %12;\n\tadd.f32 t5, t5, %13;\n\tadd.f32 t6, t6, %14;\n\tadd.f32 t7, t7, %15;\n\t"
        "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%1], t1;\n\tst.shared.f32 [%2], t2;\n\tst.shared.f32 [%3], t3;\n\t"
        "st.shared.f32 [%4], t4;\n\tst.shared.f32 [%5], t5;\n\tst.shared.f32 [%6], t6;\n\tst.shared.f32 [%7], t7;\n\t}\n"
        ::"r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]),
          "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
    __syncwarp();   // later groups stay behind these stores (see rmw8_consecutive_f32)
}
// The same for 8 consecutive entries (one address register, immediate offsets).  The warp barrier at the end
// keeps the next group's loads behind these stores: with base + immediate addresses the assembler can see that
// one THREAD's next loads do not touch these entries and would hoist them, but another lane's do.
__device__ __forceinline__ void rmw8_consecutive_f32(uint32_t a, const float* v) {
    asm volatile(
        "{\n\t.reg .f32 t0, t1, t2, t3, t4, t5, t6, t7;\n\t"
        "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%0+4];\n\tld.shared.f32 t2, [%0+8];\n\tld.shared.f32 t3, [%0+12];\n\t"
        "ld.shared.f32 t4, [%0+16];\n\tld.shared.f32 t5, [%0+20];\n\tld.shared.f32 t6, [%0+24];\n\tld.shared.f32 t7, [%0+28];\n\t"
        "add.f32 t0, t0, %1;\n\tadd.f32 t1, t1, %2;\n\tadd.f32 t2, t2, %3;\n\tadd.f32 t3, t3, %4;\n\t"
        "add.f32 t4, t4, %5;\n\tadd.f32 t5, t5, %6;\n\tadd.f32 t6, t6, %7;\n\tadd.f32 t7, t7, %8;\n\t"
        "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%0+4], t1;\n\tst.shared.f32 [%0+8], t2;\n\tst.shared.f32 [%0+12], t3;\n\t"
        "st.shared.f32 [%0+16], t4;\n\tst.shared.f32 [%0+20], t5;\n\tst.shared.f32 [%0+24], t6;\n\tst.shared.f32 [%0+28], t7;\n\t}\n"
        ::"r"(a), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
    __syncwarp();
}
// The same for the first N < 8 of 8 consecutive entries (the others belong to pairs without a token).
template <int N>
__device__ __forceinline__ void rmw_consecutive_f32(uint32_t a, const float* v) {
    if (N == 1) {
        asm volatile(
            "{\n\t.reg .f32 t0;\n\t"
            "ld.shared.f32 t0, [%0];\n\t"
            "add.f32 t0, t0, %1;\n\t"
            "st.shared.f32 [%0], t0;\n\t}\n"
            ::"r"(a), "f"(v[0]) : "memory");
    }
    if (N == 2) {
        asm volatile(
            "{\n\t.reg .f32 t0, t1;\n\t"
            "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%0+4];\n\t"
            "add.f32 t0, t0, %1;\n\tadd.f32 t1, t1, %2;\n\t"
            "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%0+4], t1;\n\t}\n"
            ::"r"(a), "f"(v[0]), "f"(v[1]) : "memory");
    }
    if (N == 3) {
        asm volatile(
            "{\n\t.reg .f32 t0, t1, t2;\n\t"
            "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%0+4];\n\tld.shared.f32 t2, [%0+8];\n\t"
            "add.f32 t0, t0, %1;\n\tadd.f32 t1, t1, %2;\n\tadd.f32 t2, t2, %3;\n\t"
            "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%0+4], t1;\n\tst.shared.f32 [%0+8], t2;\n\t}\n"
            ::"r"(a), "f"(v[0]), "f"(v[1]), "f"(v[2]) : "memory");
    }
    if (N == 4) {
        asm volatile(
            "{\n\t.reg .f32 t0, t1, t2, t3;\n\t"
            "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%0+4];\n\tld.shared.f32 t2, [%0+8];\n\tld.shared.f32 t3, [%0+12];\n\t"
            "add.f32 t0, t0, %1;\n\tadd.f32 t1, t1, %2;\n\tadd.f32 t2, t2, %3;\n\tadd.f32 t3, t3, %4;\n\t"
            "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%0+4], t1;\n\tst.shared.f32 [%0+8], t2;\n\tst.shared.f32 [%0+12], t3;\n\t}\n"
            ::"r"(a), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]) : "memory");
    }
    if (N == 5) {
        asm volatile(
            "{\n\t.reg .f32 t0, t1, t2, t3, t4;\n\t"
            "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%0+4];\n\tld.shared.f32 t2, [%0+8];\n\tld.shared.f32 t3, [%0+12];\n\tld.shared.f32 t4, [%0+16];\n\t"
            "add.f32 t0, t0, %1;\n\tadd.f32 t1, t1, %2;\n\tadd.f32 t2, t2, %3;\n\tadd.f32 t3, t3, %4;\n\tadd.f32 t4, t4, %5;\n\t"
            "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%0+4], t1;\n\tst.shared.f32 [%0+8], t2;\n\tst.shared.f32 [%0+12], t3;\n\tst.shared.f32 [%0+16], t4;\n\t}\n"
            ::"r"(a), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]) : "memory");
    }
    if (N == 6) {
        asm volatile(
            "{\n\t.reg .f32 t0, t1, t2, t3, t4, t5;\n\t"
            "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%0+4];\n\tld.shared.f32 t2, [%0+8];\n\tld.shared.f32 t3, [%0+12];\n\tld.shared.f32 t4, [%0+16];\n\tld.shared.f32 t5, [%0+20];\n\t"
            "add.f32 t0, t0, %1;\n\tadd.f32 t1, t1, %2;\n\tadd.f32 t2, t2, %3;\n\tadd.f32 t3, t3, %4;\n\tadd.f32 t4, t4, %5;\n\tadd.f32 t5, t5, %6;\n\t"
            "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%0+4], t1;\n\tst.shared.f32 [%0+8], t2;\n\tst.shared.f32 [%0+12], t3;\n\tst.shared.f32 [%0+16], t4;\n\tst.shared.f32 [%0+20], t5;\n\t}\n"
            ::"r"(a), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]) : "memory");
    }
    if (N == 7) {
        asm volatile(
            "{\n\t.reg .f32 t0, t1, t2, t3, t4, t5, t6;\n\t"
            "ld.shared.f32 t0, [%0];\n\tld.shared.f32 t1, [%0+4];\n\tld.shared.f32 t2, [%0+8];\n\tld.shared.f32 t3, [%0+12];\n\tld.shared.f32 t4, [%0+16];\n\tld.shared.f32 t5, [%0+20];\n\tld.shared.f32 t6, [%0+24];\n\t"
            "add.f32 t0, t0, %1;\n\tadd.f32 t1, t1, %2;\n\tadd.f32 t2, t2, %3;\n\tadd.f32 t3, t3, %4;\n\tadd.f32 t4, t4, %5;\n\tadd.f32 t5, t5, %6;\n\tadd.f32 t6, t6, %7;\n\t"
            "st.shared.f32 [%0], t0;\n\tst.shared.f32 [%0+4], t1;\n\tst.shared.f32 [%0+8], t2;\n\tst.shared.f32 [%0+12], t3;\n\tst.shared.f32 [%0+16], t4;\n\tst.shared.f32 [%0+20], t5;\n\tst.shared.f32 [%0+24], t6;\n\t}\n"
            ::"r"(a), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]) : "memory");
    }
    __syncwarp();
}
template <int OFF>
__device__ __forceinline__ float lds_f32_at(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1+%2];\n" : "=f"(v) : "r"(addr), "n"(OFF));
    return v;
}
// mode 8 / 4: groups of 8 / 4 consecutive columns at once; else one column at a time
__device__ __forceinline__ void dbias_add16(int mode, const uint32_t (&addr)[16], const float (&ds)[16]) {
    if (mode == 8) {
        rmw8_shared_f32(&addr[0], &ds[0]);
        rmw8_shared_f32(&addr[8], &ds[8]);
    } else if (mode == 4) {
#pragma unroll
        for (int e = 0; e < 16; e += 4) rmw4_shared_f32(&addr[e], &ds[e]);
    } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) rmw_shared_f32(addr[e], ds[e]);
    }
}

// What one elementwise thread knows about its key row.
struct RowCtx {
    uint32_t bias_row;   // shared address: bias table + the row's part of the index (the -inf zone if the row has no token)
    uint32_t dbias_row;  // shared address: this warp's bias-gradient table + the row's part of the index
    uint32_t scratch;    // shared address: this lane's scratch float behind the table
    int label;
    bool valid;
};

// 16 query columns [c, c + 16) of one key row: P = exp2(S scale + bias - lse), dS = P (dP - delta), both
// packed to bf16; dS also in fp32 with the shared address of its bias-gradient entry (the lane's scratch
// float for a pair without a token, whose dS is 0).
template <bool MASKED, bool RAGGED>
__device__ __forceinline__ void cols16(const uint32_t (&rs)[16], const uint32_t (&rp)[16], int c, const RowCtx& rc, uint32_t st_a,
                                       float scale, uint32_t (&pk_p)[8], uint32_t (&pk_ds)[8], float (&ds)[16], uint32_t (&addr)[16]) {
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
#pragma unroll
    for (int e4 = 0; e4 < 4; ++e4) {
        const float4 a = lds_f4(st_a + kOffLse + 4 * (c + e4 * 4));
        const float4 b = lds_f4(st_a + kOffDelta + 4 * (c + e4 * 4));
        l2[e4 * 4] = a.x; l2[e4 * 4 + 1] = a.y; l2[e4 * 4 + 2] = a.z; l2[e4 * 4 + 3] = a.w;
        dl[e4 * 4] = b.x; dl[e4 * 4 + 1] = b.y; dl[e4 * 4 + 2] = b.z; dl[e4 * 4 + 3] = b.w;
    }
    float p[16];
#pragma unroll
    for (int e = 0; e < 16; e += 2) {
        float x0, x1, t0, t1;
        fma2(x0, x1, __uint_as_float(rs[e]), __uint_as_float(rs[e + 1]), scale, bv[e], bv[e + 1]);
        sub2(x0, x1, x0, x1, l2[e], l2[e + 1]);
        if (MASKED && kl[e] != rc.label) x0 = -INFINITY;
        if (MASKED && kl[e + 1] != rc.label) x1 = -INFINITY;
        p[e] = fast_exp2(x0);
        p[e + 1] = fast_exp2(x1);
        sub2(t0, t1, __uint_as_float(rp[e]), __uint_as_float(rp[e + 1]), dl[e], dl[e + 1]);
        mul2(ds[e], ds[e + 1], p[e], p[e + 1], t0, t1);
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        addr[e] = rc.dbias_row + co[e];
        if (RAGGED && (!rc.valid || l2[e] == INFINITY)) addr[e] = rc.scratch;
    }
#pragma unroll
    for (int e2 = 0; e2 < 8; ++e2) {
        pk_p[e2] = pack_elem(p[2 * e2], p[2 * e2 + 1]);
        pk_ds[e2] = pack_elem(ds[2 * e2], ds[2 * e2 + 1]);
    }
}

// The same for a full 16 x 16 window without mask labels: the 16 columns [c, c + 16) are one window row, so
// their bias codes are consecutive and every table address is one base plus an immediate offset (no per-column
// offsets to load, no address arithmetic).  `code0x4` = 4 * bias code of column c.  Returns the shared
// address of the first column's bias-gradient entry; the others follow 4 bytes apart.
__device__ __forceinline__ void load16_row(int c, int code0x4, const RowCtx& rc, uint32_t st_a, float (&bv)[16], float (&l2)[16],
                                           float (&dl)[16]) {
    const uint32_t bb = rc.bias_row + code0x4;
    bv[0] = lds_f32_at<0>(bb);   bv[1] = lds_f32_at<4>(bb);   bv[2] = lds_f32_at<8>(bb);   bv[3] = lds_f32_at<12>(bb);
    bv[4] = lds_f32_at<16>(bb);  bv[5] = lds_f32_at<20>(bb);  bv[6] = lds_f32_at<24>(bb);  bv[7] = lds_f32_at<28>(bb);
    bv[8] = lds_f32_at<32>(bb);  bv[9] = lds_f32_at<36>(bb);  bv[10] = lds_f32_at<40>(bb); bv[11] = lds_f32_at<44>(bb);
    bv[12] = lds_f32_at<48>(bb); bv[13] = lds_f32_at<52>(bb); bv[14] = lds_f32_at<56>(bb); bv[15] = lds_f32_at<60>(bb);
#pragma unroll
    for (int e4 = 0; e4 < 4; ++e4) {
        const float4 a = lds_f4(st_a + kOffLse + 4 * (c + e4 * 4));
        const float4 b = lds_f4(st_a + kOffDelta + 4 * (c + e4 * 4));
        l2[e4 * 4] = a.x; l2[e4 * 4 + 1] = a.y; l2[e4 * 4 + 2] = a.z; l2[e4 * 4 + 3] = a.w;
        dl[e4 * 4] = b.x; dl[e4 * 4 + 1] = b.y; dl[e4 * 4 + 2] = b.z; dl[e4 * 4 + 3] = b.w;
    }
}
// BW < 16: only the first BW of the 16 query columns hold a token; the others have P = dS = 0 and cost nothing.
template <int BW = 16>
__device__ __forceinline__ void math16_row(const uint32_t (&rs)[16], const uint32_t (&rp)[16], const float (&bv)[16], const float (&l2)[16],
                                           const float (&dl)[16], float scale, uint32_t (&pk_p)[8], uint32_t (&pk_ds)[8], float (&ds)[16]) {
    // two-wide fp32 operations: one instruction per pair of columns
    float p[16];
#pragma unroll
    for (int e = 0; e < 16; e += 2) {
        if (e >= BW) {
            p[e] = p[e + 1] = ds[e] = ds[e + 1] = 0.f;
            continue;
        }
        float x0, x1, t0, t1;
        fma2(x0, x1, __uint_as_float(rs[e]), __uint_as_float(rs[e + 1]), scale, bv[e], bv[e + 1]);
        sub2(x0, x1, x0, x1, l2[e], l2[e + 1]);
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

// One block of a two-tile window of width BW (9 .. 15) in the layout of 16 slots per window row: this warp's steps h
// and h + 2 (one window row of queries each; the window's last block may lack the second), as in the 16-wide case.
// A query column beyond the width has lse = +inf in the slot table, so an odd width's last pair needs no special case.
template <int BW>
__device__ __forceinline__ void pad_block16(uint32_t t_s, uint32_t t_dp, int h, int ca, int cb2, int cs, bool has_b, const RowCtx& rc,
                                            uint32_t st_a, float scale, uint32_t (&pk_dsa)[8], uint32_t (&pk_dsb)[8]) {
    uint32_t sa[16], pa[16], pk_p[8];
    float ds[16], bv[16], l2[16], dl[16];
    tmem_ld16(t_s + 16 * h, sa);
    tmem_ld16(t_dp + 16 * h, pa);
    tmem_ld_wait();
    const int code_a = 4 * cs * (ca >> 4), code_b = 4 * cs * (cb2 >> 4);
    load16_row(ca, code_a, rc, st_a, bv, l2, dl);
    math16_row<BW>(sa, pa, bv, l2, dl, scale, pk_p, pk_dsa, ds);
    uint32_t a0 = rc.dbias_row + code_a;
    tmem_st8(t_s + 16 * h, pk_p);
    tmem_st8(t_dp + 16 * h, pk_dsa);
    if (has_b) {
        tmem_ld16(t_s + 16 * (h + 2), sa);
        tmem_ld16(t_dp + 16 * (h + 2), pa);
        load16_row(cb2, code_b, rc, st_a, bv, l2, dl);       // the second step's table values, in flight during the updates
    }
    rmw8_consecutive_f32(a0, &ds[0]);
    rmw_consecutive_f32<BW - 8>(a0 + 32, &ds[8]);
    if (has_b) {
        tmem_ld_wait();
        math16_row<BW>(sa, pa, bv, l2, dl, scale, pk_p, pk_dsb, ds);
        a0 = rc.dbias_row + code_b;
        tmem_st8(t_s + 16 * (h + 2), pk_p);
        tmem_st8(t_dp + 16 * (h + 2), pk_dsb);
        rmw8_consecutive_f32(a0, &ds[0]);
        rmw_consecutive_f32<BW - 8>(a0 + 32, &ds[8]);
    }
}

// PADW = the window side, 9 .. 15, of a launch that lays the slots out 16 to a window row (see make_item; 0 otherwise):
// full-width two-tile windows without mask labels then take the immediate-offset table addressing and the grouped bias-gradient updates of the 16-wide case.
// Every slot, with or without a token, carries the bias code 16-wide geometry gives it (48 a + b with a, b up to 15,
// the code stride of side 16), so that the update addresses of a warp's 32 key rows stay distinct; a pair without a token adds 0.  Such
// codes reach up to 16 - w table rows and 7 entries in front of the table and 7 entries behind it: each warp's
// bias-gradient table starts `dbias_margin(w)` floats into its block (the tables of these sides leave that room).
template <int PADW>
__global__ void __launch_bounds__(kThreads, 1)
swin_bwd_fused_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                      const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o,
                      const float* __restrict__ bias_prep, const float* __restrict__ lse, const float* __restrict__ delta,
                      __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                      float* __restrict__ dbias_parts, long long n_items, int ctas_per_head) {
    constexpr bool PAD = PADW != 0;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t smem0 = smem_u32(smem);
    const uint32_t bar0 = smem0 + kOffBars;
    auto bar_full = [&](int s) { return bar0 + 8u * s; };           // stage s holds an item's operands
    auto bar_empty = [&](int s) { return bar0 + 8u * (2 + s); };    // stage s may be overwritten
    auto bar_sdp = [&](int b) { return bar0 + 8u * (4 + b); };      // S and dP of a block are in buffer b
    auto bar_ds = [&](int b) { return bar0 + 8u * (6 + b); };       // bf16 P / dS of a block are in buffer b (and dS in shared memory)
    auto bar_acc = [&](int s) { return bar0 + 8u * (8 + s); };      // dV / dK of a key tile are final in accumulator set s
    auto bar_accfree = [&](int s) { return bar0 + 8u * (10 + s); }; // ... and have been read back
    const uint32_t bar_dsfree = bar0 + 8u * 12;                      // the dQ MMAs of a block pair have read the shared dS tile
    const uint32_t bar_dq = bar0 + 8u * 13;                          // every MMA of the item is complete (dQ final)
    const uint32_t bar_dqfree = bar0 + 8u * 14;                      // dQ has been read back
    unsigned char* tail = smem + kOffBars + 8 * 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail);
    volatile int* cta_abort = reinterpret_cast<volatile int*>(tail + 8);

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = tid >> 5;                   // role number = hardware warp
    const int head = blockIdx.x % g.heads;
    const int cta_in_head = blockIdx.x / g.heads;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar_full(s), kLoaderThreads);
            mbar_init(bar_empty(s), kEpiThreads);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_sdp(b), 1);
            mbar_init(bar_ds(b), kWorkThreads);
            mbar_init(bar_acc(b), 1);
            mbar_init(bar_accfree(b), kEpiThreads);
        }
        mbar_init(bar_dsfree, 1);
        mbar_init(bar_dq, 1);
        mbar_init(bar_dqfree, kEpiThreads);
        *cta_abort = 0;
        fence_barrier_init();
    }
    // the head's prepared bias table, and zeroed bias-gradient tables
    for (int i = tid; i < kFwdBiasFloats; i += kThreads)
        reinterpret_cast<float*>(smem + kOffBias)[i] = bias_prep[(size_t)head * kFwdBiasFloats + i];
    for (int i = tid; i < 8 * kDBiasFloats; i += kThreads) reinterpret_cast<float*>(smem + kOffDBias)[i] = 0.f;
    // the shared dS tile starts finite: columns that no block writes only reach dQ rows that are never stored
    for (int i = tid; i < 4 * kDSGroupBytes / 4; i += kThreads) reinterpret_cast<uint32_t*>(smem + kOffDS)[i] = 0u;
    fence_proxy_async();
    if (warp == kIssuerWarp) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int cs = code_stride(g.w, PAD);
    const int c0 = (g.w - 1) * (cs + 1);
    const size_t HW = (size_t)g.H * g.W;

    if (warp >= kEpiWarp0) {
        // ------------------------------------------------------------------ read-out warps
        // A tile's dV / dK and an item's dQ leave tensor memory here, as soon as their last MMA has completed,
        // while the elementwise warps are already working on the next blocks.  Each output row (64 bytes) is
        // staged in the item's own V / K / Q row, which no MMA reads any more, and stored from there as whole rows.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsEpi));
        const int quarter = warp & 3;
        const uint32_t tq = tmem_base + (((uint32_t)(32 * quarter)) << 16);
        const float out_scale = g.scale_log2e * kLn2;          // dQ and dK carry the score scale
        // 32 accumulator columns of this lane's row -> bf16 -> the row's place in the staging tile
        auto stage_row = [&](uint32_t taddr, uint32_t rows_a, float f) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t r[16];
                tmem_ld16(taddr + 16 * half, r);
                tmem_ld_wait();
                sts_u4(rows_a + tile_off<kD>(lane, 2 * half),
                       pack_elem(__uint_as_float(r[0]) * f, __uint_as_float(r[1]) * f), pack_elem(__uint_as_float(r[2]) * f, __uint_as_float(r[3]) * f),
                       pack_elem(__uint_as_float(r[4]) * f, __uint_as_float(r[5]) * f), pack_elem(__uint_as_float(r[6]) * f, __uint_as_float(r[7]) * f));
                sts_u4(rows_a + tile_off<kD>(lane, 2 * half + 1),
                       pack_elem(__uint_as_float(r[8]) * f, __uint_as_float(r[9]) * f), pack_elem(__uint_as_float(r[10]) * f, __uint_as_float(r[11]) * f),
                       pack_elem(__uint_as_float(r[12]) * f, __uint_as_float(r[13]) * f), pack_elem(__uint_as_float(r[14]) * f, __uint_as_float(r[15]) * f));
            }
        };
        // the warp's 32 staged rows -> global memory, four lanes per row; `tok` = this lane's row's grid token (-1: none)
        auto store_rows = [&](uint32_t rows_a, __nv_bfloat16* out, size_t sample_off, int tok) {
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int rr = 8 * jj + (lane >> 2), c4 = lane & 3;
                const int tok_r = __shfl_sync(0xffffffffu, tok, rr);
                const int4 a = lds_i4(rows_a + tile_off<kD>(rr, c4));
                if (tok_r >= 0)
                    *reinterpret_cast<int4*>(out + (sample_off + (size_t)tok_r) * g.ts + head * kD + c4 * 8) = a;
            }
        };
        int kuse = 0, n_tile = 0;
        bool ok = true;
        ItemCursor cur_it = cursor_init(cta_in_head, ctas_per_head, 1, g.Mw, g.Mh);
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, ++kuse, cursor_advance(cur_it, 1, g.Mw, g.Mh)) {
            int npad, ntiles;
            size_t sample_off;
            {
                const Item x = make_item(g, cur_it, PAD);
                npad = x.npad; ntiles = x.ntiles; sample_off = (size_t)x.b * HW;
            }
            const int s = kuse % kStages;
            const uint32_t st_a = smem0 + s * kStageBytes;
            if (!mbar_wait_all_relaxed(bar_full(s), (kuse / kStages) & 1, cta_abort)) break;      // the slot -> token table of the stage
            for (int t = 0; t < ntiles; ++t, ++n_tile) {
                const int set = n_tile & 1;
                ok = mbar_wait_all_relaxed(bar_acc(set), (n_tile >> 1) & 1, cta_abort);
                if (!ok) break;
                tc_fence_after();
                const int slot = 32 * ((4 * t + quarter + key_interleave(PAD ? 16 : g.w, ntiles) * lane) & (4 * ntiles - 1)) + lane;      // interleaved key order
                const int tok = lds_i32(st_a + kOffTok + 4 * slot);
                const uint32_t rows_a = st_a + (uint32_t)((t * 128 + 32 * quarter) * kRowBytes);
                stage_row(tq + kColDV + 64 * set, rows_a + kOffV, 1.f);
                stage_row(tq + kColDK + 64 * set, rows_a + kOffK, out_scale);
                tc_fence_before();
                mbar_arrive(bar_accfree(set));
                __syncwarp();
                store_rows(rows_a + kOffV, dv, sample_off, tok);
                store_rows(rows_a + kOffK, dk, sample_off, tok);
            }
            if (!ok) break;
            ok = mbar_wait_all_relaxed(bar_dq, kuse & 1, cta_abort);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int hq = 0; hq < 2; ++hq)
                if (hq * 128 < npad) stage_row(tq + kColDQ + 32 * hq, st_a + kOffQ + (uint32_t)((hq * 128 + 32 * quarter) * kRowBytes), out_scale);
            tc_fence_before();
            mbar_arrive(bar_dqfree);
            __syncwarp();
#pragma unroll
            for (int hq = 0; hq < 2; ++hq)
                if (hq * 128 < npad) {
                    const int tokq = lds_i32(st_a + kOffTok + 4 * (hq * 128 + 32 * quarter + lane));
                    store_rows(st_a + kOffQ + (uint32_t)((hq * 128 + 32 * quarter) * kRowBytes), dq, sample_off, tokq);
                }
            mbar_arrive(bar_empty(s));       // the stage's rows and tables are not needed any more
        }
    } else if (warp >= kIssuerWarp) {
    // warpgroup 2 (issuer + loaders) gives registers back: one instruction for the whole warpgroup
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kRegsOther));
    if (warp != kIssuerWarp) {
        // ------------------------------------------------------------------ loaders
        const int lt = (warp - kLoaderWarp0) * 32 + lane;
        int kuse = 0, pending_s = -1;
        ItemCursor cur_it = cursor_init(cta_in_head, ctas_per_head, 1, g.Mw, g.Mh);
        for (long long it = cta_in_head; it < n_items; it += ctas_per_head, ++kuse, cursor_advance(cur_it, 1, g.Mw, g.Mh)) {
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
            const size_t sample_off = (size_t)x.b * HW;
            // slot metadata; the lse / delta gathers stay in flight while the row copies are issued below
            constexpr int kSlotIters = (kMaxSlots + kLoaderThreads - 1) / kLoaderThreads;
            float l2v[kSlotIters], dlv[kSlotIters];
            // Slots advance by a fixed step, so their window offsets (a, b) = (slot / width, slot mod width) are
            // carried along instead of divided out each time (a division is a long chain through the reciprocal unit).
            const int ew = PAD ? 16 : x.r.ew;               // slots per window row
            const int bw = x.r.ew;                          // PAD: offsets b >= bw hold no token
            const int q_s = kLoaderThreads / ew, r_s = kLoaderThreads - q_s * ew;              // slot loop: step of kLoaderThreads
            const int q_r = (kLoaderThreads / 4) / ew, r_r = (kLoaderThreads / 4) - q_r * ew;  // row loop: step of kLoaderThreads / 4
            int a_s = lt / ew, b_s = lt - a_s * ew;
#pragma unroll
            for (int i = 0; i < kSlotIters; ++i, a_s += q_s, b_s += r_s) {
                if (b_s >= ew) { b_s -= ew; ++a_s; }
                const int slot = lt + i * kLoaderThreads;
                l2v[i] = INFINITY;                       // no token: P = exp2(.. - inf) = 0
                dlv[i] = 0.f;
                if (slot >= kMaxSlots) continue;
                int code = 0, label = 0xff, tok = -1;
                if (slot < x.r.n && (!PAD || b_s < bw)) {
                    tok = offset_token_tc(g, x.r, a_s, b_s, cs, code, label);
                    const size_t li = (sample_off + (size_t)tok) * g.heads + head;
                    l2v[i] = __ldg(lse + li);
                    dlv[i] = __ldg(delta + li);
                } else if (PAD) {
                    code = a_s * cs + b_s;               // the slot's place in 16-wide geometry (see the kernel's header)
                }
                reinterpret_cast<int*>(st + kOffColOff)[slot] = 4 * code;
                reinterpret_cast<int*>(st + kOffLab)[slot] = label;
                reinterpret_cast<int*>(st + kOffTok)[slot] = tok;
            }
            // K and V rows of every key tile in use (rows without a token as zeros: they are MMA operands and
            // must stay finite); Q and dO rows up to the padded column count
            // Key rows are interleaved: with M = 4 * (tiles in use) 32-slot groups, lane l of elementwise warp
            // W = 4 t + qd (key row 128 t + 32 qd + l) holds slot 32 ((W + l) mod M) + l (see the bias-gradient updates).
            const int chunk = lt & 3;
            const int hc = head * kD + chunk * 8;
            const int nrows = x.ntiles * 128;
            const int M = 4 * x.ntiles;
            const int kc = key_interleave(PAD ? 16 : g.w, x.ntiles);
            int a_r = (lt >> 2) / ew, b_r = (lt >> 2) - a_r * ew;
            for (int row = lt >> 2; row < nrows; row += kLoaderThreads / 4, a_r += q_r, b_r += r_r) {
                if (b_r >= ew) { b_r -= ew; ++a_r; }
                const int kl = row & 31, kw = ((row >> 5) - kc * kl) & (M - 1), krow = 128 * (kw >> 2) + 32 * (kw & 3) + kl;
                const __nv_bfloat16 *sq = q, *sk = k, *sv = v, *sg = d_o;
                int bytes = 0;
                if (row < x.r.n && (!PAD || b_r < bw)) {
                    int code, label;
                    const int tok = offset_token_tc(g, x.r, a_r, b_r, cs, code, label);
                    const size_t t_abs = sample_off + (size_t)tok;
                    const size_t off = t_abs * g.ts + hc;
                    sq = q + off; sk = k + off; sv = v + off;
                    sg = d_o + t_abs * (g.heads * kD) + hc;            // dO is dense even where q, k, v are packed
                    bytes = 16;
                }
                const uint32_t so = st_a + tile_off<kD>(row, chunk), sok = st_a + tile_off<kD>(krow, chunk);
                cp_async16(sok + kOffK, sk, bytes);
                cp_async16(sok + kOffV, sv, bytes);
                if (row < x.npad) {
                    cp_async16(so + kOffQ, sq, bytes);
                    cp_async16(so + kOffDO, sg, bytes);
                }
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
        // ------------------------------------------------------------------ MMA issuer
        // The whole warp runs the loop (warp-uniform control flow and operands); one elected lane issues.
        // The CTA's blocks form one sequence across tiles and items: block J uses S / dP buffer J & 1, and its
        // S^T / dP^T are issued two blocks ahead (from the previous item's last blocks where needed, as soon as
        // the item's stage is loaded), so the elementwise warps find them ready.
        const uint32_t idesc_acc = make_idesc_elem(128, kD, 0, 1);   // A from TMEM, B = 16 rows x 32 (MN-major)
        const uint32_t idesc_dq = make_idesc_elem(128, kD, 1, 1);    // A = dS^T tile read transposed, B = 16 K rows x 32
        // shared-memory descriptors: one common high word, low words = start address (16-byte units)
        const uint32_t d_hi = sdesc_hi(make_sdesc_sw64(smem0, 512));
        const uint32_t d_q = sdesc_lo(make_sdesc_sw64(smem0 + kOffQ, 512)), d_k = sdesc_lo(make_sdesc_sw64(smem0 + kOffK, 512));
        const uint32_t d_v = sdesc_lo(make_sdesc_sw64(smem0 + kOffV, 512)), d_do = sdesc_lo(make_sdesc_sw64(smem0 + kOffDO, 512));
        const uint32_t d_ds = sdesc_lo(make_sdesc_sw64_mn(smem0 + kOffDS, kDSGroupBytes, 512));
        uint32_t ph_ds = 0;              // bit b: parity of the next completion of bar_ds(b)
        int J = 0;                       // number of the current block in the CTA's sequence
        int n_issued = 0;                // S^T / dP^T have been issued for blocks [0, n_issued)
        int kuse = 0, n_tile = 0;
        bool ok = true;
        // S^T = K Q^T and dP^T = V dO^T of query block b of key tile t (item in stage `stage`, npad_i columns) into buffer `buf`
        auto issue_sdp = [&](int stage, int npad_i, int t, int b, int buf) {
            const int ncols = min(CB, npad_i - b * CB);
            const uint32_t so = (uint32_t)((stage * kStageBytes) >> 4);
            const uint32_t ro = so + (uint32_t)((t * 128 * kRowBytes) >> 4), co = so + (uint32_t)((b * CB * kRowBytes) >> 4);
            const uint32_t idesc = make_idesc_elem(128, ncols, 0, 0);
            const uint32_t t_s = tmem_base + buf * kColBuf, t_dp = t_s + CB;
            if (elect_one()) {
                mma_ss_h<false>(t_s, d_k + ro, d_q + co, d_hi, idesc);
                mma_ss_h<true>(t_s, d_k + ro + 2, d_q + co + 2, d_hi, idesc);
                mma_ss_h<false>(t_dp, d_v + ro, d_do + co, d_hi, idesc);
                mma_ss_h<true>(t_dp, d_v + ro + 2, d_do + co + 2, d_hi, idesc);
                mma_commit(bar_sdp(buf));
            }
            __syncwarp();
        };
        ItemCursor nx_it = cursor_init(cta_in_head, ctas_per_head, 1, g.Mw, g.Mh);     // runs one item ahead
        int npad = 0, ntiles = 0, nblk = 1;
        if (cta_in_head < n_items) {
            const Item x = make_item(g, nx_it, PAD);
            npad = x.npad; ntiles = x.ntiles; nblk = x.nblk;
            cursor_advance(nx_it, 1, g.Mw, g.Mh);
        }
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, ++kuse) {
            const int s = kuse % kStages;
            const int nb = ntiles * nblk;
            // the item after this one
            int nb_n = 0, npad_n = 0, nblk_n = 1, ntiles_n = 0;
            if (it + ctas_per_head < n_items) {
                const Item xn = make_item(g, nx_it, PAD);
                cursor_advance(nx_it, 1, g.Mw, g.Mh);
                nb_n = xn.ntiles * xn.nblk; npad_n = xn.npad; nblk_n = xn.nblk; ntiles_n = xn.ntiles;
            }
            const int J0 = J;
            ok = mbar_wait_all(bar_full(s), (kuse / kStages) & 1, cta_abort);
            if (!ok) break;
            fence_proxy_async();
            tc_fence_after();
            // S / dP of blocks [n_issued, limit): blocks of this item, or of the next one (other stage, once it is loaded)
            auto issue_upto = [&](int limit) -> bool {
                for (int jt = n_issued; jt < limit; ++jt) {
                    int local = jt - J0;
                    if (local < nb) {
                        const int t = local >= nblk ? 1 : 0;
                        issue_sdp(s, npad, t, local - t * nblk, jt & 1);
                    } else {
                        local -= nb;
                        const int sn = (kuse + 1) % kStages;
                        if (!mbar_wait_all(bar_full(sn), ((kuse + 1) / kStages) & 1, cta_abort)) return false;
                        fence_proxy_async();
                        const int t = local >= nblk_n ? 1 : 0;
                        issue_sdp(sn, npad_n, t, local - t * nblk_n, jt & 1);
                    }
                }
                if (limit > n_issued) n_issued = limit;
                return true;
            };
            if (kuse == 0) ok = issue_upto(min(2, nb + nb_n));     // the first two blocks have no earlier block to be issued from
            const uint32_t so = (uint32_t)((s * kStageBytes) >> 4);
            for (int t = 0; t < ntiles && ok; ++t) {
                const int set = n_tile & 1;
                for (int b = 0; b < nblk; ++b, ++J) {
                    const int buf = J & 1;
                    const int nks = min(CB, npad - b * CB) >> 4;
                    ok = mbar_wait_all(bar_ds(buf), (ph_ds >> buf) & 1, cta_abort);          // all eight warps are done with block J
                    ph_ds ^= 1u << buf;
                    if (ok && b == 0 && n_tile >= 2)     // the accumulator set must have been read back (tile n_tile - 2)
                        ok = mbar_wait_all(bar_accfree(set), ((n_tile >> 1) - 1) & 1, cta_abort);
                    if (!ok) break;
                    tc_fence_after();
                    // dV += P^T dO, dK += dS^T Q over the block's query columns
                    if (elect_one()) {
                        const uint32_t a_dv = tmem_base + kColDV + 64 * set, a_dk = tmem_base + kColDK + 64 * set;
                        const uint32_t t_p = tmem_base + buf * kColBuf, t_dst = t_p + CB;
                        const uint32_t b_do = d_do + so + (uint32_t)((b * CB * kRowBytes) >> 4), b_q = d_q + so + (uint32_t)((b * CB * kRowBytes) >> 4);
                        if (b == 0) {
                            mma_ts_h<false>(a_dv, t_p, b_do, d_hi, idesc_acc);
                            mma_ts_h<false>(a_dk, t_dst, b_q, d_hi, idesc_acc);
                        } else {
                            mma_ts_h<true>(a_dv, t_p, b_do, d_hi, idesc_acc);
                            mma_ts_h<true>(a_dk, t_dst, b_q, d_hi, idesc_acc);
                        }
                        if (nks == 4) {
                            mma_ts_h<true>(a_dv, t_p + 16, b_do + 64, d_hi, idesc_acc);
                            mma_ts_h<true>(a_dk, t_dst + 16, b_q + 64, d_hi, idesc_acc);
                            mma_ts_h<true>(a_dv, t_p + 32, b_do + 128, d_hi, idesc_acc);
                            mma_ts_h<true>(a_dk, t_dst + 32, b_q + 128, d_hi, idesc_acc);
                            mma_ts_h<true>(a_dv, t_p + 48, b_do + 192, d_hi, idesc_acc);
                            mma_ts_h<true>(a_dk, t_dst + 48, b_q + 192, d_hi, idesc_acc);
                        } else {
                            for (int ks = 1; ks < nks; ++ks) {
                                mma_ts_h<true>(a_dv, t_p + 16 * ks, b_do + 64 * ks, d_hi, idesc_acc);
                                mma_ts_h<true>(a_dk, t_dst + 16 * ks, b_q + 64 * ks, d_hi, idesc_acc);
                            }
                        }
                    }
                    __syncwarp();
                    if ((b & 1) || b == nblk - 1) {
                        // dQ (queries of this pair of blocks) += dS K over the tile's keys
                        if (t == 0 && b < 2 && kuse > 0) {   // the item's first write of dQ: the previous item's was read
                            ok = mbar_wait_all(bar_dqfree, (kuse - 1) & 1, cta_abort);
                            if (!ok) break;
                            tc_fence_after();
                        }
                        if (elect_one()) {
                            const uint32_t a_dq = tmem_base + kColDQ + 32 * (b >> 1);
                            const uint32_t b_k = d_k + so + (uint32_t)((t * 128 * kRowBytes) >> 4);
                            if (t == 0) mma_ss_h<false>(a_dq, d_ds, b_k, d_hi, idesc_dq);
                            else mma_ss_h<true>(a_dq, d_ds, b_k, d_hi, idesc_dq);
#pragma unroll
                            for (int ks = 1; ks < 8; ++ks)     // all 8 key steps: the interleaved key order spreads the keys over all rows
                                mma_ss_h<true>(a_dq, d_ds + 64 * ks, b_k + 64 * ks, d_hi, idesc_dq);
                            mma_commit(bar_dsfree);
                            if (b == nblk - 1) {
                                mma_commit(bar_acc(set));                  // the tile's dV / dK (and the dQ MMAs, which read its K rows)
                                if (t == ntiles - 1) mma_commit(bar_dq);   // the item's last MMAs
                            }
                        }
                        __syncwarp();
                    }
                    // S^T / dP^T two blocks ahead (this buffer is free again: its P / dS reads were issued above).  They
                    // come after the dQ MMAs: the elementwise warps need the shared dS tile back one block from
                    // now, the new S / dP only two blocks from now.
                    ok = issue_upto(min(J + 3, J0 + nb + nb_n));
                    if (!ok) break;
                }
                ++n_tile;
            }
            npad = npad_n; ntiles = ntiles_n; nblk = nblk_n;     // the next item becomes the current one
        }
    }
    } else {
        // ------------------------------------------------------------------ elementwise warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kRegsWork));
        const int h = warp >> 2;                 // which 16-column steps of a block: h and h + 2
        const int quarter = warp & 3;            // TMEM lane quarter = 32 key rows of the tile
        const uint32_t lane_addr = ((uint32_t)(32 * quarter)) << 16;
        const float scale = g.scale_log2e;
        int kuse = 0, n_pair = 0;
        uint32_t ph_sdp = 0;             // bit b: parity of the next completion of bar_sdp(b)
        bool ok = true;
        int J = 0;                       // number of this block in the CTA's sequence; its S / dP buffer is J & 1
        ItemCursor cur_it = cursor_init(cta_in_head, ctas_per_head, 1, g.Mw, g.Mh);
        for (long long it = cta_in_head; ok && it < n_items; it += ctas_per_head, ++kuse, cursor_advance(cur_it, 1, g.Mw, g.Mh)) {
            const Item x = make_item(g, cur_it, PAD);
            const int s = kuse % kStages;
            const uint32_t st_a = smem0 + s * kStageBytes;
            if (!mbar_wait_all(bar_full(s), (kuse / kStages) & 1, cta_abort)) break;
            for (int t = 0; t < x.ntiles && ok; ++t) {
                const int krow = 32 * quarter + lane;            // key row inside the tile
                const int M = 4 * x.ntiles;
                const int slot = 32 * ((4 * t + quarter + key_interleave(PAD ? 16 : g.w, x.ntiles) * lane) & (M - 1)) + lane;     // interleaved key order
                // Bias-gradient updates.  In a full-width window (width = w) the bias code of a slot is the slot
                // number plus 32 per window row, so code mod 32 = slot mod 32 = lane: the 32 updates of one warp
                // instruction (32 keys, one query) fall into 32 different banks and entries.  If w also divides 32
                // (window rows never straddle a 32-slot group), two keys of a warp in the same window row lie in
                // the same group with lanes congruent mod M, i.e. >= M slots = codes apart, keys in different rows
                // are >= 33 codes apart, and G <= min(M, w) consecutive queries of a group aligned to G sit in one
                // window row 1 .. G - 1 codes apart: the 32 x G updates of such a query group never meet and are
                // issued together.  For sides that do not divide 32 the slots 32 g - 1 and 32 g (lanes 31 and 0 of one
                // warp under c = 1) may share a window row; with c = 5 and two tiles (M = 8) any two lanes of a warp
                // hold slots at least 5 apart, and groups of 4 queries are collision-free for every full-width
                // window of side 9 .. 16 (checked exhaustively on the host over all heights; the parity tests cover
                // sides 12 and 14).  Other windows are updated one query at a time.
                int rmw_mode = 1;
                if (!PAD && x.r.ew == g.w && g.w >= 4) {
                    if ((32 % g.w) == 0) rmw_mode = (M == 8 && g.w >= 8) ? 8 : 4;
                    else if (M == 8) rmw_mode = 4;
                }
                // full 16 x 16 window: update groups of 8 apply as well; PAD: every two-tile window without mask labels
                const bool row16 = PAD ? (M == 8 && !x.masked && x.r.ew == PADW) : (g.w == 16 && x.r.n == 256 && !x.masked);
                const int coloff_i = lds_i32(st_a + kOffColOff + 4 * slot);
                const int tok = lds_i32(st_a + kOffTok + 4 * slot);
                RowCtx rc;
                rc.label = lds_i32(st_a + kOffLab + 4 * slot);
                rc.valid = tok >= 0;
                // bias index = code_query - code_key + c0; a key row without a token reads the table's -inf zone
                rc.bias_row = smem0 + kOffBias + (rc.valid ? 4 * c0 - coloff_i : 4 * (2 * c0 + 1));
                rc.dbias_row = smem0 + kOffDBias + 4 * (warp * kDBiasFloats + c0 + (PAD ? dbias_margin(g.w) : 0)) - coloff_i;
                rc.scratch = smem0 + kOffDBias + 4 * (warp * kDBiasFloats + kDBiasEntries + lane);
                for (int b = 0; b < x.nblk; ++b) {
                    const int buf = J & 1;
                    const int nsteps = min(CB, x.npad - b * CB) >> 4;
                    const bool has_a = h < nsteps, has_b = h + 2 < nsteps;
                    ok = mbar_wait_all(bar_sdp(buf), (ph_sdp >> buf) & 1, cta_abort);
                    if (!ok) break;
                    ph_sdp ^= 1u << buf;
                    tc_fence_after();
                    const uint32_t t_s = tmem_base + lane_addr + buf * kColBuf, t_dp = t_s + CB;
                    // step h: load, compute, write back; the loads of step h + 2 are in flight during the
                    // bias-gradient updates of step h
                    uint32_t sa[16], pa[16], pk_p[8], pk_dsa[8], pk_dsb[8], addr[16];
                    float ds[16];
                    const int ca = b * CB + 16 * h, cb2 = ca + 32;
                    if (row16 && PAD) {
                        if (has_a) pad_block16<PAD ? PADW : 15>(t_s, t_dp, h, ca, cb2, cs, has_b, rc, st_a, scale, pk_dsa, pk_dsb);
                    } else if (row16) {
                        // full 16 x 16 window (four steps per block, no mask): one window row per step
                        tmem_ld16(t_s + 16 * h, sa);
                        tmem_ld16(t_dp + 16 * h, pa);
                        tmem_ld_wait();
                        float bv[16], l2[16], dl[16];
                        const int code_a = 4 * cs * (ca >> 4), code_b = 4 * cs * (cb2 >> 4);
                        load16_row(ca, code_a, rc, st_a, bv, l2, dl);
                        math16_row(sa, pa, bv, l2, dl, scale, pk_p, pk_dsa, ds);
                        uint32_t a0 = rc.dbias_row + code_a;
                        tmem_st8(t_s + 16 * h, pk_p);
                        tmem_st8(t_dp + 16 * h, pk_dsa);
                        tmem_ld16(t_s + 16 * (h + 2), sa);
                        tmem_ld16(t_dp + 16 * (h + 2), pa);
                        load16_row(cb2, code_b, rc, st_a, bv, l2, dl);       // the second step's table values, in flight during the updates
                        rmw8_consecutive_f32(a0, &ds[0]);
                        rmw8_consecutive_f32(a0 + 32, &ds[8]);
                        tmem_ld_wait();
                        math16_row(sa, pa, bv, l2, dl, scale, pk_p, pk_dsb, ds);
                        a0 = rc.dbias_row + code_b;
                        tmem_st8(t_s + 16 * (h + 2), pk_p);
                        tmem_st8(t_dp + 16 * (h + 2), pk_dsb);
                        rmw8_consecutive_f32(a0, &ds[0]);
                        rmw8_consecutive_f32(a0 + 32, &ds[8]);
                    } else if (has_a) {
                        tmem_ld16(t_s + 16 * h, sa);
                        tmem_ld16(t_dp + 16 * h, pa);
                        tmem_ld_wait();
                        if (x.masked) cols16<true, true>(sa, pa, ca, rc, st_a, scale, pk_p, pk_dsa, ds, addr);
                        else if (x.ragged) cols16<false, true>(sa, pa, ca, rc, st_a, scale, pk_p, pk_dsa, ds, addr);
                        else cols16<false, false>(sa, pa, ca, rc, st_a, scale, pk_p, pk_dsa, ds, addr);
                        tmem_st8(t_s + 16 * h, pk_p);
                        tmem_st8(t_dp + 16 * h, pk_dsa);
                        if (has_b) {
                            tmem_ld16(t_s + 16 * (h + 2), sa);
                            tmem_ld16(t_dp + 16 * (h + 2), pa);
                        }
                        dbias_add16(rmw_mode, addr, ds);
                    }
                    if (has_b && !row16) {
                        tmem_ld_wait();
                        if (x.masked) cols16<true, true>(sa, pa, cb2, rc, st_a, scale, pk_p, pk_dsb, ds, addr);
                        else if (x.ragged) cols16<false, true>(sa, pa, cb2, rc, st_a, scale, pk_p, pk_dsb, ds, addr);
                        else cols16<false, false>(sa, pa, cb2, rc, st_a, scale, pk_p, pk_dsb, ds, addr);
                        tmem_st8(t_s + 16 * (h + 2), pk_p);
                        tmem_st8(t_dp + 16 * (h + 2), pk_dsb);
                        dbias_add16(rmw_mode, addr, ds);
                    }
                    // dS^T into the shared tile of this pair of blocks (32-query groups 2 (b & 1) and 2 (b & 1) + 1;
                    // step h -> group 2 (b & 1), step h + 2 -> the next group; 16-byte chunks 2 h and 2 h + 1)
                    if ((b & 1) == 0 && n_pair > 0) {
                        ok = mbar_wait_all(bar_dsfree, (n_pair - 1) & 1, cta_abort);
                        if (!ok) break;
                    }
                    {
                        const uint32_t base = smem0 + kOffDS + 2 * (b & 1) * kDSGroupBytes;
                        if (has_a) {
                            sts_u4(base + tile_off<kD>(krow, 2 * h), pk_dsa[0], pk_dsa[1], pk_dsa[2], pk_dsa[3]);
                            sts_u4(base + tile_off<kD>(krow, 2 * h + 1), pk_dsa[4], pk_dsa[5], pk_dsa[6], pk_dsa[7]);
                        }
                        if (has_b) {
                            sts_u4(base + kDSGroupBytes + tile_off<kD>(krow, 2 * h), pk_dsb[0], pk_dsb[1], pk_dsb[2], pk_dsb[3]);
                            sts_u4(base + kDSGroupBytes + tile_off<kD>(krow, 2 * h + 1), pk_dsb[4], pk_dsb[5], pk_dsb[6], pk_dsb[7]);
                        }
                    }
                    if ((b & 1) || b == x.nblk - 1) ++n_pair;
                    tmem_st_wait();
                    tc_fence_before();
                    fence_proxy_async();
                    mbar_arrive(bar_ds(buf));
                    ++J;
                }
                if (!ok) break;
            }
        }
    }

    // teardown: every role ends up here, also after an expired wait
    cp_async_wait<0>();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == kIssuerWarp) tmem_dealloc(tmem_base, 512);
    {
        // this CTA's table = sum of its warps' tables (fixed order), written to the CTA's slot of the workspace
        const float* tbl = reinterpret_cast<const float*>(smem + kOffDBias);
        for (int e = tid; e < kDBiasFloats; e += kThreads) {
            float acc = 0.f;
#pragma unroll
            for (int wq = 0; wq < 8; ++wq) acc += tbl[wq * kDBiasFloats + e];
            dbias_parts[(size_t)blockIdx.x * kDBiasFloats + e] = acc;       // (PAD: the table starts dbias_margin(w) floats in)
        }
    }
    if (tid == 0 && *cta_abort) atomicExch(&g_bwd_tc_timeout, 1);
}

// dbias[(da, db), head] = sum over the head's CTAs of their tables (entry (da + w - 1) * cs + (db + w - 1)).
// Fixed summation order over warps and CTAs: the bias gradient is reproducible run to run.
__global__ void __launch_bounds__(256)
swin_bwd_dbias_finalize_kernel(const float* __restrict__ parts, float* __restrict__ dbias, int w, int heads, int ctas_per_head,
                               int margin, int cs) {
    const int nw = 2 * w - 1;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;       // (table row, head)
    if (i >= nw * nw * heads) return;
    const int head = i % heads, r = i / heads;
    const int e = margin + (r / nw) * cs + (r % nw);
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

#ifndef TERRA_ELEM_F16
bool bwd_tc_supported(const Geo& g) { return g.d == 32 && g.nmax <= kMaxSlots && g.w <= 16 && g.heads <= 148; }

// workspace: delta [B*H*W*heads] fp32, the prepared bias tables [heads * kFwdBiasFloats] fp32, one
// bias-gradient table per CTA
size_t bwd_tc_workspace_bytes(const Geo& g) {
    const size_t delta = (((size_t)g.B * g.H * g.W * g.heads * sizeof(float)) + 255) / 256 * 256;
    return delta + (size_t)g.heads * kFwdBiasFloats * sizeof(float) + (size_t)kMaxGrid * kDBiasFloats * sizeof(float);
}
#endif  // !TERRA_ELEM_F16

cudaError_t launch_bwd_tc(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                          const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, float* dbias,
                          void* workspace, int sm_count, cudaStream_t stream) {
    float* delta = reinterpret_cast<float*>(workspace);
    const size_t delta_bytes = (((size_t)g.B * g.H * g.W * g.heads * sizeof(float)) + 255) / 256 * 256;
    float* prep = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) + delta_bytes);
    cudaError_t e = TERRA_ELEM_FN(launch_bwd_delta)(g, o, d_o, delta, stream);
    if (e != cudaSuccess) return e;
    e = launch_bias_prep(g, bias, prep, stream);
    if (e != cudaSuccess) return e;
    float* parts = prep + (size_t)g.heads * kFwdBiasFloats;
    const long long items = (long long)g.B * g.Mh * g.Mw;
    long long cph = (sm_count < kMaxGrid ? sm_count : kMaxGrid) / g.heads;
    if (cph < 1) cph = 1;
    if (cph > items) cph = items;
    const unsigned grid = (unsigned)(cph * g.heads);
    const bool pad = pad16_layout(g);       // window sides 9 .. 15: 16 slots per window row
    auto kern = swin_bwd_fused_kernel<0>;
    if (pad) {
        switch (g.w) {
            case 9: kern = swin_bwd_fused_kernel<9>; break;
            case 10: kern = swin_bwd_fused_kernel<10>; break;
            case 11: kern = swin_bwd_fused_kernel<11>; break;
            case 12: kern = swin_bwd_fused_kernel<12>; break;
            case 13: kern = swin_bwd_fused_kernel<13>; break;
            case 14: kern = swin_bwd_fused_kernel<14>; break;
            default: kern = swin_bwd_fused_kernel<15>; break;
        }
    }
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    prof_begin("swin_bwd_fused_kernel", stream);
    kern<<<grid, kThreads, kSmemBytes, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, prep, lse, delta,
        (__nv_bfloat16*)dq, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, parts, items, (int)cph);
    count_launch(stream);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int nrows = (2 * g.w - 1) * (2 * g.w - 1) * g.heads;
    swin_bwd_dbias_finalize_kernel<<<(nrows + 255) / 256, 256, 0, stream>>>(parts, dbias, g.w, g.heads, (int)cph, pad ? dbias_margin(g.w) : 0,
                                                                            pad ? 48 : g.w + 32);
    count_launch(stream);
    return cudaGetLastError();
}

}  // namespace terra
