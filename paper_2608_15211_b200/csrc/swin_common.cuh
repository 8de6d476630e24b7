// Shared device-side definitions of the shifted-window attention kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace terra {

// Window geometry of one call, resolved on the host (paper Section IV-D symbols).
struct Geo {
    int B, H, W;          // batch, token grid (H_T x W_T)
    int heads, d;         // heads, head dim
    int ts;               // elements between consecutive tokens of q, k, v (and of dq, dk, dv): heads * d for separate
                          // dense tensors, 3 * heads * d for the packed [B, H, W, 3, heads, d] layout; o, dO, lse are dense
    int w;                // window side
    int sh, sw;           // shifts, already reduced mod H / mod W
    int ph, pw;           // periodic flags
    int Mh, Mw;           // window grid: ceil(H / w) x ceil(W / w)
    int nmax;             // tokens in a full window: min(w, H) * min(w, W)
    int f16;              // activations and gradients are fp16 instead of bf16 (the paper trains in fp16 mixed precision)
    float scale_log2e;    // score scale * log2(e)
};

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Per-slot metadata packed in one int: bias code a * (2w - 1) + b in the low 16 bits, the shift-mask
// label in bits 16..17.  bias row of (query i, key j) = code_i - code_j + (w - 1) * 2w.
__device__ __forceinline__ int meta_code(int m) { return m & 0xffff; }
__device__ __forceinline__ int meta_label(int m) { return m >> 16; }

// it = quo * div + rem.  Item numbers almost always fit 32 bits, where the division is a handful of
// instructions; the 64-bit one (a long software routine) is kept for the sizes that need it.
__device__ __forceinline__ void split_item(long long it, int div, long long& quo, int& rem) {
    if (((unsigned long long)it >> 32) == 0) {
        const unsigned i = (unsigned)it, q = i / (unsigned)div;
        quo = q;
        rem = (int)(i - q * (unsigned)div);
    } else {
        quo = it / div;
        rem = (int)(it - quo * div);
    }
}

struct WindowRef {
    int wr, wc;   // window row / column
    int eh, ew;   // true extent (truncated at the last row / column)
    int n;        // eh * ew
};

__device__ __forceinline__ WindowRef window_ref(const Geo& g, int win) {
    WindowRef r;
    r.wr = win / g.Mw;
    r.wc = win - r.wr * g.Mw;
    r.eh = min(g.w, g.H - r.wr * g.w);
    r.ew = min(g.w, g.W - r.wc * g.w);
    r.n = r.eh * r.ew;
    return r;
}

__device__ __forceinline__ WindowRef window_ref_rc(const Geo& g, int wr, int wc) {
    WindowRef r;
    r.wr = wr;
    r.wc = wc;
    r.eh = min(g.w, g.H - wr * g.w);
    r.ew = min(g.w, g.W - wc * g.w);
    r.n = r.eh * r.ew;
    return r;
}

// A persistent CTA's items are it0, it0 + step, it0 + 2 step, ...  The item number is kept as mixed-radix
// digits (head | window column | window row | sample, fastest first; radix of the head digit 1 where the head
// is fixed), and going to the next item adds the step's digits with carries: no division per item (an integer
// division is a long dependent chain through the reciprocal unit, which the softmax warps keep busy).
struct ItemCursor {
    int head, wc, wr, b;
    int s_head, s_wc, s_wr, s_b;
};
__device__ __forceinline__ void cursor_digits(long long it, int heads_radix, int Mw, int Mh, int& head, int& wc, int& wr, int& b) {
    long long rest, rest2, rest3;
    split_item(it, heads_radix, rest, head);
    split_item(rest, Mw, rest2, wc);
    split_item(rest2, Mh, rest3, wr);
    b = (int)rest3;
}
__device__ __forceinline__ ItemCursor cursor_init(long long it0, long long step, int heads_radix, int Mw, int Mh) {
    ItemCursor c;
    cursor_digits(it0, heads_radix, Mw, Mh, c.head, c.wc, c.wr, c.b);
    cursor_digits(step, heads_radix, Mw, Mh, c.s_head, c.s_wc, c.s_wr, c.s_b);
    return c;
}
__device__ __forceinline__ void cursor_advance(ItemCursor& c, int heads_radix, int Mw, int Mh) {
    c.head += c.s_head;
    int carry = c.head >= heads_radix;
    c.head -= carry ? heads_radix : 0;
    c.wc += c.s_wc + carry;
    carry = c.wc >= Mw;
    c.wc -= carry ? Mw : 0;
    c.wr += c.s_wr + carry;
    carry = c.wr >= Mh;
    c.wr -= carry ? Mh : 0;
    c.b += c.s_b + carry;
}

// Slot of a window -> grid token u * W + v (undoing the roll) and packed metadata.
__device__ __forceinline__ int slot_token(const Geo& g, const WindowRef& r, int slot, int& meta) {
    int a = slot / r.ew;
    int b = slot - a * r.ew;
    int u = r.wr * g.w + a + g.sh;
    if (u >= g.H) u -= g.H;
    int v = r.wc * g.w + b + g.sw;
    if (v >= g.W) v -= g.W;
    int label = ((!g.ph && u < g.sh) ? 2 : 0) + ((!g.pw && v < g.sw) ? 1 : 0);
    meta = (a * (2 * g.w - 1) + b) | (label << 16);
    return u * g.W + v;
}

// ---- small PTX wrappers -----------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// 16-byte async copy; src_bytes = 0 writes zeros (used for rows past the window's end).
// 4-byte asynchronous copy (lse, delta values that travel with a tile's rows)
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// D (16x8, fp32) += A (16x16, fp16, row) * B (16x8, fp16, col)
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// The kernel files are compiled twice, for bf16 and (with TERRA_ELEM_F16 defined by a one-line wrapper file) for fp16
// activations: same code, the element type enters through these operations, the tcgen05 instruction descriptor's
// operand formats (make_idesc_elem) and the name suffix.
#ifdef TERRA_ELEM_F16
#define TERRA_ELEM_FN(name) name##_f16
#define mma_elem mma_f16
#define pack_elem pack_f16
#define kElemOnesPair 0x3C003C00u         /* two fp16 ones */
__device__ __forceinline__ float2 elem2_to_float2(uint32_t v) { return __half22float2(*reinterpret_cast<const __half2*>(&v)); }
#else
#define TERRA_ELEM_FN(name) name
#define mma_elem mma_bf16
#define pack_elem pack_bf16
#define kElemOnesPair 0x3F803F80u         /* two bf16 ones */
__device__ __forceinline__ float2 elem2_to_float2(uint32_t v) { return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v)); }
#endif
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory tile of bf16 rows, D elements each, 16-byte chunks XOR-swizzled so that ldmatrix
// over 8 consecutive rows touches every bank once.  Returns the byte offset of (row, chunk).
template <int D>
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    constexpr int CPR = D / 8;                       // 16-byte chunks per row: 4 (d=32) or 8 (d=64)
    int sw = (CPR == 4) ? ((row >> 1) & 3) : (row & 7);
    return static_cast<uint32_t>(row * (D * 2) + ((chunk ^ sw) << 4));
}

}  // namespace terra
