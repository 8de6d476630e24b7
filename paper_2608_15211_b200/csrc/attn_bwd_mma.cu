// Backward shifted-window attention, register-tile path (warp-level mma.sync).
// The file is compiled for bf16 and, through attn_bwd_mma_f16.cu, for fp16 activations.
//
// Three launches: (1) delta = rowsum(dO * O); (2) key-tile CTAs produce dK and dV; (3) query-tile
// CTAs produce dQ and the relative-position-bias gradient.  (2) and (3) are one kernel template: a
// CTA owns 64 rows of one side of the window (keys or queries), streams the other side through
// shared memory in 64-row blocks, recomputes P from the saved log-sum-exp and forms
// dS = P * (dP - delta).  No atomics touch dQ / dK / dV, so those are reproducible run to run.
// Bias gradient: a query-tile CTA is persistent and bound to one (head, query tile).  For full-width
// windows the position of a (query, key) pair inside the tile decides its table row, whatever the
// window, so the CTA first adds dS element by element into a 64 x n shared-memory image that it owns
// (no atomics, no conflicts) over all its windows, and bins that image into the (2w-1)^2 table once at
// the end.  Narrow edge windows, and windows too large for the image, add straight into the table with
// shared-memory atomics.  Each CTA then flushes its table with global atomics.
#include "swin_common.cuh"
#include "swin_kernels.h"

namespace terra {

namespace {

constexpr int BM = 64;
constexpr int BN = 64;
constexpr int NTHREADS = 128;

template <int D>
__device__ __forceinline__ void load_rows(unsigned char* s_tile, const __nv_bfloat16* base, const int* s_tok,
                                          int slot0, size_t sample_off, int tstride, int head, int tid) {
    constexpr int CPR = D / 8;
    for (int idx = tid; idx < BN * CPR; idx += NTHREADS) {
        int row = idx / CPR, chunk = idx - row * CPR;
        int tok = s_tok[slot0 + row];
        const __nv_bfloat16* src = base;
        int bytes = 0;
        if (tok >= 0) {
            src = base + (sample_off + (size_t)tok) * tstride + head * D + chunk * 8;
            bytes = 16;
        }
        cp_async16(smem_u32(s_tile + tile_off<D>(row, chunk)), src, bytes);
    }
}

// Head dim 128: the fragments of the CTA's own rows (two operands x 8 k-steps) and two 16 x 128 accumulators do not
// fit the register file together, so the own-row fragments are re-read from their shared-memory tiles at each use.
template <int D>
constexpr bool kFragsInRegs = D <= 64;

// acc (16 x 64 per warp) = own rows x streamed block^T; the own rows' fragments come from registers (af) or, for
// head dim 128, from their shared-memory tile (own)
template <int D>
__device__ __forceinline__ void rows_times_block_t(float (&acc)[BN / 8][4], const uint32_t (&af)[kFragsInRegs<D> ? D / 16 : 1][4],
                                                   const unsigned char* own, const unsigned char* blk, int warp, int lane) {
#pragma unroll
    for (int i = 0; i < BN / 8; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
        uint32_t a[4];
        if constexpr (kFragsInRegs<D>) {
            a[0] = af[ks][0]; a[1] = af[ks][1]; a[2] = af[ks][2]; a[3] = af[ks][3];
        } else {
            const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            ldmatrix_x4(a, smem_u32(own + tile_off<D>(row, 2 * ks + (lane >> 4))));
        }
#pragma unroll
        for (int np = 0; np < BN / 16; ++np) {
            uint32_t bf[4];
            int r = np * 16 + (lane & 7) + (lane >> 4) * 8;
            ldmatrix_x4(bf, smem_u32(blk + tile_off<D>(r, 2 * ks + ((lane >> 3) & 1))));
            mma_elem(acc[2 * np], a, bf[0], bf[1]);
            mma_elem(acc[2 * np + 1], a, bf[2], bf[3]);
        }
    }
}

// out (16 x D per warp) += coef (16 x 64, fp32 fragments, rounded to bf16) x streamed block (64 x D)
template <int D>
__device__ __forceinline__ void coef_times_block(float (&out)[D / 8][4], const float (&coef)[BN / 8][4],
                                                 const unsigned char* blk, int lane) {
#pragma unroll
    for (int ks = 0; ks < BN / 16; ++ks) {
        uint32_t pf[4];
        pf[0] = pack_elem(coef[2 * ks][0], coef[2 * ks][1]);
        pf[1] = pack_elem(coef[2 * ks][2], coef[2 * ks][3]);
        pf[2] = pack_elem(coef[2 * ks + 1][0], coef[2 * ks + 1][1]);
        pf[3] = pack_elem(coef[2 * ks + 1][2], coef[2 * ks + 1][3]);
#pragma unroll
        for (int dp = 0; dp < D / 16; ++dp) {
            uint32_t bf[4];
            int r = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            ldmatrix_x4_trans(bf, smem_u32(blk + tile_off<D>(r, 2 * dp + (lane >> 4))));
            mma_elem(out[2 * dp], pf, bf[0], bf[1]);
            mma_elem(out[2 * dp + 1], pf, bf[2], bf[3]);
        }
    }
}

template <int D>
__device__ __forceinline__ void stage_rows(unsigned char* tile, const float (&acc)[D / 8][4], float mul,
                                           int warp, int gq, int tq) {
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
        int lr = warp * 16 + gq;
        *reinterpret_cast<uint32_t*>(tile + tile_off<D>(lr, i) + tq * 4) = pack_elem(acc[i][0] * mul, acc[i][1] * mul);
        *reinterpret_cast<uint32_t*>(tile + tile_off<D>(lr + 8, i) + tq * 4) = pack_elem(acc[i][2] * mul, acc[i][3] * mul);
    }
}

template <int D>
__device__ __forceinline__ void scatter_rows(const unsigned char* tile, __nv_bfloat16* dst, const int* s_tok, int slot0,
                                             int n, size_t sample_off, int tstride, int head, int tid) {
    constexpr int CPR = D / 8;
    for (int idx = tid; idx < BM * CPR; idx += NTHREADS) {
        int row = idx / CPR, chunk = idx - row * CPR;
        int slot = slot0 + row;
        if (slot < n) {
            uint4 val = *reinterpret_cast<const uint4*>(tile + tile_off<D>(row, chunk));
            *reinterpret_cast<uint4*>(dst + (sample_off + (size_t)s_tok[slot]) * tstride + head * D + chunk * 8) = val;
        }
    }
}

// KV = true : CTA owns 64 keys   (own tiles K, V;  streams Q, dO) -> dK, dV
// KV = false: CTA owns 64 queries (own tiles Q, dO; streams K, V) -> dQ, dBias
constexpr int kStageStride = 40;   // floats per row of the dS staging tile (32 columns used)

// BIG = windows of more than 1024 tokens (window sides 33 .. 128): the slot tables cover the CTA's own 64 rows plus
// the streamed block in flight (two stages) instead of the whole window, the bias is read from the caller's table in
// global memory, and the bias gradient goes to global memory with atomics (summed over diagonals first where the
// window is complete along its width).
template <int D, bool KV, bool BIG>
__global__ void __launch_bounds__(NTHREADS)
swin_bwd_mma_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ d_o,
                    const float* __restrict__ bias, const float* __restrict__ lse, const float* __restrict__ delta,
                    __nv_bfloat16* __restrict__ out1, __nv_bfloat16* __restrict__ out2, float* __restrict__ dbias,
                    int tiles, int ctas_per_group, int acc_stride) {
    constexpr int KS = D / 16;
    constexpr int DT = D / 8;
    constexpr int TILE_BYTES = BN * D * 2;
    extern __shared__ __align__(128) unsigned char smem[];

    const int nbias = (2 * g.w - 1) * (2 * g.w - 1);
    const int npad_max = ((g.nmax + BN - 1) / BN) * BN;
    // tables: small windows [npad_max] slots of the window; BIG: [0, 64) the CTA's own rows, [64, 192) two streamed blocks
    const int ntab = BIG ? 3 * BN : npad_max;
    int* s_tok = reinterpret_cast<int*>(smem);
    int* s_meta = s_tok + ntab;
    float* s_lse = reinterpret_cast<float*>(s_meta + ntab);
    float* s_delta = s_lse + ntab;
    float* s_bias = s_delta + ntab;
    float* s_dbias = s_bias + (BIG ? 0 : nbias);
    unsigned char* s_r1 = smem + (((size_t)ntab * 16 + (BIG ? 0 : (size_t)nbias * 8) + 127) / 128) * 128;
    unsigned char* s_r2 = s_r1 + TILE_BYTES;
    unsigned char* s_c1 = s_r2 + TILE_BYTES;          // two stages
    unsigned char* s_c2 = s_c1 + 2 * TILE_BYTES;      // two stages
    float* s_acc = reinterpret_cast<float*>(s_c2 + 2 * TILE_BYTES);   // 64 x acc_stride image of summed dS (query tiles only)
    float* s_stage = s_acc + BM * acc_stride;                         // 4 warps x 16 x kStageStride staging tile (query tiles only)

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    // KV: group = head, the CTA walks (batch, window, tile).  Query side: group = (head, tile), the CTA
    // walks (batch, window), so one CTA always sees the same rows of a window.
    const int groups = KV ? g.heads : g.heads * tiles;
    const int group = blockIdx.x % groups;
    const int head = KV ? group : group / tiles;
    const int fixed_tile = KV ? 0 : group % tiles;
    const int M = g.Mh * g.Mw;
    const int c0 = (g.w - 1) * 2 * g.w;
    const long long n_items = KV ? (long long)g.B * M * tiles : (long long)g.B * M;
    const bool use_acc = !KV && acc_stride > 0;

    const __nv_bfloat16* own1 = KV ? k : q;
    const __nv_bfloat16* own2 = KV ? v : d_o;
    const __nv_bfloat16* str1 = KV ? q : k;
    const __nv_bfloat16* str2 = KV ? d_o : v;
    // token strides: q, k, v and the gradients may be slices of a packed tensor; dO is dense
    const int ts_own2 = KV ? g.ts : g.heads * D, ts_str2 = KV ? g.heads * D : g.ts;

    if (!BIG)
        for (int i = tid; i < nbias; i += NTHREADS) {
            s_bias[i] = bias[(size_t)i * g.heads + head] * kLog2e;
            s_dbias[i] = 0.f;
        }
    if (use_acc)
        for (int i = tid; i < BM * acc_stride; i += NTHREADS) s_acc[i] = 0.f;

    for (long long item = blockIdx.x / groups; item < n_items; item += ctas_per_group) {
        const int tile = KV ? (int)(item % tiles) : fixed_tile;
        const int win = KV ? (int)((item / tiles) % M) : (int)(item % M);
        const int b = KV ? (int)(item / ((long long)tiles * M)) : (int)(item / M);
        const WindowRef r = window_ref(g, win);
        const int r0 = tile * BM;
        if (r0 >= r.n) continue;
        const int nblk = (r.n + BN - 1) / BN;
        const int npad = nblk * BN;
        const size_t sample_off = (size_t)b * g.H * g.W;

        __syncthreads();   // previous item's readers of the slot tables and tiles are done
        // fills `count` table entries at `base` with the window's slots first .. first + count - 1
        auto fill_table = [&](int base, int first, int count) {
            for (int i = tid; i < count; i += NTHREADS) {
                const int sl = first + i;
                int meta = 0xff << 16, tok = -1;
                float l2 = INFINITY, dl = 0.f;      // padded queries: P = exp2(x - inf) = 0
                if (sl < r.n) {
                    tok = slot_token(g, r, sl, meta);
                    size_t li = (sample_off + (size_t)tok) * g.heads + head;
                    l2 = lse[li] * kLog2e;
                    dl = delta[li];
                }
                s_tok[base + i] = tok;
                s_meta[base + i] = meta;
                s_lse[base + i] = l2;
                s_delta[base + i] = dl;
            }
        };
        if (BIG) {
            fill_table(0, r0, BM);
            fill_table(BM, 0, BN);
        } else {
            fill_table(0, 0, npad);
        }
        __syncthreads();
        // table index of the CTA's own rows / of the rows of streamed block blk
        const int obase = BIG ? 0 : r0;
        auto cbase = [&](int blk) { return BIG ? BM + (blk & 1) * BN : blk * BN; };

        load_rows<D>(s_r1, own1, s_tok, obase, sample_off, g.ts, head, tid);
        load_rows<D>(s_r2, own2, s_tok, obase, sample_off, ts_own2, head, tid);
        load_rows<D>(s_c1, str1, s_tok, cbase(0), sample_off, g.ts, head, tid);
        load_rows<D>(s_c2, str2, s_tok, cbase(0), sample_off, ts_str2, head, tid);
        cp_async_commit();

        uint32_t f1[kFragsInRegs<D> ? KS : 1][4], f2[kFragsInRegs<D> ? KS : 1][4];
        float acc1[DT][4], acc2[KV ? DT : 1][4];
#pragma unroll
        for (int i = 0; i < DT; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc1[i][e] = 0.f;
#pragma unroll
        for (int i = 0; i < (KV ? DT : 1); ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc2[i][e] = 0.f;

        const int row_tab[2] = {obase + warp * 16 + gq, obase + warp * 16 + gq + 8};
        const int meta_r[2] = {s_meta[row_tab[0]], s_meta[row_tab[1]]};
        const float lse_r[2] = {s_lse[row_tab[0]], s_lse[row_tab[1]]};
        const float del_r[2] = {s_delta[row_tab[0]], s_delta[row_tab[1]]};

        for (int blk = 0; blk < nblk; ++blk) {
            const int stage = blk & 1;
            if (blk + 1 < nblk) {
                if (BIG) {   // the other stage's table is free: its block was finished before the barrier that ended the last step
                    fill_table(cbase(blk + 1), (blk + 1) * BN, BN);
                    __syncthreads();
                }
                load_rows<D>(s_c1 + (stage ^ 1) * TILE_BYTES, str1, s_tok, cbase(blk + 1), sample_off, g.ts, head, tid);
                load_rows<D>(s_c2 + (stage ^ 1) * TILE_BYTES, str2, s_tok, cbase(blk + 1), sample_off, ts_str2, head, tid);
                cp_async_commit();
                cp_async_wait<1>();
            } else {
                cp_async_wait<0>();
            }
            __syncthreads();
            if constexpr (kFragsInRegs<D>) {
                if (blk == 0) {
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                        ldmatrix_x4(f1[ks], smem_u32(s_r1 + tile_off<D>(row, 2 * ks + (lane >> 4))));
                        ldmatrix_x4(f2[ks], smem_u32(s_r2 + tile_off<D>(row, 2 * ks + (lane >> 4))));
                    }
                }
            }
            const unsigned char* c1 = s_c1 + stage * TILE_BYTES;
            const unsigned char* c2 = s_c2 + stage * TILE_BYTES;

            float acc_s[BN / 8][4], acc_dp[BN / 8][4];
            rows_times_block_t<D>(acc_s, f1, s_r1, c1, warp, lane);     // S (or S^T) before scale and bias
            rows_times_block_t<D>(acc_dp, f2, s_r2, c2, warp, lane);    // dP (or dP^T)

            // P = exp2(S * scale * log2e + bias * log2e - lse * log2e);  dS = P * (dP - delta)
#pragma unroll
            for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = cbase(blk) + nt * 8 + 2 * tq + (e & 1);
                    const int mc = s_meta[col];
                    const int mr = meta_r[e >> 1];
                    const bool ok = meta_label(mr) == meta_label(mc);
                    // bias row uses query offset minus key offset
                    const int bidx = KV ? (meta_code(mc) - meta_code(mr) + c0) : (meta_code(mr) - meta_code(mc) + c0);
                    const float l2 = KV ? s_lse[col] : lse_r[e >> 1];
                    const float dl = KV ? s_delta[col] : del_r[e >> 1];
                    const float bv = BIG ? (ok ? __ldg(bias + (size_t)bidx * g.heads + head) * kLog2e : 0.f) : s_bias[bidx];
                    float p = fast_exp2(acc_s[nt][e] * g.scale_log2e + bv - l2);
                    p = ok ? p : 0.f;
                    const float ds = p * (acc_dp[nt][e] - dl);
                    acc_s[nt][e] = p;
                    acc_dp[nt][e] = ds;
                }
            }
            if (!KV) {
                if (use_acc && r.ew == g.w) {
                    // this thread owns these image cells: plain read-modify-write with 8-byte accesses,
                    // all loads first so that they overlap
                    float2* cell0 = reinterpret_cast<float2*>(s_acc + (warp * 16 + gq) * acc_stride + blk * BN + 2 * tq);
                    float2 cur[BN / 8][2];
#pragma unroll
                    for (int nt = 0; nt < BN / 8; ++nt) {
                        cur[nt][0] = cell0[nt * 4];
                        cur[nt][1] = cell0[nt * 4 + 4 * acc_stride];
                    }
#pragma unroll
                    for (int nt = 0; nt < BN / 8; ++nt) {
                        cur[nt][0].x += acc_dp[nt][0]; cur[nt][0].y += acc_dp[nt][1];
                        cur[nt][1].x += acc_dp[nt][2]; cur[nt][1].y += acc_dp[nt][3];
                    }
#pragma unroll
                    for (int nt = 0; nt < BN / 8; ++nt) {
                        cell0[nt * 4] = cur[nt][0];
                        cell0[nt * 4 + 4 * acc_stride] = cur[nt][1];
                    }
                } else {
                    // The warp's 16 x 64 dS tile goes through a staging tile so that one atomic instruction
                    // covers 32 consecutive columns of one row: 32 different table entries, no retries inside
                    // the warp (in the MMA fragment layout a warp instruction hits only 14 distinct entries).
                    // The staging tile holds 32 columns: the block's two halves go through it one after the other.
                    float* stage = s_stage + warp * 16 * kStageStride;
                    const int slot0 = r0 + warp * 16;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
#pragma unroll
                        for (int nt = 4 * half; nt < 4 * half + 4; ++nt) {
                            // 8-byte stores; with a row stride of 40 floats the 16 lanes of a half warp hit 32 different banks
                            const int col = (nt - 4 * half) * 8 + 2 * tq;
                            *reinterpret_cast<float2*>(stage + gq * kStageStride + col) = make_float2(acc_dp[nt][0], acc_dp[nt][1]);
                            *reinterpret_cast<float2*>(stage + (gq + 8) * kStageStride + col) = make_float2(acc_dp[nt][2], acc_dp[nt][3]);
                        }
                        __syncwarp();
                        if (BIG) {
                            if (r.ew == g.w && (g.w & 31) == 0) {
                                // Complete along the width, side a multiple of 32: the warp's 16 rows are consecutive offsets
                                // b_q of one window row a_q, and this half of the block is 32 consecutive offsets b_k of one
                                // window row a_k.  All pairs with the same b_q - b_k share one table entry: sum each of the
                                // 47 diagonals, then one global atomic per diagonal.
                                const int a_q = slot0 / g.w, bq0 = slot0 - a_q * g.w;
                                const int k0 = blk * BN + half * 32;
                                const int a_k = k0 / g.w, bk0 = k0 - a_k * g.w;
                                const int row_base = (a_q - a_k) * (2 * g.w - 1) + c0 + bq0 - bk0;
                                float s0 = 0.f, s1 = 0.f;
#pragma unroll
                                for (int rr = 0; rr < 16; ++rr) {
                                    const bool first = rr <= lane;
                                    const float val = stage[rr * kStageStride + (first ? 31 - lane + rr : rr - lane - 1)];
                                    if (first) s0 += val; else s1 += val;
                                }
                                if (s0 != 0.f) atomicAdd(&dbias[(size_t)(row_base - 31 + lane) * g.heads + head], s0);
                                if (lane < 15 && s1 != 0.f) atomicAdd(&dbias[(size_t)(row_base + 1 + lane) * g.heads + head], s1);
                            } else {
                                const int code_c = meta_code(s_meta[cbase(blk) + half * 32 + lane]);
                                for (int rr = 0; rr < 16; ++rr) {
                                    const int code_r = meta_code(s_meta[obase + warp * 16 + rr]) + c0;
                                    const float v0 = stage[rr * kStageStride + lane];
                                    if (v0 != 0.f) atomicAdd(&dbias[(size_t)(code_r - code_c) * g.heads + head], v0);
                                }
                            }
                        } else if (g.w == 32 && r.ew == 32) {
                            // Full-width 32-wide window: the warp's 16 rows are consecutive offsets b_q of one window row
                            // a_q, and this half of the block is one window row a_k of keys with b_k = 0..31.  All pairs
                            // with the same b_q - b_k share one table entry: sum each of the 47 diagonals first, then one
                            // atomic per diagonal instead of one per pair.
                            const int a_q = slot0 >> 5, bq0 = slot0 & 31;
                            const int a_k = 2 * blk + half;
                            const int row_base = (a_q - a_k) * (2 * g.w - 1) + c0;
                            // lane l sums diagonal l (rows rr <= l) and, for l < 15, diagonal l + 32 (rows rr > l): 16 loads
                            // per lane cover all 47 diagonals
                            float s0 = 0.f, s1 = 0.f;
#pragma unroll
                            for (int rr = 0; rr < 16; ++rr) {
                                const bool first = rr <= lane;
                                const float val = stage[rr * kStageStride + (first ? 31 - lane + rr : rr - lane - 1)];
                                if (first) s0 += val; else s1 += val;
                            }
                            if (s0 != 0.f) atomicAdd(&s_dbias[row_base + bq0 - 31 + lane], s0);
                            if (lane < 15 && s1 != 0.f) atomicAdd(&s_dbias[row_base + bq0 + 1 + lane], s1);
                        } else {
                            const int code_c = meta_code(s_meta[cbase(blk) + half * 32 + lane]);
                            for (int rr = 0; rr < 16; ++rr) {
                                const int code_r = meta_code(s_meta[obase + warp * 16 + rr]) + c0;
                                const float v0 = stage[rr * kStageStride + lane];
                                if (v0 != 0.f) atomicAdd(&s_dbias[code_r - code_c], v0);
                            }
                        }
                        __syncwarp();
                    }
                }
            }
            if constexpr (KV) {
                coef_times_block<D>(acc1, acc_dp, c1, lane);    // dK += dS^T Q
                coef_times_block<D>(acc2, acc_s, c2, lane);     // dV += P^T dO
            } else {
                coef_times_block<D>(acc1, acc_dp, c1, lane);    // dQ += dS K
            }
            __syncthreads();
        }

        // stage in the own-tile slots (their fragments live in registers), then scatter to the grid
        const float scale = g.scale_log2e * kLn2;
        stage_rows<D>(s_r1, acc1, scale, warp, gq, tq);
        if constexpr (KV) stage_rows<D>(s_r2, acc2, 1.f, warp, gq, tq);
        __syncthreads();
        scatter_rows<D>(s_r1, out1, s_tok + obase - r0, r0, r.n, sample_off, g.ts, head, tid);
        if constexpr (KV) scatter_rows<D>(s_r2, out2, s_tok + obase - r0, r0, r.n, sample_off, g.ts, head, tid);
    }

    if (!KV) {
        __syncthreads();
        if (use_acc) {
            // bin the image: cell (row, col) of a full-width window belongs to table row code(row) - code(col) + c0
            const int n_full = g.nmax;
            for (int cell = tid; cell < BM * n_full; cell += NTHREADS) {
                const int row = cell / n_full, col = cell - row * n_full;
                const int slot = fixed_tile * BM + row;
                if (slot >= n_full) continue;
                const float val = s_acc[row * acc_stride + col];
                if (val == 0.f) continue;
                const int code_r = (slot / g.w) * (2 * g.w - 1) + slot % g.w;
                const int code_c = (col / g.w) * (2 * g.w - 1) + col % g.w;
                atomicAdd(&s_dbias[code_r - code_c + c0], val);
            }
            __syncthreads();
        }
        if (!BIG)
            for (int i = tid; i < nbias; i += NTHREADS) {
                float val = s_dbias[i];
                if (val != 0.f) atomicAdd(&dbias[(size_t)i * g.heads + head], val);
            }
    }
}

// out (16 x D per warp, the warp's 16 key rows) += coef^T x block, where coef is a 64 x 64 tile in shared memory
// ([query][key], 128-byte rows in the swizzled layout of a 64-column tile) and block the 64 x D rows of the queries
template <int D>
__device__ __forceinline__ void coef_t_times_block(float (&out)[D / 8][4], const unsigned char* coef, const unsigned char* blk,
                                                   int warp, int lane) {
#pragma unroll
    for (int ks = 0; ks < BN / 16; ++ks) {
        // A fragment (16 keys x 16 queries) = transpose of coef[16 ks .. + 15][16 warp .. + 15]
        uint32_t pf[4];
        const int mat = lane >> 3;
        ldmatrix_x4_trans(pf, smem_u32(coef + tile_off<64>(ks * 16 + (mat >> 1) * 8 + (lane & 7), 2 * warp + (mat & 1))));
#pragma unroll
        for (int dp = 0; dp < D / 16; ++dp) {
            uint32_t bf[4];
            int r = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            ldmatrix_x4_trans(bf, smem_u32(blk + tile_off<D>(r, 2 * dp + (lane >> 4))));
            mma_elem(out[2 * dp], pf, bf[0], bf[1]);
            mma_elem(out[2 * dp + 1], pf, bf[2], bf[3]);
        }
    }
}

// The whole backward of windows of at most 64 tokens in one kernel (the paper's 8 x 8 windows), any head dim: a CTA holds the
// window's Q, K, V, dO and O rows of one head, so every tensor is read once and dQ, dK, dV are written once (the
// split into a key side and a query side reads the inputs twice, and a third time for delta).
//   delta = rowsum(dO * O)                                 (per query row, from the two tiles)
//   query-major, a warp owns 16 query rows:  S = Q K^T, dP = dO V^T, P = exp2(S scale + bias - lse), dS = P (dP - delta),
//   the bias gradient (as in the query-side kernel above), dQ = dS K; P and dS go to shared memory as 64 x 64 tiles
//   key-major, a warp owns 16 key rows:      dV = P^T dO, dK = dS^T Q  (A fragments by transposing loads of those tiles)
// Persistent CTAs bound to one head walk over (batch, window).  Shared memory: the four operand tiles, one more that
// holds O first and P | dS afterwards, the slot tables, the summed-dS image and the staging tile of the bias gradient.
template <int D>
__global__ void __launch_bounds__(NTHREADS, 2)
swin_bwd_small_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                      const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ o,
                      const __nv_bfloat16* __restrict__ d_o, const float* __restrict__ bias, const float* __restrict__ lse,
                      __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                      float* __restrict__ dbias, int ctas_per_head, int acc_stride) {
    constexpr int KS = D / 16;
    constexpr int DT = D / 8;
    constexpr int TILE_BYTES = BN * D * 2;
    constexpr int X_BYTES = TILE_BYTES > 16384 ? TILE_BYTES : 16384;      // O, then P (8 KB) | dS (8 KB)
    extern __shared__ __align__(128) unsigned char smem[];

    const int nbias = (2 * g.w - 1) * (2 * g.w - 1);
    int* s_tok = reinterpret_cast<int*>(smem);
    int* s_meta = s_tok + BN;
    float* s_lse = reinterpret_cast<float*>(s_meta + BN);
    float* s_delta = s_lse + BN;
    float* s_bias = s_delta + BN;
    float* s_dbias = s_bias + nbias;
    unsigned char* s_q = smem + (((size_t)BN * 16 + (size_t)nbias * 8 + 127) / 128) * 128;
    unsigned char* s_k = s_q + TILE_BYTES;
    unsigned char* s_v = s_k + TILE_BYTES;
    unsigned char* s_g = s_v + TILE_BYTES;            // dO
    unsigned char* s_x = s_g + TILE_BYTES;
    unsigned char* s_p = s_x;                         // P as a 64 x 64 tile
    unsigned char* s_ds = s_x + 8192;                 // dS as a 64 x 64 tile
    float* s_acc = reinterpret_cast<float*>(s_x + X_BYTES);              // 64 x acc_stride image of summed dS
    float* s_stage = s_acc + BM * acc_stride;                            // 4 warps x 16 x kStageStride

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const int head = blockIdx.x % g.heads;
    const int M = g.Mh * g.Mw;
    const int c0 = (g.w - 1) * 2 * g.w;
    const long long n_items = (long long)g.B * M;
    const int dense = g.heads * D;                    // token stride of o and dO

    for (int i = tid; i < nbias; i += NTHREADS) {
        s_bias[i] = bias[(size_t)i * g.heads + head] * kLog2e;
        s_dbias[i] = 0.f;
    }
    for (int i = tid; i < BM * acc_stride; i += NTHREADS) s_acc[i] = 0.f;

    for (long long item = blockIdx.x / g.heads; item < n_items; item += ctas_per_head) {
        const int win = (int)(item % M);
        const int b = (int)(item / M);
        const WindowRef r = window_ref(g, win);
        const size_t sample_off = (size_t)b * g.H * g.W;

        __syncthreads();   // the previous item's readers of the tables and tiles are done
        if (tid < BN) {
            int meta = 0xff << 16, tok = -1;
            if (tid < r.n) {
                tok = slot_token(g, r, tid, meta);
                // the row's log-sum-exp travels with the tiles (no load that the copies below would have to wait for)
                cp_async4(smem_u32(&s_lse[tid]), lse + (sample_off + (size_t)tok) * g.heads + head);
            } else {
                s_lse[tid] = INFINITY;              // padded queries: P = exp2(x - inf) = 0
            }
            s_tok[tid] = tok;
            s_meta[tid] = meta;
        }
        __syncthreads();
        load_rows<D>(s_q, q, s_tok, 0, sample_off, g.ts, head, tid);
        load_rows<D>(s_k, k, s_tok, 0, sample_off, g.ts, head, tid);
        load_rows<D>(s_v, v, s_tok, 0, sample_off, g.ts, head, tid);
        load_rows<D>(s_g, d_o, s_tok, 0, sample_off, dense, head, tid);
        load_rows<D>(s_x, o, s_tok, 0, sample_off, dense, head, tid);
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();

        // ---- delta of the warp's 16 query rows: two lanes per row, half a row each
        {
            const int row = warp * 16 + (lane >> 1);
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < DT / 2; ++c) {
                const int chunk = (lane & 1) * (DT / 2) + c;
                const uint4 a = *reinterpret_cast<const uint4*>(s_x + tile_off<D>(row, chunk));
                const uint4 bb = *reinterpret_cast<const uint4*>(s_g + tile_off<D>(row, chunk));
                const uint32_t* pa = reinterpret_cast<const uint32_t*>(&a);
                const uint32_t* pb = reinterpret_cast<const uint32_t*>(&bb);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 x = elem2_to_float2(pa[e]), y = elem2_to_float2(pb[e]);
                    acc += x.x * y.x + x.y * y.y;
                }
            }
            acc += __shfl_xor_sync(0xffffffffu, acc, 1);
            if ((lane & 1) == 0) s_delta[row] = acc;
        }
        __syncthreads();   // O has been read by every warp: its tile becomes P | dS

        // ---- query-major part
        const int row_tab[2] = {warp * 16 + gq, warp * 16 + gq + 8};
        const int meta_r[2] = {s_meta[row_tab[0]], s_meta[row_tab[1]]};
        const float lse_r[2] = {s_lse[row_tab[0]] * kLog2e, s_lse[row_tab[1]] * kLog2e};
        const float del_r[2] = {s_delta[row_tab[0]], s_delta[row_tab[1]]};
        float acc1[DT][4];
        {
            // fragments of the warp's own Q and dO rows (head dim 128: read from shared memory at each use instead)
            uint32_t f1[kFragsInRegs<D> ? KS : 1][4], f2[kFragsInRegs<D> ? KS : 1][4];
            if constexpr (kFragsInRegs<D>) {
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                    ldmatrix_x4(f1[ks], smem_u32(s_q + tile_off<D>(row, 2 * ks + (lane >> 4))));
                    ldmatrix_x4(f2[ks], smem_u32(s_g + tile_off<D>(row, 2 * ks + (lane >> 4))));
                }
            }
            float acc_s[BN / 8][4], acc_dp[BN / 8][4];
            rows_times_block_t<D>(acc_s, f1, s_q, s_k, warp, lane);
            rows_times_block_t<D>(acc_dp, f2, s_g, s_v, warp, lane);
#pragma unroll
            for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col = nt * 8 + 2 * tq + (e & 1);
                    const int mc = s_meta[col];
                    const int mr = meta_r[e >> 1];
                    const bool ok = meta_label(mr) == meta_label(mc);
                    const int bidx = meta_code(mr) - meta_code(mc) + c0;
                    float p = fast_exp2(acc_s[nt][e] * g.scale_log2e + s_bias[bidx] - lse_r[e >> 1]);
                    p = ok ? p : 0.f;
                    acc_s[nt][e] = p;
                    acc_dp[nt][e] = p * (acc_dp[nt][e] - del_r[e >> 1]);
                }
            }
            // bias gradient
            if (r.ew == g.w) {
                // full-width window: this thread owns these cells of the image (binned into the table at the end)
                float2* cell0 = reinterpret_cast<float2*>(s_acc + (warp * 16 + gq) * acc_stride + 2 * tq);
                float2 cur[BN / 8][2];
#pragma unroll
                for (int nt = 0; nt < BN / 8; ++nt) {
                    cur[nt][0] = cell0[nt * 4];
                    cur[nt][1] = cell0[nt * 4 + 4 * acc_stride];
                }
#pragma unroll
                for (int nt = 0; nt < BN / 8; ++nt) {
                    cur[nt][0].x += acc_dp[nt][0]; cur[nt][0].y += acc_dp[nt][1];
                    cur[nt][1].x += acc_dp[nt][2]; cur[nt][1].y += acc_dp[nt][3];
                }
#pragma unroll
                for (int nt = 0; nt < BN / 8; ++nt) {
                    cell0[nt * 4] = cur[nt][0];
                    cell0[nt * 4 + 4 * acc_stride] = cur[nt][1];
                }
            } else {
                // narrow edge window: through the staging tile, one shared-memory atomic per pair, 32 different table
                // entries per instruction
                float* stage = s_stage + warp * 16 * kStageStride;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int nt = 4 * half; nt < 4 * half + 4; ++nt) {
                        const int col = (nt - 4 * half) * 8 + 2 * tq;
                        *reinterpret_cast<float2*>(stage + gq * kStageStride + col) = make_float2(acc_dp[nt][0], acc_dp[nt][1]);
                        *reinterpret_cast<float2*>(stage + (gq + 8) * kStageStride + col) = make_float2(acc_dp[nt][2], acc_dp[nt][3]);
                    }
                    __syncwarp();
                    const int code_c = meta_code(s_meta[half * 32 + lane]);
                    for (int rr = 0; rr < 16; ++rr) {
                        const int code_r = meta_code(s_meta[warp * 16 + rr]) + c0;
                        const float v0 = stage[rr * kStageStride + lane];
                        if (v0 != 0.f) atomicAdd(&s_dbias[code_r - code_c], v0);
                    }
                    __syncwarp();
                }
            }
            // P and dS as 64 x 64 tiles for the key-major part
            stage_rows<64>(s_p, acc_s, 1.f, warp, gq, tq);
            stage_rows<64>(s_ds, acc_dp, 1.f, warp, gq, tq);
            // dQ = dS K
#pragma unroll
            for (int i = 0; i < DT; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc1[i][e] = 0.f;
            coef_times_block<D>(acc1, acc_dp, s_k, lane);
        }
        __syncthreads();   // P, dS are complete; K and V have been read by every warp
        const float scale = g.scale_log2e * kLn2;
        stage_rows<D>(s_v, acc1, scale, warp, gq, tq);           // dQ into the V tile

        // ---- key-major part
#pragma unroll
        for (int i = 0; i < DT; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc1[i][e] = 0.f;
        coef_t_times_block<D>(acc1, s_p, s_g, warp, lane);       // dV = P^T dO
        stage_rows<D>(s_k, acc1, 1.f, warp, gq, tq);             // dV into the K tile
#pragma unroll
        for (int i = 0; i < DT; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc1[i][e] = 0.f;
        coef_t_times_block<D>(acc1, s_ds, s_q, warp, lane);      // dK = dS^T Q
        __syncthreads();   // Q has been read by every warp
        stage_rows<D>(s_q, acc1, scale, warp, gq, tq);           // dK into the Q tile
        __syncthreads();
        scatter_rows<D>(s_v, dq, s_tok, 0, r.n, sample_off, g.ts, head, tid);
        scatter_rows<D>(s_k, dv, s_tok, 0, r.n, sample_off, g.ts, head, tid);
        scatter_rows<D>(s_q, dk, s_tok, 0, r.n, sample_off, g.ts, head, tid);
    }

    __syncthreads();
    // bin the image: cell (row, col) of a full-width window belongs to table row code(row) - code(col) + c0
    const int n_full = g.nmax;
    for (int cell = tid; cell < BM * n_full; cell += NTHREADS) {
        const int row = cell / n_full, col = cell - row * n_full;
        if (row >= n_full) continue;
        const float val = s_acc[row * acc_stride + col];
        if (val == 0.f) continue;
        const int code_r = (row / g.w) * (2 * g.w - 1) + row % g.w;
        const int code_c = (col / g.w) * (2 * g.w - 1) + col % g.w;
        atomicAdd(&s_dbias[code_r - code_c + c0], val);
    }
    __syncthreads();
    for (int i = tid; i < nbias; i += NTHREADS) {
        float val = s_dbias[i];
        if (val != 0.f) atomicAdd(&dbias[(size_t)i * g.heads + head], val);
    }
}

// delta[b, token, head] = sum_c dO[b, token, head, c] * O[b, token, head, c]
template <int D>
__global__ void __launch_bounds__(256)
swin_bwd_delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                      float* __restrict__ delta, long long rows) {
    constexpr int LPR = D / 8;   // lanes per row, each lane takes one 16-byte chunk
    long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long row = gid / LPR;
    int chunk = (int)(gid % LPR);
    float acc = 0.f;
    if (row < rows) {
        uint4 a = *reinterpret_cast<const uint4*>(o + row * D + chunk * 8);
        uint4 b = *reinterpret_cast<const uint4*>(d_o + row * D + chunk * 8);
        const uint32_t* pa = reinterpret_cast<const uint32_t*>(&a);
        const uint32_t* pb = reinterpret_cast<const uint32_t*>(&b);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 x = elem2_to_float2(pa[i]), y = elem2_to_float2(pb[i]);
            acc += x.x * y.x + x.y * y.y;
        }
    }
#pragma unroll
    for (int off = LPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (row < rows && chunk == 0) delta[row] = acc;
}

// Row stride (floats) of the summed-dS image, or 0 when the window is too large for it.  The stride is
// 8 mod 32 so that the 16 lanes of one 8-byte access wave hit 32 different banks.
int acc_stride_for(const Geo& g) {
    int npad_max = ((g.nmax + BN - 1) / BN) * BN;
    return npad_max <= 256 ? npad_max + 8 : 0;
}

size_t bwd_smem_bytes(const Geo& g, bool query_side) {
    int npad_max = ((g.nmax + BN - 1) / BN) * BN;
    int nbias = (2 * g.w - 1) * (2 * g.w - 1);
    size_t head = g.w > 32 ? (size_t)3 * BN * 16 : (((size_t)npad_max * 16 + (size_t)nbias * 8 + 127) / 128) * 128;
    size_t acc = query_side ? ((size_t)BM * acc_stride_for(g) + (size_t)BM * kStageStride) * sizeof(float) : 0;
    return head + 6 * (size_t)BN * g.d * 2 + acc;
}

template <int D, bool KV, bool BIG>
cudaError_t launch_one_sized(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* bias,
                       const float* lse, const float* delta, void* out1, void* out2, float* dbias, int sm_count,
                       cudaStream_t stream) {
    auto kern = swin_bwd_mma_kernel<D, KV, BIG>;
    const size_t smem = bwd_smem_bytes(g, !KV);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, NTHREADS, smem);
    if (e != cudaSuccess) return e;
    if (occ < 1) occ = 1;
    const int tiles = (g.nmax + BM - 1) / BM;
    const int groups = KV ? g.heads : g.heads * tiles;          // what a persistent CTA is bound to
    const long long items = KV ? (long long)g.B * g.Mh * g.Mw * tiles : (long long)g.B * g.Mh * g.Mw;
    long long cpg = ((long long)sm_count * occ) / groups;
    if (cpg < 1) cpg = 1;
    if (cpg > items) cpg = items;
    prof_begin(KV ? "swin_bwd_mma_kernel<key tiles>" : "swin_bwd_mma_kernel<query tiles>", stream);
    kern<<<(unsigned)(cpg * groups), NTHREADS, smem, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)d_o, bias,
        lse, delta, (__nv_bfloat16*)out1, (__nv_bfloat16*)out2, dbias, tiles, (int)cpg, KV ? 0 : acc_stride_for(g));
    count_launch(stream);
    return cudaGetLastError();
}

template <int D, bool KV>
cudaError_t launch_one(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* bias,
                       const float* lse, const float* delta, void* out1, void* out2, float* dbias, int sm_count,
                       cudaStream_t stream) {
    return g.w > 32 ? launch_one_sized<D, KV, true>(g, q, k, v, d_o, bias, lse, delta, out1, out2, dbias, sm_count, stream)
                    : launch_one_sized<D, KV, false>(g, q, k, v, d_o, bias, lse, delta, out1, out2, dbias, sm_count, stream);
}

size_t bwd_small_smem_bytes(const Geo& g) {
    const int nbias = (2 * g.w - 1) * (2 * g.w - 1);
    const size_t head = (((size_t)BN * 16 + (size_t)nbias * 8 + 127) / 128) * 128;
    const size_t tile = (size_t)BN * g.d * 2;
    return head + 4 * tile + (tile > 16384 ? tile : 16384) + ((size_t)BM * (BN + 8) + (size_t)BM * kStageStride) * sizeof(float);
}

}  // namespace

// windows of at most 64 tokens: the one-kernel backward
bool TERRA_ELEM_FN(bwd_small_supported)(const Geo& g) { return g.nmax <= BN && g.w <= 32; }

cudaError_t TERRA_ELEM_FN(launch_bwd_small)(const Geo& g, const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                            const float* bias, const float* lse, void* dq, void* dk, void* dv, float* dbias,
                                            int sm_count, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(dbias, 0, sizeof(float) * (size_t)(2 * g.w - 1) * (2 * g.w - 1) * g.heads, stream);
    if (e != cudaSuccess) return e;
    auto kern = g.d == 32 ? swin_bwd_small_kernel<32> : g.d == 64 ? swin_bwd_small_kernel<64> : swin_bwd_small_kernel<128>;
    const size_t smem = bwd_small_smem_bytes(g);
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, NTHREADS, smem);
    if (e != cudaSuccess) return e;
    if (occ < 1) occ = 1;
    const long long items = (long long)g.B * g.Mh * g.Mw;
    long long cph = ((long long)sm_count * occ) / g.heads;
    if (cph < 1) cph = 1;
    if (cph > items) cph = items;
    prof_begin("swin_bwd_small_kernel", stream);
    kern<<<(unsigned)(cph * g.heads), NTHREADS, smem, stream>>>(
        g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (const __nv_bfloat16*)o,
        (const __nv_bfloat16*)d_o, bias, lse, (__nv_bfloat16*)dq, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, dbias, (int)cph, BN + 8);
    count_launch(stream);
    return cudaGetLastError();
}

cudaError_t TERRA_ELEM_FN(launch_bwd_delta)(const Geo& g, const void* o, const void* d_o, float* delta, cudaStream_t stream) {
    const long long rows = (long long)g.B * g.H * g.W * g.heads;
    const int lpr = g.d / 8;
    const long long threads = rows * lpr;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    prof_begin("swin_bwd_delta_kernel", stream);
    if (g.d == 32)
        swin_bwd_delta_kernel<32><<<blocks, 256, 0, stream>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, delta, rows);
    else if (g.d == 64)
        swin_bwd_delta_kernel<64><<<blocks, 256, 0, stream>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, delta, rows);
    else
        swin_bwd_delta_kernel<128><<<blocks, 256, 0, stream>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, delta, rows);
    count_launch(stream);
    return cudaGetLastError();
}

cudaError_t TERRA_ELEM_FN(launch_bwd_mma)(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                           const float* lse, const float* delta, const void* d_o,
                           void* dq, void* dk, void* dv, float* dbias, int sm_count, cudaStream_t stream,
                           bool query_side_only) {
    cudaError_t e = cudaMemsetAsync(dbias, 0, sizeof(float) * (size_t)(2 * g.w - 1) * (2 * g.w - 1) * g.heads, stream);
    if (e != cudaSuccess) return e;
    if (query_side_only) {    // dK, dV come from another kernel
        if (g.d == 128) return launch_one<128, false>(g, q, k, v, d_o, bias, lse, delta, dq, nullptr, dbias, sm_count, stream);
        return g.d == 32 ? launch_one<32, false>(g, q, k, v, d_o, bias, lse, delta, dq, nullptr, dbias, sm_count, stream)
                         : launch_one<64, false>(g, q, k, v, d_o, bias, lse, delta, dq, nullptr, dbias, sm_count, stream);
    }
    if (g.d == 128) {
        e = launch_one<128, true>(g, q, k, v, d_o, bias, lse, delta, dk, dv, nullptr, sm_count, stream);
        if (e != cudaSuccess) return e;
        return launch_one<128, false>(g, q, k, v, d_o, bias, lse, delta, dq, nullptr, dbias, sm_count, stream);
    }
    if (g.d == 32) {
        e = launch_one<32, true>(g, q, k, v, d_o, bias, lse, delta, dk, dv, nullptr, sm_count, stream);
        if (e != cudaSuccess) return e;
        return launch_one<32, false>(g, q, k, v, d_o, bias, lse, delta, dq, nullptr, dbias, sm_count, stream);
    }
    e = launch_one<64, true>(g, q, k, v, d_o, bias, lse, delta, dk, dv, nullptr, sm_count, stream);
    if (e != cudaSuccess) return e;
    return launch_one<64, false>(g, q, k, v, d_o, bias, lse, delta, dq, nullptr, dbias, sm_count, stream);
}

}  // namespace terra
