// Forward shifted-window attention, register-tile path (warp-level mma.sync).
//
// One CTA = one (batch, window, head, 64-query tile).  The window's keys and values stream through
// shared memory in 64-key blocks with an online softmax, so any window size up to 32 x 32 fits.
// Roll, window gather, shift mask, relative-position bias, softmax, PV and the scatter back to the
// contiguous grid all happen here; nothing window-major is ever written to global memory.
// The file is compiled for bf16 and, through attn_fwd_mma_f16.cu, for fp16 activations.
// This path covers every window class (truncated edges, the split latitude-wrap row, w up to 32,
// head dim 32 / 64 / 128; head dim 128, the width of the paper's Table V models, runs here only).
#include "swin_common.cuh"
#include "swin_kernels.h"

namespace terra {

namespace {

constexpr int BM = 64;   // queries per CTA (4 warps x 16 rows)
constexpr int BN = 64;   // keys per streamed block
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

// BIG = windows of more than 1024 tokens (window sides 33 .. 128): the slot tables of a whole window and the head's
// bias table no longer fit shared memory, so the tables cover the CTA's 64 query rows plus the key block in flight
// (two stages) and the bias is read from the caller's table in global memory.
template <int D, bool BIG>
__device__ __forceinline__ void
swin_fwd_mma_body(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, const float* __restrict__ bias,
                    __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int qtiles) {
    constexpr int KS = D / 16;       // k-steps of Q K^T
    constexpr int DT = D / 8;        // 8-wide output tiles of O
    constexpr int TILE_BYTES = BN * D * 2;
    extern __shared__ __align__(128) unsigned char smem[];

    int item = blockIdx.x;
    const int qt = item % qtiles; item /= qtiles;
    const int head = item % g.heads; item /= g.heads;
    const int M = g.Mh * g.Mw;
    const int win = item % M;
    const int b = item / M;
    const WindowRef r = window_ref(g, win);
    const int q0 = qt * BM;
    if (q0 >= r.n) return;
    const int nkb = (r.n + BN - 1) / BN;
    const int npad = nkb * BN;
    const int nbias = (2 * g.w - 1) * (2 * g.w - 1);
    const int npad_max = ((g.nmax + BN - 1) / BN) * BN;

    // table layout: small windows [npad_max] slots of the window; BIG: [0, 64) the query rows, [64, 192) two key blocks
    const int ntab = BIG ? 3 * BN : npad_max;
    int* s_tok = reinterpret_cast<int*>(smem);
    int* s_meta = s_tok + ntab;
    float* s_bias = reinterpret_cast<float*>(s_meta + ntab);
    unsigned char* s_q = smem + (((size_t)ntab * 8 + (BIG ? 0 : (size_t)nbias * 4) + 127) / 128) * 128;
    // K and V: two stages each; one where no window has more than one key block (then more CTAs fit an SM)
    const int nstages = (BIG || npad_max > BN) ? 2 : 1;
    unsigned char* s_k = s_q + TILE_BYTES;
    unsigned char* s_v = s_k + nstages * TILE_BYTES;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const size_t sample_off = (size_t)b * g.H * g.W;

    // fills 64 table entries at `base` with the window's slots first .. first + 63
    auto fill_table = [&](int base, int first) {
        if (tid < BN) {
            int meta = 0xff << 16, tok = -1;
            if (first + tid < r.n) tok = slot_token(g, r, first + tid, meta);
            s_tok[base + tid] = tok;
            s_meta[base + tid] = meta;
        }
    };
    if (BIG) {
        fill_table(0, q0);
        fill_table(BN, 0);
    } else {
        for (int s = tid; s < npad; s += NTHREADS) {
            int meta = 0xff << 16, tok = -1;
            if (s < r.n) tok = slot_token(g, r, s, meta);
            s_tok[s] = tok;
            s_meta[s] = meta;
        }
        for (int i = tid; i < nbias; i += NTHREADS) s_bias[i] = bias[(size_t)i * g.heads + head] * kLog2e;
    }
    __syncthreads();
    // table index of query row `row` of this CTA / of row `row` of key block kb
    const int qbase = BIG ? 0 : q0;
    auto kbase = [&](int kb) { return BIG ? BN + (kb & 1) * BN : kb * BN; };

    load_rows<D>(s_q, q, s_tok, qbase, sample_off, g.ts, head, tid);
    load_rows<D>(s_k, k, s_tok, kbase(0), sample_off, g.ts, head, tid);
    load_rows<D>(s_v, v, s_tok, kbase(0), sample_off, g.ts, head, tid);
    cp_async_commit();

    uint32_t qf[KS][4];
    float acc_o[DT][4];
#pragma unroll
    for (int i = 0; i < DT; ++i)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc_o[i][e] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

    const int row_slot[2] = {q0 + warp * 16 + gq, q0 + warp * 16 + gq + 8};
    const int meta_r[2] = {s_meta[qbase + warp * 16 + gq], s_meta[qbase + warp * 16 + gq + 8]};
    const int c0 = (g.w - 1) * 2 * g.w;

    for (int kb = 0; kb < nkb; ++kb) {
        const int stage = kb & 1;
        if (kb + 1 < nkb) {
            if (BIG) {       // the other stage's table is free: its block was finished before the barrier that ended the last step
                fill_table(kbase(kb + 1), (kb + 1) * BN);
                __syncthreads();
            }
            load_rows<D>(s_k + (stage ^ 1) * TILE_BYTES, k, s_tok, kbase(kb + 1), sample_off, g.ts, head, tid);
            load_rows<D>(s_v + (stage ^ 1) * TILE_BYTES, v, s_tok, kbase(kb + 1), sample_off, g.ts, head, tid);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (kb == 0) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                ldmatrix_x4(qf[ks], smem_u32(s_q + tile_off<D>(row, 2 * ks + (lane >> 4))));
            }
        }
        const unsigned char* sk = s_k + stage * TILE_BYTES;
        const unsigned char* sv = s_v + stage * TILE_BYTES;

        float acc_s[BN / 8][4];
#pragma unroll
        for (int i = 0; i < BN / 8; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc_s[i][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int np = 0; np < BN / 16; ++np) {
                uint32_t bf[4];
                int key = np * 16 + (lane & 7) + (lane >> 4) * 8;
                ldmatrix_x4(bf, smem_u32(sk + tile_off<D>(key, 2 * ks + ((lane >> 3) & 1))));
                mma_elem(acc_s[2 * np], qf[ks], bf[0], bf[1]);
                mma_elem(acc_s[2 * np + 1], qf[ks], bf[2], bf[3]);
            }
        }

        // scale + relative-position bias + shift mask, in the log2 domain
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                int mj = s_meta[kbase(kb) + nt * 8 + 2 * tq + (e & 1)];
                int mi = meta_r[e >> 1];
                bool ok = meta_label(mi) == meta_label(mj);
                const int bidx = meta_code(mi) - meta_code(mj) + c0;
                const float bv = BIG ? (ok ? __ldg(bias + (size_t)bidx * g.heads + head) * kLog2e : 0.f) : s_bias[bidx];
                float sc = acc_s[nt][e] * g.scale_log2e + bv;
                sc = ok ? sc : -INFINITY;
                acc_s[nt][e] = sc;
                mx[e >> 1] = fmaxf(mx[e >> 1], sc);
            }
        }
        float corr[2], m_use[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            float m_new = fmaxf(m_run[h], mx[h]);
            m_use[h] = (m_new == -INFINITY) ? 0.f : m_new;     // a fully masked block leaves the state alone
            corr[h] = fast_exp2(m_run[h] - m_use[h]);
            m_run[h] = m_new;
            l_run[h] *= corr[h];
        }
#pragma unroll
        for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float p = fast_exp2(acc_s[nt][e] - m_use[e >> 1]);
                acc_s[nt][e] = p;
                l_run[e >> 1] += p;
            }
        }
#pragma unroll
        for (int i = 0; i < DT; ++i) {
            acc_o[i][0] *= corr[0]; acc_o[i][1] *= corr[0];
            acc_o[i][2] *= corr[1]; acc_o[i][3] *= corr[1];
        }
        // O += P V
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
            uint32_t pf[4];
            pf[0] = pack_elem(acc_s[2 * ks][0], acc_s[2 * ks][1]);
            pf[1] = pack_elem(acc_s[2 * ks][2], acc_s[2 * ks][3]);
            pf[2] = pack_elem(acc_s[2 * ks + 1][0], acc_s[2 * ks + 1][1]);
            pf[3] = pack_elem(acc_s[2 * ks + 1][2], acc_s[2 * ks + 1][3]);
#pragma unroll
            for (int dp = 0; dp < DT / 2; ++dp) {
                uint32_t bf[4];
                int key = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                ldmatrix_x4_trans(bf, smem_u32(sv + tile_off<D>(key, 2 * dp + (lane >> 4))));
                mma_elem(acc_o[2 * dp], pf, bf[0], bf[1]);
                mma_elem(acc_o[2 * dp + 1], pf, bf[2], bf[3]);
            }
        }
        __syncthreads();
    }

    // normalise, stage the 64 x D output tile in shared memory (Q's slot), scatter rows to the grid
    float inv[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float l = l_run[h];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        l_run[h] = l;
        inv[h] = 1.f / l;
    }
#pragma unroll
    for (int i = 0; i < DT; ++i) {
        int lr = warp * 16 + gq;
        // chunk i holds columns 8i..8i+7; this thread owns columns 2tq, 2tq+1 of it
        *reinterpret_cast<uint32_t*>(s_q + tile_off<D>(lr, i) + tq * 4) = pack_elem(acc_o[i][0] * inv[0], acc_o[i][1] * inv[0]);
        *reinterpret_cast<uint32_t*>(s_q + tile_off<D>(lr + 8, i) + tq * 4) = pack_elem(acc_o[i][2] * inv[1], acc_o[i][3] * inv[1]);
    }
    if (tq == 0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            int slot = row_slot[h];
            if (slot < r.n)
                lse[(sample_off + (size_t)s_tok[slot - q0 + qbase]) * g.heads + head] = (m_run[h] + log2f(l_run[h])) * kLn2;
        }
    }
    __syncthreads();
    constexpr int CPR = D / 8;
    for (int idx = tid; idx < BM * CPR; idx += NTHREADS) {
        int row = idx / CPR, chunk = idx - row * CPR;
        int slot = q0 + row;
        if (slot < r.n) {
            uint4 val = *reinterpret_cast<const uint4*>(s_q + tile_off<D>(row, chunk));
            *reinterpret_cast<uint4*>(o + ((sample_off + (size_t)s_tok[qbase + row]) * g.heads + head) * D + chunk * 8) = val;
        }
    }
}

template <int D, bool BIG>
__global__ void __launch_bounds__(NTHREADS)
swin_fwd_mma_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                    const __nv_bfloat16* __restrict__ v, const float* __restrict__ bias,
                    __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int qtiles) {
    swin_fwd_mma_body<D, BIG>(g, q, k, v, bias, o, lse, qtiles);
}

// Windows of at most 64 tokens (the paper's 8 x 8 windows), every head dim: persistent CTAs bound to one head walk over
// (batch, window); a window is one 64-row tile of Q, K and V.  The tiles are double-buffered: while a window is
// computed and its output rows are written, the next window's rows are already on their way, so a CTA always has
// loads in flight (these shapes are bound by HBM).  No online softmax: the whole score row is in registers.
template <int D>
__global__ void __launch_bounds__(NTHREADS, 2)
swin_fwd_small_kernel(const Geo g, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                      const __nv_bfloat16* __restrict__ v, const float* __restrict__ bias,
                      __nv_bfloat16* __restrict__ o, float* __restrict__ lse, int ctas_per_head) {
    constexpr int KS = D / 16;
    constexpr int DT = D / 8;
    constexpr int TILE_BYTES = BN * D * 2;
    constexpr int BUF_BYTES = 3 * TILE_BYTES;
    extern __shared__ __align__(128) unsigned char smem[];

    const int nbias = (2 * g.w - 1) * (2 * g.w - 1);
    int* s_tok = reinterpret_cast<int*>(smem);                // [2][64]
    int* s_meta = s_tok + 2 * BN;                             // [2][64]
    float* s_bias = reinterpret_cast<float*>(s_meta + 2 * BN);
    unsigned char* s_tiles = smem + (((size_t)BN * 16 + (size_t)nbias * 4 + 127) / 128) * 128;   // [2][Q | K | V]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const int head = blockIdx.x % g.heads;
    const int M = g.Mh * g.Mw;
    const int c0 = (g.w - 1) * 2 * g.w;
    const long long n_items = (long long)g.B * M;
    const long long first = blockIdx.x / g.heads;

    for (int i = tid; i < nbias; i += NTHREADS) s_bias[i] = bias[(size_t)i * g.heads + head] * kLog2e;

    // slot tables of item `item` into buffer `b`
    auto fill_tables = [&](long long item, int b) {
        if (tid < BN) {
            const WindowRef r = window_ref(g, (int)(item % M));
            int meta = 0xff << 16, tok = -1;
            if (tid < r.n) tok = slot_token(g, r, tid, meta);
            s_tok[b * BN + tid] = tok;
            s_meta[b * BN + tid] = meta;
        }
    };
    // the copies of item `item` into buffer `b` (its tables must be visible), one group
    auto issue_loads = [&](long long item, int b) {
        const size_t sample_off = (size_t)(item / M) * g.H * g.W;
        unsigned char* t = s_tiles + b * BUF_BYTES;
        load_rows<D>(t, q, s_tok + b * BN, 0, sample_off, g.ts, head, tid);
        load_rows<D>(t + TILE_BYTES, k, s_tok + b * BN, 0, sample_off, g.ts, head, tid);
        load_rows<D>(t + 2 * TILE_BYTES, v, s_tok + b * BN, 0, sample_off, g.ts, head, tid);
        cp_async_commit();
    };
    if (first < n_items) {
        fill_tables(first, 0);
        __syncthreads();
        issue_loads(first, 0);
    }
    int buf = 0;
    for (long long item = first; item < n_items; item += ctas_per_head, buf ^= 1) {
        const long long next = item + ctas_per_head;
        // the other buffer was last read by the scatter of the item before this one, which ended with a barrier
        if (next < n_items) fill_tables(next, buf ^ 1);
        __syncthreads();
        if (next < n_items) {
            issue_loads(next, buf ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const WindowRef r = window_ref(g, (int)(item % M));
        const size_t sample_off = (size_t)(item / M) * g.H * g.W;
        unsigned char* s_q = s_tiles + buf * BUF_BYTES;
        const unsigned char* s_k = s_q + TILE_BYTES;
        const unsigned char* s_v = s_q + 2 * TILE_BYTES;
        const int* tokb = s_tok + buf * BN;
        const int* metab = s_meta + buf * BN;

        // S = Q K^T for the warp's 16 query rows
        float acc_s[BN / 8][4];
#pragma unroll
        for (int i = 0; i < BN / 8; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc_s[i][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t qf[4];
            const int row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
            ldmatrix_x4(qf, smem_u32(s_q + tile_off<D>(row, 2 * ks + (lane >> 4))));
#pragma unroll
            for (int np = 0; np < BN / 16; ++np) {
                uint32_t bf[4];
                const int key = np * 16 + (lane & 7) + (lane >> 4) * 8;
                ldmatrix_x4(bf, smem_u32(s_k + tile_off<D>(key, 2 * ks + ((lane >> 3) & 1))));
                mma_elem(acc_s[2 * np], qf, bf[0], bf[1]);
                mma_elem(acc_s[2 * np + 1], qf, bf[2], bf[3]);
            }
        }
        // scale + relative-position bias + shift mask, in the log2 domain; row maxima
        const int meta_r[2] = {metab[warp * 16 + gq], metab[warp * 16 + gq + 8]};
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int mj = metab[nt * 8 + 2 * tq + (e & 1)];
                const int mi = meta_r[e >> 1];
                const bool ok = meta_label(mi) == meta_label(mj);
                float sc = acc_s[nt][e] * g.scale_log2e + s_bias[meta_code(mi) - meta_code(mj) + c0];
                sc = ok ? sc : -INFINITY;
                acc_s[nt][e] = sc;
                mx[e >> 1] = fmaxf(mx[e >> 1], sc);
            }
        }
        float m_use[2], l_row[2] = {0.f, 0.f};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            m_use[h] = (mx[h] == -INFINITY) ? 0.f : mx[h];     // a row without a token sees no key
        }
#pragma unroll
        for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float p = fast_exp2(acc_s[nt][e] - m_use[e >> 1]);
                acc_s[nt][e] = p;
                l_row[e >> 1] += p;
            }
        }
        // O = P V
        float acc_o[DT][4];
#pragma unroll
        for (int i = 0; i < DT; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc_o[i][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < BN / 16; ++ks) {
            uint32_t pf[4];
            pf[0] = pack_elem(acc_s[2 * ks][0], acc_s[2 * ks][1]);
            pf[1] = pack_elem(acc_s[2 * ks][2], acc_s[2 * ks][3]);
            pf[2] = pack_elem(acc_s[2 * ks + 1][0], acc_s[2 * ks + 1][1]);
            pf[3] = pack_elem(acc_s[2 * ks + 1][2], acc_s[2 * ks + 1][3]);
#pragma unroll
            for (int dp = 0; dp < DT / 2; ++dp) {
                uint32_t bf[4];
                const int key = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                ldmatrix_x4_trans(bf, smem_u32(s_v + tile_off<D>(key, 2 * dp + (lane >> 4))));
                mma_elem(acc_o[2 * dp], pf, bf[0], bf[1]);
                mma_elem(acc_o[2 * dp + 1], pf, bf[2], bf[3]);
            }
        }
        float inv[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            float l = l_row[h];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            l_row[h] = l;
            inv[h] = 1.f / l;
        }
        __syncthreads();   // every warp has read its Q fragments: the Q tile becomes the output tile
#pragma unroll
        for (int i = 0; i < DT; ++i) {
            const int lr = warp * 16 + gq;
            *reinterpret_cast<uint32_t*>(s_q + tile_off<D>(lr, i) + tq * 4) = pack_elem(acc_o[i][0] * inv[0], acc_o[i][1] * inv[0]);
            *reinterpret_cast<uint32_t*>(s_q + tile_off<D>(lr + 8, i) + tq * 4) = pack_elem(acc_o[i][2] * inv[1], acc_o[i][3] * inv[1]);
        }
        if (tq == 0) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int slot = warp * 16 + gq + 8 * h;
                if (slot < r.n) lse[(sample_off + (size_t)tokb[slot]) * g.heads + head] = (mx[h] + log2f(l_row[h])) * kLn2;
            }
        }
        __syncthreads();
        constexpr int CPR = D / 8;
        for (int idx = tid; idx < BM * CPR; idx += NTHREADS) {
            const int row = idx / CPR, chunk = idx - row * CPR;
            if (row < r.n) {
                const uint4 val = *reinterpret_cast<const uint4*>(s_q + tile_off<D>(row, chunk));
                *reinterpret_cast<uint4*>(o + ((sample_off + (size_t)tokb[row]) * g.heads + head) * D + chunk * 8) = val;
            }
        }
        __syncthreads();   // the buffer's tiles and tables are free for the item after next
    }
}

size_t fwd_smem_bytes(const Geo& g) {
    int npad_max = ((g.nmax + BN - 1) / BN) * BN;
    int nbias = (2 * g.w - 1) * (2 * g.w - 1);
    size_t head = g.w > 32 ? (size_t)3 * BN * 8 : (((size_t)npad_max * 8 + (size_t)nbias * 4 + 127) / 128) * 128;
    const int nstages = (g.w > 32 || npad_max > BN) ? 2 : 1;
    return head + (size_t)(1 + 2 * nstages) * BN * g.d * 2;
}

}  // namespace

cudaError_t TERRA_ELEM_FN(launch_fwd_mma)(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                           void* o, float* lse, cudaStream_t stream) {
    if (g.nmax <= BN && g.w <= 32) {
        // windows of at most 64 tokens: the persistent double-buffered kernel
        auto kern = g.d == 32 ? swin_fwd_small_kernel<32> : g.d == 64 ? swin_fwd_small_kernel<64> : swin_fwd_small_kernel<128>;
        const int nbias = (2 * g.w - 1) * (2 * g.w - 1);
        const size_t smem = (((size_t)BN * 16 + (size_t)nbias * 4 + 127) / 128) * 128 + 6 * (size_t)BN * g.d * 2;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        int occ = 0, dev = 0, sms = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, NTHREADS, smem);
        if (e == cudaSuccess) e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        if (occ < 1) occ = 1;
        const long long items = (long long)g.B * g.Mh * g.Mw;
        long long cph = ((long long)sms * occ) / g.heads;
        if (cph < 1) cph = 1;
        if (cph > items) cph = items;
        prof_begin("swin_fwd_small_kernel", stream);
        kern<<<(unsigned)(cph * g.heads), NTHREADS, smem, stream>>>(g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k,
                                                                   (const __nv_bfloat16*)v, bias, (__nv_bfloat16*)o, lse, (int)cph);
        count_launch(stream);
        return cudaGetLastError();
    }
    const int qtiles = (g.nmax + BM - 1) / BM;
    const long long items = (long long)g.B * g.Mh * g.Mw * g.heads * qtiles;
    const size_t smem = fwd_smem_bytes(g);
    auto kern = g.w > 32 ? ((g.d == 32) ? swin_fwd_mma_kernel<32, true> : (g.d == 64) ? swin_fwd_mma_kernel<64, true> : swin_fwd_mma_kernel<128, true>)
                         : ((g.d == 32) ? swin_fwd_mma_kernel<32, false> : (g.d == 64) ? swin_fwd_mma_kernel<64, false> : swin_fwd_mma_kernel<128, false>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    prof_begin("swin_fwd_mma_kernel", stream);
    kern<<<(unsigned)items, NTHREADS, smem, stream>>>(g, (const __nv_bfloat16*)q, (const __nv_bfloat16*)k,
                                                      (const __nv_bfloat16*)v, bias, (__nv_bfloat16*)o, lse, qtiles);
    count_launch(stream);
    return cudaGetLastError();
}

}  // namespace terra
