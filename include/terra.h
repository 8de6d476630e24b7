/*
 * terra.h -- C ABI of the B200 (sm_100a) shifted-window attention block.
 *
 * The block is the Swin-style window attention of the TERRA forecaster (paper Section IV-A:
 * W-MSA / SW-MSA inside each Transformer block), fed from the spatially contiguous lat-lon token
 * grid that the convolutional sampling modules produce and returned to it (Section IV-D: the token
 * route converts between the contiguous layout and the window-major layout using the global token
 * coordinate (u, v), window (floor(u/w), floor(v/w)) and offset (u mod w, v mod w); the shift route
 * changes the token coordinate, and the backward pass applies the inverse mapping).
 *
 * Conventions fixed by this library where the paper is silent:
 *   - the shift is a cyclic roll by -shift: token (u, v) sits at u' = (u - shift_h) mod H,
 *     v' = (v - shift_w) mod W, and windows tile the (u', v') frame, row-major (Section V-A);
 *   - the last window row / column is truncated when w does not divide H / W (no padding tokens);
 *   - on a non-periodic axis tokens that wrapped across the edge (u < shift_h, v < shift_w) only
 *     attend to each other (shift mask); a periodic axis has no mask;
 *   - scores are scale * <q, k> + T[(a_q - a_k + w - 1) * (2w - 1) + (b_q - b_k + w - 1), head]
 *     with (a, b) the in-window offsets; masked pairs get probability exactly zero.
 *
 * All pointers are DEVICE pointers unless stated otherwise, 16-byte aligned, owned by the caller.
 * The device that holds them must be the CURRENT device of the calling thread (cudaSetDevice): every entry
 * point launches on the current device and takes its SM count, and the built-in scratch of
 * terra_swin_attn_fwd_noalloc, from it.
 * Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream)
 * and return without synchronising.  No call allocates device memory; scratch comes from the
 * caller's workspace.  Every function returns a terra_status; nothing throws, nothing falls back to
 * the CPU.  Outputs must not alias inputs.
 */
#ifndef TERRA_H_
#define TERRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TERRA_OK = 0,
    TERRA_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, element count out of range   */
    TERRA_ERR_UNSUPPORTED = 2,   /* head_dim not in {32, 64, 128}, window too large, not an sm_100 GPU */
    TERRA_ERR_ALIGNMENT = 3,     /* a pointer is not 16-byte aligned                              */
    TERRA_ERR_WORKSPACE = 4,     /* workspace NULL or smaller than terra_swin_workspace_bytes     */
    TERRA_ERR_CUDA = 5,          /* a CUDA call failed; text via terra_last_cuda_error            */
    TERRA_ERR_DEVICE_TIMEOUT = 6,/* a bounded wait inside a kernel expired (see terra_swin_check) */
    TERRA_ERR_NOALLOC_LIMIT = 7  /* terra_swin_attn_fwd_noalloc: more heads than its fixed scratch holds */
} terra_status;

/*
 * Element type of the activations and their gradients: bf16, or fp16, which is what the paper trains in (Section
 * VII-A: FP16 mixed precision).  Every kernel of the library exists in a build for either type and the same kernel is
 * chosen for a shape whatever the type.  Scores, softmax, accumulation, lse, bias_table and dbias are fp32 either
 * way.  A descriptor zero-initialised beyond `scale` selects bf16.
 */
#define TERRA_DTYPE_BF16 0
#define TERRA_DTYPE_F16 1

/* Largest `heads` terra_swin_attn_fwd_noalloc accepts on the shapes that need scratch. */
#define TERRA_NOALLOC_MAX_HEADS 64

/* Problem statement: token grid, window, heads (paper Table I symbols; H, W here are H_T, W_T). */
typedef struct {
    int32_t B;                      /* batch (samples / rollout steps), >= 1                      */
    int32_t H, W;                   /* token grid: latitude rows x longitude columns              */
    int32_t heads, head_dim;        /* attention heads; per-head width: 32, 64 or 128 (Table V)   */
    int32_t window;                 /* w: square window side, 1 <= w <= 128                       */
    int32_t shift_h, shift_w;       /* >= 0, taken mod H and mod W                                */
    int32_t periodic_h, periodic_w; /* 0 / 1; the paper's grids: latitude 0, longitude 1          */
    float scale;                    /* score scale; <= 0 selects 1/sqrt(head_dim)                 */
    int32_t dtype;                  /* element type of q, k, v, o, d_o, dq, dk, dv: TERRA_DTYPE_*   */
} terra_swin_desc;

/*
 * Sizes of the route arrays (Section IV-D window grid: M_h = ceil(H/w), M_w = ceil(W/w)).
 * Host-only.  Any output may be NULL.
 *   n_tokens = H * W, n_windows = M_h * M_w, max_window_tokens = min(w, H) * min(w, W).
 */
int terra_route_sizes(const terra_swin_desc* desc, int64_t* n_tokens, int32_t* n_windows,
                      int32_t* max_window_tokens);

/*
 * Token route (Section IV-D, with the shift route folded in): the integer map between the
 * contiguous grid and the window-major layout, for one sample (all samples share it).
 *   win_offsets [n_windows + 1]  first slot of window g = wr * M_w + wc; last entry = H * W
 *   perm        [H * W]          perm[slot] = u * W + v, the grid token stored in that slot; slots
 *                                inside a window run row-major over the window's true extent
 *   inv_perm    [H * W]          inv_perm[u * W + v] = slot
 *   pos         [H * W]          pos[slot] = a * w + b, the in-window offset
 *   label       [H * W]          label[slot] = 2 * [lat non-periodic and u < shift_h]
 *                                              + [lon non-periodic and v < shift_w]
 * int32 device arrays; any may be NULL to skip it.  Exact integer work.
 */
int terra_window_route(const terra_swin_desc* desc, int32_t* perm, int32_t* inv_perm,
                       int32_t* win_offsets, int32_t* pos, int32_t* label, void* stream);

/* Scratch bytes the forward (backward = 0) or backward (backward = 1) call needs.  Host-only. */
int terra_swin_workspace_bytes(const terra_swin_desc* desc, int backward, size_t* bytes);

/*
 * Forward shifted-window attention (Section IV-A W-MSA / SW-MSA; route + attention + inverse route
 * in one pass).
 *   q, k, v      bf16 (fp16 with TERRA_DTYPE_F16, like every "bf16" below) [B, H, W, heads, head_dim], innermost
 *                contiguous (the contiguous grid layout)
 *   bias_table   fp32 [(2w-1)^2, heads]
 *   o            bf16 [B, H, W, heads, head_dim]   attention output at the token's grid position
 *   lse          fp32 [B, H, W, heads]             natural-log sum-exp of each score row (for bwd)
 *   workspace    >= terra_swin_workspace_bytes(desc, 0) bytes (may be NULL when that is 0)
 */
int terra_swin_attn_fwd(const terra_swin_desc* desc, const void* q, const void* k, const void* v,
                        const float* bias_table, void* o, float* lse,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward of terra_swin_attn_fwd (Section IV-D: gradients return through the inverse routes).
 *   q, k, v, o, lse   as given to / produced by the forward call
 *   d_o               bf16 [B, H, W, heads, head_dim]   upstream gradient
 *   dq, dk, dv        bf16 [B, H, W, heads, head_dim]   overwritten
 *   dbias             fp32 [(2w-1)^2, heads]            overwritten (summed over batch and windows; in a fixed
 *                                                       order, hence reproducible run to run, for head_dim 32
 *                                                       with window <= 16; with atomics, hence in no fixed
 *                                                       order, for the other shapes)
 *   workspace         >= terra_swin_workspace_bytes(desc, 1) bytes
 */
int terra_swin_attn_bwd(const terra_swin_desc* desc, const void* q, const void* k, const void* v,
                        const float* bias_table, const void* o, const float* lse, const void* d_o,
                        void* dq, void* dk, void* dv, float* dbias,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * The same two passes on the packed layout of a fused QKV projection (the block sits between that GEMM and the
 * output projection, Section IV-A; the paper has no layout statement, this is the library's): the GEMM's output
 * is consumed in place and the gradient comes back in the layout that GEMM's backward reads, with no re-layout
 * pass in between.
 *   qkv    bf16 [B, H, W, 3, heads, head_dim]   q = [..., 0, :, :], k = [..., 1, :, :], v = [..., 2, :, :]
 *   dqkv   bf16 [B, H, W, 3, heads, head_dim]   overwritten: dq, dk, dv in the same three slots
 *   o, lse, d_o, bias_table, dbias, workspace   as in terra_swin_attn_fwd / terra_swin_attn_bwd (o and d_o dense
 *                                               [B, H, W, heads, head_dim]); same sizes from terra_swin_workspace_bytes
 * Results are those of the unpacked calls on the three slices, bit for bit; same error codes.
 */
int terra_swin_attn_fwd_packed(const terra_swin_desc* desc, const void* qkv, const float* bias_table, void* o, float* lse,
                               void* workspace, size_t workspace_bytes, void* stream);
int terra_swin_attn_bwd_packed(const terra_swin_desc* desc, const void* qkv, const float* bias_table, const void* o,
                               const float* lse, const void* d_o, void* dqkv, float* dbias,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Forward pass without a workspace argument.  (The paper has no counterpart: this exists for the way the
 * library is embedded, not for the method.)
 *
 * Who needs it: code that runs where device memory may not be requested -- a plug-in inside a serving
 * process whose memory is owned by a pool it cannot reach, a real-time loop that was handed all of its
 * buffers up front, a callback from which cudaMalloc is off limits.  Such a caller still brings the inputs
 * and outputs, but has nowhere to get the forward kernel's scratch (one prepared bias table per head) from.
 * Here that scratch is a fixed array compiled into the library: TERRA_NOALLOC_MAX_HEADS * 9216 bytes
 * (576 KiB) on every GPU that loads the library, held until the process exits.  The call itself allocates
 * nothing: no cudaMalloc / cudaFree, no allocating library routine.  One thing happens once per device: under
 * CUDA's lazy module loading the FIRST call on a device is what makes the driver load the code module that
 * holds the array and place it in that device's memory.  So make one warm-up call per device during
 * initialisation -- outside any callback, real-time section or stream capture -- and only later calls are
 * free of loading and allocation.
 *
 * Arguments, layouts and error codes are those of terra_swin_attn_fwd.  Results: the same within the
 * library's tolerance; bit-equal to terra_swin_attn_fwd for head_dim 32 with window <= 16, where both run the
 * same kernel (the tensor-core kernel for windows of more than 64 tokens, the register-tile kernel for smaller
 * ones), and for every shape whose windows hold at most 64 tokens.  For every other shape this entry point runs
 * the register-tile forward kernel (`swin_fwd_mma_kernel`, which needs no scratch) while terra_swin_attn_fwd
 * may pick a faster chunked tensor-core kernel that does need a workspace: equal within tolerance, not bit for
 * bit, and slower.
 * Extra rules:
 *   - heads > TERRA_NOALLOC_MAX_HEADS is refused with TERRA_ERR_NOALLOC_LIMIT when the shape uses the
 *     scratch (head_dim 32, window <= 16, windows of more than 64 tokens); other shapes need no scratch and are
 *     not limited;
 *   - the first call on each device looks the array's device address up (the device must be current);
 *     make that first call before any stream capture begins;
 *   - all calls on a device share the one array and every call rewrites the part it uses, so nothing has to
 *     be cleared in between; but two calls that overlap on the GPU (different streams) race on it and give
 *     wrong results -- keep calls to this entry point ordered on one stream per device.
 */
int terra_swin_attn_fwd_noalloc(const terra_swin_desc* desc, const void* q, const void* k, const void* v,
                                const float* bias_table, void* o, float* lse, void* stream);

/*
 * Waits for `stream` and reports whether any kernel of this library gave up on a bounded wait since
 * the last check (the kernels never spin forever: a wait on a barrier has a cycle limit, after which the
 * CTA stops working, releases its tensor memory and raises a device-side word).  Returns TERRA_OK or
 * TERRA_ERR_DEVICE_TIMEOUT (and clears the word).  The paper has no counterpart; this is the library's
 * own failure report.
 */
int terra_swin_check(void* stream);

/*
 * Self-test of the failure report above (the paper has no counterpart): launches one small CTA that waits on
 * a barrier nobody arrives on, with a limit of `limit_cycles` SM clocks (1 .. 2e9).  The wait expires, the
 * kernel ends normally, and the next terra_swin_check returns TERRA_ERR_DEVICE_TIMEOUT.  Nothing hangs or
 * faults; the context stays usable.
 */
int terra_selftest_bounded_wait(long long limit_cycles, void* stream);

/*
 * Per-kernel timing for benchmarks (the paper has no counterpart).  While enabled, the library brackets each
 * of its main kernel launches with CUDA events on the launching stream.  terra_profile_enable(1) clears the
 * record and starts, (0) clears and stops; terra_profile_count gives the number of recorded launches;
 * terra_profile_get waits for launch `index` and returns its kernel name (truncated to name_bytes) and
 * duration in milliseconds.  Host-only; off by default; not meant for use during stream capture.
 */
int terra_profile_enable(int on);
int terra_profile_count(void);
int terra_profile_get(int index, char* name, int name_bytes, float* ms);

/*
 * Complete-window ("padded") mode (Section IV-B and Eq. 3: the paper pads the grid so that every window is complete,
 * and the padded tokens are ordinary tokens of the Transformer blocks).  The attention entry points truncate the last
 * window row / column of a grid that the window side does not divide; a caller who wants the paper's padded
 * execution instead keeps its activations on the padded token grid H_pad x W_pad (multiples of the window side; for
 * the fixed assignment of Eq. 3 multiples of w m and w n) and describes THAT grid to the attention calls.  These two
 * calls move a tensor between the two grids:
 *   terra_pad_grid   y [B, H_pad, W_pad, token_bytes] = x [B, H, W, token_bytes] in the top-left corner, zeros elsewhere
 *   terra_crop_grid  x [B, H, W, token_bytes] = the top-left corner of y (the backward of the padding, and the way
 *                    results leave the padded grid)
 * token_bytes = bytes per token (for [.., heads, head_dim] bf16: heads * head_dim * 2; for lse: heads * 4), a multiple of 4; device
 * pointers, 16-byte aligned, no overlap.  H_pad >= H, W_pad >= W.  Errors: TERRA_ERR_INVALID_ARG,
 * TERRA_ERR_ALIGNMENT, TERRA_ERR_CUDA.
 */
int terra_pad_grid(const void* x, void* y, int32_t B, int32_t H, int32_t W, int32_t H_pad, int32_t W_pad,
                   int64_t token_bytes, void* stream);
int terra_crop_grid(const void* y, void* x, int32_t B, int32_t H, int32_t W, int32_t H_pad, int32_t W_pad,
                    int64_t token_bytes, void* stream);

/*
 * Window ownership across window-parallel (WP) ranks (Section V-A).  Host-only integer helpers; they launch
 * nothing and touch no device.  This library runs one GPU; these state which windows a rank of a WP group
 * would own, so that a caller sharding windows over several processes uses the paper's rule.
 *
 * terra_fixed_assignment_padding (Eq. 3): the fixed round-robin assignment over an m x n WP mesh needs every
 * rank to hold the same number of complete windows, so the INPUT field (H x W grid points, before patching) is
 * padded to  H_hat = ceil(H / (p alpha w m)) p alpha w m,  W_hat = ceil(W / (p alpha w n)) p alpha w n
 * (p patch size, alpha sampling factor, w window side in tokens).  m = n = 1 gives the padding to complete
 * windows alone, which is all the ragged assignment needs.  All arguments >= 1; results via H_hat, W_hat
 * (either may be NULL).  TERRA_ERR_INVALID_ARG on a non-positive argument or a product that overflows int64.
 *
 * terra_ragged_window_range (Eq. 4): with the M = M_h M_w complete windows numbered row-major, rank r of
 * `ranks` owns the contiguous range [L, R),  L = floor(r M / ranks),  R = floor((r + 1) M / ranks).  Every
 * window is owned exactly once and two ranks' counts differ by at most one.  M >= 0, ranks >= 1,
 * 0 <= r < ranks; else TERRA_ERR_INVALID_ARG.  Either output may be NULL.
 */
int terra_fixed_assignment_padding(int64_t H, int64_t W, int32_t p, int32_t alpha, int32_t w, int32_t m, int32_t n,
                                   int64_t* H_hat, int64_t* W_hat);
int terra_ragged_window_range(int64_t M, int32_t ranks, int32_t r, int64_t* L, int64_t* R);

/* Static text for a terra_status.  Host-only. */
const char* terra_strerror(int status);

/* Text of the last CUDA error this library saw on the calling thread ("" if none).  Host-only. */
const char* terra_last_cuda_error(void);

/* Number of kernels the library has launched in this process (monotonic).  Host-only. */
int64_t terra_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TERRA_H_ */
