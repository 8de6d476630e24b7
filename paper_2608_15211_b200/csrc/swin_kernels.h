// Host-side launch interface between the C ABI (api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "swin_common.cuh"

namespace terra {

void count_launch(cudaStream_t stream);   // after every launch: bumps the launch counter, closes an open timing scope
// Optional per-kernel timing (terra_profile_*): opens a scope (CUDA event on `stream`) that the next
// count_launch closes.  Does nothing unless profiling is enabled.
void prof_begin(const char* name, cudaStream_t stream);

cudaError_t launch_route(const Geo& g, int32_t* perm, int32_t* inv_perm, int32_t* win_offsets,
                         int32_t* pos, int32_t* label, cudaStream_t stream);

cudaError_t launch_fwd_mma(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                           void* o, float* lse, cudaStream_t stream);
// the register-tile kernels for fp16 activations and gradients (same arguments)
cudaError_t launch_fwd_mma_f16(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                               void* o, float* lse, cudaStream_t stream);
bool bwd_small_supported_f16(const Geo& g);
cudaError_t launch_bwd_small_f16(const Geo& g, const void* q, const void* k, const void* v, const void* o, const void* d_o,
                                 const float* bias, const float* lse, void* dq, void* dk, void* dv, float* dbias,
                                 int sm_count, cudaStream_t stream);
// the tcgen05 kernels compiled for fp16 activations (same shapes, workspaces and helpers as the bf16 ones)
cudaError_t launch_fwd_tc_f16(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                              void* o, float* lse, void* workspace, int sm_count, cudaStream_t stream);
cudaError_t read_tc_status_f16(int* timed_out, cudaStream_t stream);
cudaError_t launch_bwd_tc_f16(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                              const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, float* dbias,
                              void* workspace, int sm_count, cudaStream_t stream);
cudaError_t read_bwd_tc_status_f16(int* timed_out);
cudaError_t launch_fwd_tc64_f16(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                                void* o, float* lse, void* workspace, int sm_count, cudaStream_t stream);
cudaError_t read_fwd_tc64_status_f16(int* timed_out);
cudaError_t launch_bwd_kv64_f16(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                                const float* lse, const float* delta, void* dk, void* dv, int sm_count, cudaStream_t stream);
cudaError_t read_bwd_kv64_status_f16(int* timed_out);
cudaError_t launch_bwd_kv64_qside_f16(const Geo& g, const void* q, const void* k, const void* v, const void* d_o,
                                      const float* prep_reflected, const float* lse, const float* delta, void* dq, float* dbias,
                                      int sm_count, cudaStream_t stream);
cudaError_t launch_bwd_q64_f16(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                               const float* lse, const float* delta, void* dq, float* dbias, int sm_count, cudaStream_t stream);
cudaError_t read_bwd_q64_status_f16(int* timed_out);
cudaError_t launch_bwd_delta_f16(const Geo& g, const void* o, const void* d_o, float* delta, cudaStream_t stream);
cudaError_t launch_bwd_mma_f16(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                               const float* lse, const float* delta, const void* d_o,
                               void* dq, void* dk, void* dv, float* dbias, int sm_count, cudaStream_t stream,
                               bool query_side_only = false);

// tcgen05 forward path (head dim 32, window side <= 16)
constexpr int kFwdBiasFloats = 2304;   // prepared bias table per head (padded rows, -inf zone, maximum in the last float)
bool fwd_tc_supported(const Geo& g);
bool pad16_layout(const Geo& g);       // window sides 9 .. 15: slots laid out 16 to a window row, bias codes with stride 48
size_t fwd_tc_workspace_bytes(const Geo& g);
cudaError_t launch_fwd_tc(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                          void* o, float* lse, void* workspace, int sm_count, cudaStream_t stream);
// synchronises the stream, reads and clears the device-side "a bounded wait expired" word
cudaError_t read_tc_status(int* timed_out, cudaStream_t stream);

// TMA variants of the two kernels above (grids of 16-wide windows whose window rows are runs of consecutive tokens):
// the shape test, and the encoder of a [tokens][channels] tensor map with a box of 32 channels x box_tokens tokens
bool tma_row_shape(const Geo& g);
bool make_row_map(void* cu_tensor_map, const Geo& g, const void* base, int token_stride, int box_tokens);

// tcgen05 forward path for head dim 64 and windows of up to 1024 tokens (keys streamed in chunks, two passes)
bool fwd_tc64_supported(const Geo& g);
size_t fwd_tc64_workspace_bytes(const Geo& g);
cudaError_t launch_fwd_tc64(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                            void* o, float* lse, void* workspace, int sm_count, cudaStream_t stream);
cudaError_t read_fwd_tc64_status(int* timed_out);     // after the stream has been synchronised
// (window sides 64 and 128: whole table rows; `reflect`: the table reflected through its centre)
cudaError_t launch_bias_prep64(const Geo& g, const float* bias, float* prep, cudaStream_t stream, bool reflect = false);

// tcgen05 key side (dK, dV) of the backward pass for head dim 64 and windows of up to 1024 tokens; `prep` = the
// tables of launch_bias_prep64, `delta` as for the register-tile kernels
bool bwd_kv64_supported(const Geo& g);
cudaError_t launch_bwd_kv64(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                            const float* lse, const float* delta, void* dk, void* dv, int sm_count, cudaStream_t stream);
cudaError_t read_bwd_kv64_status(int* timed_out);
// the query side (dQ, dBias) of complete windows of side 64 and 128 with the same kernel; `prep_reflected` = the
// tables of launch_bias_prep64 with reflect = true; dbias is overwritten
cudaError_t launch_bwd_kv64_qside(const Geo& g, const void* q, const void* k, const void* v, const void* d_o,
                                  const float* prep_reflected, const float* lse, const float* delta, void* dq, float* dbias,
                                  int sm_count, cudaStream_t stream);

// tcgen05 query side (dQ, dBias) of the same regime for complete 32 x 32 windows (window side 32, grid extents
// multiples of 32); dbias is overwritten
bool bwd_q64_supported(const Geo& g);
cudaError_t launch_bwd_q64(const Geo& g, const void* q, const void* k, const void* v, const void* d_o, const float* prep,
                           const float* lse, const float* delta, void* dq, float* dbias, int sm_count, cudaStream_t stream);
cudaError_t read_bwd_q64_status(int* timed_out);

cudaError_t launch_bounded_wait_selftest(long long limit_cycles, cudaStream_t stream);
cudaError_t launch_bias_prep(const Geo& g, const float* bias, float* prep, cudaStream_t stream);

// tcgen05 backward path (head dim 32, window side <= 16)
bool bwd_tc_supported(const Geo& g);
size_t bwd_tc_workspace_bytes(const Geo& g);
cudaError_t launch_bwd_tc(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                          const void* o, const float* lse, const void* d_o, void* dq, void* dk, void* dv, float* dbias,
                          void* workspace, int sm_count, cudaStream_t stream);
cudaError_t read_bwd_tc_status(int* timed_out);

// delta[b, token, head] = sum_c dO * O   (fp32, same indexing as lse)
// the whole backward in one kernel for windows of at most 64 tokens (no delta kernel, no workspace)
bool bwd_small_supported(const Geo& g);
cudaError_t launch_bwd_small(const Geo& g, const void* q, const void* k, const void* v, const void* o, const void* d_o,
                             const float* bias, const float* lse, void* dq, void* dk, void* dv, float* dbias,
                             int sm_count, cudaStream_t stream);
cudaError_t launch_bwd_delta(const Geo& g, const void* o, const void* d_o, float* delta, cudaStream_t stream);

// dK, dV (key-tile CTAs) and dQ, dBias (query-tile CTAs)
cudaError_t launch_bwd_mma(const Geo& g, const void* q, const void* k, const void* v, const float* bias,
                           const float* lse, const float* delta, const void* d_o,
                           void* dq, void* dk, void* dv, float* dbias, int sm_count, cudaStream_t stream,
                           bool query_side_only = false);

}  // namespace terra
