// Forward entry point for callers that cannot hand the library a workspace: the scratch of the forward
// kernel (one prepared bias table per head) lives in a fixed array inside the library's device image.
#include <mutex>

#include "../../include/terra.h"
#include "swin_kernels.h"

namespace terra {

int resolve_attention_geo(const terra_swin_desc* d, Geo* out);
int current_device_sm_count(int* sm_count);
int report_cuda_failure(cudaError_t e, const char* where);

namespace {

constexpr int kNoAllocMaxHeads = TERRA_NOALLOC_MAX_HEADS;
constexpr int kMaxDevices = 64;

// Every GPU that loads the library carries this array (TERRA_NOALLOC_MAX_HEADS * 9216 bytes) until the
// process exits.  Host code must not use the name as a pointer: it is only a handle for
// cudaGetSymbolAddress, which yields the array's address on the device that is current at that moment.
static __device__ __align__(256) float g_noalloc_bias_scratch[kNoAllocMaxHeads * kFwdBiasFloats];

std::mutex g_setup_mutex;
float* g_scratch_on_device[kMaxDevices] = {};

// First call on a device: look the array's device address up (with that device current) and keep it.
int scratch_for_current_device(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return report_cuda_failure(e, "cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return TERRA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_on_device[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_bias_scratch);
        if (e != cudaSuccess) return report_cuda_failure(e, "cudaGetSymbolAddress(no-alloc scratch)");
        if (!p) return TERRA_ERR_CUDA;
        g_scratch_on_device[dev] = static_cast<float*>(p);
    }
    *out = g_scratch_on_device[dev];
    return TERRA_OK;
}

}  // namespace
}  // namespace terra

using namespace terra;

extern "C" int terra_swin_attn_fwd_noalloc(const terra_swin_desc* desc, const void* q, const void* k, const void* v,
                                           const float* bias_table, void* o, float* lse, void* stream) {
    Geo g;
    int rc = resolve_attention_geo(desc, &g);
    if (rc) return rc;
    if (!q || !k || !v || !bias_table || !o || !lse) return TERRA_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, bias_table, o, lse};
    for (const void* p : ptrs)
        if ((reinterpret_cast<uintptr_t>(p) & 15u) != 0) return TERRA_ERR_ALIGNMENT;
    int sms = 0;
    rc = current_device_sm_count(&sms);
    if (rc) return rc;
    cudaError_t e;
    if (fwd_tc_supported(g) && g.nmax > 64) {        // (windows of at most 64 tokens: the register-tile kernel, as in the regular forward)
        // the one shape-dependent limit of this entry point: the fixed scratch holds this many heads
        if (g.heads > kNoAllocMaxHeads) return TERRA_ERR_NOALLOC_LIMIT;
        float* scratch = nullptr;
        rc = scratch_for_current_device(&scratch);
        if (rc) return rc;
        e = g.f16 ? launch_fwd_tc_f16(g, q, k, v, bias_table, o, lse, scratch, sms, (cudaStream_t)stream)
                  : launch_fwd_tc(g, q, k, v, bias_table, o, lse, scratch, sms, (cudaStream_t)stream);
    } else {
        // this kernel needs no scratch
        e = g.f16 ? launch_fwd_mma_f16(g, q, k, v, bias_table, o, lse, (cudaStream_t)stream)
                  : launch_fwd_mma(g, q, k, v, bias_table, o, lse, (cudaStream_t)stream);
    }
    return e == cudaSuccess ? TERRA_OK : report_cuda_failure(e, "terra_swin_attn_fwd_noalloc");
}
