// Complete-window ("padded") mode: the paper pads the grid so that every window is complete (Section IV-B; Eq. 3) and
// runs the Transformer blocks on the padded token grid.  These two kernels move a [B, H, W, C] tensor into the top-left
// corner of a zero-filled [B, H_pad, W_pad, C] one and back; the attention entry points then see a grid that the window
// side divides.
#include <stdint.h>

#include "../../include/terra.h"
#include "swin_kernels.h"

namespace terra {

int report_cuda_failure(cudaError_t e, const char* where);

namespace {

// PAD: y[b, u, v, :] = u < H && v < W ? x[b, u, v, :] : 0 over the padded grid; else x[b, u, v, :] = y[b, u, v, :] over the grid
template <bool PAD, typename T>
__global__ void __launch_bounds__(256)
swin_pad_crop_kernel(const T* __restrict__ src, T* __restrict__ dst, int H, int W, int Hp, int Wp, int chunks, long long total) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int c = (int)(i % chunks);
    long long t = i / chunks;
    const int Wo = PAD ? Wp : W, Ho = PAD ? Hp : H;        // extents of the tensor this kernel writes
    const int v = (int)(t % Wo);
    t /= Wo;
    const int u = (int)(t % Ho);
    const long long b = t / Ho;
    if (PAD) {
        T val = T();
        if (u < H && v < W) val = src[((b * H + u) * W + v) * chunks + c];
        dst[i] = val;
    } else {
        dst[i] = src[((b * Hp + u) * Wp + v) * chunks + c];
    }
}

int pad_crop(bool pad, const void* src, void* dst, int32_t B, int32_t H, int32_t W, int32_t Hp, int32_t Wp, int64_t token_bytes,
             void* stream) {
    if (!src || !dst || B < 1 || H < 1 || W < 1 || Hp < H || Wp < W || token_bytes < 4 || (token_bytes & 3)) return TERRA_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15u) != 0) return TERRA_ERR_ALIGNMENT;
    const bool wide = (token_bytes & 15) == 0;                  // 16 bytes per thread where the token size allows, else 4
    const long long per_token = token_bytes / (wide ? 16 : 4);
    if (per_token > 0x7fffffffLL) return TERRA_ERR_INVALID_ARG;
    const int chunks = (int)per_token;
    const long long total = (long long)B * (pad ? Hp : H) * (pad ? Wp : W) * chunks;
    if (total > (1LL << 40)) return TERRA_ERR_INVALID_ARG;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    cudaStream_t st = (cudaStream_t)stream;
    if (pad && wide) swin_pad_crop_kernel<true, uint4><<<blocks, 256, 0, st>>>((const uint4*)src, (uint4*)dst, H, W, Hp, Wp, chunks, total);
    else if (pad) swin_pad_crop_kernel<true, uint32_t><<<blocks, 256, 0, st>>>((const uint32_t*)src, (uint32_t*)dst, H, W, Hp, Wp, chunks, total);
    else if (wide) swin_pad_crop_kernel<false, uint4><<<blocks, 256, 0, st>>>((const uint4*)src, (uint4*)dst, H, W, Hp, Wp, chunks, total);
    else swin_pad_crop_kernel<false, uint32_t><<<blocks, 256, 0, st>>>((const uint32_t*)src, (uint32_t*)dst, H, W, Hp, Wp, chunks, total);
    count_launch((cudaStream_t)stream);
    const cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? TERRA_OK : report_cuda_failure(e, pad ? "terra_pad_grid" : "terra_crop_grid");
}

}  // namespace
}  // namespace terra

extern "C" int terra_pad_grid(const void* x, void* y, int32_t B, int32_t H, int32_t W, int32_t H_pad, int32_t W_pad,
                              int64_t token_bytes, void* stream) {
    return terra::pad_crop(true, x, y, B, H, W, H_pad, W_pad, token_bytes, stream);
}

extern "C" int terra_crop_grid(const void* y, void* x, int32_t B, int32_t H, int32_t W, int32_t H_pad, int32_t W_pad,
                               int64_t token_bytes, void* stream) {
    return terra::pad_crop(false, y, x, B, H, W, H_pad, W_pad, token_bytes, stream);
}
