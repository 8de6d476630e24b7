// Token route: the integer map between the contiguous lat-lon grid and the window-major layout
// (paper Section IV-D coordinates, with the window shift folded in as a cyclic roll).
#include "swin_common.cuh"
#include "swin_kernels.h"

namespace terra {

namespace {

// first slot of window (wr, wc): full window rows above it, then the windows to its left in this row
__device__ __forceinline__ int window_first_slot(const Geo& g, int wr, int wc) {
    int eh = min(g.w, g.H - wr * g.w);
    return wr * g.w * g.W + eh * wc * g.w;
}

__global__ void route_tokens_kernel(const Geo g, int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                                    int32_t* __restrict__ pos, int32_t* __restrict__ label) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;   // grid token u * W + v
    if (t >= g.H * g.W) return;
    const int u = t / g.W, v = t - u * g.W;
    int up = u - g.sh; if (up < 0) up += g.H;
    int vp = v - g.sw; if (vp < 0) vp += g.W;
    const int wr = up / g.w, wc = vp / g.w;
    const int a = up - wr * g.w, b = vp - wc * g.w;
    const int ew = min(g.w, g.W - wc * g.w);
    const int slot = window_first_slot(g, wr, wc) + a * ew + b;
    if (perm) perm[slot] = t;
    if (inv_perm) inv_perm[t] = slot;
    if (pos) pos[slot] = a * g.w + b;
    if (label) label[slot] = ((!g.ph && u < g.sh) ? 2 : 0) + ((!g.pw && v < g.sw) ? 1 : 0);
}

__global__ void route_offsets_kernel(const Geo g, int32_t* __restrict__ win_offsets) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int M = g.Mh * g.Mw;
    if (i > M) return;
    if (i == M) { win_offsets[i] = g.H * g.W; return; }
    const int wr = i / g.Mw, wc = i - wr * g.Mw;
    win_offsets[i] = window_first_slot(g, wr, wc);
}

}  // namespace

cudaError_t launch_route(const Geo& g, int32_t* perm, int32_t* inv_perm, int32_t* win_offsets,
                         int32_t* pos, int32_t* label, cudaStream_t stream) {
    if (perm || inv_perm || pos || label) {
        const int n = g.H * g.W;
        route_tokens_kernel<<<(n + 255) / 256, 256, 0, stream>>>(g, perm, inv_perm, pos, label);
        count_launch(stream);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (win_offsets) {
        const int n = g.Mh * g.Mw + 1;
        route_offsets_kernel<<<(n + 255) / 256, 256, 0, stream>>>(g, win_offsets);
        count_launch(stream);
        return cudaGetLastError();
    }
    return cudaSuccess;
}

}  // namespace terra
