// Window rows by tiled bulk copies (TMA), shared by the large-window tcgen05 kernels.
//
// On a grid of complete windows whose longitude shift is a multiple of 8, the tokens of one window row are one run of
// consecutive tokens of the tensor, or two where the rolled row crosses the longitude seam, each a multiple of 8 long.
// A tensor is described as [tokens, heads * d] with boxes of 32 columns (one 64-byte-swizzled part of a row) by 128,
// 64, 32, 16 or 8 tokens; a run is covered by the largest boxes that fit (the copy engine's time per box grows far
// slower than the box: 2 KB boxes reach a third of the bytes per clock of 8 KB boxes).
#pragma once
#include <cuda.h>

#include "swin_common.cuh"
#include "tc_common.cuh"

namespace terra {

struct RowMaps3 {
    // boxes of 32, 16, 8 tokens; then, at window sides 64 and 128, boxes of 64 and 128 tokens, and at window side 32 the
    // tensor as [token rows, token columns, heads * d] with boxes of 2 and 4 token rows x 32 token columns (2 and 4
    // window rows of a window in one copy)
    CUtensorMap m[5];
};

// host: the three maps of one tensor (`token_stride` in elements); false if the driver's encoder is not available
bool make_row_maps3(RowMaps3* maps, const Geo& g, const void* base, int token_stride);

// host: one tensor as [token rows, token columns, heads * d] with boxes of 32 columns x 1 token column x 16 token
// rows: 16 vertically adjacent tokens of one head become 16 consecutive 64-byte rows of a swizzled region
bool make_col_map(CUtensorMap* map, const Geo& g, const void* base, int token_stride);
// host: the same tensor with the token-row axis BEFORE the token-column axis ([token columns, token rows, heads * d]) and
// boxes of 32 columns x 16 token rows x 4 token columns: four runs of 16 vertically adjacent tokens in one copy.
// false if the encoder refuses the axis order (the callers then keep to make_col_map's boxes).
bool make_col_map4(CUtensorMap* map, const Geo& g, const void* base, int token_stride);

// host: the geometry the bulk-copy loaders are written for
inline bool bulk_rows_shape(const Geo& g) {
    return (g.w == 16 || g.w == 32 || g.w == 64 || g.w == 128) && g.H % g.w == 0 && g.W % g.w == 0 && g.sw % 8 == 0 &&
           (long long)g.B * g.H * g.W < 0x7fffffffLL;
}

// device: the copies of `n_run` slots (a multiple of 8) of window row `a`, from window column `b0` (a multiple of 8) on,
// of window row-index `wr` in sample `b`: 64 bytes per slot from `dst` on (a multiple of 512 bytes into a swizzled
// region), columns [xc, xc + 32) of every token; `v0` = the window's first token column after the roll.  The bytes
// are counted on `bar`.
__device__ __forceinline__ void bulk_copy_window_run(const RowMaps3& m3, uint32_t dst, const Geo& g, int b, int wr, int v0, int a,
                                                     int b0, int n_run, int xc, uint32_t bar) {
    int u = wr * g.w + a + g.sh;
    if (u >= g.H) u -= g.H;
    const int y0 = (b * g.H + u) * g.W;
    int vs = v0 + b0;
    if (vs >= g.W) vs -= g.W;
    const int n1 = min(n_run, g.W - vs);          // tokens up to the seam; the rest starts at column 0
    int y = y0 + vs, n = n1;
#pragma unroll
    for (int seg = 0; seg < 2; ++seg) {
        if (g.w >= 64) {
            while (n >= 128) { tc::tma_load_2d(dst, &m3.m[4], xc, y, bar); dst += 128 * 64; y += 128; n -= 128; }
            if (n >= 64) { tc::tma_load_2d(dst, &m3.m[3], xc, y, bar); dst += 64 * 64; y += 64; n -= 64; }
        }
        while (n >= 32) { tc::tma_load_2d(dst, &m3.m[0], xc, y, bar); dst += 32 * 64; y += 32; n -= 32; }
        if (n >= 16) { tc::tma_load_2d(dst, &m3.m[1], xc, y, bar); dst += 16 * 64; y += 16; n -= 16; }
        if (n >= 8) { tc::tma_load_2d(dst, &m3.m[2], xc, y, bar); dst += 8 * 64; }
        y = y0;
        n = n_run - n1;
    }
}
// the whole window row
__device__ __forceinline__ void bulk_copy_window_row(const RowMaps3& m3, uint32_t dst, const Geo& g, int b, int wr, int v0, int a,
                                                     int xc, uint32_t bar);
// `nrows` consecutive window rows a0, a0 + 1, .. into consecutive slots.  In a 32-wide window whose rows do not cross
// the longitude seam, groups of 4 or 2 window rows that do not cross the latitude wrap travel as one copy each.
__device__ __forceinline__ void bulk_copy_window_rows(const RowMaps3& m3, uint32_t dst, const Geo& g, int b, int wr, int v0, int a0,
                                                      int nrows, int xc, uint32_t bar) {
    const bool groups = g.w == 32 && v0 + 32 <= g.W;
    int a = a0;
    while (nrows > 0) {
        int u = wr * g.w + a + g.sh;
        if (u >= g.H) u -= g.H;
        if (groups && nrows >= 4 && u + 4 <= g.H) {
            tc::tma_load_3d(dst, &m3.m[4], xc, v0, b * g.H + u, bar);
            dst += 4 * 32 * 64; a += 4; nrows -= 4;
        } else if (groups && nrows >= 2 && u + 2 <= g.H) {
            tc::tma_load_3d(dst, &m3.m[3], xc, v0, b * g.H + u, bar);
            dst += 2 * 32 * 64; a += 2; nrows -= 2;
        } else {
            bulk_copy_window_row(m3, dst, g, b, wr, v0, a, xc, bar);
            dst += g.w * 64; ++a; --nrows;
        }
    }
}
__device__ __forceinline__ void bulk_copy_window_row(const RowMaps3& m3, uint32_t dst, const Geo& g, int b, int wr, int v0, int a,
                                                     int xc, uint32_t bar) {
    bulk_copy_window_run(m3, dst, g, b, wr, v0, a, 0, g.w, xc, bar);
}

}  // namespace terra
