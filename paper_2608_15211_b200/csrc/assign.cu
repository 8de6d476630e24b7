// Window ownership across window-parallel ranks (Section V-A, Eq. 3 and Eq. 4): host-side integer helpers.
#include <stdint.h>

#include "../../include/terra.h"

namespace {

// a * b with overflow check (both >= 1)
bool mul_ok(int64_t a, int64_t b, int64_t* out) { return !__builtin_mul_overflow(a, b, out); }

// ceil(x / unit) * unit for x, unit >= 1
bool round_up_to(int64_t x, int64_t unit, int64_t* out) {
    const int64_t q = (x + unit - 1) / unit;
    return mul_ok(q, unit, out);
}

}  // namespace

extern "C" int terra_fixed_assignment_padding(int64_t H, int64_t W, int32_t p, int32_t alpha, int32_t w, int32_t m,
                                              int32_t n, int64_t* H_hat, int64_t* W_hat) {
    if (H < 1 || W < 1 || p < 1 || alpha < 1 || w < 1 || m < 1 || n < 1) return TERRA_ERR_INVALID_ARG;
    int64_t unit;                                      // p alpha w: grid points per window side
    if (!mul_ok(p, alpha, &unit) || !mul_ok(unit, w, &unit)) return TERRA_ERR_INVALID_ARG;
    int64_t uh, uw, hh, ww;
    if (!mul_ok(unit, m, &uh) || !mul_ok(unit, n, &uw)) return TERRA_ERR_INVALID_ARG;
    if (H > INT64_MAX - uh || W > INT64_MAX - uw) return TERRA_ERR_INVALID_ARG;
    if (!round_up_to(H, uh, &hh) || !round_up_to(W, uw, &ww)) return TERRA_ERR_INVALID_ARG;
    if (H_hat) *H_hat = hh;
    if (W_hat) *W_hat = ww;
    return TERRA_OK;
}

extern "C" int terra_ragged_window_range(int64_t M, int32_t ranks, int32_t r, int64_t* L, int64_t* R) {
    if (M < 0 || ranks < 1 || r < 0 || r >= ranks) return TERRA_ERR_INVALID_ARG;
    // floor(r M / ranks) without forming r M: M = q ranks + rem  =>  r M / ranks = r q + floor(r rem / ranks)
    const int64_t q = M / ranks, rem = M % ranks;
    const int64_t lo = (int64_t)r * q + ((int64_t)r * rem) / ranks;
    const int64_t hi = (int64_t)(r + 1) * q + ((int64_t)(r + 1) * rem) / ranks;
    if (L) *L = lo;
    if (R) *R = hi;
    return TERRA_OK;
}
