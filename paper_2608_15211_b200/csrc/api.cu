// C ABI of the shifted-window attention library: argument checks, geometry, launches.
#include <atomic>
#include <mutex>
#include <vector>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "../../include/terra.h"
#include "swin_kernels.h"

namespace terra {

static std::atomic<long long> g_launches{0};

struct ProfEntry { const char* name; cudaEvent_t begin, end; bool closed; };
static std::mutex g_prof_mutex;
static bool g_prof_on = false;
static std::vector<ProfEntry> g_prof;

void prof_begin(const char* name, cudaStream_t stream) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (!g_prof_on) return;
    ProfEntry e{name, nullptr, nullptr, false};
    if (cudaEventCreate(&e.begin) != cudaSuccess || cudaEventCreate(&e.end) != cudaSuccess) return;
    cudaEventRecord(e.begin, stream);
    g_prof.push_back(e);
}

void count_launch(cudaStream_t stream) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (g_prof_on && !g_prof.empty() && !g_prof.back().closed) {
        cudaEventRecord(g_prof.back().end, stream);
        g_prof.back().closed = true;
    }
}

static void prof_clear() {
    for (auto& e : g_prof) { cudaEventDestroy(e.begin); cudaEventDestroy(e.end); }
    g_prof.clear();
}

static thread_local char g_cuda_error[256] = "";

static int cuda_fail(cudaError_t e, const char* where) {
    std::snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", where, cudaGetErrorString(e));
    return TERRA_ERR_CUDA;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Checks the descriptor and resolves the window geometry.  Host arithmetic only.
static int make_geo(const terra_swin_desc* d, bool for_attention, Geo* out) {
    if (!d) return TERRA_ERR_INVALID_ARG;
    if (d->B <= 0 || d->H <= 0 || d->W <= 0 || d->heads <= 0 || d->head_dim <= 0 || d->window <= 0 ||
        d->shift_h < 0 || d->shift_w < 0)
        return TERRA_ERR_INVALID_ARG;
    if ((long long)d->H * d->W > 0x7fffffffLL) return TERRA_ERR_INVALID_ARG;             // token index is int32
    if ((long long)d->B * d->H * d->W * d->heads > (1LL << 40)) return TERRA_ERR_INVALID_ARG;
    if (for_attention) {
        if (d->head_dim != 32 && d->head_dim != 64 && d->head_dim != 128) return TERRA_ERR_UNSUPPORTED;
        if (d->window > 128) return TERRA_ERR_UNSUPPORTED;
        if (!(d->scale == d->scale) || std::isinf(d->scale)) return TERRA_ERR_INVALID_ARG;
        if (d->dtype != TERRA_DTYPE_BF16 && d->dtype != TERRA_DTYPE_F16) return TERRA_ERR_INVALID_ARG;
    }
    Geo g;
    g.B = d->B; g.H = d->H; g.W = d->W;
    g.heads = d->heads; g.d = d->head_dim; g.w = d->window;
    g.ts = d->heads * d->head_dim;
    g.sh = d->shift_h % d->H; g.sw = d->shift_w % d->W;
    g.ph = d->periodic_h != 0; g.pw = d->periodic_w != 0;
    g.Mh = (d->H + d->window - 1) / d->window;
    g.Mw = (d->W + d->window - 1) / d->window;
    g.nmax = (d->window < d->H ? d->window : d->H) * (d->window < d->W ? d->window : d->W);
    g.f16 = for_attention && d->dtype == TERRA_DTYPE_F16;
    const float scale = d->scale > 0.f ? d->scale : 1.0f / std::sqrt((float)d->head_dim);
    g.scale_log2e = scale * kLog2e;
    *out = g;
    return TERRA_OK;
}

static int device_props(int* sm_count) {
    static thread_local int cached_dev = -1, cached_sms = 0, cached_major = 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev != cached_dev) {
        int sms = 0, major = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
        cached_dev = dev; cached_sms = sms; cached_major = major;
    }
    if (cached_major != 10) return TERRA_ERR_UNSUPPORTED;
    *sm_count = cached_sms;
    return TERRA_OK;
}

// Debugging switch: TERRA_REGISTER_PATH=1 routes every shape through the register-tile kernels.
static bool force_register_path() {
    static const bool on = [] {
        const char* v = std::getenv("TERRA_REGISTER_PATH");
        return v && v[0] == '1';
    }();
    return on;
}

// Windows of at most 64 tokens (the 8 x 8 windows of configs 1, 2 and of the paper's small and medium models) half
// fill a 128-row tcgen05 tile and are bound by HBM and launch overheads: the register-tile forward and the one-kernel
// register-tile backward are faster there at every head dim (config 2: 0.117 ms against 0.188 ms per step).
static bool small_windows(const Geo& g) { return g.nmax <= 64; }

// (every kernel exists for bf16 and for fp16 activations: `f16` only selects the build of the kernel)
static bool use_fwd_tc(const Geo& g) { return fwd_tc_supported(g) && !small_windows(g); }
// head dim 128 with windows of fewer than 256 tokens (the 8 x 8 windows of the paper's small and medium models): a
// 128-row tile would be mostly empty and the path is bound by HBM, the register-tile kernels are about twice as fast
static bool small_window_128(const Geo& g) { return (g.d == 128 && g.nmax < 256) || small_windows(g); }
static bool use_fwd_tc64(const Geo& g) { return fwd_tc64_supported(g) && !force_register_path() && !small_window_128(g); }

static size_t fwd_bytes(const Geo& g) {
    if (force_register_path()) return 0;
    if (use_fwd_tc(g)) return align_up(fwd_tc_workspace_bytes(g), 256);
    if (use_fwd_tc64(g)) return align_up(fwd_tc64_workspace_bytes(g), 256);
    return 0;
}

// TERRA_SPLIT_SMALL=1: a debugging switch that keeps small windows at head dim 128 on the two-kernel register-tile backward
static bool force_split_small() {
    static const bool on = [] {
        const char* v = std::getenv("TERRA_SPLIT_SMALL");
        return v && v[0] == '1';
    }();
    return on;
}

static bool use_bwd_tc(const Geo& g) { return bwd_tc_supported(g) && !force_register_path() && !small_windows(g); }

static bool use_bwd_kv64(const Geo& g) { return bwd_kv64_supported(g) && !force_register_path() && !small_window_128(g); }

static size_t delta_bytes(const Geo& g) {
    if (use_bwd_tc(g)) return align_up(bwd_tc_workspace_bytes(g), 256);
    const size_t delta = align_up(sizeof(float) * (size_t)g.B * g.H * g.W * g.heads, 256);
    // the tcgen05 key-side kernel of the head-dim-64 regime also wants the prepared bias tables
    // (windows of side 64 and 128: twice, the second copy reflected for the query-side use of that kernel)
    return use_bwd_kv64(g) ? delta + (g.w > 32 ? 2 : 1) * align_up(fwd_tc64_workspace_bytes(g), 256) : delta;
}

// Descriptor check + geometry, and the SM count of the current device, for entry points that live in
// other files of the library.
int resolve_attention_geo(const terra_swin_desc* d, Geo* out) { return make_geo(d, true, out); }
int current_device_sm_count(int* sm_count) { return device_props(sm_count); }
int report_cuda_failure(cudaError_t e, const char* where) { return cuda_fail(e, where); }

}  // namespace terra

using namespace terra;

extern "C" {

int terra_route_sizes(const terra_swin_desc* desc, int64_t* n_tokens, int32_t* n_windows,
                      int32_t* max_window_tokens) {
    Geo g;
    int rc = make_geo(desc, false, &g);
    if (rc) return rc;
    if (n_tokens) *n_tokens = (int64_t)g.H * g.W;
    if (n_windows) *n_windows = g.Mh * g.Mw;
    if (max_window_tokens) *max_window_tokens = g.nmax;
    return TERRA_OK;
}

int terra_window_route(const terra_swin_desc* desc, int32_t* perm, int32_t* inv_perm,
                       int32_t* win_offsets, int32_t* pos, int32_t* label, void* stream) {
    Geo g;
    int rc = make_geo(desc, false, &g);
    if (rc) return rc;
    cudaError_t e = launch_route(g, perm, inv_perm, win_offsets, pos, label, (cudaStream_t)stream);
    return e == cudaSuccess ? TERRA_OK : cuda_fail(e, "terra_window_route");
}

int terra_swin_workspace_bytes(const terra_swin_desc* desc, int backward, size_t* bytes) {
    Geo g;
    int rc = make_geo(desc, true, &g);
    if (rc) return rc;
    if (!bytes) return TERRA_ERR_INVALID_ARG;
    *bytes = backward ? delta_bytes(g) : fwd_bytes(g);
    return TERRA_OK;
}

// forward with q, k, v given as three pointers and one token stride (g.ts elements)
static int fwd_call(const Geo& g, const void* q, const void* k, const void* v,
                    const float* bias_table, void* o, float* lse,
                    void* workspace, size_t workspace_bytes, void* stream) {
    int rc;
    if (!q || !k || !v || !bias_table || !o || !lse) return TERRA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(bias_table) || !aligned16(lse))
        return TERRA_ERR_ALIGNMENT;
    const size_t need = fwd_bytes(g);
    if (need > 0 && (!workspace || workspace_bytes < need)) return TERRA_ERR_WORKSPACE;
    if (need > 0 && !aligned16(workspace)) return TERRA_ERR_ALIGNMENT;
    int sms = 0;
    rc = device_props(&sms);
    if (rc) return rc;
    cudaError_t e;
    cudaStream_t st = (cudaStream_t)stream;
    if (need > 0 && use_fwd_tc64(g) && !use_fwd_tc(g))
        e = g.f16 ? launch_fwd_tc64_f16(g, q, k, v, bias_table, o, lse, workspace, sms, st)
                  : launch_fwd_tc64(g, q, k, v, bias_table, o, lse, workspace, sms, st);
    else if (need > 0)
        e = g.f16 ? launch_fwd_tc_f16(g, q, k, v, bias_table, o, lse, workspace, sms, st)
                  : launch_fwd_tc(g, q, k, v, bias_table, o, lse, workspace, sms, st);
    else
        e = g.f16 ? launch_fwd_mma_f16(g, q, k, v, bias_table, o, lse, st) : launch_fwd_mma(g, q, k, v, bias_table, o, lse, st);
    return e == cudaSuccess ? TERRA_OK : cuda_fail(e, "terra_swin_attn_fwd");
}

int terra_swin_attn_fwd(const terra_swin_desc* desc, const void* q, const void* k, const void* v,
                        const float* bias_table, void* o, float* lse,
                        void* workspace, size_t workspace_bytes, void* stream) {
    Geo g;
    int rc = make_geo(desc, true, &g);
    if (rc) return rc;
    return fwd_call(g, q, k, v, bias_table, o, lse, workspace, workspace_bytes, stream);
}

int terra_swin_attn_fwd_packed(const terra_swin_desc* desc, const void* qkv, const float* bias_table, void* o, float* lse,
                               void* workspace, size_t workspace_bytes, void* stream) {
    Geo g;
    int rc = make_geo(desc, true, &g);
    if (rc) return rc;
    if (!qkv) return TERRA_ERR_INVALID_ARG;
    const size_t hd = (size_t)g.heads * g.d;
    g.ts = (int)(3 * hd);
    const __nv_bfloat16* base = reinterpret_cast<const __nv_bfloat16*>(qkv);
    return fwd_call(g, base, base + hd, base + 2 * hd, bias_table, o, lse, workspace, workspace_bytes, stream);
}

// backward with q, k, v and dq, dk, dv given as pointers and one token stride (g.ts elements)
static int bwd_call(const Geo& g, const void* q, const void* k, const void* v,
                    const float* bias_table, const void* o, const float* lse, const void* d_o,
                    void* dq, void* dk, void* dv, float* dbias,
                    void* workspace, size_t workspace_bytes, void* stream) {
    int rc;
    if (!q || !k || !v || !bias_table || !o || !lse || !d_o || !dq || !dk || !dv || !dbias)
        return TERRA_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, bias_table, o, lse, d_o, dq, dk, dv, dbias};
    for (const void* p : ptrs)
        if (!aligned16(p)) return TERRA_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < delta_bytes(g)) return TERRA_ERR_WORKSPACE;
    if (!aligned16(workspace)) return TERRA_ERR_ALIGNMENT;
    int sms = 0;
    rc = device_props(&sms);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (use_bwd_tc(g)) {
        cudaError_t et = g.f16 ? launch_bwd_tc_f16(g, q, k, v, bias_table, o, lse, d_o, dq, dk, dv, dbias, workspace, sms, st)
                               : launch_bwd_tc(g, q, k, v, bias_table, o, lse, d_o, dq, dk, dv, dbias, workspace, sms, st);
        return et == cudaSuccess ? TERRA_OK : cuda_fail(et, "terra_swin_attn_bwd");
    }
    if (bwd_small_supported(g) && !force_split_small()) {
        // windows of at most 64 tokens at head dim 128: one kernel reads every tensor once
        cudaError_t es = g.f16 ? launch_bwd_small_f16(g, q, k, v, o, d_o, bias_table, lse, dq, dk, dv, dbias, sms, st)
                               : launch_bwd_small(g, q, k, v, o, d_o, bias_table, lse, dq, dk, dv, dbias, sms, st);
        return es == cudaSuccess ? TERRA_OK : cuda_fail(es, "terra_swin_attn_bwd");
    }
    float* delta = reinterpret_cast<float*>(workspace);
    cudaError_t e = g.f16 ? launch_bwd_delta_f16(g, o, d_o, delta, st) : launch_bwd_delta(g, o, d_o, delta, st);
    if (e != cudaSuccess) return cuda_fail(e, "terra_swin_attn_bwd (delta)");
    // the register-tile backward, both sides or the query side only
    auto bwd_mma = [&](bool query_side_only) {
        return g.f16 ? launch_bwd_mma_f16(g, q, k, v, bias_table, lse, delta, d_o, dq, dk, dv, dbias, sms, st, query_side_only)
                     : launch_bwd_mma(g, q, k, v, bias_table, lse, delta, d_o, dq, dk, dv, dbias, sms, st, query_side_only);
    };
    if (use_bwd_kv64(g)) {
        // key side (dK, dV) on tcgen05
        float* prep = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(workspace) +
                                               align_up(sizeof(float) * (size_t)g.B * g.H * g.W * g.heads, 256));
        e = launch_bias_prep64(g, bias_table, prep, st);
        if (e == cudaSuccess)
            e = g.f16 ? launch_bwd_kv64_f16(g, q, k, v, d_o, prep, lse, delta, dk, dv, sms, st)
                      : launch_bwd_kv64(g, q, k, v, d_o, prep, lse, delta, dk, dv, sms, st);
        if (e == cudaSuccess) {
            // query side (dQ, dBias): tcgen05 for complete 32 x 32 windows and for complete windows of side 64 and 128
            // (the key-side kernel with the tensors' roles exchanged), else the register-tile kernel
            if (g.w > 32) {
                float* prep_r = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(prep) + align_up(fwd_tc64_workspace_bytes(g), 256));
                e = launch_bias_prep64(g, bias_table, prep_r, st, true);
                if (e == cudaSuccess)
                    e = g.f16 ? launch_bwd_kv64_qside_f16(g, q, k, v, d_o, prep_r, lse, delta, dq, dbias, sms, st)
                              : launch_bwd_kv64_qside(g, q, k, v, d_o, prep_r, lse, delta, dq, dbias, sms, st);
            } else if (bwd_q64_supported(g))
                e = g.f16 ? launch_bwd_q64_f16(g, q, k, v, d_o, prep, lse, delta, dq, dbias, sms, st)
                          : launch_bwd_q64(g, q, k, v, d_o, prep, lse, delta, dq, dbias, sms, st);
            else
                e = bwd_mma(true);
        }
        return e == cudaSuccess ? TERRA_OK : cuda_fail(e, "terra_swin_attn_bwd");
    }
    e = bwd_mma(false);
    return e == cudaSuccess ? TERRA_OK : cuda_fail(e, "terra_swin_attn_bwd");
}

int terra_swin_attn_bwd(const terra_swin_desc* desc, const void* q, const void* k, const void* v,
                        const float* bias_table, const void* o, const float* lse, const void* d_o,
                        void* dq, void* dk, void* dv, float* dbias,
                        void* workspace, size_t workspace_bytes, void* stream) {
    Geo g;
    int rc = make_geo(desc, true, &g);
    if (rc) return rc;
    return bwd_call(g, q, k, v, bias_table, o, lse, d_o, dq, dk, dv, dbias, workspace, workspace_bytes, stream);
}

int terra_swin_attn_bwd_packed(const terra_swin_desc* desc, const void* qkv, const float* bias_table, const void* o,
                               const float* lse, const void* d_o, void* dqkv, float* dbias,
                               void* workspace, size_t workspace_bytes, void* stream) {
    Geo g;
    int rc = make_geo(desc, true, &g);
    if (rc) return rc;
    if (!qkv || !dqkv) return TERRA_ERR_INVALID_ARG;
    const size_t hd = (size_t)g.heads * g.d;
    g.ts = (int)(3 * hd);
    const __nv_bfloat16* base = reinterpret_cast<const __nv_bfloat16*>(qkv);
    __nv_bfloat16* gbase = reinterpret_cast<__nv_bfloat16*>(dqkv);
    return bwd_call(g, base, base + hd, base + 2 * hd, bias_table, o, lse, d_o, gbase, gbase + hd, gbase + 2 * hd, dbias,
                    workspace, workspace_bytes, stream);
}

int terra_selftest_bounded_wait(long long limit_cycles, void* stream) {
    if (limit_cycles <= 0 || limit_cycles > 2000000000LL) return TERRA_ERR_INVALID_ARG;
    int sms = 0;
    int rc = device_props(&sms);
    if (rc) return rc;
    cudaError_t e = launch_bounded_wait_selftest(limit_cycles, (cudaStream_t)stream);
    return e == cudaSuccess ? TERRA_OK : cuda_fail(e, "terra_selftest_bounded_wait");
}

int terra_swin_check(void* stream) {
    int timed_out = 0;
    cudaError_t e = read_tc_status(&timed_out, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "terra_swin_check");
    int timed_out_bwd = 0;
    e = read_bwd_tc_status(&timed_out_bwd);
    if (e != cudaSuccess) return cuda_fail(e, "terra_swin_check");
    int timed_out_64 = 0;
    e = read_fwd_tc64_status(&timed_out_64);
    if (e != cudaSuccess) return cuda_fail(e, "terra_swin_check");
    int timed_out_kv = 0;
    e = read_bwd_kv64_status(&timed_out_kv);
    if (e != cudaSuccess) return cuda_fail(e, "terra_swin_check");
    int timed_out_q = 0;
    e = read_bwd_q64_status(&timed_out_q);
    if (e != cudaSuccess) return cuda_fail(e, "terra_swin_check");
    // the fp16 builds of the same kernels keep status words of their own
    int t16[5] = {0, 0, 0, 0, 0};
    e = read_tc_status_f16(&t16[0], (cudaStream_t)stream);
    if (e == cudaSuccess) e = read_bwd_tc_status_f16(&t16[1]);
    if (e == cudaSuccess) e = read_fwd_tc64_status_f16(&t16[2]);
    if (e == cudaSuccess) e = read_bwd_kv64_status_f16(&t16[3]);
    if (e == cudaSuccess) e = read_bwd_q64_status_f16(&t16[4]);
    if (e != cudaSuccess) return cuda_fail(e, "terra_swin_check");
    const bool any16 = t16[0] || t16[1] || t16[2] || t16[3] || t16[4];
    return (timed_out || timed_out_bwd || timed_out_64 || timed_out_kv || timed_out_q || any16) ? TERRA_ERR_DEVICE_TIMEOUT : TERRA_OK;
}

int terra_profile_enable(int on) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    prof_clear();
    g_prof_on = on != 0;
    return TERRA_OK;
}

int terra_profile_count(void) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    return (int)g_prof.size();
}

int terra_profile_get(int index, char* name, int name_bytes, float* ms) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (index < 0 || index >= (int)g_prof.size() || !ms) return TERRA_ERR_INVALID_ARG;
    const ProfEntry& e = g_prof[index];
    if (!e.closed) return TERRA_ERR_INVALID_ARG;
    cudaError_t err = cudaEventSynchronize(e.end);
    if (err == cudaSuccess) err = cudaEventElapsedTime(ms, e.begin, e.end);
    if (err != cudaSuccess) return cuda_fail(err, "terra_profile_get");
    if (name && name_bytes > 0) {
        std::strncpy(name, e.name, (size_t)name_bytes - 1);
        name[name_bytes - 1] = 0;
    }
    return TERRA_OK;
}

const char* terra_strerror(int status) {
    switch (status) {
        case TERRA_OK: return "ok";
        case TERRA_ERR_INVALID_ARG: return "invalid argument (null pointer, non-positive size, or size out of range)";
        case TERRA_ERR_UNSUPPORTED: return "unsupported configuration (head_dim must be 32, 64 or 128, window <= 128, GPU must be sm_100)";
        case TERRA_ERR_ALIGNMENT: return "pointer is not 16-byte aligned";
        case TERRA_ERR_WORKSPACE: return "workspace missing or too small (see terra_swin_workspace_bytes)";
        case TERRA_ERR_CUDA: return "CUDA error (see terra_last_cuda_error)";
        case TERRA_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel expired; results of that call are invalid";
        case TERRA_ERR_NOALLOC_LIMIT: return "terra_swin_attn_fwd_noalloc: heads exceeds TERRA_NOALLOC_MAX_HEADS, the size of its fixed scratch";
        default: return "unknown status";
    }
}

const char* terra_last_cuda_error(void) { return g_cuda_error; }

int64_t terra_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
