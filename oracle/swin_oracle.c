/*
 * swin_oracle.c -- CPU oracle for the shifted-window attention block.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
 * path is checked against.  It shares no code, header, table or helper with the
 * CUDA library, and only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  Arithmetic is fp64 throughout; bf16 inputs are widened exactly.
 *
 * What it follows.  The paper (Section IV-A) builds its forecaster from Swin blocks
 * with window attention (W-MSA) and shifted-window attention (SW-MSA) and refers to
 * the Swin Transformer for their definition; Section IV-D identifies every token by
 * a global grid coordinate (u, v), its window by (floor(u/w), floor(v/w)) and its
 * in-window offset by (u mod w, v mod w), flattens windows row-major (Section V-A),
 * and says that shifting changes the token coordinate and that the backward pass
 * applies the inverse mapping.  Windowed attention is exact attention under a
 * block mask, so the oracle is that definition written out: no blocking, no online
 * softmax, no reordering.
 *
 * Readings taken where the paper is silent (each is listed again in the design notes):
 *   - shift = cyclic roll by -s: token (u, v) moves to u' = (u - s_h) mod H,
 *     v' = (v - s_w) mod W, and windows are cut in the (u', v') frame;
 *   - a grid that the window does not divide keeps a truncated last window row /
 *     column (no padding tokens);
 *   - an axis that is not periodic gets the Swin shift mask: tokens that wrapped
 *     across that edge (u < s_h, resp. v < s_w) only attend to each other; a
 *     periodic axis (longitude) gets no mask;
 *   - relative-position bias T[(a_q - a_k + w - 1) * (2w - 1) + (b_q - b_k + w - 1), head]
 *     with (a, b) the offsets in the shifted frame;
 *   - masked pairs are excluded exactly (probability zero).
 *
 * Output layout.  Results are produced in the window-major layout of the token
 * route: selected windows in the order given, slots inside a window in (a, b)
 * row-major order over the window's true extent.  The route arrays map slots back
 * to grid tokens.
 *
 * Pins (tests/test_oracle_*.py): brute-force global attention under the membership
 * mask, library SDPA special cases, Swin's roll + region-mask construction,
 * softmax / convexity / shift invariants, central finite differences.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t B, H, W;            /* batch, token grid rows (lat) x cols (lon): the paper's H_T x W_T */
    int32_t heads, head_dim;
    int32_t window;             /* w */
    int32_t shift_h, shift_w;   /* >= 0, taken mod H / mod W */
    int32_t periodic_h, periodic_w;
    double scale;               /* <= 0 means 1/sqrt(head_dim) */
} oracle_desc;

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_NO_MEM = 2 };
enum { IN_BF16 = 0, IN_F64 = 1 };

static int desc_ok(const oracle_desc *d) {
    return d && d->B > 0 && d->H > 0 && d->W > 0 && d->heads > 0 && d->head_dim > 0 &&
           d->window > 0 && d->shift_h >= 0 && d->shift_w >= 0;
}
static int ceil_div(int a, int b) { return (a + b - 1) / b; }
/* extent of window row wr (resp. column wc): the last one is truncated */
static int extent(int L, int w, int idx) { int r = L - idx * w; return r < w ? r : w; }

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int oracle_route_sizes(const oracle_desc *d, int64_t *n_tokens, int32_t *n_windows,
                       int32_t *max_window_tokens) {
    if (!desc_ok(d)) return ORACLE_BAD_ARG;
    int Mh = ceil_div(d->H, d->window), Mw = ceil_div(d->W, d->window);
    if (n_tokens) *n_tokens = (int64_t)d->H * d->W;
    if (n_windows) *n_windows = Mh * Mw;
    if (max_window_tokens) *max_window_tokens = extent(d->H, d->window, 0) * extent(d->W, d->window, 0);
    return ORACLE_OK;
}

/*
 * Token route (Section IV-D coordinates + the shift reading above), per sample.
 *   win_offsets[g]           first slot of window g = wr * M_w + wc (row-major windows)
 *   perm[slot]               grid token u * W + v stored in that slot
 *   inv_perm[u * W + v]      its slot
 *   pos[slot]                a * w + b (offset inside the window, nominal stride w)
 *   label[slot]              2 * [lat not periodic and u < s_h] + [lon not periodic and v < s_w]
 * Any output may be NULL.
 */
int oracle_window_route(const oracle_desc *d, int32_t *perm, int32_t *inv_perm,
                        int32_t *win_offsets, int32_t *pos, int32_t *label) {
    if (!desc_ok(d)) return ORACLE_BAD_ARG;
    const int H = d->H, W = d->W, w = d->window;
    const int sh = d->shift_h % H, sw = d->shift_w % W;
    const int Mh = ceil_div(H, w), Mw = ceil_div(W, w);
    int32_t *offs = (int32_t *)malloc(sizeof(int32_t) * (size_t)(Mh * Mw + 1));
    if (!offs) return ORACLE_NO_MEM;
    int32_t run = 0;
    for (int wr = 0; wr < Mh; ++wr)
        for (int wc = 0; wc < Mw; ++wc) {
            offs[wr * Mw + wc] = run;
            run += extent(H, w, wr) * extent(W, w, wc);
        }
    offs[Mh * Mw] = run;
    for (int u = 0; u < H; ++u)
        for (int v = 0; v < W; ++v) {
            int up = ((u - sh) % H + H) % H;      /* coordinate after the roll */
            int vp = ((v - sw) % W + W) % W;
            int wr = up / w, wc = vp / w;          /* window coordinate */
            int a = up - wr * w, b = vp - wc * w;  /* offset inside the window */
            int slot = offs[wr * Mw + wc] + a * extent(W, w, wc) + b;
            int lab = 2 * ((!d->periodic_h && u < sh) ? 1 : 0) + ((!d->periodic_w && v < sw) ? 1 : 0);
            if (perm) perm[slot] = u * W + v;
            if (inv_perm) inv_perm[u * W + v] = slot;
            if (pos) pos[slot] = a * w + b;
            if (label) label[slot] = lab;
        }
    if (win_offsets) memcpy(win_offsets, offs, sizeof(int32_t) * (size_t)(Mh * Mw + 1));
    free(offs);
    return ORACLE_OK;
}

/* ---- input access: the grid tensors are [B, H, W, heads, head_dim] ------------------- */
static double bf16_to_double(uint16_t bits) {
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}
static double load_elem(int kind, const void *base, int64_t idx) {
    return kind == IN_BF16 ? bf16_to_double(((const uint16_t *)base)[idx]) : ((const double *)base)[idx];
}
/* rows of one (batch, window, head): out[i][c] = x[b, token(slot i), head, c] */
static void gather_rows(const oracle_desc *d, int kind, const void *x, int b, const int32_t *perm_win,
                        int n, int head, double *out) {
    const int dh = d->head_dim;
    for (int i = 0; i < n; ++i) {
        int64_t base = (((int64_t)b * d->H * d->W + perm_win[i]) * d->heads + head) * dh;
        for (int c = 0; c < dh; ++c) out[(size_t)i * dh + c] = load_elem(kind, x, base + c);
    }
}

typedef struct {
    int32_t *perm, *offs, *pos, *label;
    int M;
} route_t;

static int build_route(const oracle_desc *d, route_t *r) {
    int64_t nt;
    int32_t nw;
    oracle_route_sizes(d, &nt, &nw, NULL);
    r->M = nw;
    r->perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)nt);
    r->pos = (int32_t *)malloc(sizeof(int32_t) * (size_t)nt);
    r->label = (int32_t *)malloc(sizeof(int32_t) * (size_t)nt);
    r->offs = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nw + 1));
    if (!r->perm || !r->pos || !r->label || !r->offs) return ORACLE_NO_MEM;
    return oracle_window_route(d, r->perm, NULL, r->offs, r->pos, r->label);
}
static void free_route(route_t *r) { free(r->perm); free(r->pos); free(r->label); free(r->offs); }

/* first output slot of every selected window; sel[k] = b * M + g, or all (b, g) when sel is NULL */
static int64_t *selection_offsets(const oracle_desc *d, const route_t *r, int64_t n_sel, const int64_t *sel) {
    int64_t *o = (int64_t *)malloc(sizeof(int64_t) * (size_t)(n_sel + 1));
    if (!o) return NULL;
    int64_t run = 0;
    for (int64_t k = 0; k < n_sel; ++k) {
        int64_t id = sel ? sel[k] : k;
        int g = (int)(id % r->M);
        o[k] = run;
        run += r->offs[g + 1] - r->offs[g];
    }
    o[n_sel] = run;
    (void)d;
    return o;
}

/* relative-position bias row for query offset pi = a_q * w + b_q and key offset pj */
static int bias_row(int w, int pi, int pj) {
    int aq = pi / w, bq = pi % w, ak = pj / w, bk = pj % w;
    return (aq - ak + w - 1) * (2 * w - 1) + (bq - bk + w - 1);
}

/*
 * One softmax row: scores of query i against every key of its window.
 *   S_ij = scale * <q_i, k_j> + T[row(i, j), head]   if label_i == label_j, else excluded
 *   P_ij = exp(S_ij - m_i) / Z_i,  m_i = max_j S_ij,  Z_i = sum_j exp(S_ij - m_i)
 * Returns log-sum-exp m_i + ln Z_i; excluded entries get P = 0.
 */
static double softmax_row(const oracle_desc *d, double scale, const double *bias, int head, int n, int i,
                          const double *q, const double *k, const int32_t *pos, const int32_t *label,
                          double *P) {
    const int dh = d->head_dim, w = d->window;
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        if (label[i] != label[j]) { P[j] = -INFINITY; continue; }
        double dot = 0.0;
        for (int c = 0; c < dh; ++c) dot += q[(size_t)i * dh + c] * k[(size_t)j * dh + c];
        P[j] = scale * dot + bias[(size_t)bias_row(w, pos[i], pos[j]) * d->heads + head];
        if (P[j] > m) m = P[j];
    }
    double Z = 0.0;
    for (int j = 0; j < n; ++j) {
        P[j] = (P[j] == -INFINITY) ? 0.0 : exp(P[j] - m);
        Z += P[j];
    }
    for (int j = 0; j < n; ++j) P[j] /= Z;
    return m + log(Z);
}

/*
 * Forward: O_i = sum_j P_ij v_j and LSE_i for every selected (batch, window) and every head.
 *   q, k, v        grid layout [B, H, W, heads, head_dim]; bf16 bit patterns (in_kind 0) or fp64 (1)
 *   bias           fp64 [(2w-1)^2, heads]
 *   o              fp64 [S, heads, head_dim], S = total slots of the selected windows
 *   lse            fp64 [S, heads] (may be NULL)
 */
int oracle_attn_fwd(const oracle_desc *d, int in_kind, const void *q, const void *k, const void *v,
                    const double *bias, int64_t n_sel, const int64_t *sel, double *o, double *lse) {
    if (!desc_ok(d) || !q || !k || !v || !bias || !o || n_sel < 0) return ORACLE_BAD_ARG;
    route_t r;
    int rc = build_route(d, &r);
    if (rc) return rc;
    int64_t *so = selection_offsets(d, &r, n_sel, sel);
    if (!so) { free_route(&r); return ORACLE_NO_MEM; }
    const int dh = d->head_dim, nh = d->heads;
    const double scale = d->scale > 0 ? d->scale : 1.0 / sqrt((double)dh);
    int32_t nmax;
    oracle_route_sizes(d, NULL, NULL, &nmax);
    int fail = 0;
#pragma omp parallel
    {
        double *qw = (double *)malloc(sizeof(double) * (size_t)nmax * dh);
        double *kw = (double *)malloc(sizeof(double) * (size_t)nmax * dh);
        double *vw = (double *)malloc(sizeof(double) * (size_t)nmax * dh);
        double *P = (double *)malloc(sizeof(double) * (size_t)nmax);
        if (!qw || !kw || !vw || !P) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 1)
            for (int64_t item = 0; item < n_sel * nh; ++item) {
                int64_t ks = item / nh;
                int head = (int)(item % nh);
                int64_t id = sel ? sel[ks] : ks;
                int b = (int)(id / r.M), g = (int)(id % r.M);
                int off = r.offs[g], n = r.offs[g + 1] - off;
                gather_rows(d, in_kind, q, b, r.perm + off, n, head, qw);
                gather_rows(d, in_kind, k, b, r.perm + off, n, head, kw);
                gather_rows(d, in_kind, v, b, r.perm + off, n, head, vw);
                for (int i = 0; i < n; ++i) {
                    double l = softmax_row(d, scale, bias, head, n, i, qw, kw, r.pos + off, r.label + off, P);
                    double *orow = o + ((so[ks] + i) * nh + head) * dh;
                    for (int c = 0; c < dh; ++c) orow[c] = 0.0;
                    for (int j = 0; j < n; ++j)
                        for (int c = 0; c < dh; ++c) orow[c] += P[j] * vw[(size_t)j * dh + c];
                    if (lse) lse[(so[ks] + i) * nh + head] = l;
                }
            }
        }
        free(qw); free(kw); free(vw); free(P);
    }
    free(so);
    free_route(&r);
    return fail ? ORACLE_NO_MEM : ORACLE_OK;
}

/*
 * Backward of the forward above for an upstream gradient dO (grid layout like q):
 *   dP_ij = <dO_i, v_j>          D_i = sum_j P_ij dP_ij        dS_ij = P_ij (dP_ij - D_i)
 *   dV_j = sum_i P_ij dO_i       dQ_i = scale sum_j dS_ij k_j   dK_j = scale sum_i dS_ij q_i
 *   dT[row(i, j), head] = sum over selected (batch, window) and allowed pairs of dS_ij
 * dq, dk, dv: fp64 [S, heads, head_dim] in selection / slot order; dbias: fp64 [(2w-1)^2, heads],
 * overwritten.  The per-thread dT partials are added in thread order, so a run with a fixed thread
 * count is reproducible.
 */
int oracle_attn_bwd(const oracle_desc *d, int in_kind, const void *q, const void *k, const void *v,
                    const void *d_o, const double *bias, int64_t n_sel, const int64_t *sel,
                    double *dq, double *dk, double *dv, double *dbias) {
    if (!desc_ok(d) || !q || !k || !v || !d_o || !bias || !dq || !dk || !dv || !dbias || n_sel < 0)
        return ORACLE_BAD_ARG;
    route_t r;
    int rc = build_route(d, &r);
    if (rc) return rc;
    int64_t *so = selection_offsets(d, &r, n_sel, sel);
    if (!so) { free_route(&r); return ORACLE_NO_MEM; }
    const int dh = d->head_dim, nh = d->heads, w = d->window;
    const size_t nb = (size_t)(2 * w - 1) * (2 * w - 1) * nh;
    const double scale = d->scale > 0 ? d->scale : 1.0 / sqrt((double)dh);
    int32_t nmax;
    oracle_route_sizes(d, NULL, NULL, &nmax);
    const int nthreads = oracle_num_threads();
    double *dT_parts = (double *)calloc(nb * (size_t)nthreads, sizeof(double));
    if (!dT_parts) { free(so); free_route(&r); return ORACLE_NO_MEM; }
    int fail = 0;
#pragma omp parallel num_threads(nthreads)
    {
#ifdef _OPENMP
        double *dT = dT_parts + nb * (size_t)omp_get_thread_num();
#else
        double *dT = dT_parts;
#endif
        size_t tile = (size_t)nmax * dh;
        double *buf = (double *)malloc(sizeof(double) * (7 * tile + 2 * (size_t)nmax));
        if (!buf) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
            double *qw = buf, *kw = buf + tile, *vw = buf + 2 * tile, *gw = buf + 3 * tile;
            double *dqw = buf + 4 * tile, *dkw = buf + 5 * tile, *dvw = buf + 6 * tile;
            double *P = buf + 7 * tile, *dS = P + nmax;
#pragma omp for schedule(dynamic, 1)
            for (int64_t item = 0; item < n_sel * nh; ++item) {
                int64_t ks = item / nh;
                int head = (int)(item % nh);
                int64_t id = sel ? sel[ks] : ks;
                int b = (int)(id / r.M), g = (int)(id % r.M);
                int off = r.offs[g], n = r.offs[g + 1] - off;
                const int32_t *pos = r.pos + off, *label = r.label + off;
                gather_rows(d, in_kind, q, b, r.perm + off, n, head, qw);
                gather_rows(d, in_kind, k, b, r.perm + off, n, head, kw);
                gather_rows(d, in_kind, v, b, r.perm + off, n, head, vw);
                gather_rows(d, in_kind, d_o, b, r.perm + off, n, head, gw);
                for (size_t t = 0; t < (size_t)n * dh; ++t) dqw[t] = dkw[t] = dvw[t] = 0.0;
                for (int i = 0; i < n; ++i) {
                    softmax_row(d, scale, bias, head, n, i, qw, kw, pos, label, P);
                    double D = 0.0;
                    for (int j = 0; j < n; ++j) {
                        double dP = 0.0;
                        for (int c = 0; c < dh; ++c) dP += gw[(size_t)i * dh + c] * vw[(size_t)j * dh + c];
                        dS[j] = dP;
                        D += P[j] * dP;
                    }
                    for (int j = 0; j < n; ++j) {
                        dS[j] = P[j] * (dS[j] - D);
                        if (label[i] != label[j]) continue;   /* excluded pair: P = 0, dS = 0 */
                        dT[(size_t)bias_row(w, pos[i], pos[j]) * nh + head] += dS[j];
                        for (int c = 0; c < dh; ++c) {
                            dvw[(size_t)j * dh + c] += P[j] * gw[(size_t)i * dh + c];
                            dqw[(size_t)i * dh + c] += scale * dS[j] * kw[(size_t)j * dh + c];
                            dkw[(size_t)j * dh + c] += scale * dS[j] * qw[(size_t)i * dh + c];
                        }
                    }
                }
                for (int i = 0; i < n; ++i) {
                    size_t dst = (size_t)((so[ks] + i) * nh + head) * dh;
                    for (int c = 0; c < dh; ++c) {
                        dq[dst + c] = dqw[(size_t)i * dh + c];
                        dk[dst + c] = dkw[(size_t)i * dh + c];
                        dv[dst + c] = dvw[(size_t)i * dh + c];
                    }
                }
            }
        }
        free(buf);
    }
    for (size_t t = 0; t < nb; ++t) {
        double s = 0.0;
        for (int th = 0; th < nthreads; ++th) s += dT_parts[nb * (size_t)th + t];
        dbias[t] = s;
    }
    free(dT_parts);
    free(so);
    free_route(&r);
    return fail ? ORACLE_NO_MEM : ORACLE_OK;
}
