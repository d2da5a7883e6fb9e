/*
 * CPU oracle for 3D Deformable Slide Attention (3D-DSA), forward and backward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
 * library is checked against.  It shares no code with the CUDA path and nothing in the
 * product may call it; only the tests, the smoke check and the benchmark's CPU-baseline
 * leg do.
 *
 * What it computes (paper Sec. "3D Deformable Slide Attention", Formulation, Eq. 1 and
 * the softmax definition under it; Implementation considerations for the sampling):
 *
 *   For a query token n = (t, y, x) on a (T, H, W) grid and a head m, with a window
 *   (kt, kh, kw) of P = kt*kh*kw cells, cell p = (u*kh + v)*kw + w:
 *
 *     b(p)   = (u - kt/2, v - kh/2, w - kw/2)            integer window displacement
 *                                                        (integer division; zero offsets
 *                                                        give fixed local attention,
 *                                                        Ablations, "Effect of offsets")
 *     pi_a   = coord_a + b_a(p) + Delta[n, m, p, a]      a in (t, y, x)   (Formulation)
 *     i0_a   = floor(pi_a),  f_a = pi_a - i0_a
 *     corner c in {0,1}^3: idx_a = i0_a + c_a,  w_c = prod_a (c_a ? f_a : 1 - f_a),
 *                          valid iff 0 <= idx_a <= size_a - 1 on every axis
 *     k_p    = sum over valid c of w_c * K[idx, m, :]     trilinear sample, zero padding
 *     v_p    = sum over valid c of w_c * V[idx, m, :]     (the grid_sample 'bilinear'
 *                                                        5-D convention with zeros)
 *     s_p    = (q[n, m, :] . k_p) / sqrt(d)
 *     alpha  = softmax_p(s_p)        every one of the P samples takes part, also a
 *                                    sample with no valid corner (k_p = v_p = 0, s_p = 0)
 *     out[n, m, :] = sum_p alpha_p * v_p                  second term of Eq. 1
 *     lse[n, m]    = log sum_p exp(s_p)
 *
 *   The depthwise-convolution term of Eq. 1, the projections and the offset predictor
 *   are outside the operator.
 *
 *   Backward (chain rule through the lines above; pinned in the tests by central finite
 *   differences and by autograd through torch's grid_sample + softmax):
 *
 *     g_p = dO . v_p,  delta = sum_p alpha_p g_p,  dS_p = alpha_p (g_p - delta)
 *     dQ[n, m, :]          = (1/sqrt d) sum_p dS_p k_p
 *     dK[idx_c, m, :]     += w_c (1/sqrt d) dS_p q[n, m, :]      for valid c
 *     dV[idx_c, m, :]     += w_c alpha_p dO[n, m, :]             for valid c
 *     C_c                  = (1/sqrt d) dS_p (q . K[idx_c]) + alpha_p (dO . V[idx_c])
 *     dDelta[n, m, p, a]   = sum over valid c of (c_a ? +1 : -1)
 *                             * prod_{a' != a} (c_a' ? f_a' : 1 - f_a') * C_c
 *
 * Precision.  All arithmetic on values is fp64.  The sampling POSITION follows the
 * storage type of the offsets: for fp32 offsets (dtype F32 and BF16) the position is
 * formed in fp32, float(coord + b) + Delta with one rounding, then floorf and the fp32
 * difference f = pi - i0, because the floor is an integer decision and both sides of a
 * parity test must take it in the same precision.  For dtype F64 (offsets are doubles)
 * the position is fp64; that mode exists for the finite-difference pins.
 *
 * Layouts (row-major, channels last): K, V are the full grid [T, H, W, heads, d].
 * Queries are given as a list of rows: qtok[i] is the flat token index of row i (NULL
 * means row i is token i), q_rows [nq, heads, d], off_rows [nq, heads, P, 3] with the
 * last axis ordered (t, y, x), dout_rows [nq, heads, d].  Outputs are fp64.
 *
 * Parity status: every function here is pinned by tests/test_oracle_pins.py.  Library
 * conventions that the paper does not fix (the centre of an even window, natural-log
 * lse of the scaled logits) are conventions of this build, not pinned by the paper.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_F64 = 2 };

static int g_last_threads = 1;

int dsa3d_oracle_last_threads(void) { return g_last_threads; }

int dsa3d_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static inline double load_elt(const void *base, int dtype, int64_t idx) {
    if (dtype == ORC_F32) return (double)((const float *)base)[idx];
    if (dtype == ORC_F64) return ((const double *)base)[idx];
    /* bf16 is the upper half of an fp32 */
    uint32_t bits = (uint32_t)((const uint16_t *)base)[idx] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* Geometry of one sample: which of the 8 corners are inside the grid, their token
 * indices, the per-axis interpolation factors wt[a][c_a], and the corner weights. */
typedef struct {
    int valid[8];
    int64_t tok[8];
    double wt[3][2]; /* wt[a][0] = 1 - f_a, wt[a][1] = f_a */
    double w[8];
} sample_geom;

static void sample_geometry(const int coord[3], const int b[3], const void *off, int off_is_f64,
                            const int size[3], sample_geom *g) {
    int i0[3];
    int dead = 0;
    for (int a = 0; a < 3; ++a) {
        double f;
        if (off_is_f64) {
            double pi = (double)(coord[a] + b[a]) + ((const double *)off)[a];
            if (!(pi >= -1.0) || !(pi < (double)size[a])) { dead = 1; break; } /* NaN too */
            double fl = floor(pi);
            i0[a] = (int)fl;
            f = pi - fl;
        } else {
            float pi = (float)(coord[a] + b[a]) + ((const float *)off)[a];
            if (!(pi >= -1.0f) || !(pi < (float)size[a])) { dead = 1; break; }
            float fl = floorf(pi);
            i0[a] = (int)fl;
            float ff = pi - fl;
            f = (double)ff;
        }
        g->wt[a][0] = 1.0 - f;
        g->wt[a][1] = f;
    }
    for (int c = 0; c < 8; ++c) {
        g->valid[c] = 0;
        g->tok[c] = -1;
        g->w[c] = 0.0;
    }
    if (dead) {
        for (int a = 0; a < 3; ++a) g->wt[a][0] = g->wt[a][1] = 0.0;
        return;
    }
    for (int c = 0; c < 8; ++c) {
        int cc[3] = {(c >> 2) & 1, (c >> 1) & 1, c & 1};
        int idx[3], ok = 1;
        for (int a = 0; a < 3; ++a) {
            idx[a] = i0[a] + cc[a];
            if (idx[a] < 0 || idx[a] > size[a] - 1) ok = 0;
        }
        g->w[c] = g->wt[0][cc[0]] * g->wt[1][cc[1]] * g->wt[2][cc[2]];
        if (ok) {
            g->valid[c] = 1;
            g->tok[c] = ((int64_t)idx[0] * size[1] + idx[1]) * size[2] + idx[2];
        }
    }
}

static void window_displacement(int p, const int window[3], int b[3]) {
    int w = p % window[2];
    int v = (p / window[2]) % window[1];
    int u = p / (window[2] * window[1]);
    b[0] = u - window[0] / 2;
    b[1] = v - window[1] / 2;
    b[2] = w - window[2] / 2;
}

/* Forward of one (query row, head): fills kp, vp [P, d], s, alpha [P]; returns lse. */
static double forward_one(const void *q_rows, const void *k, const void *v, const void *off_rows,
                          int64_t row, int64_t n, int m, const int size[3], int heads, int d,
                          const int window[3], int P, int dtype, sample_geom *geom, double *kp,
                          double *vp, double *s, double *alpha) {
    const int off_is_f64 = (dtype == ORC_F64);
    const size_t off_elt = off_is_f64 ? sizeof(double) : sizeof(float);
    int coord[3];
    coord[2] = (int)(n % size[2]);
    coord[1] = (int)((n / size[2]) % size[1]);
    coord[0] = (int)(n / ((int64_t)size[2] * size[1]));
    const int64_t qbase = (row * heads + m) * (int64_t)d;
    const double scale = 1.0 / sqrt((double)d);
    for (int p = 0; p < P; ++p) {
        int b[3];
        window_displacement(p, window, b);
        const char *off = (const char *)off_rows + (size_t)(((row * heads + m) * P + p) * 3) * off_elt;
        sample_geometry(coord, b, off, off_is_f64, size, &geom[p]);
        double *kpp = kp + (size_t)p * d, *vpp = vp + (size_t)p * d;
        for (int j = 0; j < d; ++j) kpp[j] = vpp[j] = 0.0;
        for (int c = 0; c < 8; ++c) {
            if (!geom[p].valid[c]) continue;
            const int64_t kbase = (geom[p].tok[c] * heads + m) * (int64_t)d;
            for (int j = 0; j < d; ++j) {
                kpp[j] += geom[p].w[c] * load_elt(k, dtype, kbase + j);
                vpp[j] += geom[p].w[c] * load_elt(v, dtype, kbase + j);
            }
        }
        double dot = 0.0;
        for (int j = 0; j < d; ++j) dot += load_elt(q_rows, dtype, qbase + j) * kpp[j];
        s[p] = dot * scale;
    }
    double mx = s[0];
    for (int p = 1; p < P; ++p)
        if (s[p] > mx) mx = s[p];
    double l = 0.0;
    for (int p = 0; p < P; ++p) l += exp(s[p] - mx);
    const double lse = mx + log(l);
    for (int p = 0; p < P; ++p) alpha[p] = exp(s[p] - lse);
    return lse;
}

static int check_args(int T, int H, int W, int heads, int d, const int *window, int dtype) {
    if (T < 1 || H < 1 || W < 1 || heads < 1 || d < 1) return 1;
    if (!window || window[0] < 1 || window[1] < 1 || window[2] < 1) return 1;
    if (dtype != ORC_F32 && dtype != ORC_BF16 && dtype != ORC_F64) return 1;
    return 0;
}

/* out_rows [nq, heads, d], lse_rows [nq, heads], alpha_rows [nq, heads, P] (may be NULL). */
int dsa3d_oracle_forward(const void *q_rows, const void *k, const void *v, const void *off_rows,
                         const int64_t *qtok, int64_t nq, int T, int H, int W, int heads, int d,
                         const int *window, int dtype, double *out_rows, double *lse_rows,
                         double *alpha_rows) {
    if (check_args(T, H, W, heads, d, window, dtype)) return 1;
    const int size[3] = {T, H, W};
    const int P = window[0] * window[1] * window[2];
    int failed = 0;
    g_last_threads = dsa3d_oracle_max_threads();
#pragma omp parallel
    {
        sample_geom *geom = (sample_geom *)malloc(sizeof(sample_geom) * P);
        double *kp = (double *)malloc(sizeof(double) * P * d);
        double *vp = (double *)malloc(sizeof(double) * P * d);
        double *s = (double *)malloc(sizeof(double) * P * 2);
        if (!geom || !kp || !vp || !s) {
#pragma omp atomic write
            failed = 1;
        } else {
            double *alpha = s + P;
#pragma omp for collapse(2) schedule(dynamic, 16)
            for (int64_t i = 0; i < nq; ++i) {
                for (int m = 0; m < heads; ++m) {
                    const int64_t n = qtok ? qtok[i] : i;
                    const double lse = forward_one(q_rows, k, v, off_rows, i, n, m, size, heads, d,
                                                   window, P, dtype, geom, kp, vp, s, alpha);
                    double *o = out_rows + (i * heads + m) * (int64_t)d;
                    for (int j = 0; j < d; ++j) o[j] = 0.0;
                    for (int p = 0; p < P; ++p)
                        for (int j = 0; j < d; ++j) o[j] += alpha[p] * vp[(size_t)p * d + j];
                    lse_rows[i * heads + m] = lse;
                    if (alpha_rows)
                        for (int p = 0; p < P; ++p) alpha_rows[(i * heads + m) * (int64_t)P + p] = alpha[p];
                }
            }
        }
        free(geom);
        free(kp);
        free(vp);
        free(s);
    }
    return failed ? 2 : 0;
}

/* dq_rows [nq, heads, d], doff_rows [nq, heads, P, 3], fully overwritten.
 * dk_rows, dv_rows [nk, heads, d] are ACCUMULATED INTO (the caller zeroes them).
 * kslot: NULL means slot = token index (nk = T*H*W); otherwise kslot[token] is the output
 * row of that key token, or -1 if its gradient is not wanted.
 *
 * Two phases.  Phase A visits every (query row, head) independently and produces dQ,
 * dOffsets and the two per-sample scatter coefficients  ck_p = dS_p / sqrt(d)  and
 * cv_p = alpha_p.  Phase B adds  w_c ck_p q  into dK and  w_c cv_p dO  into dV; it is
 * split over (head, channel range) so that every dK/dV element belongs to one thread and
 * is summed in query-row order whatever the thread count. */
int dsa3d_oracle_backward(const void *q_rows, const void *k, const void *v, const void *off_rows,
                          const void *dout_rows, const int64_t *qtok, int64_t nq, int T, int H,
                          int W, int heads, int d, const int *window, int dtype,
                          const int64_t *kslot, double *dq_rows, double *dk_rows, double *dv_rows,
                          double *doff_rows) {
    if (check_args(T, H, W, heads, d, window, dtype)) return 1;
    const int size[3] = {T, H, W};
    const int P = window[0] * window[1] * window[2];
    const double scale = 1.0 / sqrt((double)d);
    const int off_is_f64 = (dtype == ORC_F64);
    const size_t off_elt = off_is_f64 ? sizeof(double) : sizeof(float);
    int failed = 0;
    g_last_threads = dsa3d_oracle_max_threads();
    double *coef = (double *)malloc(sizeof(double) * 2 * (size_t)nq * heads * P + 16);
    if (!coef) return 2;

    /* ---- phase A: dQ, dOffsets, scatter coefficients ---- */
#pragma omp parallel
    {
        sample_geom *geom = (sample_geom *)malloc(sizeof(sample_geom) * P);
        double *kp = (double *)malloc(sizeof(double) * P * d);
        double *vp = (double *)malloc(sizeof(double) * P * d);
        double *s = (double *)malloc(sizeof(double) * P * 4);
        double *qv = (double *)malloc(sizeof(double) * d * 2);
        if (!geom || !kp || !vp || !s || !qv) {
#pragma omp atomic write
            failed = 1;
        } else {
            double *alpha = s + P, *g = s + 2 * P, *dS = s + 3 * P;
            double *dov = qv + d;
#pragma omp for collapse(2) schedule(dynamic, 16)
            for (int64_t i = 0; i < nq; ++i) {
                for (int m = 0; m < heads; ++m) {
                    const int64_t n = qtok ? qtok[i] : i;
                    forward_one(q_rows, k, v, off_rows, i, n, m, size, heads, d, window, P, dtype,
                                geom, kp, vp, s, alpha);
                    const int64_t qbase = (i * heads + m) * (int64_t)d;
                    for (int j = 0; j < d; ++j) {
                        qv[j] = load_elt(q_rows, dtype, qbase + j);
                        dov[j] = load_elt(dout_rows, dtype, qbase + j);
                    }
                    double delta = 0.0;
                    for (int p = 0; p < P; ++p) {
                        double acc = 0.0;
                        for (int j = 0; j < d; ++j) acc += dov[j] * vp[(size_t)p * d + j];
                        g[p] = acc;
                        delta += alpha[p] * acc;
                    }
                    for (int p = 0; p < P; ++p) dS[p] = alpha[p] * (g[p] - delta);
                    double *dq = dq_rows + qbase;
                    for (int j = 0; j < d; ++j) dq[j] = 0.0;
                    for (int p = 0; p < P; ++p)
                        for (int j = 0; j < d; ++j) dq[j] += scale * dS[p] * kp[(size_t)p * d + j];
                    for (int p = 0; p < P; ++p) {
                        double *doff = doff_rows + ((i * heads + m) * (int64_t)P + p) * 3;
                        doff[0] = doff[1] = doff[2] = 0.0;
                        for (int c = 0; c < 8; ++c) {
                            if (!geom[p].valid[c]) continue;
                            const int cc[3] = {(c >> 2) & 1, (c >> 1) & 1, c & 1};
                            const int64_t kbase = (geom[p].tok[c] * heads + m) * (int64_t)d;
                            double qk = 0.0, dov_v = 0.0;
                            for (int j = 0; j < d; ++j) {
                                qk += qv[j] * load_elt(k, dtype, kbase + j);
                                dov_v += dov[j] * load_elt(v, dtype, kbase + j);
                            }
                            const double Cc = scale * dS[p] * qk + alpha[p] * dov_v;
                            for (int a = 0; a < 3; ++a) {
                                double prod = cc[a] ? 1.0 : -1.0;
                                for (int a2 = 0; a2 < 3; ++a2)
                                    if (a2 != a) prod *= geom[p].wt[a2][cc[a2]];
                                doff[a] += prod * Cc;
                            }
                        }
                        double *cf = coef + 2 * ((i * heads + m) * (int64_t)P + p);
                        cf[0] = scale * dS[p];
                        cf[1] = alpha[p];
                    }
                }
            }
        }
        free(geom);
        free(kp);
        free(vp);
        free(s);
        free(qv);
    }

    /* ---- phase B: dK, dV ---- */
    if (!failed) {
        int nchunk = (g_last_threads + heads - 1) / heads;
        if (nchunk > d) nchunk = d;
        if (nchunk < 1) nchunk = 1;
        const int cw = (d + nchunk - 1) / nchunk;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
        for (int m = 0; m < heads; ++m) {
            for (int ch = 0; ch < nchunk; ++ch) {
                const int j0 = ch * cw, j1 = (j0 + cw < d) ? j0 + cw : d;
                sample_geom geom;
                for (int64_t i = 0; i < nq; ++i) {
                    const int64_t n = qtok ? qtok[i] : i;
                    int coord[3];
                    coord[2] = (int)(n % W);
                    coord[1] = (int)((n / W) % H);
                    coord[0] = (int)(n / ((int64_t)W * H));
                    const int64_t qbase = (i * heads + m) * (int64_t)d;
                    for (int p = 0; p < P; ++p) {
                        int b[3];
                        window_displacement(p, window, b);
                        const char *off = (const char *)off_rows +
                                          (size_t)(((i * heads + m) * P + p) * 3) * off_elt;
                        sample_geometry(coord, b, off, off_is_f64, size, &geom);
                        const double *cf = coef + 2 * ((i * heads + m) * (int64_t)P + p);
                        for (int c = 0; c < 8; ++c) {
                            if (!geom.valid[c]) continue;
                            const int64_t slot = kslot ? kslot[geom.tok[c]] : geom.tok[c];
                            if (slot < 0) continue;
                            double *dk = dk_rows + (slot * heads + m) * (int64_t)d;
                            double *dv = dv_rows + (slot * heads + m) * (int64_t)d;
                            const double ck = geom.w[c] * cf[0];
                            const double cv = geom.w[c] * cf[1];
                            for (int j = j0; j < j1; ++j) {
                                dk[j] += ck * load_elt(q_rows, dtype, qbase + j);
                                dv[j] += cv * load_elt(dout_rows, dtype, qbase + j);
                            }
                        }
                    }
                }
            }
        }
    }
    free(coef);
    return failed ? 2 : 0;
}
