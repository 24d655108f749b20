/*
 * CHELA token-mixer hot path -- float64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * CUDA library is checked against.  It shares no code, header, table or
 * constant with the CUDA path and must never be called from the product path;
 * only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Everything is double precision, written as the paper's definitions:
 *   - causal linear attention  Norm(Q (K^T V))  (Eq. 2 with the causal mask of
 *     Sec. 4.1) in three separately written forms: quadratic masked form,
 *     token-by-token recurrent form, and the chunked (tiled) form of Sec. 4.1;
 *   - short depthwise causal convolution followed by SiLU (Eq. 7, inner part);
 *   - long convolution, direct sum and FFT form (Eq. 6, Sec. 2.2);
 *   - the mixer composition Z = K_l(silu(K_s(X))), Q/K/V formation
 *     (Eqs. 10-12), per-head linear attention (Eq. 8 without the gate).
 *
 * Readings of points the paper leaves open (feature map = identity, Norm =
 * gain-free RMS normalisation of each output row, mask includes the diagonal,
 * the long convolution is causal/linear rather than circular, tap j of the
 * short kernel multiplies x[t-j]) are the library's documented readings.
 * The choice of Norm itself is a reading, not fixed by the paper:
 * "parity unpinned" for that choice; the un-normalised output (norm = 0) is
 * pinned independently.
 *
 * Layouts (row-major, last index fastest):
 *   q,k : [B, L, H, d_k]     v,o : [B, L, H, d_v]
 *   x,y,z : [B, L, D]        w_short : [D, width]     k_long : [D, L]
 *   dense weights : [D_in, D_out]
 *
 * Parallelism: OpenMP over independent (batch, head) / (batch, channel) units
 * only; no blocking or reordering inside a unit beyond what each form states.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define IDX_QK(b, t, h) ((((size_t)(b) * L + (t)) * H + (h)) * dk)
#define IDX_V(b, t, h) ((((size_t)(b) * L + (t)) * H + (h)) * dv)

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Row normaliser: o = r * (mean_j r_j^2 + eps)^(-1/2); norm == 0 leaves r. */
static void norm_row(double *r, int n, int norm, double eps)
{
    if (!norm) return;
    double ss = 0.0;
    for (int j = 0; j < n; ++j) ss += r[j] * r[j];
    double inv = 1.0 / sqrt(ss / (double)n + eps);
    for (int j = 0; j < n; ++j) r[j] *= inv;
}

/* Quadratic masked form: r_t = scale * sum_{s<=t} <q_t,k_s> v_s  (Eq. 2, causal). */
void oracle_linattn_quadratic(const double *q, const double *k, const double *v, double *o,
                              int B, int H, int L, int dk, int dv,
                              double scale, int norm, double eps)
{
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int t = 0; t < L; ++t) {
                double *r = o + IDX_V(b, t, h);
                for (int j = 0; j < dv; ++j) r[j] = 0.0;
                const double *qt = q + IDX_QK(b, t, h);
                for (int s = 0; s <= t; ++s) {
                    const double *ks = k + IDX_QK(b, s, h);
                    double a = 0.0;
                    for (int i = 0; i < dk; ++i) a += qt[i] * ks[i];
                    a *= scale;
                    const double *vs = v + IDX_V(b, s, h);
                    for (int j = 0; j < dv; ++j) r[j] += a * vs[j];
                }
                norm_row(r, dv, norm, eps);
            }
}

/* Recurrent form: S_t = S_{t-1} + k_t v_t^T ; r_t = scale * S_t^T q_t.
 * state_in / state_out ([B,H,dk,dv], nullable) carry S across segments. */
void oracle_linattn_recurrent(const double *q, const double *k, const double *v, double *o,
                              int B, int H, int L, int dk, int dv,
                              double scale, int norm, double eps,
                              const double *state_in, double *state_out)
{
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            double *S = (double *)calloc((size_t)dk * dv, sizeof(double));
            size_t soff = ((size_t)b * H + h) * dk * dv;
            if (state_in) memcpy(S, state_in + soff, sizeof(double) * dk * dv);
            for (int t = 0; t < L; ++t) {
                const double *qt = q + IDX_QK(b, t, h);
                const double *kt = k + IDX_QK(b, t, h);
                const double *vt = v + IDX_V(b, t, h);
                double *r = o + IDX_V(b, t, h);
                for (int i = 0; i < dk; ++i)
                    for (int j = 0; j < dv; ++j) S[(size_t)i * dv + j] += kt[i] * vt[j];
                for (int j = 0; j < dv; ++j) {
                    double acc = 0.0;
                    for (int i = 0; i < dk; ++i) acc += S[(size_t)i * dv + j] * qt[i];
                    r[j] = scale * acc;
                }
                norm_row(r, dv, norm, eps);
            }
            if (state_out) memcpy(state_out + soff, S, sizeof(double) * dk * dv);
            free(S);
        }
}

/* Chunked form (Sec. 4.1): for chunk i over tokens [iC, min((i+1)C, L)):
 *   R_i = scale * ( Q_i S_{i-1} + tril(Q_i K_i^T) V_i ),  S_i = S_{i-1} + K_i^T V_i. */
void oracle_linattn_chunked(const double *q, const double *k, const double *v, double *o,
                            int B, int H, int L, int dk, int dv, int C,
                            double scale, int norm, double eps)
{
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            double *S = (double *)calloc((size_t)dk * dv, sizeof(double));
            double *P = (double *)malloc(sizeof(double) * (size_t)C * C);
            for (int t0 = 0; t0 < L; t0 += C) {
                int n = (L - t0 < C) ? (L - t0) : C;
                /* P = tril(Q_i K_i^T) */
                for (int a = 0; a < n; ++a)
                    for (int c = 0; c < n; ++c) {
                        double acc = 0.0;
                        if (c <= a) {
                            const double *qa = q + IDX_QK(b, t0 + a, h);
                            const double *kc = k + IDX_QK(b, t0 + c, h);
                            for (int i = 0; i < dk; ++i) acc += qa[i] * kc[i];
                        }
                        P[(size_t)a * C + c] = acc;
                    }
                /* R_i = scale * (Q_i S_{i-1} + P V_i) */
                for (int a = 0; a < n; ++a) {
                    const double *qa = q + IDX_QK(b, t0 + a, h);
                    double *r = o + IDX_V(b, t0 + a, h);
                    for (int j = 0; j < dv; ++j) {
                        double inter = 0.0, intra = 0.0;
                        for (int i = 0; i < dk; ++i) inter += qa[i] * S[(size_t)i * dv + j];
                        for (int c = 0; c < n; ++c)
                            intra += P[(size_t)a * C + c] * v[IDX_V(b, t0 + c, h) + j];
                        r[j] = scale * (inter + intra);
                    }
                    norm_row(r, dv, norm, eps);
                }
                /* S_i = S_{i-1} + K_i^T V_i */
                for (int c = 0; c < n; ++c) {
                    const double *kc = k + IDX_QK(b, t0 + c, h);
                    const double *vc = v + IDX_V(b, t0 + c, h);
                    for (int i = 0; i < dk; ++i)
                        for (int j = 0; j < dv; ++j) S[(size_t)i * dv + j] += kc[i] * vc[j];
                }
            }
            free(P);
            free(S);
        }
}

static double silu(double u) { return u / (1.0 + exp(-u)); }

/* Short depthwise causal conv (+ optional SiLU), inner part of Eq. 7:
 *   y[b,t,c] = act( bias[c] + sum_{j<width} w[c,j] * x[b,t-j,c] ),  x[t<0] = 0. */
void oracle_shortconv(const double *x, const double *w, const double *bias, double *y,
                      int B, int L, int D, int width, int act)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < L; ++t)
            for (int c = 0; c < D; ++c) {
                double acc = bias ? bias[c] : 0.0;
                for (int j = 0; j < width; ++j)
                    if (t - j >= 0)
                        acc += w[(size_t)c * width + j] * x[((size_t)b * L + (t - j)) * D + c];
                y[((size_t)b * L + t) * D + c] = act ? silu(acc) : acc;
            }
}

/* Long conv, direct definition (causal linear convolution):
 *   z[b,t,c] = sum_{s=0..t} k[c,s] * a[b,t-s,c]. */
void oracle_longconv_direct(const double *a, const double *k, double *z, int B, int L, int D)
{
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < D; ++c)
            for (int t = 0; t < L; ++t) {
                double acc = 0.0;
                for (int s = 0; s <= t; ++s)
                    acc += k[(size_t)c * L + s] * a[((size_t)b * L + (t - s)) * D + c];
                z[((size_t)b * L + t) * D + c] = acc;
            }
}

/* In-place iterative radix-2 complex FFT, n a power of two; sign = -1 forward, +1 inverse
 * (no 1/n scaling here). */
static void fft_radix2(double *re, double *im, int n, int sign)
{
    for (int i = 1, j = 0; i < n; ++i) {
        int bit = n >> 1;
        for (; j & bit; bit >>= 1) j ^= bit;
        j ^= bit;
        if (i < j) {
            double tr = re[i]; re[i] = re[j]; re[j] = tr;
            double ti = im[i]; im[i] = im[j]; im[j] = ti;
        }
    }
    const double pi = 3.14159265358979323846264338327950288;
    for (int len = 2; len <= n; len <<= 1) {
        int half = len >> 1;
        for (int i = 0; i < n; i += len)
            for (int m = 0; m < half; ++m) {
                double ang = sign * 2.0 * pi * (double)m / (double)len;
                double wr = cos(ang), wi = sin(ang);
                double xr = re[i + m + half], xi = im[i + m + half];
                double tr = wr * xr - wi * xi, ti = wr * xi + wi * xr;
                re[i + m + half] = re[i + m] - tr;
                im[i + m + half] = im[i + m] - ti;
                re[i + m] += tr;
                im[i + m] += ti;
            }
    }
}

/* Long conv through the FFT theorem (Eq. 6), zero-padded to N = 2*nextpow2(L) so the
 * circular product equals the causal linear convolution on the first L samples. */
void oracle_longconv_fft(const double *a, const double *k, double *z, int B, int L, int D)
{
    int N = 1;
    while (N < L) N <<= 1;
    N <<= 1;
#pragma omp parallel
    {
        double *ur = (double *)malloc(sizeof(double) * N), *ui = (double *)malloc(sizeof(double) * N);
        double *kr = (double *)malloc(sizeof(double) * N), *ki = (double *)malloc(sizeof(double) * N);
#pragma omp for collapse(2) schedule(dynamic)
        for (int b = 0; b < B; ++b)
            for (int c = 0; c < D; ++c) {
                for (int t = 0; t < N; ++t) {
                    ur[t] = (t < L) ? a[((size_t)b * L + t) * D + c] : 0.0;
                    kr[t] = (t < L) ? k[(size_t)c * L + t] : 0.0;
                    ui[t] = 0.0;
                    ki[t] = 0.0;
                }
                fft_radix2(ur, ui, N, -1);
                fft_radix2(kr, ki, N, -1);
                for (int f = 0; f < N; ++f) {
                    double pr = ur[f] * kr[f] - ui[f] * ki[f];
                    double pi_ = ur[f] * ki[f] + ui[f] * kr[f];
                    ur[f] = pr;
                    ui[f] = pi_;
                }
                fft_radix2(ur, ui, N, +1);
                for (int t = 0; t < L; ++t) z[((size_t)b * L + t) * D + c] = ur[t] / (double)N;
            }
        free(ur); free(ui); free(kr); free(ki);
    }
}

/* y[M,N] = act( x[M,K] * w[K,N] + bias[N] ), plain triple loop. */
void oracle_dense(const double *x, const double *w, const double *bias, double *y,
                  size_t M, int K, int N, int act)
{
#pragma omp parallel for schedule(static)
    for (size_t m = 0; m < M; ++m) {
        double *yr = y + m * N;
        for (int n = 0; n < N; ++n) yr[n] = bias ? bias[n] : 0.0;
        for (int kk = 0; kk < K; ++kk) {
            double xv = x[m * K + kk];
            const double *wr = w + (size_t)kk * N;
            for (int n = 0; n < N; ++n) yr[n] += xv * wr[n];
        }
        if (act)
            for (int n = 0; n < N; ++n) yr[n] = silu(yr[n]);
    }
}

/* y[m,c] = alpha[c] * x[m,c] + beta[c]  (Eqs. 10-11, per-channel scalers and offsets). */
void oracle_affine(const double *x, const double *alpha, const double *beta, double *y,
                   size_t M, int D)
{
#pragma omp parallel for schedule(static)
    for (size_t m = 0; m < M; ++m)
        for (int c = 0; c < D; ++c)
            y[m * D + c] = alpha[c] * x[m * D + c] + (beta ? beta[c] : 0.0);
}

/* Mixer composition (Eq. 7, Eqs. 10-12, Eq. 8 without the gate):
 *   A = silu(shortconv(X)); Z = longconv(A);
 *   Q = Z W_q + b_q, K = Z W_k + b_k (dense), or Q = alpha_q.Z + beta_q (qk_diag);
 *   V = silu?(X W_v + b_v); heads = contiguous column blocks of width D/H;
 *   O = Norm(causal linear attention) per head, heads merged back to [B,L,D].
 * use_fft selects the FFT or direct long convolution.  z_out (nullable) receives Z. */
void oracle_mixer(const double *x, const double *w_short, int width, const double *k_long,
                  const double *w_q, const double *w_k, const double *w_v,
                  const double *b_q, const double *b_k, const double *b_v,
                  int qk_diag, int v_silu, double *o, double *z_out,
                  int B, int L, int D, int H, int norm, double eps, int use_fft)
{
    size_t M = (size_t)B * L, n = M * D;
    double *a = (double *)malloc(sizeof(double) * n);
    double *z = (double *)malloc(sizeof(double) * n);
    double *qq = (double *)malloc(sizeof(double) * n);
    double *kk = (double *)malloc(sizeof(double) * n);
    double *vv = (double *)malloc(sizeof(double) * n);
    oracle_shortconv(x, w_short, NULL, a, B, L, D, width, 1);
    if (use_fft) oracle_longconv_fft(a, k_long, z, B, L, D);
    else oracle_longconv_direct(a, k_long, z, B, L, D);
    if (z_out) memcpy(z_out, z, sizeof(double) * n);
    if (qk_diag) {
        oracle_affine(z, w_q, b_q, qq, M, D);
        oracle_affine(z, w_k, b_k, kk, M, D);
    } else {
        oracle_dense(z, w_q, b_q, qq, M, D, D, 0);
        oracle_dense(z, w_k, b_k, kk, M, D, D, 0);
    }
    oracle_dense(x, w_v, b_v, vv, M, D, D, v_silu);
    /* [B,L,D] with head h = columns [h*d,(h+1)*d) is exactly [B,L,H,d]. */
    oracle_linattn_recurrent(qq, kk, vv, o, B, H, L, D / H, D / H, 1.0, norm, eps, NULL, NULL);
    free(a); free(z); free(qq); free(kk); free(vv);
}

/* Gated mixer (Eqs. 8, 9, 13, 14): with O = oracle_mixer(...) and Z its short-long convolution output,
 *   G_a = silu(Z W_a + b_a), G_o = sigmoid(Z W_o + b_o), U = O . G_a . G_o + X . (1 - G_o). */
void oracle_mixer_gated(const double *x, const double *w_short, int width, const double *k_long,
                        const double *w_q, const double *w_k, const double *w_v,
                        const double *b_q, const double *b_k, const double *b_v,
                        const double *w_a, const double *b_a, const double *w_o, const double *b_o,
                        int qk_diag, int v_silu, double *u,
                        int B, int L, int D, int H, int norm, double eps, int use_fft)
{
    size_t M = (size_t)B * L, n = M * D;
    double *o = (double *)malloc(sizeof(double) * n);
    double *z = (double *)malloc(sizeof(double) * n);
    double *ga = (double *)malloc(sizeof(double) * n);
    double *go = (double *)malloc(sizeof(double) * n);
    oracle_mixer(x, w_short, width, k_long, w_q, w_k, w_v, b_q, b_k, b_v, qk_diag, v_silu, o, z, B, L, D, H, norm, eps, use_fft);
    oracle_dense(z, w_a, b_a, ga, M, D, D, 1);
    oracle_dense(z, w_o, b_o, go, M, D, D, 0);
    for (size_t i = 0; i < n; ++i) {
        double g = 1.0 / (1.0 + exp(-go[i]));
        u[i] = o[i] * ga[i] * g + x[i] * (1.0 - g);
    }
    free(o); free(z); free(ga); free(go);
}

/* Backward of causal linear attention, written from the definition (Eq. 2 with the causal mask and the
 * row normaliser): for a loss with gradient d_o[t] with respect to o_t,
 *   r_t = scale * sum_{s<=t} <q_t,k_s> v_s,  n_t = sqrt(mean_j r_tj^2 + eps),  o_t = r_t / n_t
 *   g_t = dLoss/dr_t = (d_o[t] - o_t * <o_t, d_o[t]> / d_v) / n_t          (g_t = d_o[t] without the normaliser)
 *   dq_t = scale * sum_{s<=t} <g_t,v_s> k_s
 *   dk_s = scale * sum_{t>=s} <g_t,v_s> q_t
 *   dv_s = scale * sum_{t>=s} <q_t,k_s> g_t
 * Plain O(L^2) loops per (batch, head). */
void oracle_linattn_backward(const double *q, const double *k, const double *v, const double *d_o,
                             double *dq, double *dk_out, double *dv_out,
                             int B, int H, int L, int dk, int dv, double scale, int norm, double eps)
{
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            double *g = (double *)malloc(sizeof(double) * (size_t)L * dv);
            double *r = (double *)malloc(sizeof(double) * dv);
            for (int t = 0; t < L; ++t) {
                for (int j = 0; j < dv; ++j) r[j] = 0.0;
                const double *qt = q + IDX_QK(b, t, h);
                for (int s = 0; s <= t; ++s) {
                    const double *ks = k + IDX_QK(b, s, h);
                    double a = 0.0;
                    for (int i = 0; i < dk; ++i) a += qt[i] * ks[i];
                    const double *vs = v + IDX_V(b, s, h);
                    for (int j = 0; j < dv; ++j) r[j] += scale * a * vs[j];
                }
                const double *dot = d_o + IDX_V(b, t, h);
                double *gt = g + (size_t)t * dv;
                if (norm) {
                    double ss = 0.0, od = 0.0;
                    for (int j = 0; j < dv; ++j) ss += r[j] * r[j];
                    double n = sqrt(ss / (double)dv + eps);
                    for (int j = 0; j < dv; ++j) od += (r[j] / n) * dot[j];
                    for (int j = 0; j < dv; ++j) gt[j] = (dot[j] - (r[j] / n) * od / (double)dv) / n;
                } else {
                    for (int j = 0; j < dv; ++j) gt[j] = dot[j];
                }
            }
            for (int t = 0; t < L; ++t) {
                double *dqt = dq + IDX_QK(b, t, h);
                for (int i = 0; i < dk; ++i) dqt[i] = 0.0;
                for (int s = 0; s <= t; ++s) {
                    const double *vs = v + IDX_V(b, s, h);
                    const double *ks = k + IDX_QK(b, s, h);
                    double c = 0.0;
                    for (int j = 0; j < dv; ++j) c += g[(size_t)t * dv + j] * vs[j];
                    for (int i = 0; i < dk; ++i) dqt[i] += scale * c * ks[i];
                }
            }
            for (int s = 0; s < L; ++s) {
                double *dks = dk_out + IDX_QK(b, s, h);
                double *dvs = dv_out + IDX_V(b, s, h);
                for (int i = 0; i < dk; ++i) dks[i] = 0.0;
                for (int j = 0; j < dv; ++j) dvs[j] = 0.0;
                const double *vs = v + IDX_V(b, s, h);
                const double *ks = k + IDX_QK(b, s, h);
                for (int t = s; t < L; ++t) {
                    const double *qt = q + IDX_QK(b, t, h);
                    const double *gt = g + (size_t)t * dv;
                    double c = 0.0, a = 0.0;
                    for (int j = 0; j < dv; ++j) c += gt[j] * vs[j];
                    for (int i = 0; i < dk; ++i) a += qt[i] * ks[i];
                    for (int i = 0; i < dk; ++i) dks[i] += scale * c * qt[i];
                    for (int j = 0; j < dv; ++j) dvs[j] += scale * a * gt[j];
                }
            }
            free(g);
            free(r);
        }
}
