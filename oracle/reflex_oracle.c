/*
 * CPU oracle for the Reflex action-expert hot path. TEST INFRASTRUCTURE ONLY: nothing in the
 * product path may call, link or load this file. Plain C, double accumulators, no blocking,
 * no fusion, no reordering beyond what each definition states. Inputs are fp32 arrays that
 * already hold values rounded to the storage dtype; outputs are double.
 *
 * Each function names the passage of the paper it follows.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>

/* ------------------------------------------------------------------------------------------
 * Attention by definition (Eq. 1; Appendix A, Proposition 1): queries are the T dynamic-suffix
 * tokens, the context is the explicit concatenation [pinned prefix ; sliding history in FIFO
 * order ; dynamic suffix] handed in as one contiguous array of n_ctx rows.
 *   q    [T][Hq][d]         kctx, vctx [n_ctx][Hkv][d]        out [T][Hq][d]
 * Query head h reads KV head h / (Hq/Hkv). n_prefix = rows before the dynamic block. With
 * dyn_mask = 1 dynamic key j is hidden from dynamic query i when j > i (causal inside the
 * suffix, the "standard causal self-attention" of Proposition 1); dyn_mask = 0 is Eq. 1 as
 * printed (no mask). Returns 0, or -1 on allocation failure.
 * ------------------------------------------------------------------------------------------ */
int reflex_oracle_attention_def(const float *q, const float *kctx, const float *vctx,
                                int T, int Hq, int Hkv, int d, int n_ctx, int n_prefix,
                                int dyn_mask, double scale, double *out)
{
    const int G = Hq / Hkv;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(static)
    for (int i = 0; i < T; ++i) {
        for (int h = 0; h < Hq; ++h) {
            const int kv = h / G;
            const float *qr = q + ((size_t)i * Hq + h) * d;
            double *s = (double *)malloc(sizeof(double) * (size_t)(n_ctx > 0 ? n_ctx : 1));
            if (!s) { fail = 1; continue; }
            double mx = -INFINITY;
            for (int j = 0; j < n_ctx; ++j) {
                const int hidden = dyn_mask && j >= n_prefix && (j - n_prefix) > i;
                if (hidden) { s[j] = -INFINITY; continue; }
                const float *kr = kctx + ((size_t)j * Hkv + kv) * d;
                double dot = 0.0;
                for (int e = 0; e < d; ++e) dot += (double)qr[e] * (double)kr[e];
                s[j] = dot * scale;
                if (s[j] > mx) mx = s[j];
            }
            double denom = 0.0;
            for (int j = 0; j < n_ctx; ++j) {
                s[j] = (s[j] == -INFINITY) ? 0.0 : exp(s[j] - mx);
                denom += s[j];
            }
            double *o = out + ((size_t)i * Hq + h) * d;
            for (int e = 0; e < d; ++e) {
                double acc = 0.0;
                for (int j = 0; j < n_ctx; ++j)
                    acc += s[j] * (double)vctx[((size_t)j * Hkv + kv) * d + e];
                o[e] = acc / denom;
            }
            free(s);
        }
    }
    return fail ? -1 : 0;
}

/* One region's softmax partial for one (query, head): running max m, sum l = sum exp(s-m),
 * acc = sum exp(s-m) v. Rows whose `valid` flag is 0 do not take part at all. */
static void region_partial(const float *qr, const float *k, const float *v, int rows, int Hkv, int kv, int d,
                           const unsigned char *valid, double scale, double *m, double *l, double *acc)
{
    *m = -INFINITY; *l = 0.0;
    for (int e = 0; e < d; ++e) acc[e] = 0.0;
    for (int j = 0; j < rows; ++j) {
        if (!valid[j]) continue;
        const float *kr = k + ((size_t)j * Hkv + kv) * d;
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += (double)qr[e] * (double)kr[e];
        const double s = dot * scale;
        if (s > *m) *m = s;
    }
    if (*m == -INFINITY) return;
    for (int j = 0; j < rows; ++j) {
        if (!valid[j]) continue;
        const float *kr = k + ((size_t)j * Hkv + kv) * d;
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += (double)qr[e] * (double)kr[e];
        const double p = exp(dot * scale - *m);
        *l += p;
        const float *vr = v + ((size_t)j * Hkv + kv) * d;
        for (int e = 0; e < d; ++e) acc[e] += p * (double)vr[e];
    }
}

/* ------------------------------------------------------------------------------------------
 * Partitioned attention (Eq. 1 evaluated region by region; the weights-over-partitions
 * argument in the proof of Proposition 1). The three regions stay where they live:
 *   static  k_s,v_s [S_cap][Hkv][d], rows [0, S) valid
 *   ring    k_r,v_r [N][Hkv][d] in PHYSICAL slot order; slot p is valid iff
 *           ((p - (head - count)) mod N) < count, head = next write slot, count = live tokens
 *   dynamic k_d,v_d [T][Hkv][d]
 * Each region yields (m_r, l_r, acc_r); they are merged with
 *   m = max_r m_r,  l = sum_r l_r e^{m_r-m},  o = sum_r acc_r e^{m_r-m} / l.
 * ------------------------------------------------------------------------------------------ */
int reflex_oracle_attention_part(const float *q,
                                 const float *k_s, const float *v_s, int S,
                                 const float *k_r, const float *v_r, int N, int head, int count,
                                 const float *k_d, const float *v_d,
                                 int T, int Hq, int Hkv, int d, int dyn_mask, double scale, double *out)
{
    const int G = Hq / Hkv;
    int fail = 0;
    unsigned char *valid_s = (unsigned char *)malloc((size_t)(S > 0 ? S : 1));
    unsigned char *valid_r = (unsigned char *)malloc((size_t)(N > 0 ? N : 1));
    if (!valid_s || !valid_r) { free(valid_s); free(valid_r); return -1; }
    for (int j = 0; j < S; ++j) valid_s[j] = 1;
    for (int p = 0; p < N; ++p) {
        int age = (p - (head - count)) % N;
        if (age < 0) age += N;
        valid_r[p] = (unsigned char)(age < count);
    }
#pragma omp parallel for collapse(2) schedule(static)
    for (int i = 0; i < T; ++i) {
        for (int h = 0; h < Hq; ++h) {
            const int kv = h / G;
            const float *qr = q + ((size_t)i * Hq + h) * d;
            double *acc = (double *)malloc(sizeof(double) * 3 * (size_t)d);
            unsigned char *valid_d = (unsigned char *)malloc((size_t)T);
            if (!acc || !valid_d) { fail = 1; free(acc); free(valid_d); continue; }
            for (int j = 0; j < T; ++j) valid_d[j] = (unsigned char)!(dyn_mask && j > i);
            double m[3], l[3];
            region_partial(qr, k_s, v_s, S, Hkv, kv, d, valid_s, scale, &m[0], &l[0], acc);
            region_partial(qr, k_r, v_r, N, Hkv, kv, d, valid_r, scale, &m[1], &l[1], acc + d);
            region_partial(qr, k_d, v_d, T, Hkv, kv, d, valid_d, scale, &m[2], &l[2], acc + 2 * d);
            double mm = -INFINITY;
            for (int r = 0; r < 3; ++r) if (m[r] > mm) mm = m[r];
            double w[3], ll = 0.0;
            for (int r = 0; r < 3; ++r) {
                w[r] = (m[r] == -INFINITY) ? 0.0 : exp(m[r] - mm);
                ll += l[r] * w[r];
            }
            double *o = out + ((size_t)i * Hq + h) * d;
            for (int e = 0; e < d; ++e)
                o[e] = (acc[e] * w[0] + acc[d + e] * w[1] + acc[2 * d + e] * w[2]) / ll;
            free(acc); free(valid_d);
        }
    }
    free(valid_s); free(valid_r);
    return fail ? -1 : 0;
}

/* ------------------------------------------------------------------------------------------
 * AdaRMSNorm (Eq. 2; Appendix B.3): y = x / RMS(x) * gamma(c),
 *   RMS(x) = sqrt(mean_i x_i^2 + eps),  gamma(c) = 1 + W2 SiLU(W1 c + b1) + b2,
 *   SiLU(z) = z / (1 + e^-z).
 *   x [R][D]  c [Cd]  W1 [Hd][Cd]  b1 [Hd]  W2 [D][Hd]  b2 [D]  ->  y [R][D], gamma [D] (optional)
 * One conditioning vector serves all R rows (one stream at one denoising step).
 * ------------------------------------------------------------------------------------------ */
int reflex_oracle_adarmsnorm(const float *x, const float *c, const float *W1, const float *b1,
                             const float *W2, const float *b2, int R, int D, int Cd, int Hd,
                             double eps, double *y, double *gamma_out)
{
    double *hid = (double *)malloc(sizeof(double) * (size_t)(Hd > 0 ? Hd : 1));
    double *gamma = (double *)malloc(sizeof(double) * (size_t)D);
    if (!hid || !gamma) { free(hid); free(gamma); return -1; }
    for (int j = 0; j < Hd; ++j) {
        double z = (double)b1[j];
        for (int e = 0; e < Cd; ++e) z += (double)W1[(size_t)j * Cd + e] * (double)c[e];
        hid[j] = z / (1.0 + exp(-z));
    }
    for (int i = 0; i < D; ++i) {
        double g = (double)b2[i];
        for (int j = 0; j < Hd; ++j) g += (double)W2[(size_t)i * Hd + j] * hid[j];
        gamma[i] = 1.0 + g;
    }
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r) {
        const float *xr = x + (size_t)r * D;
        double ss = 0.0;
        for (int i = 0; i < D; ++i) ss += (double)xr[i] * (double)xr[i];
        const double rms = sqrt(ss / (double)D + eps);
        for (int i = 0; i < D; ++i) y[(size_t)r * D + i] = (double)xr[i] / rms * gamma[i];
    }
    if (gamma_out) for (int i = 0; i < D; ++i) gamma_out[i] = gamma[i];
    free(hid); free(gamma);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Adaptive norm followed by the packed projection (Sec. 3.3 "System Optimizations": the query,
 * key and value projections as one matrix W_QKV = [W_Q; W_K; W_V]; Sec. 4 "Operator Fusion
 * Impact": the adaptive norm combined with the linear layer after it). By definition
 *   y = AdaRMSNorm(x; gamma)   (Eq. 2, y kept in double: the fused form never materialises it)
 *   out[r][n] = sum_i y[r][i] * Wp[n][i]
 *   x [R][D]  gamma [D] (from reflex_oracle_adarmsnorm)  Wp [Nout][D] (row n = output feature n)
 *   -> out [R][Nout]; the caller slices the columns into Q, K and V.
 * ------------------------------------------------------------------------------------------ */
int reflex_oracle_adarmsnorm_linear(const float *x, const double *gamma, const float *Wp, int R, int D,
                                    int Nout, double eps, double *out)
{
    double *y = (double *)malloc(sizeof(double) * (size_t)R * (size_t)D);
    if (!y) return -1;
    for (int r = 0; r < R; ++r) {
        const float *xr = x + (size_t)r * D;
        double ss = 0.0;
        for (int i = 0; i < D; ++i) ss += (double)xr[i] * (double)xr[i];
        const double rms = sqrt(ss / (double)D + eps);
        for (int i = 0; i < D; ++i) y[(size_t)r * D + i] = (double)xr[i] / rms * gamma[i];
    }
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r)
        for (int n = 0; n < Nout; ++n) {
            double acc = 0.0;
            for (int i = 0; i < D; ++i) acc += y[(size_t)r * D + i] * (double)Wp[(size_t)n * D + i];
            out[(size_t)r * Nout + n] = acc;
        }
    free(y);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Adaptive norm followed by the combined gate and up projections of a SwiGLU block (Sec. 3.3
 * "System Optimizations": the Gate and Up projections of SwiGLU blocks fused into one kernel;
 * Sec. 4 "Operator Fusion Impact": the norm combined with the linear layer after it):
 *   y = AdaRMSNorm(x; gamma)                      (Eq. 2, in double)
 *   h[r][f] = SiLU(sum_i y[r][i] Wg[f][i]) * (sum_i y[r][i] Wu[f][i]),  SiLU(z) = z / (1 + e^-z)
 *   x [R][D]  gamma [D]  Wg, Wu [F][D]  ->  h [R][F]
 * ------------------------------------------------------------------------------------------ */
int reflex_oracle_adarmsnorm_swiglu(const float *x, const double *gamma, const float *Wg, const float *Wu,
                                    int R, int D, int F, double eps, double *h)
{
    double *y = (double *)malloc(sizeof(double) * (size_t)R * (size_t)D);
    if (!y) return -1;
    for (int r = 0; r < R; ++r) {
        const float *xr = x + (size_t)r * D;
        double ss = 0.0;
        for (int i = 0; i < D; ++i) ss += (double)xr[i] * (double)xr[i];
        const double rms = sqrt(ss / (double)D + eps);
        for (int i = 0; i < D; ++i) y[(size_t)r * D + i] = (double)xr[i] / rms * gamma[i];
    }
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r)
        for (int f = 0; f < F; ++f) {
            double g = 0.0, u = 0.0;
            for (int i = 0; i < D; ++i) {
                g += y[(size_t)r * D + i] * (double)Wg[(size_t)f * D + i];
                u += y[(size_t)r * D + i] * (double)Wu[(size_t)f * D + i];
            }
            h[(size_t)r * F + f] = g / (1.0 + exp(-g)) * u;
        }
    free(y);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Flow-matching update (Sec. 2.1 "ODE integration", Sec. 3.2 x ~ N(0,I) at t = 1, Appendix C
 * "Flow matching steps 10"): forward Euler with K uniform steps from t = 1 to t = 0,
 *   x <- x + dt * v,  dt = -1/K.
 * ------------------------------------------------------------------------------------------ */
/* ------------------------------------------------------------------------------------------
 * A plain projection of the action expert with its residual connection (Sec. 3.3 lists the expert's
 * linear layers; the attention output projection and the down projection of the SwiGLU block each
 * add their result to the residual stream):
 *     out[r][n] = res[r][n] + sum_i a[r][i] * W[n][i]
 *   a [M][K], W [N][K] (one row per output feature), res [M][N] or NULL (no residual), out [M][N].
 * Plain triple loop, double accumulator, nothing rounded.
 * ------------------------------------------------------------------------------------------ */
int reflex_oracle_linear_residual(const float *a, const float *W, const float *res, int M, int K, int N, double *out)
{
#pragma omp parallel for schedule(static)
    for (int r = 0; r < M; ++r) {
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int i = 0; i < K; ++i) acc += (double)a[(size_t)r * K + i] * (double)W[(size_t)n * K + i];
            out[(size_t)r * N + n] = acc + (res ? (double)res[(size_t)r * N + n] : 0.0);
        }
    }
    return 0;
}

void reflex_oracle_flow_step(double *x, const float *v, long n, int K)
{
    const double dt = -1.0 / (double)K;
    for (long i = 0; i < n; ++i) x[i] += dt * (double)v[i];
}

/* Flow time at the start of denoising step k, from integers (never accumulated): t_k = 1 - k/K. */
double reflex_oracle_flow_time(int k, int K) { return 1.0 - (double)k / (double)K; }

int reflex_oracle_max_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
