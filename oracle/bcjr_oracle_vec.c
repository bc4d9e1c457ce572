/*
 * CPU oracle for the trellis with VECTOR emissions: every state emits V numbers per step.
 *
 * TEST INFRASTRUCTURE ONLY, like bcjr_oracle.c: plain float64, no code shared with the CUDA
 * path, called only by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * The paper quotes its configuration as "L=16, k=2, V=2" (Section 3.1, Section 4 "Quantization
 * configuration") and its kernel section speaks of a 128-step recursion with 16 predecessors
 * per state for 256-weight blocks: a trellis that consumes V = 2 weights per step and shifts
 * k*V = 4 new bits into a 16-bit state.  Section 3.1 itself only writes the scalar emission,
 * so the vector form below is a READING of the paper, fixed as follows:
 *   - states 0..S-1, S = 2^Lb; per step `kb` = k*V input bits: s' = ((s << kb) | b) mod S;
 *   - state s emits the vector (c[s][0], ..., c[s][V-1]); a block of n weights (n a multiple of
 *     V) is a path of n/V states, step t covering the weights w[V*t .. V*t + V);
 *   - log-potential of a step (Eq. 4 summed over the step's weights):
 *         e_t(s) = -(1/T) * sum_v 1/2 (w[V*t + v] - c[s][v])^2 ;
 *   - everything else is Eq. 5-7 and Section 3.2 / 3.5 unchanged: messages, marginals
 *     gamma_t(s), soft codeword  what[V*t + v] = sum_s c[s][v] gamma_t(s), the exact gradient of
 *     l = sum_i g[i] what[i] with T constant, and the Viterbi path minimising the squared error.
 * With V = 1 every function reduces to its scalar counterpart in bcjr_oracle.c.
 *
 * Parity pins (tests/test_oracle_vec_pins.py): enumeration of every path, central finite
 * differences of that enumeration, the V = 1 reduction, a constant second column (the step
 * energy then differs from the scalar one by a constant), the memoryless case Lb = kb
 * (independent softmaxes), and exhaustive search for Viterbi.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_EINVAL -1
#define ORACLE_ENOMEM -2
#define VMAX 4

static int vec_tables(int Lb, int kb, int32_t **pred_out, int32_t **succ_out)
{
    const int64_t S = (int64_t)1 << Lb, K = (int64_t)1 << kb;
    int32_t *succ = (int32_t *)malloc(sizeof(int32_t) * S * K);
    int32_t *pred = (int32_t *)malloc(sizeof(int32_t) * S * K);
    int32_t *fill = (int32_t *)calloc(S, sizeof(int32_t));
    if (!succ || !pred || !fill) { free(succ); free(pred); free(fill); return ORACLE_ENOMEM; }
    for (int64_t s = 0; s < S; ++s)
        for (int64_t b = 0; b < K; ++b)
            succ[s * K + b] = (int32_t)(((s << kb) | b) & (S - 1));
    for (int64_t s = 0; s < S; ++s)                /* increasing s: predecessors listed in increasing order */
        for (int64_t b = 0; b < K; ++b) {
            int32_t to = succ[s * K + b];
            pred[(int64_t)to * K + fill[to]++] = (int32_t)s;
        }
    free(fill);
    *pred_out = pred; *succ_out = succ;
    return ORACLE_OK;
}

static int vec_dims(int Lb, int kb, int V, int n, int64_t B, double T)
{
    if (V < 1 || V > VMAX || kb < 1 || kb > 4 || Lb < kb || Lb > 16 || n < V || n % V || B < 0) return ORACLE_EINVAL;
    if (!(T > 0.0) || !isfinite(T)) return ORACLE_EINVAL;
    return ORACLE_OK;
}

static double vec_lse(const double *x, int m)
{
    double mx = x[0];
    for (int i = 1; i < m; ++i) if (x[i] > mx) mx = x[i];
    double acc = 0.0;
    for (int i = 0; i < m; ++i) acc += exp(x[i] - mx);
    return mx + log(acc);
}

/* e_t(s) = -(1/T) sum_v 1/2 (w_v - c[s][v])^2 */
static double vec_logpot(const double *w, const double *cs, int V, double T)
{
    double e = 0.0;
    for (int v = 0; v < V; ++v) { double d = w[v] - cs[v]; e += 0.5 * d * d; }
    return -e / T;
}

/* alpha[t*S + s], beta[t*S + s] for steps t = 0..nt-1 (log domain, Eq. 5) */
static void vec_forward_backward(const double *w, const double *c, int nt, int V, int64_t S, int K, double T,
                                 const int32_t *pred, const int32_t *succ, double *alpha, double *beta)
{
    double tmp[16];
    for (int64_t s = 0; s < S; ++s) alpha[s] = vec_logpot(w, c + s * V, V, T);
    for (int t = 1; t < nt; ++t)
        for (int64_t s = 0; s < S; ++s) {
            for (int j = 0; j < K; ++j) tmp[j] = alpha[(int64_t)(t - 1) * S + pred[s * K + j]];
            alpha[(int64_t)t * S + s] = vec_logpot(w + (int64_t)t * V, c + s * V, V, T) + vec_lse(tmp, K);
        }
    for (int64_t s = 0; s < S; ++s) beta[(int64_t)(nt - 1) * S + s] = 0.0;
    for (int t = nt - 2; t >= 0; --t)
        for (int64_t s = 0; s < S; ++s) {
            for (int b = 0; b < K; ++b) {
                int32_t s2 = succ[s * K + b];
                tmp[b] = vec_logpot(w + (int64_t)(t + 1) * V, c + (int64_t)s2 * V, V, T) + beta[(int64_t)(t + 1) * S + s2];
            }
            beta[(int64_t)t * S + s] = vec_lse(tmp, K);
        }
}

/* W [B*n], c [S*V] (row s = the V numbers state s emits), soft [B*n], logZ [B] or NULL */
int oracle_vec_soft_quantize(const double *W, const double *c, int Lb, int kb, int V, int n, int64_t B,
                             double T, double *soft, double *logZ)
{
    int rc = vec_dims(Lb, kb, V, n, B, T);
    if (rc) return rc;
    const int64_t S = (int64_t)1 << Lb; const int K = 1 << kb; const int nt = n / V;
    int32_t *pred, *succ;
    if ((rc = vec_tables(Lb, kb, &pred, &succ))) return rc;
    int fail = 0;
#pragma omp parallel
    {
        double *alpha = (double *)malloc(sizeof(double) * nt * S);
        double *beta = (double *)malloc(sizeof(double) * nt * S);
        double *ab = (double *)malloc(sizeof(double) * S);
        if (!alpha || !beta || !ab) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 1)
            for (int64_t blk = 0; blk < B; ++blk) {
                const double *w = W + blk * n;
                vec_forward_backward(w, c, nt, V, S, K, T, pred, succ, alpha, beta);
                if (logZ) logZ[blk] = vec_lse(alpha + (int64_t)(nt - 1) * S, (int)S);
                for (int t = 0; t < nt; ++t) {
                    for (int64_t s = 0; s < S; ++s) ab[s] = alpha[(int64_t)t * S + s] + beta[(int64_t)t * S + s];
                    double lzt = vec_lse(ab, (int)S);               /* Eq. 6-7: softmax over s, then the expectation */
                    double acc[VMAX] = {0.0, 0.0, 0.0, 0.0};
                    for (int64_t s = 0; s < S; ++s) {
                        double gam = exp(ab[s] - lzt);
                        for (int v = 0; v < V; ++v) acc[v] += c[s * V + v] * gam;
                    }
                    for (int v = 0; v < V; ++v) soft[blk * n + (int64_t)t * V + v] = acc[v];
                }
            }
        }
        free(alpha); free(beta); free(ab);
    }
    free(pred); free(succ);
    return fail ? ORACLE_ENOMEM : ORACLE_OK;
}

/*
 * Gradients of l = sum_i g[i] what[i]:  grad_W [B*n];  grad_c [S*V], summed over blocks.
 * G(path) = sum_t sum_v g[V*t + v] c[s_t][v];  dl/de_t(s) = delta_t(s) = gamma_t(s) (E[G | s_t = s] - E[G]),
 * E[G | s_t = s] = A_t(s) + Bx_t(s) (prefix up to and including t, suffix after t), with the
 * same one-step conditionals as in the scalar oracle.  Chain rule through e_t(s):
 *   de_t(s)/dw[V*t + v] = -(w[V*t + v] - c[s][v]) / T,   de_t(s)/dc[s][v] = +(w[V*t + v] - c[s][v]) / T,
 * plus the direct term g[V*t + v] gamma_t(s) for the table.
 */
int oracle_vec_backward(const double *W, const double *c, const double *g, int Lb, int kb, int V, int n,
                        int64_t B, double T, double *grad_W, double *grad_c)
{
    int rc = vec_dims(Lb, kb, V, n, B, T);
    if (rc) return rc;
    const int64_t S = (int64_t)1 << Lb; const int K = 1 << kb; const int nt = n / V;
    int32_t *pred, *succ;
    if ((rc = vec_tables(Lb, kb, &pred, &succ))) return rc;
    for (int64_t i = 0; i < S * V; ++i) grad_c[i] = 0.0;
    int fail = 0;
#pragma omp parallel
    {
        double *alpha = (double *)malloc(sizeof(double) * nt * S);
        double *beta = (double *)malloc(sizeof(double) * nt * S);
        double *A = (double *)malloc(sizeof(double) * nt * S);
        double *Bx = (double *)malloc(sizeof(double) * nt * S);
        double *gam = (double *)malloc(sizeof(double) * nt * S);
        double *gc = (double *)calloc(S * V, sizeof(double));
        if (!alpha || !beta || !A || !Bx || !gam || !gc) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 1)
            for (int64_t blk = 0; blk < B; ++blk) {
                const double *w = W + blk * n;
                const double *gb = g + blk * n;
                vec_forward_backward(w, c, nt, V, S, K, T, pred, succ, alpha, beta);
                double lz = vec_lse(alpha + (int64_t)(nt - 1) * S, (int)S);
                double Gbar = 0.0;
                for (int t = 0; t < nt; ++t)
                    for (int64_t s = 0; s < S; ++s) {
                        double p = exp(alpha[(int64_t)t * S + s] + beta[(int64_t)t * S + s] - lz);
                        gam[(int64_t)t * S + s] = p;
                        for (int v = 0; v < V; ++v) Gbar += gb[t * V + v] * c[s * V + v] * p;
                    }
                /* emitted value of state s at step t: h_t(s) = sum_v g[V*t + v] c[s][v] */
                for (int64_t s = 0; s < S; ++s) {
                    double h = 0.0;
                    for (int v = 0; v < V; ++v) h += gb[v] * c[s * V + v];
                    A[s] = h;
                }
                for (int t = 1; t < nt; ++t)
                    for (int64_t s = 0; s < S; ++s) {
                        double acc = 0.0, h = 0.0;
                        double et = vec_logpot(w + (int64_t)t * V, c + s * V, V, T);
                        for (int j = 0; j < K; ++j) {
                            int32_t sp = pred[s * K + j];
                            double P = exp(alpha[(int64_t)(t - 1) * S + sp] + et - alpha[(int64_t)t * S + s]);
                            acc += P * A[(int64_t)(t - 1) * S + sp];
                        }
                        for (int v = 0; v < V; ++v) h += gb[t * V + v] * c[s * V + v];
                        A[(int64_t)t * S + s] = h + acc;
                    }
                for (int64_t s = 0; s < S; ++s) Bx[(int64_t)(nt - 1) * S + s] = 0.0;
                for (int t = nt - 2; t >= 0; --t)
                    for (int64_t s = 0; s < S; ++s) {
                        double acc = 0.0;
                        for (int b = 0; b < K; ++b) {
                            int32_t s2 = succ[s * K + b];
                            double P = exp(vec_logpot(w + (int64_t)(t + 1) * V, c + (int64_t)s2 * V, V, T)
                                           + beta[(int64_t)(t + 1) * S + s2] - beta[(int64_t)t * S + s]);
                            double h = 0.0;
                            for (int v = 0; v < V; ++v) h += gb[(t + 1) * V + v] * c[(int64_t)s2 * V + v];
                            acc += P * (h + Bx[(int64_t)(t + 1) * S + s2]);
                        }
                        Bx[(int64_t)t * S + s] = acc;
                    }
                for (int t = 0; t < nt; ++t) {
                    double gw[VMAX] = {0.0, 0.0, 0.0, 0.0};
                    for (int64_t s = 0; s < S; ++s) {
                        double p = gam[(int64_t)t * S + s];
                        double delta = p * (A[(int64_t)t * S + s] + Bx[(int64_t)t * S + s] - Gbar);
                        for (int v = 0; v < V; ++v) {
                            double diff = (w[t * V + v] - c[s * V + v]) / T;
                            gw[v] += delta * (-diff);
                            gc[s * V + v] += gb[t * V + v] * p + delta * diff;
                        }
                    }
                    for (int v = 0; v < V; ++v) grad_W[blk * n + (int64_t)t * V + v] = gw[v];
                }
            }
#pragma omp critical
            for (int64_t i = 0; i < S * V; ++i) grad_c[i] += gc[i];
        }
        free(alpha); free(beta); free(A); free(Bx); free(gam); free(gc);
    }
    free(pred); free(succ);
    return fail ? ORACLE_ENOMEM : ORACLE_OK;
}

/*
 * Viterbi (Section 3.2) with vector emissions: argmin over legal paths of
 * sum_t sum_v (w[V*t + v] - c[s_t][v])^2.  Float32 inputs, IEEE double metric without fused
 * multiply-add: e = d_0*d_0, then e += d_v*d_v for v = 1..V-1, m_t(s) = min_pred + e.
 * Ties: lowest predecessor, lowest final state.
 *   states [B*nt] uint16, hard [B*n] float32 (the emitted numbers, copies of table entries),
 *   path_bits [B*stride]: Lb + kb (nt - 1) bits, most significant first (s_1, then kb bits per step).
 */
int oracle_vec_viterbi(const float *Wf, const float *cf, int Lb, int kb, int V, int n, int64_t B,
                       uint16_t *states, float *hard, uint8_t *path_bits, int64_t stride, double *cost)
{
    int rc = vec_dims(Lb, kb, V, n, B, 1.0);
    if (rc) return rc;
    const int64_t S = (int64_t)1 << Lb; const int K = 1 << kb; const int nt = n / V;
    const int64_t nbits = Lb + (int64_t)kb * (nt - 1);
    if (path_bits && stride < (nbits + 7) / 8) return ORACLE_EINVAL;
    int32_t *pred, *succ;
    if ((rc = vec_tables(Lb, kb, &pred, &succ))) return rc;
    int fail = 0;
#pragma omp parallel
    {
        double *m = (double *)malloc(sizeof(double) * 2 * S);
        int32_t *from = (int32_t *)malloc(sizeof(int32_t) * (int64_t)nt * S);
        int32_t *st = (int32_t *)malloc(sizeof(int32_t) * nt);
        if (!m || !from || !st) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 1)
            for (int64_t blk = 0; blk < B; ++blk) {
                const float *w = Wf + blk * n;
                double *cur = m, *nxt = m + S;
                for (int t = 0; t < nt; ++t) {
                    for (int64_t s = 0; s < S; ++s) {
                        volatile double e = 0.0;
                        for (int v = 0; v < V; ++v) {
                            volatile double d = (double)w[t * V + v] - (double)cf[s * V + v];
                            volatile double dd = d * d;
                            e = v == 0 ? dd : e + dd;
                        }
                        if (t == 0) { cur[s] = e; continue; }
                        int32_t best = pred[s * K];
                        double bm = cur[best];
                        for (int j = 1; j < K; ++j) {
                            int32_t sp = pred[s * K + j];
                            if (cur[sp] < bm) { bm = cur[sp]; best = sp; }
                        }
                        nxt[s] = bm + e;
                        from[(int64_t)t * S + s] = best;
                    }
                    if (t > 0) { double *sw = cur; cur = nxt; nxt = sw; }
                }
                int32_t bs = 0;
                for (int64_t s = 1; s < S; ++s) if (cur[s] < cur[bs]) bs = (int32_t)s;
                if (cost) cost[blk] = cur[bs];
                st[nt - 1] = bs;
                for (int t = nt - 1; t >= 1; --t) st[t - 1] = from[(int64_t)t * S + st[t]];
                for (int t = 0; t < nt; ++t) {
                    if (states) states[blk * nt + t] = (uint16_t)st[t];
                    if (hard) for (int v = 0; v < V; ++v) hard[blk * n + (int64_t)t * V + v] = cf[(int64_t)st[t] * V + v];
                }
                if (path_bits) {
                    uint8_t *pb = path_bits + blk * stride;
                    memset(pb, 0, (size_t)stride);
                    int64_t pos = 0;
                    for (int i = Lb - 1; i >= 0; --i, ++pos)
                        if ((st[0] >> i) & 1) pb[pos >> 3] |= (uint8_t)(1u << (7 - (pos & 7)));
                    for (int t = 1; t < nt; ++t)
                        for (int i = kb - 1; i >= 0; --i, ++pos)
                            if ((st[t] >> i) & 1) pb[pos >> 3] |= (uint8_t)(1u << (7 - (pos & 7)));
                }
            }
        }
        free(m); free(from); free(st);
    }
    free(pred); free(succ);
    return fail ? ORACLE_ENOMEM : ORACLE_OK;
}
