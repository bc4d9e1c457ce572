/*
 * CPU oracle for the BCJR soft codeword, its gradients and the Viterbi hard code.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain float64 statement of what
 * the CUDA library must compute.  It shares no code with the CUDA path, is never
 * called by it, and is used only by the tests, the smoke check and the benchmark's
 * CPU-baseline leg.
 *
 * Everything follows the paper's Section 3 literally, one weight block at a time:
 *   - trellis (Section 3.1): states 0..S-1 with S = 2^Lb, transition
 *     s' = f(s, b) = ((s << k) | b) mod S for the k input bits b, scalar emission c[s];
 *     a path s_1..s_n emits the codeword (c[s_1], ..., c[s_n]);
 *   - Boltzmann path distribution (Eq. 4): p(path) ~ exp(-(1/T) sum_t 1/2 (w_t - c[s_t])^2)
 *     over legal paths, free first state, free last state;
 *   - forward/backward messages in the log domain (Eq. 5 and the "numerical
 *     stability" paragraph), state marginals (Eq. 6) and the soft codeword (Eq. 7);
 *   - gradient of l = sum_t g_t * what_t with T held constant (Section 3.5): the
 *     distribution is an exponential family in the log-potentials e_t(s), so
 *     dl/de_t(s) = Cov(G, 1[s_t = s]) with G = sum_t g_t c[s_t], followed by the chain
 *     rule through e_t(s) = -(1/(2T)) (w_t - c[s])^2 and, for the table, the direct
 *     term g_t * gamma_t(s);
 *   - Viterbi (Section 3.2): dynamic programme on the distortion sum_t (w_t - c[s_t])^2
 *     followed by a backtrack.
 *
 * Explicit predecessor / successor tables are built from f, as the paper's own
 * implementation does; nothing is blocked, fused or reordered.
 *
 * Parity pins (see tests/): brute-force enumeration of every path, central finite
 * differences, marginals summing to one, an independent Viterbi, and special cases
 * that reduce to scipy's softmax / logsumexp.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_EINVAL -1
#define ORACLE_ENOMEM -2

/* pred[s*K + j] = j-th state that can precede s;  succ[s*K + b] = f(s, b). */
static int build_tables(int Lb, int k, int32_t **pred_out, int32_t **succ_out)
{
    const int64_t S = (int64_t)1 << Lb, K = (int64_t)1 << k;
    int32_t *succ = (int32_t *)malloc(sizeof(int32_t) * S * K);
    int32_t *pred = (int32_t *)malloc(sizeof(int32_t) * S * K);
    int32_t *fill = (int32_t *)calloc(S, sizeof(int32_t));
    if (!succ || !pred || !fill) { free(succ); free(pred); free(fill); return ORACLE_ENOMEM; }
    for (int64_t s = 0; s < S; ++s)
        for (int64_t b = 0; b < K; ++b)
            succ[s * K + b] = (int32_t)(((s << k) | b) & (S - 1));
    /* invert f: visiting s in increasing order lists the predecessors of every state
       in increasing order */
    for (int64_t s = 0; s < S; ++s)
        for (int64_t b = 0; b < K; ++b) {
            int32_t to = succ[s * K + b];
            pred[(int64_t)to * K + fill[to]++] = (int32_t)s;
        }
    free(fill);
    *pred_out = pred; *succ_out = succ;
    return ORACLE_OK;
}

static int check_dims(int Lb, int k, int n, int64_t B, double T)
{
    if (k < 1 || k > 4 || Lb < k || Lb > 16 || n < 1 || B < 0) return ORACLE_EINVAL;
    if (!(T > 0.0) || !isfinite(T)) return ORACLE_EINVAL;
    return ORACLE_OK;
}

static double lse(const double *x, int m)
{
    double mx = x[0];
    for (int i = 1; i < m; ++i) if (x[i] > mx) mx = x[i];
    double acc = 0.0;
    for (int i = 0; i < m; ++i) acc += exp(x[i] - mx);
    return mx + log(acc);
}

/* log-potential of Eq. 4: e_t(s) = -(1/T) * 1/2 * (w_t - c[s])^2 */
static inline double logpot(double w, double c, double T)
{
    double d = w - c;
    return -(0.5 * d * d) / T;
}

/* alpha[t*S + s] = log alpha_{t+1}(s), beta likewise (0-based t here, 1-based in the paper). */
static void forward_backward(const double *w, const double *c, int n, int64_t S, int K, double T,
                             const int32_t *pred, const int32_t *succ,
                             double *alpha, double *beta)
{
    double tmp[16];
    for (int64_t s = 0; s < S; ++s) alpha[s] = logpot(w[0], c[s], T);
    for (int t = 1; t < n; ++t)
        for (int64_t s = 0; s < S; ++s) {
            for (int j = 0; j < K; ++j) tmp[j] = alpha[(int64_t)(t - 1) * S + pred[s * K + j]];
            alpha[(int64_t)t * S + s] = logpot(w[t], c[s], T) + lse(tmp, K);
        }
    for (int64_t s = 0; s < S; ++s) beta[(int64_t)(n - 1) * S + s] = 0.0;
    for (int t = n - 2; t >= 0; --t)
        for (int64_t s = 0; s < S; ++s) {
            for (int b = 0; b < K; ++b) {
                int32_t s2 = succ[s * K + b];
                tmp[b] = logpot(w[t + 1], c[s2], T) + beta[(int64_t)(t + 1) * S + s2];
            }
            beta[(int64_t)t * S + s] = lse(tmp, K);
        }
}

/*
 * Soft codeword (Eq. 7) and log partition function for B blocks.
 *   W [B*n], c [S], soft [B*n], logZ [B] (may be NULL),
 *   gamma_out [n*S] (may be NULL; marginals of block `gamma_block`),
 *   logZ_t_out [n] (may be NULL; log sum_s alpha_t beta_t of block `gamma_block`, Eq. 6 "any t").
 */
int oracle_soft_quantize(const double *W, const double *c, int Lb, int k, int n, int64_t B,
                         double T, double *soft, double *logZ,
                         int64_t gamma_block, double *gamma_out, double *logZ_t_out)
{
    int rc = check_dims(Lb, k, n, B, T);
    if (rc) return rc;
    const int64_t S = (int64_t)1 << Lb; const int K = 1 << k;
    int32_t *pred, *succ;
    if ((rc = build_tables(Lb, k, &pred, &succ))) return rc;
    int fail = 0;
#pragma omp parallel
    {
        double *alpha = (double *)malloc(sizeof(double) * n * S);
        double *beta = (double *)malloc(sizeof(double) * n * S);
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
                forward_backward(w, c, n, S, K, T, pred, succ, alpha, beta);
                double lz = lse(alpha + (int64_t)(n - 1) * S, (int)S);
                if (logZ) logZ[blk] = lz;
                for (int t = 0; t < n; ++t) {
                    for (int64_t s = 0; s < S; ++s)
                        ab[s] = alpha[(int64_t)t * S + s] + beta[(int64_t)t * S + s];
                    /* Eq. 7: softmax over s of (log alpha + log beta), then the expectation */
                    double lzt = lse(ab, (int)S);
                    double acc = 0.0;
                    for (int64_t s = 0; s < S; ++s) {
                        double gam = exp(ab[s] - lzt);
                        acc += c[s] * gam;
                        if (gamma_out && blk == gamma_block) gamma_out[(int64_t)t * S + s] = gam;
                    }
                    soft[blk * n + t] = acc;
                    if (logZ_t_out && blk == gamma_block) logZ_t_out[t] = lzt;
                }
            }
        }
        free(alpha); free(beta); free(ab);
    }
    free(pred); free(succ);
    return fail ? ORACLE_ENOMEM : ORACLE_OK;
}

/*
 * Gradients of l = sum_{blocks,t} g_t * what_t.
 *   grad_W [B*n]; grad_c [S] = sum over all blocks (overwritten).
 * With G(path) = sum_t g_t c[s_t] and Gbar = E[G]:
 *   dl/de_t(s) = delta_t(s) = gamma_t(s) * (E[G | s_t = s] - Gbar),
 *   E[G | s_t = s] = A_t(s) + Bx_t(s): expected emitted sum of the prefix (including t)
 *   and of the suffix (after t), which are independent given s_t:
 *     A_1(s) = g_1 c[s],  A_t(s) = g_t c[s] + sum_{s' in pred(s)} P(s_{t-1}=s' | s_t=s) A_{t-1}(s'),
 *       P(s_{t-1}=s' | s_t=s) = alpha_{t-1}(s') exp(e_t(s)) / alpha_t(s);
 *     Bx_n(s) = 0,  Bx_t(s) = sum_{s' in succ(s)} P(s_{t+1}=s' | s_t=s) (g_{t+1} c[s'] + Bx_{t+1}(s')),
 *       P(s_{t+1}=s' | s_t=s) = exp(e_{t+1}(s')) beta_{t+1}(s') / beta_t(s).
 *   grad_W[t]  = sum_s delta_t(s) * de_t(s)/dw_t,   de_t(s)/dw_t  = -(w_t - c[s]) / T
 *   grad_c[u] += g_t gamma_t(u) + delta_t(u) * de_t(u)/dc[u],  de_t(u)/dc[u] = +(w_t - c[u]) / T
 */
int oracle_backward(const double *W, const double *c, const double *g, int Lb, int k, int n,
                    int64_t B, double T, double *grad_W, double *grad_c)
{
    int rc = check_dims(Lb, k, n, B, T);
    if (rc) return rc;
    const int64_t S = (int64_t)1 << Lb; const int K = 1 << k;
    int32_t *pred, *succ;
    if ((rc = build_tables(Lb, k, &pred, &succ))) return rc;
    for (int64_t s = 0; s < S; ++s) grad_c[s] = 0.0;
    int fail = 0;
#pragma omp parallel
    {
        double *alpha = (double *)malloc(sizeof(double) * n * S);
        double *beta = (double *)malloc(sizeof(double) * n * S);
        double *A = (double *)malloc(sizeof(double) * n * S);
        double *Bx = (double *)malloc(sizeof(double) * n * S);
        double *gam = (double *)malloc(sizeof(double) * n * S);
        double *soft = (double *)malloc(sizeof(double) * n);
        double *gc = (double *)calloc(S, sizeof(double));
        if (!alpha || !beta || !A || !Bx || !gam || !soft || !gc) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for schedule(dynamic, 1)
            for (int64_t blk = 0; blk < B; ++blk) {
                const double *w = W + blk * n;
                const double *gb = g + blk * n;
                forward_backward(w, c, n, S, K, T, pred, succ, alpha, beta);
                double lz = lse(alpha + (int64_t)(n - 1) * S, (int)S);
                double Gbar = 0.0;
                for (int t = 0; t < n; ++t) {
                    double acc = 0.0;
                    for (int64_t s = 0; s < S; ++s) {
                        double p = exp(alpha[(int64_t)t * S + s] + beta[(int64_t)t * S + s] - lz);
                        gam[(int64_t)t * S + s] = p;
                        acc += c[s] * p;
                    }
                    soft[t] = acc;
                    Gbar += gb[t] * acc;
                }
                for (int64_t s = 0; s < S; ++s) A[s] = gb[0] * c[s];
                for (int t = 1; t < n; ++t)
                    for (int64_t s = 0; s < S; ++s) {
                        double acc = 0.0;
                        double et = logpot(w[t], c[s], T);
                        for (int j = 0; j < K; ++j) {
                            int32_t sp = pred[s * K + j];
                            double P = exp(alpha[(int64_t)(t - 1) * S + sp] + et - alpha[(int64_t)t * S + s]);
                            acc += P * A[(int64_t)(t - 1) * S + sp];
                        }
                        A[(int64_t)t * S + s] = gb[t] * c[s] + acc;
                    }
                for (int64_t s = 0; s < S; ++s) Bx[(int64_t)(n - 1) * S + s] = 0.0;
                for (int t = n - 2; t >= 0; --t)
                    for (int64_t s = 0; s < S; ++s) {
                        double acc = 0.0;
                        for (int b = 0; b < K; ++b) {
                            int32_t s2 = succ[s * K + b];
                            double P = exp(logpot(w[t + 1], c[s2], T) + beta[(int64_t)(t + 1) * S + s2]
                                           - beta[(int64_t)t * S + s]);
                            acc += P * (gb[t + 1] * c[s2] + Bx[(int64_t)(t + 1) * S + s2]);
                        }
                        Bx[(int64_t)t * S + s] = acc;
                    }
                for (int t = 0; t < n; ++t) {
                    double gw = 0.0;
                    for (int64_t s = 0; s < S; ++s) {
                        double p = gam[(int64_t)t * S + s];
                        double delta = p * (A[(int64_t)t * S + s] + Bx[(int64_t)t * S + s] - Gbar);
                        double de_dw = -(w[t] - c[s]) / T;
                        double de_dc = (w[t] - c[s]) / T;
                        gw += delta * de_dw;
                        gc[s] += gb[t] * p + delta * de_dc;
                    }
                    grad_W[blk * n + t] = gw;
                }
            }
#pragma omp critical
            for (int64_t s = 0; s < S; ++s) grad_c[s] += gc[s];
        }
        free(alpha); free(beta); free(A); free(Bx); free(gam); free(soft); free(gc);
    }
    free(pred); free(succ);
    return fail ? ORACLE_ENOMEM : ORACLE_OK;
}

/*
 * Viterbi hard code (Section 3.2): argmin over legal paths of sum_t (w_t - c[s_t])^2.
 *   Wf, cf: the float32 inputs themselves; the metric is accumulated in IEEE double,
 *   d = (double)w - (double)c;  m_t(s) = min_{s' in pred(s)} m_{t-1}(s') + d*d,
 *   with no fused multiply-add.  Ties: lowest predecessor, lowest final state.
 *   states [B*n] (uint16), hard [B*n] (float32 copies of table entries),
 *   path_bits [B*stride]: Lb + k(n-1) bits, MSB first: s_1 in Lb bits, then for each later
 *   step the k new input bits; bit i sits in byte i>>3 at position 7-(i&7); padding zero.
 *   cost [B] (may be NULL): the minimal distortion.
 */
int oracle_viterbi(const float *Wf, const float *cf, int Lb, int k, int n, int64_t B,
                   uint16_t *states, float *hard, uint8_t *path_bits, int64_t stride, double *cost)
{
    int rc = check_dims(Lb, k, n, B, 1.0);
    if (rc) return rc;
    const int64_t S = (int64_t)1 << Lb; const int K = 1 << k;
    const int64_t nbits = Lb + (int64_t)k * (n - 1);
    if (path_bits && stride < (nbits + 7) / 8) return ORACLE_EINVAL;
    int32_t *pred, *succ;
    if ((rc = build_tables(Lb, k, &pred, &succ))) return rc;
    int fail = 0;
#pragma omp parallel
    {
        double *m = (double *)malloc(sizeof(double) * 2 * S);
        int32_t *from = (int32_t *)malloc(sizeof(int32_t) * (int64_t)n * S);
        int32_t *st = (int32_t *)malloc(sizeof(int32_t) * n);
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
                for (int64_t s = 0; s < S; ++s) {
                    volatile double d = (double)w[0] - (double)cf[s];
                    volatile double e = d * d;
                    cur[s] = e;
                }
                for (int t = 1; t < n; ++t) {
                    for (int64_t s = 0; s < S; ++s) {
                        int32_t best = pred[s * K];
                        double bm = cur[best];
                        for (int j = 1; j < K; ++j) {
                            int32_t sp = pred[s * K + j];
                            if (cur[sp] < bm) { bm = cur[sp]; best = sp; }
                        }
                        volatile double d = (double)w[t] - (double)cf[s];
                        volatile double e = d * d;
                        nxt[s] = bm + e;
                        from[(int64_t)t * S + s] = best;
                    }
                    double *sw = cur; cur = nxt; nxt = sw;
                }
                int32_t bs = 0;
                for (int64_t s = 1; s < S; ++s) if (cur[s] < cur[bs]) bs = (int32_t)s;
                if (cost) cost[blk] = cur[bs];
                st[n - 1] = bs;
                for (int t = n - 1; t >= 1; --t) st[t - 1] = from[(int64_t)t * S + st[t]];
                for (int t = 0; t < n; ++t) {
                    if (states) states[blk * n + t] = (uint16_t)st[t];
                    if (hard) hard[blk * n + t] = cf[st[t]];
                }
                if (path_bits) {
                    uint8_t *pb = path_bits + blk * stride;
                    memset(pb, 0, (size_t)stride);
                    int64_t pos = 0;
                    for (int i = Lb - 1; i >= 0; --i, ++pos)
                        if ((st[0] >> i) & 1) pb[pos >> 3] |= (uint8_t)(1u << (7 - (pos & 7)));
                    for (int t = 1; t < n; ++t)
                        for (int i = k - 1; i >= 0; --i, ++pos)
                            if ((st[t] >> i) & 1) pb[pos >> 3] |= (uint8_t)(1u << (7 - (pos & 7)));
                }
            }
        }
        free(m); free(from); free(st);
    }
    free(pred); free(succ);
    return fail ? ORACLE_ENOMEM : ORACLE_OK;
}

/* Number of OpenMP threads the calls above will use (1 when built without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int oracle_num_threads(void) { return omp_get_max_threads(); }
void oracle_set_num_threads(int t) { if (t > 0) omp_set_num_threads(t); }
#else
int oracle_num_threads(void) { return 1; }
void oracle_set_num_threads(int t) { (void)t; }
#endif
