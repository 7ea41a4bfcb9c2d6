/*
 * lt_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU statement of what the attention hot path computes.
 * Only tests, the smoke check and the benchmark's cpu-baseline / reference legs
 * may load this library; the CUDA library shares no code with it.
 *
 * What it follows.  The paper's Attention Backward (Section 4.1, "Memory-resident
 * Attention Backward", Algorithm 1) lists the quantities
 *     GP = GO V^T,  GS = SoftmaxBackward(P, GP),  GV = P^T GO,
 *     GQ = GS K,    GK = GS^T Q
 * and says the probability tile P is forward state.  The tile schedule of
 * Algorithm 1 is a re-association of exact sums, so the oracle is the plain
 * definition with no tiling, no online softmax and no saved P:
 *
 *   s_ij  = scale * sum_d Q[i,d] K[j,d]         (visible j: all j, or j <= i if causal)
 *   LSE_i = ln sum_j exp(s_ij)                  (natural log, over visible j)
 *   p_ij  = exp(s_ij - LSE_i)                   (0 for hidden j)
 *   O_i   = sum_j p_ij V_j
 *   dp_ij = sum_d dO[i,d] V[j,d]                (Algorithm 1 line 6, GP)
 *   delta_i = sum_d dO[i,d] O[i,d]              (= sum_j p_ij dp_ij)
 *   ds_ij = p_ij (dp_ij - delta_i)              (Algorithm 1 line 6, SoftmaxBackward)
 *   dQ_i  = scale * sum_j ds_ij K_j             (Algorithm 1 line 11)
 *   dK_j  = scale * sum_{h in group} sum_i ds_ij Q_i   (Algorithm 1 lines 13-15)
 *   dV_j  =         sum_{h in group} sum_i p_ij dO_i   (Algorithm 1 lines 8-9)
 *
 * Grouped-query attention: query head h uses key/value head h / (Hq/Hkv).
 * Layout: every tensor is contiguous [B, H, S, D], D innermost; LSE is [B, Hq, S].
 * All arithmetic is double precision; callers pass fp16-rounded values widened
 * to double when they want the "fp64 math on fp16 inputs" reference.
 *
 * Two modes of the backward:
 *   O_in == NULL : everything (P, O, LSE, delta) is recomputed from Q, K, V.
 *   O_in != NULL : LSE_in and O_in are taken as given forward state (diagnostic:
 *                  separates forward error from backward error).
 *
 * Parallelism: OpenMP over the B*Hq (batch, query head) units, each with private
 * dK/dV buffers that are summed over the group in fixed head order afterwards,
 * so results do not depend on the thread count.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define LT_ORACLE_OK 0
#define LT_ORACLE_BAD_ARG 1
#define LT_ORACLE_NO_MEM 2

static int bad_dims(int B, int Hq, int Hkv, int S, int D)
{
    return B <= 0 || Hq <= 0 || Hkv <= 0 || S <= 0 || D <= 0 || (Hq % Hkv) != 0;
}

int lt_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Scores of one query row against its visible keys, then LSE and p (in place). */
static double row_softmax(const double *q, const double *Kh, int nvis, int D,
                          double scale, double *p)
{
    double m = -INFINITY;
    for (int j = 0; j < nvis; ++j) {
        const double *k = Kh + (size_t)j * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += q[d] * k[d];
        p[j] = scale * acc;
        if (p[j] > m) m = p[j];
    }
    double sum = 0.0;
    for (int j = 0; j < nvis; ++j) sum += exp(p[j] - m);
    double lse = m + log(sum);
    for (int j = 0; j < nvis; ++j) p[j] = exp(p[j] - lse);
    return lse;
}

int lt_oracle_attn_fwd_f64(const double *Q, const double *K, const double *V,
                           double *O, double *LSE,
                           int B, int Hq, int Hkv, int S, int D, int causal, double scale)
{
    if (!Q || !K || !V || !O || !LSE || bad_dims(B, Hq, Hkv, S, D)) return LT_ORACLE_BAD_ARG;
    const int G = Hq / Hkv;
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < B * Hq; ++u) {
        const int b = u / Hq, h = u % Hq, g = h / G;
        const double *Qh = Q + (size_t)u * S * D;
        const double *Kh = K + ((size_t)b * Hkv + g) * S * D;
        const double *Vh = V + ((size_t)b * Hkv + g) * S * D;
        double *Oh = O + (size_t)u * S * D;
        double *p = (double *)malloc(sizeof(double) * (size_t)S);
        if (!p) { err = 1; continue; }
        for (int i = 0; i < S; ++i) {
            const int nvis = causal ? i + 1 : S;
            LSE[(size_t)u * S + i] = row_softmax(Qh + (size_t)i * D, Kh, nvis, D, scale, p);
            double *o = Oh + (size_t)i * D;
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (int j = 0; j < nvis; ++j) {
                const double *v = Vh + (size_t)j * D;
                for (int d = 0; d < D; ++d) o[d] += p[j] * v[d];
            }
        }
        free(p);
    }
    return err ? LT_ORACLE_NO_MEM : LT_ORACLE_OK;
}

int lt_oracle_attn_bwd_f64(const double *Q, const double *K, const double *V, const double *dO,
                           const double *O_in, const double *LSE_in,
                           double *dQ, double *dK, double *dV,
                           int B, int Hq, int Hkv, int S, int D, int causal, double scale)
{
    if (!Q || !K || !V || !dO || !dQ || !dK || !dV || bad_dims(B, Hq, Hkv, S, D)) return LT_ORACLE_BAD_ARG;
    if ((O_in == NULL) != (LSE_in == NULL)) return LT_ORACLE_BAD_ARG;
    const int G = Hq / Hkv;
    const size_t SD = (size_t)S * D;
    /* private per-(b,h) dK/dV, reduced over the group afterwards in head order */
    double *dKp = (double *)calloc((size_t)B * Hq * SD, sizeof(double));
    double *dVp = (double *)calloc((size_t)B * Hq * SD, sizeof(double));
    if (!dKp || !dVp) { free(dKp); free(dVp); return LT_ORACLE_NO_MEM; }
    int err = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < B * Hq; ++u) {
        const int b = u / Hq, h = u % Hq, g = h / G;
        const double *Qh = Q + (size_t)u * SD;
        const double *dOh = dO + (size_t)u * SD;
        const double *Kh = K + ((size_t)b * Hkv + g) * SD;
        const double *Vh = V + ((size_t)b * Hkv + g) * SD;
        double *dQh = dQ + (size_t)u * SD;
        double *dKh = dKp + (size_t)u * SD;
        double *dVh = dVp + (size_t)u * SD;
        double *p = (double *)malloc(sizeof(double) * (size_t)S);
        double *o = (double *)malloc(sizeof(double) * (size_t)D);
        if (!p || !o) { err = 1; free(p); free(o); continue; }
        for (int i = 0; i < S; ++i) {
            const int nvis = causal ? i + 1 : S;
            const double *q = Qh + (size_t)i * D;
            const double *go = dOh + (size_t)i * D;
            double delta = 0.0;
            if (O_in) {
                /* given forward state: p from the supplied LSE, delta from the supplied O */
                const double lse = LSE_in[(size_t)u * S + i];
                for (int j = 0; j < nvis; ++j) {
                    const double *k = Kh + (size_t)j * D;
                    double acc = 0.0;
                    for (int d = 0; d < D; ++d) acc += q[d] * k[d];
                    p[j] = exp(scale * acc - lse);
                }
                const double *oi = O_in + (size_t)u * SD + (size_t)i * D;
                for (int d = 0; d < D; ++d) delta += go[d] * oi[d];
            } else {
                row_softmax(q, Kh, nvis, D, scale, p);
                for (int d = 0; d < D; ++d) o[d] = 0.0;
                for (int j = 0; j < nvis; ++j) {
                    const double *v = Vh + (size_t)j * D;
                    for (int d = 0; d < D; ++d) o[d] += p[j] * v[d];
                }
                for (int d = 0; d < D; ++d) delta += go[d] * o[d];
            }
            double *dq = dQh + (size_t)i * D;
            for (int d = 0; d < D; ++d) dq[d] = 0.0;
            for (int j = 0; j < nvis; ++j) {
                const double *k = Kh + (size_t)j * D;
                const double *v = Vh + (size_t)j * D;
                double dp = 0.0;
                for (int d = 0; d < D; ++d) dp += go[d] * v[d];
                const double ds = p[j] * (dp - delta);
                double *dk = dKh + (size_t)j * D;
                double *dv = dVh + (size_t)j * D;
                for (int d = 0; d < D; ++d) {
                    dq[d] += ds * k[d];
                    dk[d] += ds * q[d];
                    dv[d] += p[j] * go[d];
                }
            }
            for (int d = 0; d < D; ++d) dq[d] *= scale;
        }
        free(p);
        free(o);
    }
    /* group sum, fixed order */
    for (int b = 0; b < B; ++b)
        for (int g = 0; g < Hkv; ++g) {
            double *dk = dK + ((size_t)b * Hkv + g) * SD;
            double *dv = dV + ((size_t)b * Hkv + g) * SD;
            for (size_t e = 0; e < SD; ++e) { dk[e] = 0.0; dv[e] = 0.0; }
            for (int r = 0; r < G; ++r) {
                const size_t u = (size_t)b * Hq + (size_t)g * G + r;
                const double *sk = dKp + u * SD;
                const double *sv = dVp + u * SD;
                for (size_t e = 0; e < SD; ++e) { dk[e] += sk[e]; dv[e] += sv[e]; }
            }
            for (size_t e = 0; e < SD; ++e) dk[e] *= scale;
        }
    free(dKp);
    free(dVp);
    return err ? LT_ORACLE_NO_MEM : LT_ORACLE_OK;
}

/* delta_i = sum_d dO[i,d] O[i,d] for n rows of width D (the preprocess step alone). */
int lt_oracle_delta_f64(const double *dO, const double *O, double *delta, long long n, int D)
{
    if (!dO || !O || !delta || n < 0 || D <= 0) return LT_ORACLE_BAD_ARG;
    for (long long i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += dO[(size_t)i * D + d] * O[(size_t)i * D + d];
        delta[i] = acc;
    }
    return LT_ORACLE_OK;
}
