/*
 * fp64 CPU oracle for scaled-dot-product attention, forward and backward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code with the CUDA path and must
 * never be called from it; only the tests, the smoke check and the CPU-baseline
 * leg of the benchmark use it.
 *
 * What it computes, per (batch, head) pair, for Q,K,V,dO in R^{n x d}:
 *
 *   S_ij  = scale * sum_k Q_ik K_jk            (causal: S_ij = -inf for j > i)
 *   m_i   = max_j S_ij ;  E_ij = exp(S_ij - m_i) ;  l_i = sum_j E_ij
 *   P_ij  = E_ij / l_i                          (the n x n array the paper calls A)
 *   L_i   = m_i + log l_i                       (natural-log logsumexp)
 *   O_ik  = sum_j P_ij V_jk                     (the paper's Out)
 *   dP_ij = sum_k dO_ik V_jk
 *   D_i   = sum_j P_ij dP_ij
 *   dS_ij = P_ij (dP_ij - D_i)                  (the paper's GS, analytic softmax backward)
 *   dQ_ik = scale * sum_j dS_ij K_jk            (GQ)
 *   dK_jk = scale * sum_i dS_ij Q_ik            (GK)
 *   dV_jk = sum_i P_ij dO_ik                    (GV)
 *
 * The paper names these arrays (Q, K, V, Out, A, GS, GQ, GK, GV; Sec. 3 traffic
 * table, Sec. 4 backward/fused kernels) but prints no formula for them; the
 * formulas above are the textbook definition of softmax attention and its
 * gradient, with S and P held explicitly as full n x n arrays.
 *
 * Structure follows the paper's repaired CPU kernels (Sec. 4, the crash fix):
 * two race-free passes with heap buffers, the first parallel over query rows i
 * (every row of P, dS, O, dQ has one writer), the second parallel over key
 * columns j (every row of dK, dV has one writer).  No reductions onto shared
 * arrays, no blocking, no online softmax.
 *
 * Layout: every tensor is contiguous [B,H,n,d] (d fastest) in double; L is [B,H,n].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int moa_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One head.  P and dS are caller-provided n*n scratch/outputs (row-major [i][j]).
 * Dout (n) may be NULL. */
void moa_oracle_attn_head(int n, int d, int causal, double scale,
                          const double *Q, const double *K, const double *V, const double *dO,
                          double *O, double *L, double *dQ, double *dK, double *dV,
                          double *P, double *dS, double *Dout)
{
    /* pass 1: parallel over query rows */
#pragma omp parallel for schedule(dynamic, 4)
    for (int i = 0; i < n; ++i) {
        double *Pi = P + (size_t)i * n;
        double *dSi = dS + (size_t)i * n;
        const double *Qi = Q + (size_t)i * d;
        const double *dOi = dO + (size_t)i * d;

        /* scores */
        for (int j = 0; j < n; ++j) {
            if (causal && j > i) {
                Pi[j] = -INFINITY;
            } else {
                const double *Kj = K + (size_t)j * d;
                double acc = 0.0;
                for (int k = 0; k < d; ++k) acc += Qi[k] * Kj[k];
                Pi[j] = scale * acc;
            }
        }
        /* row softmax */
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) if (Pi[j] > m) m = Pi[j];
        double l = 0.0;
        for (int j = 0; j < n; ++j) { Pi[j] = exp(Pi[j] - m); l += Pi[j]; }
        for (int j = 0; j < n; ++j) Pi[j] = Pi[j] / l;
        L[i] = m + log(l);

        /* O = P V */
        double *Oi = O + (size_t)i * d;
        for (int k = 0; k < d; ++k) Oi[k] = 0.0;
        for (int j = 0; j < n; ++j) {
            const double *Vj = V + (size_t)j * d;
            const double p = Pi[j];
            for (int k = 0; k < d; ++k) Oi[k] += p * Vj[k];
        }

        /* dP, D, dS */
        double Di = 0.0;
        for (int j = 0; j < n; ++j) {
            const double *Vj = V + (size_t)j * d;
            double acc = 0.0;
            for (int k = 0; k < d; ++k) acc += dOi[k] * Vj[k];
            dSi[j] = acc;               /* dP_ij for now */
            Di += Pi[j] * acc;
        }
        if (Dout) Dout[i] = Di;
        for (int j = 0; j < n; ++j) dSi[j] = Pi[j] * (dSi[j] - Di);

        /* dQ = scale * dS K */
        double *dQi = dQ + (size_t)i * d;
        for (int k = 0; k < d; ++k) dQi[k] = 0.0;
        for (int j = 0; j < n; ++j) {
            const double *Kj = K + (size_t)j * d;
            const double g = dSi[j];
            for (int k = 0; k < d; ++k) dQi[k] += g * Kj[k];
        }
        for (int k = 0; k < d; ++k) dQi[k] *= scale;
    }

    /* pass 2: parallel over key columns, reading the persisted P and dS */
#pragma omp parallel for schedule(dynamic, 4)
    for (int j = 0; j < n; ++j) {
        double *dKj = dK + (size_t)j * d;
        double *dVj = dV + (size_t)j * d;
        for (int k = 0; k < d; ++k) { dKj[k] = 0.0; dVj[k] = 0.0; }
        for (int i = 0; i < n; ++i) {
            const double g = dS[(size_t)i * n + j];
            const double p = P[(size_t)i * n + j];
            const double *Qi = Q + (size_t)i * d;
            const double *dOi = dO + (size_t)i * d;
            for (int k = 0; k < d; ++k) { dKj[k] += g * Qi[k]; dVj[k] += p * dOi[k]; }
        }
        for (int k = 0; k < d; ++k) dKj[k] *= scale;
    }
}

/* All B*H heads.  Returns 0, or -1 if the two n x n buffers cannot be allocated. */
int moa_oracle_attn(int B, int H, int n, int d, int causal, double scale,
                    const double *Q, const double *K, const double *V, const double *dO,
                    double *O, double *L, double *dQ, double *dK, double *dV)
{
    size_t nn = (size_t)n * (size_t)n;
    double *P = (double *)malloc(nn * sizeof(double));
    double *dS = (double *)malloc(nn * sizeof(double));
    if ((!P || !dS) && nn) { free(P); free(dS); return -1; }
    size_t hs = (size_t)n * d;
    for (int bh = 0; bh < B * H; ++bh) {
        moa_oracle_attn_head(n, d, causal, scale, Q + bh * hs, K + bh * hs, V + bh * hs,
                             dO + bh * hs, O + bh * hs, L + (size_t)bh * n, dQ + bh * hs,
                             dK + bh * hs, dV + bh * hs, P, dS, NULL);
    }
    free(P); free(dS);
    return 0;
}

/*
 * Sampled outputs of ONE head, for sizes where the n x n arrays of every head
 * would take too long: the same definition restricted to chosen query rows.
 * For each sampled row i the full row of S, P, dP and dS is formed (length n).
 * Outputs: O_rows, dQ_rows are [nrows, d]; L_rows is [nrows].
 */
int moa_oracle_attn_rows(int n, int d, int causal, double scale,
                         const double *Q, const double *K, const double *V, const double *dO,
                         int nrows, const int32_t *rows,
                         double *O_rows, double *L_rows, double *dQ_rows)
{
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int r = 0; r < nrows; ++r) {
        const int i = rows[r];
        double *Pi = (double *)malloc((size_t)n * sizeof(double));
        double *dSi = (double *)malloc((size_t)n * sizeof(double));
        if (!Pi || !dSi) { fail = 1; free(Pi); free(dSi); continue; }
        const double *Qi = Q + (size_t)i * d;
        const double *dOi = dO + (size_t)i * d;
        for (int j = 0; j < n; ++j) {
            if (causal && j > i) { Pi[j] = -INFINITY; continue; }
            const double *Kj = K + (size_t)j * d;
            double acc = 0.0;
            for (int k = 0; k < d; ++k) acc += Qi[k] * Kj[k];
            Pi[j] = scale * acc;
        }
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) if (Pi[j] > m) m = Pi[j];
        double l = 0.0;
        for (int j = 0; j < n; ++j) { Pi[j] = exp(Pi[j] - m); l += Pi[j]; }
        for (int j = 0; j < n; ++j) Pi[j] = Pi[j] / l;
        L_rows[r] = m + log(l);
        double *Oi = O_rows + (size_t)r * d;
        for (int k = 0; k < d; ++k) Oi[k] = 0.0;
        for (int j = 0; j < n; ++j) {
            const double *Vj = V + (size_t)j * d;
            for (int k = 0; k < d; ++k) Oi[k] += Pi[j] * Vj[k];
        }
        double Di = 0.0;
        for (int j = 0; j < n; ++j) {
            const double *Vj = V + (size_t)j * d;
            double acc = 0.0;
            for (int k = 0; k < d; ++k) acc += dOi[k] * Vj[k];
            dSi[j] = acc;
            Di += Pi[j] * acc;
        }
        for (int j = 0; j < n; ++j) dSi[j] = Pi[j] * (dSi[j] - Di);
        double *dQi = dQ_rows + (size_t)r * d;
        for (int k = 0; k < d; ++k) dQi[k] = 0.0;
        for (int j = 0; j < n; ++j) {
            const double *Kj = K + (size_t)j * d;
            for (int k = 0; k < d; ++k) dQi[k] += dSi[j] * Kj[k];
        }
        for (int k = 0; k < d; ++k) dQi[k] *= scale;
        free(Pi); free(dSi);
    }
    return fail ? -1 : 0;
}

/*
 * Sampled key columns of ONE head: dK_j and dV_j for chosen j.  Column j of P
 * needs the softmax statistics (m_i, l_i) and D_i of every row, so a first pass
 * over all rows forms each full row of S, P and dP once to get them; the second
 * pass evaluates P_ij = exp(S_ij - m_i) / l_i and dS_ij for the sampled columns
 * only.  Outputs dK_cols, dV_cols are [ncols, d].
 */
int moa_oracle_attn_cols(int n, int d, int causal, double scale,
                         const double *Q, const double *K, const double *V, const double *dO,
                         int ncols, const int32_t *cols,
                         double *dK_cols, double *dV_cols)
{
    double *mvec = (double *)malloc((size_t)n * sizeof(double));
    double *lvec = (double *)malloc((size_t)n * sizeof(double));
    double *Dvec = (double *)malloc((size_t)n * sizeof(double));
    if (!mvec || !lvec || !Dvec) { free(mvec); free(lvec); free(Dvec); return -1; }
    int fail = 0;
#pragma omp parallel
    {
        double *Pi = (double *)malloc((size_t)n * sizeof(double));
        if (!Pi) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for schedule(dynamic, 4)
        for (int i = 0; i < n; ++i) {
            if (!Pi) continue;
            const double *Qi = Q + (size_t)i * d;
            const double *dOi = dO + (size_t)i * d;
            for (int j = 0; j < n; ++j) {
                if (causal && j > i) { Pi[j] = -INFINITY; continue; }
                const double *Kj = K + (size_t)j * d;
                double acc = 0.0;
                for (int k = 0; k < d; ++k) acc += Qi[k] * Kj[k];
                Pi[j] = scale * acc;
            }
            double m = -INFINITY;
            for (int j = 0; j < n; ++j) if (Pi[j] > m) m = Pi[j];
            double l = 0.0;
            for (int j = 0; j < n; ++j) { Pi[j] = exp(Pi[j] - m); l += Pi[j]; }
            double Di = 0.0;
            for (int j = 0; j < n; ++j) {
                const double *Vj = V + (size_t)j * d;
                double acc = 0.0;
                for (int k = 0; k < d; ++k) acc += dOi[k] * Vj[k];
                Di += (Pi[j] / l) * acc;
            }
            mvec[i] = m; lvec[i] = l; Dvec[i] = Di;
        }
        free(Pi);
    }
    if (!fail) {
#pragma omp parallel for schedule(dynamic, 1)
        for (int c = 0; c < ncols; ++c) {
            const int j = cols[c];
            const double *Kj = K + (size_t)j * d;
            const double *Vj = V + (size_t)j * d;
            double *dKj = dK_cols + (size_t)c * d;
            double *dVj = dV_cols + (size_t)c * d;
            for (int k = 0; k < d; ++k) { dKj[k] = 0.0; dVj[k] = 0.0; }
            for (int i = 0; i < n; ++i) {
                if (causal && j > i) continue;      /* P_ij = 0 exactly */
                const double *Qi = Q + (size_t)i * d;
                const double *dOi = dO + (size_t)i * d;
                double s = 0.0, dp = 0.0;
                for (int k = 0; k < d; ++k) { s += Qi[k] * Kj[k]; dp += dOi[k] * Vj[k]; }
                const double p = exp(scale * s - mvec[i]) / lvec[i];
                const double g = p * (dp - Dvec[i]);
                for (int k = 0; k < d; ++k) { dKj[k] += g * Qi[k]; dVj[k] += p * dOi[k]; }
            }
            for (int k = 0; k < d; ++k) dKj[k] *= scale;
        }
    }
    free(mvec); free(lvec); free(Dvec);
    return fail ? -1 : 0;
}
