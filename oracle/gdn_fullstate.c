/*
 * ORACLE - TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 CPU statement of what the
 * beam-shared Gated DeltaNet decode computes.  Nothing in the product path may
 * import, link or call this file; it shares no code with the CUDA library.
 *
 * What it computes (paper Section 2.2, Eq. 1; Section 3.2, Eq. 2 for "the state of
 * the selected parent beam, with the shared post-prefill state as initial state"):
 * for one (beam, head) unit at decode call T-1, find the unit's records by walking
 * the per-step parent arrays backward from the beam (linked form, Section 3.3:
 * "each child reuses the ancestry of its selected parent"), then MATERIALISE the
 * full d_v x d_k state by applying Eq. 1 once per record, oldest first, starting
 * from a copy of S_0, and read it out along the query: o = S q (the output sees
 * the state AFTER the current token's update, Eq. 1 second line).
 *
 * No blocking, fusion or reordering: one matrix-vector product, one rank-1 update
 * and one scaling per record, exactly as Eq. 1 is printed.  Inputs are fp32
 * arrays (bf16 values widened exactly by the caller); every operation is fp64.
 * OpenMP only spreads independent units over host cores.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* One GDN transition step, Eq. 1:  S <- a S + b (v - a S k) k^T.
 * S is [dv][dk] row-major; u is scratch of length dv. */
static void gdn_transition(double *S, double *u, int dk, int dv, const float *k, const float *v,
                           double a, double b) {
    for (int i = 0; i < dv; ++i) {          /* u = S k */
        double acc = 0.0;
        for (int j = 0; j < dk; ++j) acc += S[(size_t)i * dk + j] * (double)k[j];
        u[i] = acc;
    }
    for (int i = 0; i < dv; ++i) {
        double delta = b * ((double)v[i] - a * u[i]);      /* Eq. 2's delta_t */
        for (int j = 0; j < dk; ++j)
            S[(size_t)i * dk + j] = a * S[(size_t)i * dk + j] + delta * (double)k[j];
    }
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Full-state decode for selected (beam, head) units of ONE request and ONE layer.
 *
 *   H, dk, dv      heads and head dimensions
 *   T              number of decode calls made so far (records on each chain), >= 0
 *   W[t]           beam width at call t
 *   S0             [H][dv][dk] fp32, the shared post-prefill state
 *   k[t], v[t]     [W[t]][H][dk] / [W[t]][H][dv] fp32: the token every beam appended at call t
 *   alpha[t], beta[t]   [W[t]][H]
 *   parents[t]     [W[t]] parent of each beam of call t in the beam of call t-1 (t >= 1;
 *                  parents[0] is ignored: at call 0 every beam's parent is S0)
 *   q              [W[T-1]][H][dk] query of the last call (for T == 0: [n][H][dk] rows
 *                  indexed by sel_beam, and the output is S0 q)
 *   sel_beam/head  the n_sel units to evaluate (beam index at call T-1, head)
 *   out            [n_sel][dv] fp64
 *   chain_out      optional [n_sel][T] int32: the unit's beam index at each call,
 *                  oldest first (the last entry is sel_beam itself)
 * Returns 0, or -1 on a parent index outside the previous beam.
 */
int oracle_gdn_decode(int H, int dk, int dv, int T, const int32_t *W, const float *S0,
                      const float *const *k, const float *const *v, const float *const *alpha,
                      const float *const *beta, const int32_t *const *parents, const float *q,
                      int n_sel, const int32_t *sel_beam, const int32_t *sel_head, double *out,
                      int32_t *chain_out, int nthreads) {
    int bad = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
#pragma omp parallel
    {
        double *S = (double *)malloc(sizeof(double) * (size_t)dv * dk);
        double *u = (double *)malloc(sizeof(double) * (size_t)dv);
        int32_t *chain = (int32_t *)malloc(sizeof(int32_t) * (size_t)(T > 0 ? T : 1));
#pragma omp for schedule(dynamic, 8)
        for (int s = 0; s < n_sel; ++s) {
            const int b = sel_beam[s], h = sel_head[s];
            /* walk parent pointers newest -> oldest */
            int cur = b, ok = 1;
            for (int t = T - 1; t >= 0; --t) {
                if (cur < 0 || cur >= W[t]) { ok = 0; break; }
                chain[t] = cur;
                if (t > 0) cur = parents[t][cur];
            }
            if (!ok) {
#pragma omp atomic write
                bad = 1;
                continue;
            }
            if (chain_out)
                for (int t = 0; t < T; ++t) chain_out[(size_t)s * T + t] = chain[t];
            /* materialise the state: copy S0, apply Eq. 1 oldest -> newest */
            const float *S0h = S0 + (size_t)h * dv * dk;
            for (size_t e = 0; e < (size_t)dv * dk; ++e) S[e] = (double)S0h[e];
            for (int t = 0; t < T; ++t) {
                const size_t row = (size_t)chain[t] * H + h;
                gdn_transition(S, u, dk, dv, k[t] + row * dk, v[t] + row * dv,
                               (double)alpha[t][row], (double)beta[t][row]);
            }
            /* o = S q */
            const float *qv = q + ((size_t)b * H + h) * dk;
            for (int i = 0; i < dv; ++i) {
                double acc = 0.0;
                for (int j = 0; j < dk; ++j) acc += S[(size_t)i * dk + j] * (double)qv[j];
                out[(size_t)s * dv + i] = acc;
            }
        }
        free(S); free(u); free(chain);
    }
    return bad ? -1 : 0;
}

/*
 * Prefill: run Eq. 1 from the zero state over N prompt tokens, per head.
 *   k [N][H][dk], v [N][H][dv], alpha, beta [N][H] fp32;  S_out [H][dv][dk] fp64.
 */
int oracle_gdn_prefill(int H, int dk, int dv, int N, const float *k, const float *v,
                       const float *alpha, const float *beta, double *S_out, int nthreads) {
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif
#pragma omp parallel
    {
        double *u = (double *)malloc(sizeof(double) * (size_t)dv);
#pragma omp for schedule(dynamic, 1)
        for (int h = 0; h < H; ++h) {
            double *S = S_out + (size_t)h * dv * dk;
            memset(S, 0, sizeof(double) * (size_t)dv * dk);
            for (int t = 0; t < N; ++t) {
                const size_t row = (size_t)t * H + h;
                gdn_transition(S, u, dk, dv, k + row * dk, v + row * dv, (double)alpha[row],
                               (double)beta[row]);
            }
        }
        free(u);
    }
    return 0;
}
