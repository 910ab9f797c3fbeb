/*
 * HGRN2 recurrence oracle: plain C, fp64, step by step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct definition
 * that the CUDA library is checked against.  Only the tests, the smoke check and
 * the benchmark's cpu_baseline / reference arm may call it.  It shares no code,
 * header, table or helper with the CUDA path and the product never routes
 * through it.
 *
 * What it computes (paper Eq. 3, multi-head variant of Section 3.2, and the
 * HGRN2 <-> GLA correspondence of Table 4), per independent (batch, head) unit:
 *
 *     S_t[k][v] = a_t[k] * S_{t-1}[k][v] + kk_t[k] * vv_t[v]
 *     y_t[v]    = sum_k q_t[k] * S_t[k][v]            (the UPDATED state feeds y_t)
 *
 * The paper writes h_t = h_{t-1} Diag{f_t} + i_t (x) (1 - f_t), y_t = h_t o_t with
 * h in R^{d x d} whose columns are indexed by the gate dimension; S here is the
 * transpose of h (rows = gate/key dimension k, columns = input/value dimension
 * v), which is the same set of numbers.
 *
 * The core is written for the UNTIED recurrence (separate a, kk) so that the
 * special case a == 1 can be pinned against plain causal linear attention; the
 * HGRN2 entry points tie the gates: q = o, a = f, kk = 1 - f, vv = i.
 * Products are taken in linear space (no logarithms), so f = 0 and f = 1 are
 * exact.  No 1/sqrt(d) scale is applied: Eq. 3 has none.
 *
 * Backward: the paper gives none (training is delegated to prior work), so it
 * is the reverse-mode derivative of the loop above, derived by hand, for the
 * scalar  L = sum_t <dy_t, y_t> + <dSN, S_N>:
 *
 *     G_N = dSN;  for t = N..1:
 *         G_t     = G_t(carried) + q_t dy_t^T              (dL/dS_t, all paths)
 *         dq_t[k] = sum_v S_t[k][v]     * dy_t[v]
 *         dk_t[k] = sum_v G_t[k][v]     * vv_t[v]
 *         dv_t[v] = sum_k kk_t[k]       * G_t[k][v]
 *         da_t[k] = sum_v G_t[k][v]     * S_{t-1}[k][v]
 *         G_{t-1}(carried) = Diag(a_t) G_t
 *     dS0 = G_0(carried)
 *
 * With tied gates d_f = da - dk (f enters as the decay and as kk = 1 - f).
 * S_t is re-created from checkpoints spaced about sqrt(N) steps apart.
 *
 * Layouts: every sequence tensor is [B][H][N][d] contiguous (d innermost);
 * states are [B][H][dk][dv] (dv innermost).  All pointers are host memory.
 * Nullable: S0 (zero state), SN, dSN (zero), dS0.
 * Return value: 0 on success, -1 on allocation failure or bad sizes.
 *
 * Parity pins (tests/test_oracle_pins.py): unrolled closed form by brute force,
 * f == 0, f == 1 (tied and untied vs. a library matmul), central finite
 * differences, adjoint identities, d_k = d_v = 1 vs. the scalar recurrence of
 * Eq. 1/2, partition of unity, state passing.  Every function here is pinned.
 */
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int hgrn2_ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One recurrence step on one unit, in place.  Eq. 3. */
static void gla_step_unit(int dk, int dv, const double *q, const double *kk, const double *vv,
                          const double *a, double *S, double *y)
{
    for (int k = 0; k < dk; ++k)
        for (int v = 0; v < dv; ++v)
            S[(size_t)k * dv + v] = a[k] * S[(size_t)k * dv + v] + kk[k] * vv[v];
    if (y) {
        for (int v = 0; v < dv; ++v) {
            double acc = 0.0;
            for (int k = 0; k < dk; ++k)
                acc += q[k] * S[(size_t)k * dv + v];
            y[v] = acc;
        }
    }
}

static void gla_fwd_unit(long N, int dk, int dv, const double *q, const double *kk, const double *vv,
                         const double *a, const double *S0, double *y, double *SN, double *S)
{
    const size_t ss = (size_t)dk * dv;
    if (S0) memcpy(S, S0, ss * sizeof(double));
    else    memset(S, 0, ss * sizeof(double));
    for (long t = 0; t < N; ++t)
        gla_step_unit(dk, dv, q + t * dk, kk + t * dk, vv + t * dv, a + t * dk, S,
                      y ? y + t * dv : NULL);
    if (SN) memcpy(SN, S, ss * sizeof(double));
}

/* Reverse-mode derivative of gla_fwd_unit.  Returns -1 if scratch cannot be allocated. */
static int gla_bwd_unit(long N, int dk, int dv, const double *q, const double *kk, const double *vv,
                        const double *a, const double *S0, const double *dy, const double *dSN,
                        double *dq, double *dkk, double *dvv, double *da, double *dS0)
{
    const size_t ss = (size_t)dk * dv;
    long L = 1;
    while (L * L < N) ++L;                 /* segment length ~ sqrt(N) */
    if (L < 1) L = 1;
    const long nseg = (N + L - 1) / L;

    double *ckpt = (double *)malloc((size_t)(nseg > 0 ? nseg : 1) * ss * sizeof(double));
    double *seg  = (double *)malloc((size_t)(L + 1) * ss * sizeof(double));
    double *G    = (double *)malloc(ss * sizeof(double));
    if (!ckpt || !seg || !G) { free(ckpt); free(seg); free(G); return -1; }

    /* forward sweep: keep the state at the start of every segment */
    double *S = seg;                       /* borrow seg[0] as the running state */
    if (S0) memcpy(S, S0, ss * sizeof(double));
    else    memset(S, 0, ss * sizeof(double));
    for (long t = 0; t < N; ++t) {
        if (t % L == 0) memcpy(ckpt + (size_t)(t / L) * ss, S, ss * sizeof(double));
        gla_step_unit(dk, dv, q + t * dk, kk + t * dk, vv + t * dv, a + t * dk, S, NULL);
    }

    if (dSN) memcpy(G, dSN, ss * sizeof(double));
    else     memset(G, 0, ss * sizeof(double));

    for (long s = nseg - 1; s >= 0; --s) {
        const long t0 = s * L;
        const long t1 = (t0 + L < N) ? t0 + L : N;
        /* seg[j] = state BEFORE step t0 + j, j = 0..(t1 - t0); seg[j+1] = state after it */
        memcpy(seg, ckpt + (size_t)s * ss, ss * sizeof(double));
        for (long t = t0; t < t1; ++t) {
            double *cur = seg + (size_t)(t - t0 + 1) * ss;
            memcpy(cur, seg + (size_t)(t - t0) * ss, ss * sizeof(double));
            gla_step_unit(dk, dv, q + t * dk, kk + t * dk, vv + t * dv, a + t * dk, cur, NULL);
        }
        for (long t = t1 - 1; t >= t0; --t) {
            const double *St   = seg + (size_t)(t - t0 + 1) * ss;   /* S_t     */
            const double *Stm1 = seg + (size_t)(t - t0) * ss;       /* S_{t-1} */
            const double *qt = q + t * dk, *kt = kk + t * dk, *vt = vv + t * dv, *at = a + t * dk;
            const double *dyt = dy + t * dv;
            for (int k = 0; k < dk; ++k)
                for (int v = 0; v < dv; ++v)
                    G[(size_t)k * dv + v] += qt[k] * dyt[v];
            for (int k = 0; k < dk; ++k) {
                double sq = 0.0, sk = 0.0, sa = 0.0;
                for (int v = 0; v < dv; ++v) {
                    sq += St[(size_t)k * dv + v] * dyt[v];
                    sk += G[(size_t)k * dv + v] * vt[v];
                    sa += G[(size_t)k * dv + v] * Stm1[(size_t)k * dv + v];
                }
                dq[t * dk + k]  = sq;
                dkk[t * dk + k] = sk;
                da[t * dk + k]  = sa;
            }
            for (int v = 0; v < dv; ++v) {
                double sv = 0.0;
                for (int k = 0; k < dk; ++k)
                    sv += kt[k] * G[(size_t)k * dv + v];
                dvv[t * dv + v] = sv;
            }
            for (int k = 0; k < dk; ++k)
                for (int v = 0; v < dv; ++v)
                    G[(size_t)k * dv + v] *= at[k];
        }
    }
    if (dS0) memcpy(dS0, G, ss * sizeof(double));
    free(ckpt); free(seg); free(G);
    return 0;
}

/* ---- untied entry points (GLA column of Table 4) --------------------------------------- */

int ref_gla_fwd(int B, int H, long N, int dk, int dv, const double *q, const double *kk,
                const double *vv, const double *a, const double *S0, double *y, double *SN)
{
    if (B < 0 || H < 0 || N < 0 || dk <= 0 || dv <= 0) return -1;
    const long U = (long)B * H;
    const size_t ss = (size_t)dk * dv;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long u = 0; u < U; ++u) {
        double *S = (double *)malloc(ss * sizeof(double));
        if (!S) {
#pragma omp atomic write
            fail = 1;
            continue;
        }
        gla_fwd_unit(N, dk, dv, q + u * N * dk, kk + u * N * dk, vv + u * N * dv, a + u * N * dk,
                     S0 ? S0 + u * ss : NULL, y ? y + u * N * dv : NULL, SN ? SN + u * ss : NULL, S);
        free(S);
    }
    return fail ? -1 : 0;
}

int ref_gla_bwd(int B, int H, long N, int dk, int dv, const double *q, const double *kk,
                const double *vv, const double *a, const double *S0, const double *dy,
                const double *dSN, double *dq, double *dkk, double *dvv, double *da, double *dS0)
{
    if (B < 0 || H < 0 || N < 0 || dk <= 0 || dv <= 0) return -1;
    const long U = (long)B * H;
    const size_t ss = (size_t)dk * dv;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (long u = 0; u < U; ++u) {
        int rc = gla_bwd_unit(N, dk, dv, q + u * N * dk, kk + u * N * dk, vv + u * N * dv,
                              a + u * N * dk, S0 ? S0 + u * ss : NULL, dy + u * N * dv,
                              dSN ? dSN + u * ss : NULL, dq + u * N * dk, dkk + u * N * dk,
                              dvv + u * N * dv, da + u * N * dk, dS0 ? dS0 + u * ss : NULL);
        if (rc != 0) {
#pragma omp atomic write
            fail = 1;
        }
    }
    return fail ? -1 : 0;
}

/* ---- HGRN2 entry points: tied gates q = o, a = f, kk = 1 - f, vv = i (Table 4) ---------- */

static double *one_minus(const double *f, size_t n)
{
    double *k = (double *)malloc((n ? n : 1) * sizeof(double));
    if (!k) return NULL;
    for (size_t j = 0; j < n; ++j) k[j] = 1.0 - f[j];
    return k;
}

int ref_hgrn2_fwd(int B, int H, long N, int dk, int dv, const double *o, const double *f,
                  const double *i, const double *S0, double *y, double *SN)
{
    if (B < 0 || H < 0 || N < 0 || dk <= 0 || dv <= 0) return -1;
    const size_t n = (size_t)B * H * N * dk;
    double *kk = one_minus(f, n);
    if (!kk) return -1;
    int rc = ref_gla_fwd(B, H, N, dk, dv, o, kk, i, f, S0, y, SN);
    free(kk);
    return rc;
}

int ref_hgrn2_bwd(int B, int H, long N, int dk, int dv, const double *o, const double *f,
                  const double *i, const double *S0, const double *dy, const double *dSN,
                  double *d_o, double *d_f, double *d_i, double *dS0)
{
    if (B < 0 || H < 0 || N < 0 || dk <= 0 || dv <= 0) return -1;
    const size_t n = (size_t)B * H * N * dk;
    double *kk  = one_minus(f, n);
    double *dkk = (double *)malloc((n ? n : 1) * sizeof(double));
    if (!kk || !dkk) { free(kk); free(dkk); return -1; }
    /* d_f first receives the decay-path gradient da, then the key path is folded in. */
    int rc = ref_gla_bwd(B, H, N, dk, dv, o, kk, i, f, S0, dy, dSN, d_o, dkk, d_i, d_f, dS0);
    if (rc == 0)
        for (size_t j = 0; j < n; ++j) d_f[j] -= dkk[j];
    free(kk); free(dkk);
    return rc;
}

/* One decode step for every unit: o, f are [B][H][dk], i and y are [B][H][dv], S in place. */
int ref_hgrn2_step(int B, int H, int dk, int dv, const double *o, const double *f, const double *i,
                   double *S, double *y)
{
    if (B < 0 || H < 0 || dk <= 0 || dv <= 0) return -1;
    const long U = (long)B * H;
    const size_t ss = (size_t)dk * dv;
    int fail = 0;
#pragma omp parallel for schedule(static)
    for (long u = 0; u < U; ++u) {
        double *kk = (double *)malloc((size_t)dk * sizeof(double));
        if (!kk) {
#pragma omp atomic write
            fail = 1;
            continue;
        }
        for (int k = 0; k < dk; ++k) kk[k] = 1.0 - f[u * dk + k];
        gla_step_unit(dk, dv, o + u * dk, kk, i + u * dv, f + u * dk, S + u * ss, y + u * dv);
        free(kk);
    }
    return fail ? -1 : 0;
}
