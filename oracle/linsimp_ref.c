/*
 * fp64 CPU oracle for linearized 2-simplicial attention (LinSimp), plain C.
 *
 * TEST INFRASTRUCTURE ONLY: the same recurrent definition as linsimp_ref.py,
 * written as explicit loops so that it can be read against the paper and so
 * that it is fast enough to check slices of the full-size workloads and to be
 * the timed CPU baseline.  It shares no code with the CUDA library.
 *
 *   phi(x)  = exp(Omega x - |x|^2/2)/sqrt(m)                    (Eq. prf)
 *   M_i = M_{i-1} + phi(k_i) v_i^T ,  a_i = a_{i-1} + phi(k_i)  (Eqs. Mstate, astate)
 *   C_i = {max(0,i-W+1) .. i}                                   (Sec. 3.3)
 *   N_i = sum_c [phi(q_i*r_c)^T M_i]*u_c , Z_i = sum_c phi(q_i*r_c)^T a_i
 *   o_i = N_i/(Z_i+eps)                       (Eqs. Ni, Zi, linearized-output)
 *
 * A "unit" is one (batch, head) sequence; units are independent and are the
 * only thing parallelised (OpenMP, one unit per thread at a time).
 * Layout: q,k,r,v,u,dO and gradients [n_units][T][d] (value width = d);
 * omega [n_omega][d][m], unit n uses bank n % n_omega; states M [m][d], a [m]
 * including the 1/sqrt(m) factor.  Rows < t0 are history: their keys/values
 * are already inside (M0,a0) and they serve only as anchors.
 * Pinned by tests against linsimp_ref.py and, through it, by that file's pins.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* log features l_p = sum_a omega[a][p] x[a] - |x|^2/2, then phi_p = exp(l_p)/sqrt(m) */
static void feature_map(const double *x, const double *omega, int d, int m, double *out)
{
    double nrm = 0.0;
    for (int a = 0; a < d; ++a) nrm += x[a] * x[a];
    for (int p = 0; p < m; ++p) out[p] = 0.0;
    for (int a = 0; a < d; ++a) {
        const double xa = x[a];
        const double *row = omega + (size_t)a * m;
        for (int p = 0; p < m; ++p) out[p] += row[p] * xa;
    }
    const double s = 1.0 / sqrt((double)m);
    for (int p = 0; p < m; ++p) out[p] = exp(out[p] - 0.5 * nrm) * s;
}

static void state_update(double *M, double *a, const double *chi, const double *v, int d, int m)
{
    for (int p = 0; p < m; ++p) {
        a[p] += chi[p];
        double *Mp = M + (size_t)p * d;
        const double cp = chi[p];
        for (int e = 0; e < d; ++e) Mp[e] += cp * v[e];
    }
}

int linsimp_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Prefix state alone (Eqs. Mstate, astate): M [n][m][d], a [n][m] after all T rows (added to M0, a0 if given). */
int linsimp_oracle_prefix_state(int n_units, int T, int d, int m,
                                const double *k, const double *v, const double *omega, int n_omega,
                                const double *M0, const double *a0, double *Mout, double *aout)
{
    if (n_units < 0 || T < 0 || d < 1 || m < 1 || n_omega < 1) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int n = 0; n < n_units; ++n) {
        const double *om = omega + (size_t)(n % n_omega) * d * m;
        double *M = Mout + (size_t)n * m * d, *a = aout + (size_t)n * m;
        double *chi = malloc(sizeof(double) * m);
        if (!chi) {
            failed = 1;
        } else {
            for (size_t x = 0; x < (size_t)m * d; ++x) M[x] = M0 ? M0[(size_t)n * m * d + x] : 0.0;
            for (int p = 0; p < m; ++p) a[p] = a0 ? a0[(size_t)n * m + p] : 0.0;
            for (int j = 0; j < T; ++j) {
                feature_map(k + ((size_t)n * T + j) * d, om, d, m, chi);
                state_update(M, a, chi, v + ((size_t)n * T + j) * d, d, m);
            }
        }
        free(chi);
    }
    return failed ? -2 : 0;
}

/* Forward.  o [n][T][d]; Zout nullable [n][T]; Mout/aout nullable final states. */
int linsimp_oracle_fwd(int n_units, int T, int d, int m, int W, double eps,
                       const double *q, const double *k, const double *v,
                       const double *r, const double *u,
                       const double *omega, int n_omega,
                       const double *M0, const double *a0, int t0,
                       double *o, double *Zout, double *Mout, double *aout)
{
    if (n_units < 0 || T < 0 || d < 1 || m < 1 || W < 1 || n_omega < 1) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int n = 0; n < n_units; ++n) {
        const size_t off = (size_t)n * T * d;
        const double *om = omega + (size_t)(n % n_omega) * d * m;
        double *M = calloc((size_t)m * d, sizeof(double));
        double *a = calloc((size_t)m, sizeof(double));
        double *chi = malloc(sizeof(double) * m);
        double *psi = malloc(sizeof(double) * m);
        double *x = malloc(sizeof(double) * d);
        double *g = malloc(sizeof(double) * d);
        double *N = malloc(sizeof(double) * d);
        if (!M || !a || !chi || !psi || !x || !g || !N) {
            failed = 1;
        } else {
            if (M0) memcpy(M, M0 + (size_t)n * m * d, sizeof(double) * m * d);
            if (a0) memcpy(a, a0 + (size_t)n * m, sizeof(double) * m);
            for (int i = 0; i < t0 && i < T; ++i)
                for (int e = 0; e < d; ++e) o[off + (size_t)i * d + e] = 0.0;
            for (int i = t0; i < T; ++i) {
                feature_map(k + off + (size_t)i * d, om, d, m, chi);
                state_update(M, a, chi, v + off + (size_t)i * d, d, m);
                for (int e = 0; e < d; ++e) N[e] = 0.0;
                double Z = 0.0;
                const int c0 = i - W + 1 > 0 ? i - W + 1 : 0;
                for (int c = c0; c <= i; ++c) {
                    const double *qi = q + off + (size_t)i * d;
                    const double *rc = r + off + (size_t)c * d;
                    const double *uc = u + off + (size_t)c * d;
                    for (int b = 0; b < d; ++b) x[b] = qi[b] * rc[b];
                    feature_map(x, om, d, m, psi);
                    for (int e = 0; e < d; ++e) g[e] = 0.0;
                    for (int p = 0; p < m; ++p) {
                        const double pp = psi[p];
                        const double *Mp = M + (size_t)p * d;
                        for (int e = 0; e < d; ++e) g[e] += pp * Mp[e];
                        Z += pp * a[p];
                    }
                    for (int e = 0; e < d; ++e) N[e] += g[e] * uc[e];
                }
                for (int e = 0; e < d; ++e) o[off + (size_t)i * d + e] = N[e] / (Z + eps);
                if (Zout) Zout[(size_t)n * T + i] = Z;
            }
            if (Mout) memcpy(Mout + (size_t)n * m * d, M, sizeof(double) * m * d);
            if (aout) memcpy(aout + (size_t)n * m, a, sizeof(double) * m);
        }
        free(M); free(a); free(chi); free(psi); free(x); free(g); free(N);
    }
    return failed ? -2 : 0;
}

/* Backward of sum(dO*o): sweep 1 forward over queries (dq, dr, du), sweep 2
 * backward over keys/values (dk, dv) with D = sum_{i>=j} dM_i, e = sum_{i>=j} da_i.
 * All five gradient arrays are overwritten. */
int linsimp_oracle_bwd(int n_units, int T, int d, int m, int W, double eps,
                       const double *q, const double *k, const double *v,
                       const double *r, const double *u,
                       const double *omega, int n_omega,
                       const double *M0, const double *a0, int t0,
                       const double *dO,
                       double *dq, double *dk, double *dv, double *dr, double *du)
{
    if (n_units < 0 || T < 0 || d < 1 || m < 1 || W < 1 || n_omega < 1) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int n = 0; n < n_units; ++n) {
        const size_t off = (size_t)n * T * d;
        const double *om = omega + (size_t)(n % n_omega) * d * m;
        double *M = calloc((size_t)m * d, sizeof(double));
        double *a = calloc((size_t)m, sizeof(double));
        double *D = calloc((size_t)m * d, sizeof(double));
        double *ee = calloc((size_t)m, sizeof(double));
        double *chi = malloc(sizeof(double) * m);
        double *psi = malloc(sizeof(double) * m);
        double *dl = malloc(sizeof(double) * m);
        double *x = malloc(sizeof(double) * d);
        double *g = malloc(sizeof(double) * d);
        double *dg = malloc(sizeof(double) * d);
        double *N = malloc(sizeof(double) * d);
        double *gw = malloc(sizeof(double) * (size_t)W * d);   /* g_ic of one query */
        double *dNs = calloc((size_t)T * d + 1, sizeof(double));
        double *dZs = calloc((size_t)T + 1, sizeof(double));
        if (!M || !a || !D || !ee || !chi || !psi || !dl || !x || !g || !dg || !N || !gw || !dNs || !dZs) {
            failed = 1;
        } else {
            if (M0) memcpy(M, M0 + (size_t)n * m * d, sizeof(double) * m * d);
            if (a0) memcpy(a, a0 + (size_t)n * m, sizeof(double) * m);
            memset(dq + off, 0, sizeof(double) * T * d);
            memset(dk + off, 0, sizeof(double) * T * d);
            memset(dv + off, 0, sizeof(double) * T * d);
            memset(dr + off, 0, sizeof(double) * T * d);
            memset(du + off, 0, sizeof(double) * T * d);
            /* sweep 1 */
            for (int i = t0; i < T; ++i) {
                const double *qi = q + off + (size_t)i * d;
                feature_map(k + off + (size_t)i * d, om, d, m, chi);
                state_update(M, a, chi, v + off + (size_t)i * d, d, m);
                const int c0 = i - W + 1 > 0 ? i - W + 1 : 0;
                /* pass A: N, Z, and g_ic kept for du */
                for (int e = 0; e < d; ++e) N[e] = 0.0;
                double Z = 0.0;
                for (int c = c0; c <= i; ++c) {
                    const double *rc = r + off + (size_t)c * d;
                    const double *uc = u + off + (size_t)c * d;
                    double *gc = gw + (size_t)(c - c0) * d;
                    for (int b = 0; b < d; ++b) x[b] = qi[b] * rc[b];
                    feature_map(x, om, d, m, psi);
                    for (int e = 0; e < d; ++e) gc[e] = 0.0;
                    for (int p = 0; p < m; ++p) {
                        const double *Mp = M + (size_t)p * d;
                        for (int e = 0; e < d; ++e) gc[e] += psi[p] * Mp[e];
                        Z += psi[p] * a[p];
                    }
                    for (int e = 0; e < d; ++e) N[e] += gc[e] * uc[e];
                }
                const double den = Z + eps;
                double dot = 0.0;
                for (int e = 0; e < d; ++e) dot += dO[off + (size_t)i * d + e] * (N[e] / den);
                double *dNi = dNs + (size_t)i * d;
                for (int e = 0; e < d; ++e) dNi[e] = dO[off + (size_t)i * d + e] / den;
                const double dZi = -dot / den;
                dZs[i] = dZi;
                /* pass B: gradients through each anchor */
                for (int c = c0; c <= i; ++c) {
                    const double *rc = r + off + (size_t)c * d;
                    const double *uc = u + off + (size_t)c * d;
                    const double *gc = gw + (size_t)(c - c0) * d;
                    for (int e = 0; e < d; ++e) {
                        du[off + (size_t)c * d + e] += dNi[e] * gc[e];
                        dg[e] = dNi[e] * uc[e];
                    }
                    for (int b = 0; b < d; ++b) x[b] = qi[b] * rc[b];
                    feature_map(x, om, d, m, psi);
                    double sdl = 0.0;
                    for (int p = 0; p < m; ++p) {
                        const double *Mp = M + (size_t)p * d;
                        double dpsi = dZi * a[p];
                        for (int e = 0; e < d; ++e) dpsi += Mp[e] * dg[e];
                        dl[p] = dpsi * psi[p];
                        sdl += dl[p];
                    }
                    for (int b = 0; b < d; ++b) {
                        const double *row = om + (size_t)b * m;
                        double dx = -sdl * x[b];             /* d l/d z = omega - z */
                        for (int p = 0; p < m; ++p) dx += row[p] * dl[p];
                        dq[off + (size_t)i * d + b] += dx * rc[b];
                        dr[off + (size_t)c * d + b] += dx * qi[b];
                    }
                }
            }
            /* sweep 2 */
            for (int i = T - 1; i >= t0; --i) {
                const double *qi = q + off + (size_t)i * d;
                const double *dNi = dNs + (size_t)i * d;
                const int c0 = i - W + 1 > 0 ? i - W + 1 : 0;
                for (int c = c0; c <= i; ++c) {
                    const double *rc = r + off + (size_t)c * d;
                    const double *uc = u + off + (size_t)c * d;
                    for (int b = 0; b < d; ++b) x[b] = qi[b] * rc[b];
                    feature_map(x, om, d, m, psi);
                    for (int e = 0; e < d; ++e) dg[e] = dNi[e] * uc[e];
                    for (int p = 0; p < m; ++p) {
                        double *Dp = D + (size_t)p * d;
                        for (int e = 0; e < d; ++e) Dp[e] += psi[p] * dg[e];   /* dM_i */
                        ee[p] += dZs[i] * psi[p];                              /* da_i */
                    }
                }
                const double *ki = k + off + (size_t)i * d;
                const double *vi = v + off + (size_t)i * d;
                feature_map(ki, om, d, m, chi);
                double sdl = 0.0;
                for (int e = 0; e < d; ++e) g[e] = 0.0;
                for (int p = 0; p < m; ++p) {
                    const double *Dp = D + (size_t)p * d;
                    double dchi = ee[p];
                    for (int e = 0; e < d; ++e) {
                        dchi += Dp[e] * vi[e];
                        g[e] += Dp[e] * chi[p];
                    }
                    dl[p] = dchi * chi[p];
                    sdl += dl[p];
                }
                for (int e = 0; e < d; ++e) dv[off + (size_t)i * d + e] = g[e];
                for (int b = 0; b < d; ++b) {
                    const double *row = om + (size_t)b * m;
                    double acc = -sdl * ki[b];
                    for (int p = 0; p < m; ++p) acc += row[p] * dl[p];
                    dk[off + (size_t)i * d + b] = acc;
                }
            }
        }
        free(M); free(a); free(D); free(ee); free(chi); free(psi); free(dl);
        free(x); free(g); free(dg); free(N); free(gw); free(dNs); free(dZs);
    }
    return failed ? -2 : 0;
}

/* One decode step per unit (Theorem 1).  M [n][m][d], a [n][m] in/out;
 * ring_r, ring_u [n][W][d] in/out; pos[n] = tokens seen so far.  The state is
 * updated, token pos is stored at slot pos % W, then min(pos+1, W) anchors are read. */
int linsimp_oracle_decode(int n_units, int d, int m, int W, double eps,
                          const double *q, const double *k, const double *v,
                          const double *r, const double *u,
                          const double *omega, int n_omega,
                          double *M, double *a, double *ring_r, double *ring_u,
                          const int *pos, double *o)
{
    if (n_units < 0 || d < 1 || m < 1 || W < 1 || n_omega < 1) return -1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int n = 0; n < n_units; ++n) {
        const double *om = omega + (size_t)(n % n_omega) * d * m;
        double *Mn = M + (size_t)n * m * d, *an = a + (size_t)n * m;
        double *rr = ring_r + (size_t)n * W * d, *ru = ring_u + (size_t)n * W * d;
        double *chi = malloc(sizeof(double) * m);
        double *psi = malloc(sizeof(double) * m);
        double *x = malloc(sizeof(double) * d);
        double *g = malloc(sizeof(double) * d);
        double *N = calloc((size_t)d, sizeof(double));
        if (!chi || !psi || !x || !g || !N) {
            failed = 1;
        } else {
            const int t = pos[n];
            feature_map(k + (size_t)n * d, om, d, m, chi);
            state_update(Mn, an, chi, v + (size_t)n * d, d, m);
            memcpy(rr + (size_t)(t % W) * d, r + (size_t)n * d, sizeof(double) * d);
            memcpy(ru + (size_t)(t % W) * d, u + (size_t)n * d, sizeof(double) * d);
            const int cnt = t + 1 < W ? t + 1 : W;
            double Z = 0.0;
            for (int s = 0; s < cnt; ++s) {
                const int slot = ((t - s) % W + W) % W;
                const double *rc = rr + (size_t)slot * d, *uc = ru + (size_t)slot * d;
                for (int b = 0; b < d; ++b) x[b] = q[(size_t)n * d + b] * rc[b];
                feature_map(x, om, d, m, psi);
                for (int e = 0; e < d; ++e) g[e] = 0.0;
                for (int p = 0; p < m; ++p) {
                    const double *Mp = Mn + (size_t)p * d;
                    for (int e = 0; e < d; ++e) g[e] += psi[p] * Mp[e];
                    Z += psi[p] * an[p];
                }
                for (int e = 0; e < d; ++e) N[e] += g[e] * uc[e];
            }
            for (int e = 0; e < d; ++e) o[(size_t)n * d + e] = N[e] / (Z + eps);
        }
        free(chi); free(psi); free(x); free(g); free(N);
    }
    return failed ? -2 : 0;
}
