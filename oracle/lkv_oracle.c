/*
 * lkv_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, fp64, token-by-token CPU statement of what the recurrent-layer
 * half of hybrid position-independent caching computes.  It exists only so that
 * the tests, the smoke check and the benchmark's cpu_baseline leg have something
 * independent to compare the CUDA library with.  It shares no code, header,
 * table or helper with the CUDA path and nothing in the product may call it.
 *
 * Every function is the definition written out: no blocking, no chunkwise
 * re-association, no WY/UT transform.  The only parallelism is an OpenMP loop
 * over heads, which never interact.
 *
 * Conventions (the paper leaves them open; each is fixed by a pin in the CPU
 * tests or recorded as "parity unpinned"):
 *   - state S of one head is d_k x d_v, row-major, d_v contiguous;
 *   - GDN update term  u_t = beta_t k_t v_t^T          (Eq. 1 with Eq. 3);
 *   - Mamba-2 update   u_t = dt_t  B_t x_t^T, a_t = exp(dt_t A_h)   (Eq. 2);
 *   - read-out uses the post-update state: o_t = scale * S_t^T q_t,
 *     y_t = S_t^T C_t                           (parity unpinned: convention);
 *   - value head h uses q/k head  h / (H_v / H_k)  (parity unpinned: convention);
 *   - a chunk's transition is the ordered product with the LATER token on the
 *     left, T_C = T_{t_L} ... T_{t_1}           (Eq. 5; pinned by brute force);
 *   - Eq. 6 is evaluated as the back-to-back application of Eq. 5 in context
 *     order, starting from the empty state.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int lkvo_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void lkvo_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/*
 * Gated DeltaNet, one sequence, token by token (Eq. 1 with the GDN transition of
 * Eq. 3):   S_t = alpha_t (I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T,
 * alpha_t = exp(g_t).  Expanding the product with S' = alpha_t S_{t-1} gives
 * S_t = S' + beta_t k_t (v_t - S'^T k_t)^T, which is what the loop does.
 *
 * q, k  : [T, Hk, dk]      v : [T, Hv, dv]      g, beta : [T, Hv]
 * S0    : [Hv, dk, dv] or NULL (empty state)
 * o     : [T, Hv, dv]      S_T : [Hv, dk, dv]
 */
void lkvo_gdn_seq(const double *q, const double *k, const double *v,
                  const double *g, const double *beta, const double *S0,
                  double scale, int T, int Hk, int Hv, int dk, int dv,
                  double *o, double *S_T)
{
    const int rep = Hv / Hk;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < Hv; ++h) {
        const int hk = h / rep;
        double *S = S_T + (size_t)h * dk * dv;
        double *r = (double *)malloc(sizeof(double) * (size_t)dv);
        if (S0)
            memcpy(S, S0 + (size_t)h * dk * dv, sizeof(double) * (size_t)dk * dv);
        else
            memset(S, 0, sizeof(double) * (size_t)dk * dv);
        for (int t = 0; t < T; ++t) {
            const double *kt = k + ((size_t)t * Hk + hk) * dk;
            const double *qt = q + ((size_t)t * Hk + hk) * dk;
            const double *vt = v + ((size_t)t * Hv + h) * dv;
            const double alpha = exp(g[(size_t)t * Hv + h]);
            const double b = beta[(size_t)t * Hv + h];
            /* S' = alpha S */
            for (int i = 0; i < dk * dv; ++i) S[i] *= alpha;
            /* r = v - S'^T k */
            for (int j = 0; j < dv; ++j) r[j] = vt[j];
            for (int i = 0; i < dk; ++i) {
                const double ki = kt[i];
                const double *Si = S + (size_t)i * dv;
                for (int j = 0; j < dv; ++j) r[j] -= Si[j] * ki;
            }
            /* S = S' + beta k r^T */
            for (int i = 0; i < dk; ++i) {
                const double c = b * kt[i];
                double *Si = S + (size_t)i * dv;
                for (int j = 0; j < dv; ++j) Si[j] += c * r[j];
            }
            /* o = scale S^T q */
            double *ot = o + ((size_t)t * Hv + h) * dv;
            for (int j = 0; j < dv; ++j) ot[j] = 0.0;
            for (int i = 0; i < dk; ++i) {
                const double qi = qt[i];
                const double *Si = S + (size_t)i * dv;
                for (int j = 0; j < dv; ++j) ot[j] += Si[j] * qi;
            }
            for (int j = 0; j < dv; ++j) ot[j] *= scale;
        }
        free(r);
    }
}

/*
 * Mamba-2 (SSD), one sequence, token by token (Eq. 1 with the scalar transition
 * of Eq. 2):   S_t = a_t S_{t-1} + dt_t B_t x_t^T,  a_t = exp(dt_t A_h),
 * y_t = S_t^T C_t.
 *
 * x : [T, H, P]   dt : [T, H]   A : [H]   B, C : [T, G, N]
 * S0 : [H, N, P] or NULL        y : [T, H, P]   S_T : [H, N, P]
 */
void lkvo_ssd_seq(const double *x, const double *dt, const double *A,
                  const double *B, const double *C, const double *S0,
                  int T, int H, int P, int N, int G, double *y, double *S_T)
{
    const int rep = H / G;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < H; ++h) {
        const int grp = h / rep;
        double *S = S_T + (size_t)h * N * P;
        if (S0)
            memcpy(S, S0 + (size_t)h * N * P, sizeof(double) * (size_t)N * P);
        else
            memset(S, 0, sizeof(double) * (size_t)N * P);
        for (int t = 0; t < T; ++t) {
            const double d = dt[(size_t)t * H + h];
            const double a = exp(d * A[h]);
            const double *xt = x + ((size_t)t * H + h) * P;
            const double *Bt = B + ((size_t)t * G + grp) * N;
            const double *Ct = C + ((size_t)t * G + grp) * N;
            double *yt = y + ((size_t)t * H + h) * P;
            for (int p = 0; p < P; ++p) yt[p] = 0.0;
            for (int n = 0; n < N; ++n) {
                double *Sn = S + (size_t)n * P;
                const double c = d * Bt[n];
                const double cn = Ct[n];
                for (int p = 0; p < P; ++p) {
                    Sn[p] = a * Sn[p] + c * xt[p];
                    yt[p] += Sn[p] * cn;
                }
            }
        }
    }
}

/*
 * Accumulated GDN transition of one chunk (the T_C of Eq. 5): start from the
 * identity and left-multiply by each token's T_t = alpha_t (I - beta_t k_t k_t^T)
 * in token order, so the last token ends up leftmost.
 *
 * k : [T, Hk, dk]   g, beta : [T, Hv]   Tc : [Hv, dk, dk] row-major
 */
void lkvo_gdn_transition(const double *k, const double *g, const double *beta,
                         int T, int Hk, int Hv, int dk, double *Tc)
{
    const int rep = Hv / Hk;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < Hv; ++h) {
        const int hk = h / rep;
        double *M = Tc + (size_t)h * dk * dk;
        double *w = (double *)malloc(sizeof(double) * (size_t)dk);
        for (int i = 0; i < dk; ++i)
            for (int c = 0; c < dk; ++c) M[(size_t)i * dk + c] = (i == c) ? 1.0 : 0.0;
        for (int t = 0; t < T; ++t) {
            const double *kt = k + ((size_t)t * Hk + hk) * dk;
            const double alpha = exp(g[(size_t)t * Hv + h]);
            const double b = beta[(size_t)t * Hv + h];
            /* w = k^T M  (row vector) */
            for (int c = 0; c < dk; ++c) w[c] = 0.0;
            for (int i = 0; i < dk; ++i) {
                const double ki = kt[i];
                const double *Mi = M + (size_t)i * dk;
                for (int c = 0; c < dk; ++c) w[c] += ki * Mi[c];
            }
            /* M = alpha (M - beta k w) */
            for (int i = 0; i < dk; ++i) {
                const double c0 = b * kt[i];
                double *Mi = M + (size_t)i * dk;
                for (int c = 0; c < dk; ++c) Mi[c] = alpha * (Mi[c] - c0 * w[c]);
            }
        }
        free(w);
    }
}

/*
 * Accumulated Mamba-2 transition of one chunk in log form: every token's
 * transition is the scalar exp(dt_t A_h) (Eq. 2), so the chunk's is
 * exp(lambda_h) with lambda_h = A_h * sum_t dt_t.
 *
 * dt : [T, H]   A : [H]   lam : [H]
 */
void lkvo_mamba_logdecay(const double *dt, const double *A, int T, int H, double *lam)
{
    for (int h = 0; h < H; ++h) {
        double s = 0.0;
        for (int t = 0; t < T; ++t) s += dt[(size_t)t * H + h];
        lam[h] = A[h] * s;
    }
}

/*
 * Exact composition for GDN (Eq. 6, evaluated as Eq. 5 applied chunk after chunk
 * from the empty state):  S <- S_{c_1};  S <- T_{c_j} S + S_{c_j}, j = 2..K.
 *
 * states : pool [n_chunks, H, dk, dv]   trans : pool [n_chunks, H, dk, dk]
 * ids    : int32[K] pool indices in context order
 * S0     : [H, dk, dv];  K == 0 gives the empty (zero) state.
 */
void lkvo_init_exact_gdn(const double *states, const double *trans, const int32_t *ids,
                         int K, int H, int dk, int dv, double *S0)
{
    const size_t ss = (size_t)dk * dv, ts = (size_t)dk * dk;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < H; ++h) {
        double *S = S0 + (size_t)h * ss;
        double *tmp = (double *)malloc(sizeof(double) * ss);
        memset(S, 0, sizeof(double) * ss);
        for (int j = 0; j < K; ++j) {
            const double *Sj = states + ((size_t)ids[j] * H + h) * ss;
            if (j == 0) {
                memcpy(S, Sj, sizeof(double) * ss);
                continue;
            }
            const double *Tj = trans + ((size_t)ids[j] * H + h) * ts;
            for (int i = 0; i < dk; ++i) {
                double *row = tmp + (size_t)i * dv;
                for (int c = 0; c < dv; ++c) row[c] = Sj[(size_t)i * dv + c];
                for (int m = 0; m < dk; ++m) {
                    const double tim = Tj[(size_t)i * dk + m];
                    const double *Sm = S + (size_t)m * dv;
                    for (int c = 0; c < dv; ++c) row[c] += tim * Sm[c];
                }
            }
            memcpy(S, tmp, sizeof(double) * ss);
        }
        free(tmp);
    }
}

/*
 * Exact composition for Mamba-2: the same chain with the scalar transition
 * exp(lambda_{c_j, h}).
 *
 * states : pool [n_chunks, H, N, P]   lam : pool [n_chunks, H]
 */
void lkvo_init_exact_mamba(const double *states, const double *lam, const int32_t *ids,
                           int K, int H, int N, int P, double *S0)
{
    const size_t ss = (size_t)N * P;
    for (int h = 0; h < H; ++h) {
        double *S = S0 + (size_t)h * ss;
        memset(S, 0, sizeof(double) * ss);
        for (int j = 0; j < K; ++j) {
            const double *Sj = states + ((size_t)ids[j] * H + h) * ss;
            if (j == 0) {
                memcpy(S, Sj, sizeof(double) * ss);
                continue;
            }
            const double a = exp(lam[(size_t)ids[j] * H + h]);
            for (size_t e = 0; e < ss; ++e) S[e] = a * S[e] + Sj[e];
        }
    }
}
