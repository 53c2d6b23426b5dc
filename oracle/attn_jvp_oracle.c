/*
 * fp64 C oracle for attention with a Jacobian-vector product and its backward pass.
 *
 * TEST INFRASTRUCTURE ONLY.  Slow, plain, one score row at a time; shares no code with the
 * CUDA path and is never linked into the product library.  Only tests, the smoke check and
 * the CPU-baseline leg of the benchmark build and call it.
 *
 * Per (batch, head) and per query row i it materialises one row of every N-long quantity the
 * paper's App. C names and then applies the definitions literally:
 *
 *   a_j  = alpha * <Q_i, K_j>                  P_j = exp(a_j - max a) / sum_j exp(a_j - max a)
 *   t_j  = alpha * (<tQ_i, K_j> + <Q_i, tK_j>) mu  = sum_j P_j t_j        n_j = t_j - mu
 *   O_i  = sum_j P_j V_j                       tO_i = sum_j P_j n_j V_j + sum_j P_j tV_j
 *   lse  = max a + log sum_j exp(a_j - max a)
 *
 * Backward (cotangents G = dL/dO, Hc = dL/dtO).  Sigma_1 and Sigma_2 are the P-weighted sums of
 * App. C "Step 1" (not the rowsum(Hc*O) shortcut); d0 is the row term of a standard attention
 * backward, which the paper adds to the tangent-path gradients:
 *
 *   D_j  = <Hc_i, V_j>      gv_j = <G_i, V_j>      htv_j = <Hc_i, tV_j>
 *   Sg1  = sum_j P_j D_j    Sg2  = sum_j P_j (htv_j + D_j n_j)     d0 = sum_j P_j gv_j
 *   w_j  = P_j (D_j - Sg1)                                   (Steps 2/3 bracket)
 *   da_j = P_j (gv_j + htv_j - d0 - Sg2) + w_j n_j           (Steps 4/5 bracket + primal part)
 *   dV_j  += P_j G_i + P_j n_j Hc_i      dtV_j += P_j Hc_i               (Step 6 + primal part)
 *   dQ_i   = alpha sum_j (da_j K_j + w_j tK_j)     dtQ_i = alpha sum_j w_j K_j
 *   dK_j  += alpha (da_j Q_i + w_j tQ_i)           dtK_j += alpha w_j Q_i
 *
 * Layout: every tensor is packed (B, H, N, d) row-major double; lse and mu are (B, H, N) double.
 * Threads split the B*H heads; inside a head the loops are sequential, so sums have a fixed order.
 */
#include <math.h>
#include <pthread.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int is_bwd;
    long BH, N, d;
    double alpha;
    const double *Q, *K, *V, *tQ, *tK, *tV, *G, *Hc;
    double *O, *tO, *lse, *mu;
    double *dQ, *dK, *dV, *dtQ, *dtK, *dtV;
    long next; /* next head to take, guarded by lock */
    pthread_mutex_t lock;
    int failed;
} job_t;

static double dot(const double *x, const double *y, long d) {
    double s = 0.0;
    for (long c = 0; c < d; ++c) s += x[c] * y[c];
    return s;
}

/* Row i of head `h`: fills p[], n[] (length N) and returns lse and mu through pointers. */
static void score_row(const job_t *jb, long h, long i, double *a, double *p, double *t, double *n,
                      double *lse_out, double *mu_out) {
    const long N = jb->N, d = jb->d;
    const double *Qi = jb->Q + (h * N + i) * d, *tQi = jb->tQ + (h * N + i) * d;
    double amax = -INFINITY;
    for (long j = 0; j < N; ++j) {
        const double *Kj = jb->K + (h * N + j) * d, *tKj = jb->tK + (h * N + j) * d;
        a[j] = jb->alpha * dot(Qi, Kj, d);
        t[j] = jb->alpha * (dot(tQi, Kj, d) + dot(Qi, tKj, d));
        if (a[j] > amax) amax = a[j];
    }
    double denom = 0.0;
    for (long j = 0; j < N; ++j) {
        p[j] = exp(a[j] - amax);
        denom += p[j];
    }
    double mu = 0.0;
    for (long j = 0; j < N; ++j) {
        p[j] /= denom;
        mu += p[j] * t[j];
    }
    for (long j = 0; j < N; ++j) n[j] = t[j] - mu;
    *lse_out = amax + log(denom);
    *mu_out = mu;
}

static void fwd_head(const job_t *jb, long h, double *scratch) {
    const long N = jb->N, d = jb->d;
    double *a = scratch, *p = a + N, *t = p + N, *n = t + N;
    for (long i = 0; i < N; ++i) {
        double lse, mu;
        score_row(jb, h, i, a, p, t, n, &lse, &mu);
        double *Oi = jb->O + (h * N + i) * d, *tOi = jb->tO + (h * N + i) * d;
        for (long c = 0; c < d; ++c) { Oi[c] = 0.0; tOi[c] = 0.0; }
        for (long j = 0; j < N; ++j) {
            const double *Vj = jb->V + (h * N + j) * d, *tVj = jb->tV + (h * N + j) * d;
            const double pj = p[j], pdj = p[j] * n[j];
            for (long c = 0; c < d; ++c) {
                Oi[c] += pj * Vj[c];
                tOi[c] += pdj * Vj[c] + pj * tVj[c];
            }
        }
        jb->lse[h * N + i] = lse;
        jb->mu[h * N + i] = mu;
    }
}

static void bwd_head(const job_t *jb, long h, double *scratch) {
    const long N = jb->N, d = jb->d;
    double *a = scratch, *p = a + N, *t = p + N, *n = t + N;
    double *D = n + N, *gv = D + N, *htv = gv + N;
    const double alpha = jb->alpha;
    for (long j = 0; j < N; ++j)
        for (long c = 0; c < d; ++c) {
            long o = (h * N + j) * d + c;
            jb->dK[o] = 0.0; jb->dV[o] = 0.0; jb->dtK[o] = 0.0; jb->dtV[o] = 0.0;
        }
    for (long i = 0; i < N; ++i) {
        double lse, mu;
        score_row(jb, h, i, a, p, t, n, &lse, &mu);
        const double *Qi = jb->Q + (h * N + i) * d, *tQi = jb->tQ + (h * N + i) * d;
        const double *Gi = jb->G + (h * N + i) * d, *Hi = jb->Hc + (h * N + i) * d;
        double sg1 = 0.0, sg2 = 0.0, d0 = 0.0;
        for (long j = 0; j < N; ++j) {
            const double *Vj = jb->V + (h * N + j) * d, *tVj = jb->tV + (h * N + j) * d;
            D[j] = dot(Hi, Vj, d);
            gv[j] = dot(Gi, Vj, d);
            htv[j] = dot(Hi, tVj, d);
            sg1 += p[j] * D[j];
            sg2 += p[j] * (htv[j] + D[j] * n[j]);
            d0 += p[j] * gv[j];
        }
        double *dQi = jb->dQ + (h * N + i) * d, *dtQi = jb->dtQ + (h * N + i) * d;
        for (long c = 0; c < d; ++c) { dQi[c] = 0.0; dtQi[c] = 0.0; }
        for (long j = 0; j < N; ++j) {
            const double w = p[j] * (D[j] - sg1);
            const double da = p[j] * (gv[j] + htv[j] - d0 - sg2) + w * n[j];
            const double pj = p[j], pdj = p[j] * n[j];
            const double *Kj = jb->K + (h * N + j) * d, *tKj = jb->tK + (h * N + j) * d;
            double *dKj = jb->dK + (h * N + j) * d, *dtKj = jb->dtK + (h * N + j) * d;
            double *dVj = jb->dV + (h * N + j) * d, *dtVj = jb->dtV + (h * N + j) * d;
            for (long c = 0; c < d; ++c) {
                dQi[c] += da * Kj[c] + w * tKj[c];
                dtQi[c] += w * Kj[c];
                dKj[c] += alpha * (da * Qi[c] + w * tQi[c]);
                dtKj[c] += alpha * (w * Qi[c]);
                dVj[c] += pj * Gi[c] + pdj * Hi[c];
                dtVj[c] += pj * Hi[c];
            }
        }
        for (long c = 0; c < d; ++c) { dQi[c] *= alpha; dtQi[c] *= alpha; }
    }
}

static void *worker(void *arg) {
    job_t *jb = (job_t *)arg;
    double *scratch = (double *)malloc(sizeof(double) * 7 * (size_t)jb->N);
    if (!scratch) {
        pthread_mutex_lock(&jb->lock);
        jb->failed = 1;
        pthread_mutex_unlock(&jb->lock);
        return NULL;
    }
    for (;;) {
        pthread_mutex_lock(&jb->lock);
        long h = jb->next++;
        pthread_mutex_unlock(&jb->lock);
        if (h >= jb->BH) break;
        if (jb->is_bwd) bwd_head(jb, h, scratch); else fwd_head(jb, h, scratch);
    }
    free(scratch);
    return NULL;
}

static int run(job_t *jb, int nthreads) {
    if (jb->BH <= 0 || jb->N <= 0 || jb->d <= 0) return -1;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > jb->BH) nthreads = (int)jb->BH;
    if (nthreads > 256) nthreads = 256;
    pthread_t tid[256];
    jb->next = 0;
    jb->failed = 0;
    pthread_mutex_init(&jb->lock, NULL);
    int started = 0;
    for (int k = 0; k < nthreads; ++k)
        if (pthread_create(&tid[k], NULL, worker, jb) == 0) ++started; else break;
    if (started == 0) worker(jb); /* fall back to the calling thread */
    for (int k = 0; k < started; ++k) pthread_join(tid[k], NULL);
    pthread_mutex_destroy(&jb->lock);
    return jb->failed ? -2 : started > 0 ? started : 1;
}

/* Returns the number of threads used (> 0) or a negative error. */
int oracle_attn_jvp_fwd(long BH, long N, long d, double alpha, const double *Q, const double *K,
                        const double *V, const double *tQ, const double *tK, const double *tV,
                        double *O, double *tO, double *lse, double *mu, int nthreads) {
    job_t jb;
    memset(&jb, 0, sizeof jb);
    jb.is_bwd = 0; jb.BH = BH; jb.N = N; jb.d = d; jb.alpha = alpha;
    jb.Q = Q; jb.K = K; jb.V = V; jb.tQ = tQ; jb.tK = tK; jb.tV = tV;
    jb.O = O; jb.tO = tO; jb.lse = lse; jb.mu = mu;
    return run(&jb, nthreads);
}

int oracle_attn_jvp_bwd(long BH, long N, long d, double alpha, const double *Q, const double *K,
                        const double *V, const double *tQ, const double *tK, const double *tV,
                        const double *G, const double *Hc, double *dQ, double *dK, double *dV,
                        double *dtQ, double *dtK, double *dtV, int nthreads) {
    job_t jb;
    memset(&jb, 0, sizeof jb);
    jb.is_bwd = 1; jb.BH = BH; jb.N = N; jb.d = d; jb.alpha = alpha;
    jb.Q = Q; jb.K = K; jb.V = V; jb.tQ = tQ; jb.tK = tK; jb.tV = tV; jb.G = G; jb.Hc = Hc;
    jb.dQ = dQ; jb.dK = dK; jb.dV = dV; jb.dtQ = dtQ; jb.dtK = dtK; jb.dtV = dtV;
    return run(&jb, nthreads);
}
