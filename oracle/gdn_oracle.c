/*
 * CPU fp64 oracle for the gated-delta-rule linear recurrence and its gradient.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call this file; it exists so that the
 * CUDA kernels can be compared against a plain, slow, token-by-token statement of the method.
 * It shares no code with the CUDA path.
 *
 * What it computes (paper Eq. 1 restricted to per-(token, head) scalar gates; Table 2 lists the
 * family members as gate settings).  Per (sequence, head) chain, state h of shape d_k x d_v:
 *
 *     ht_t = exp(g_t) * h_{t-1}                      decay
 *     p_t  = ht_t^T k_t                              what the state already predicts for key k_t
 *     u_t  = w_t * v_t - b_t * p_t                   delta-rule correction (erase gate b, write gate w)
 *     h_t  = ht_t + k_t u_t^T                        rank-one write
 *     o_t  = scale * h_t^T q_t                       read-out
 *
 * GDN is b_t = w_t = beta_t; the scalar-gate linear recurrence (SSD-like row of Table 2) is b = 0,
 * w = 1; g = 0 on top of that is plain causal linear attention.
 *
 * Gradient: for the scalar L = sum_t <dO_t, o_t> + <dh_T, h_T> the reverse-time adjoint of the five
 * lines above, walked from t = T down to 1 (the paper's Appendix A states only its shape:
 * "dS_t = Diag(e^{g_t}) dS_{t+1} + rank-one delta correction, walked backward"; the steps below are
 * that adjoint written out).  dg is the gradient with respect to the log-decay g, not exp(g).
 *
 * Parity pins (tests, no GPU needed): central finite differences, T = 1 closed form, reductions to
 * gated / plain linear attention computed as masked matrix products, the delta-rule write invariant
 * h_t^T k_t = v_t for unit keys with b = w = 1, linearity identities, split and packing consistency,
 * and equality with an independent chunked fp64 formulation.  Nothing here is "parity unpinned".
 *
 * Memory layout (all host pointers, all double, row-major):
 *     q, k [Ttot, H, d_k]   v, o, dO [Ttot, H, d_v]   g, b, w [Ttot, H]
 *     h0, hT, dhT, dh0 [N, H, d_k, d_v]               cu_seqlens int32 [N + 1] (cu[0] = 0, cu[N] = Ttot)
 * Return value: 0 on success, negative on argument error.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_SEG 64 /* forward states are kept every ORACLE_SEG tokens and re-materialised in between */

typedef struct {
    int N, H, dk, dv;
    const int32_t* cu;
    double scale;
    const double *q, *k, *v, *g, *b, *w, *h0, *dO, *dhT;
    double *o, *hT, *dq, *dkk, *dvv, *dg, *db, *dw, *dh0;
    int want_bwd;
    int next_chain; /* work counter, guarded by mu */
    pthread_mutex_t mu;
    int failed;
} job_t;

/* One forward step in place: h <- exp(g) h ; u = w v - b h^T k ; h += k u^T.  Returns u in `u`
 * and, when ht_out != NULL, the decayed state ht (before the write). */
static void fwd_step(int dk, int dv, double* h, const double* kt, const double* vt, double g, double b,
                     double w, double* u, double* ht_out) {
    const double a = exp(g);
    for (int i = 0; i < dk * dv; ++i) h[i] *= a;
    if (ht_out) memcpy(ht_out, h, sizeof(double) * (size_t)dk * dv);
    for (int c = 0; c < dv; ++c) {
        double p = 0.0;
        for (int r = 0; r < dk; ++r) p += h[r * dv + c] * kt[r];
        u[c] = w * vt[c] - b * p;
    }
    for (int r = 0; r < dk; ++r)
        for (int c = 0; c < dv; ++c) h[r * dv + c] += kt[r] * u[c];
}

static int run_chain(job_t* J, int n, int hd) {
    const int H = J->H, dk = J->dk, dv = J->dv;
    const int t0 = J->cu[n], t1 = J->cu[n + 1], len = t1 - t0;
    const size_t S = (size_t)dk * dv;
    const size_t soff = ((size_t)n * H + hd) * S;
    const int nseg = (len + ORACLE_SEG - 1) / ORACLE_SEG;

    double* h = (double*)malloc(sizeof(double) * S);
    double* u = (double*)malloc(sizeof(double) * dv);
    double* seg0 = J->want_bwd ? (double*)malloc(sizeof(double) * S * (size_t)(nseg > 0 ? nseg : 1)) : NULL;
    if (!h || !u || (J->want_bwd && !seg0)) { free(h); free(u); free(seg0); return -1; }

    if (J->h0) memcpy(h, J->h0 + soff, sizeof(double) * S); else memset(h, 0, sizeof(double) * S);

    /* ---- forward sweep ---- */
    for (int t = 0; t < len; ++t) {
        if (J->want_bwd && t % ORACLE_SEG == 0) memcpy(seg0 + (size_t)(t / ORACLE_SEG) * S, h, sizeof(double) * S);
        const size_t x = (size_t)(t0 + t) * H + hd;
        fwd_step(dk, dv, h, J->k + x * dk, J->v + x * dv, J->g[x], J->b[x], J->w[x], u, NULL);
        if (J->o) {
            const double* qt = J->q + x * dk;
            double* ot = J->o + x * dv;
            for (int c = 0; c < dv; ++c) {
                double s = 0.0;
                for (int r = 0; r < dk; ++r) s += h[r * dv + c] * qt[r];
                ot[c] = J->scale * s;
            }
        }
    }
    if (J->hT) memcpy(J->hT + soff, h, sizeof(double) * S);
    if (!J->want_bwd) { free(h); free(u); return 0; }

    /* ---- reverse sweep ---- */
    double* dh = (double*)malloc(sizeof(double) * S);
    double* hs = (double*)malloc(sizeof(double) * S * ORACLE_SEG);  /* h_t for the tokens of one segment */
    double* hts = (double*)malloc(sizeof(double) * S * ORACLE_SEG); /* ht_t (decayed, before the write) */
    double* us = (double*)malloc(sizeof(double) * (size_t)dv * ORACLE_SEG);
    double* du = (double*)malloc(sizeof(double) * dv);
    if (!dh || !hs || !hts || !us || !du) { free(h); free(u); free(seg0); free(dh); free(hs); free(hts); free(us); free(du); return -1; }
    if (J->dhT) memcpy(dh, J->dhT + soff, sizeof(double) * S); else memset(dh, 0, sizeof(double) * S);

    for (int sgm = nseg - 1; sgm >= 0; --sgm) {
        const int a0 = sgm * ORACLE_SEG;
        const int a1 = (a0 + ORACLE_SEG < len) ? a0 + ORACLE_SEG : len;
        memcpy(h, seg0 + (size_t)sgm * S, sizeof(double) * S);
        for (int t = a0; t < a1; ++t) {
            const size_t x = (size_t)(t0 + t) * H + hd;
            const int j = t - a0;
            fwd_step(dk, dv, h, J->k + x * dk, J->v + x * dv, J->g[x], J->b[x], J->w[x], us + (size_t)j * dv, hts + (size_t)j * S);
            memcpy(hs + (size_t)j * S, h, sizeof(double) * S);
        }
        for (int t = a1 - 1; t >= a0; --t) {
            const size_t x = (size_t)(t0 + t) * H + hd;
            const int j = t - a0;
            const double *qt = J->q + x * dk, *kt = J->k + x * dk, *vt = J->v + x * dv, *dOt = J->dO + x * dv;
            const double *ht_ = hts + (size_t)j * S, *h_ = hs + (size_t)j * S, *ut = us + (size_t)j * dv;
            const double b = J->b[x], w = J->w[x], sc = J->scale;
            double *dq = J->dq + x * dk, *dkt = J->dkk + x * dk, *dvt = J->dvv + x * dv;

            /* o_t = scale h_t^T q_t */
            for (int r = 0; r < dk; ++r) {
                double s = 0.0;
                for (int c = 0; c < dv; ++c) { s += h_[r * dv + c] * dOt[c]; dh[r * dv + c] += sc * qt[r] * dOt[c]; }
                dq[r] = sc * s;
            }
            /* h_t = ht_t + k_t u_t^T */
            for (int c = 0; c < dv; ++c) {
                double s = 0.0;
                for (int r = 0; r < dk; ++r) s += dh[r * dv + c] * kt[r];
                du[c] = s;
            }
            double dw_ = 0.0, db_ = 0.0;
            /* u_t = w v_t - b p_t,  p_t = ht_t^T k_t */
            for (int c = 0; c < dv; ++c) {
                double p = 0.0;
                for (int r = 0; r < dk; ++r) p += ht_[r * dv + c] * kt[r];
                dvt[c] = w * du[c];
                dw_ += du[c] * vt[c];
                db_ -= du[c] * p;
            }
            double dg_ = 0.0;
            const double a = exp(J->g[x]);
            for (int r = 0; r < dk; ++r) {
                double s1 = 0.0, s2 = 0.0;
                for (int c = 0; c < dv; ++c) {
                    s1 += dh[r * dv + c] * ut[c];       /* from h_t = ... + k u^T      */
                    s2 += ht_[r * dv + c] * du[c];      /* from p = ht^T k, dp = -b du */
                    const double dht = dh[r * dv + c] - b * kt[r] * du[c]; /* gradient w.r.t. ht_t */
                    dg_ += dht * ht_[r * dv + c];       /* ht = exp(g) h_{t-1}  =>  d ht / d g = ht */
                    dh[r * dv + c] = a * dht;           /* gradient w.r.t. h_{t-1} */
                }
                dkt[r] = s1 - b * s2;
            }
            J->dg[x] = dg_;
            J->db[x] = db_;
            J->dw[x] = dw_;
        }
    }
    if (J->dh0) memcpy(J->dh0 + soff, dh, sizeof(double) * S);
    free(h); free(u); free(seg0); free(dh); free(hs); free(hts); free(us); free(du);
    return 0;
}

static void* worker(void* arg) {
    job_t* J = (job_t*)arg;
    const int total = J->N * J->H;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        const int c = J->next_chain++;
        pthread_mutex_unlock(&J->mu);
        if (c >= total) break;
        if (run_chain(J, c / J->H, c % J->H) != 0) {
            pthread_mutex_lock(&J->mu);
            J->failed = 1;
            pthread_mutex_unlock(&J->mu);
        }
    }
    return NULL;
}

static int run_job(job_t* J, int n_threads) {
    if (J->N < 0 || J->H <= 0 || J->dk <= 0 || J->dv <= 0 || !J->cu) return -1;
    if (J->cu[0] != 0) return -2;
    for (int n = 0; n < J->N; ++n) if (J->cu[n + 1] < J->cu[n]) return -2;
    const int total = J->N * J->H;
    if (n_threads < 1) n_threads = 1;
    if (n_threads > total) n_threads = total > 0 ? total : 1;
    if (n_threads > 256) n_threads = 256;
    J->next_chain = 0;
    J->failed = 0;
    pthread_mutex_init(&J->mu, NULL);
    pthread_t th[256];
    int started = 0;
    for (int i = 1; i < n_threads; ++i) {
        if (pthread_create(&th[started], NULL, worker, J) == 0) ++started;
    }
    worker(J);
    for (int i = 0; i < started; ++i) pthread_join(th[i], NULL);
    pthread_mutex_destroy(&J->mu);
    return J->failed ? -3 : 0;
}

/* Forward only: o (may be NULL) and the final state hT (may be NULL). */
int gdn_oracle_fwd(int N, const int32_t* cu_seqlens, int H, int dk, int dv, double scale,
                   const double* q, const double* k, const double* v, const double* g, const double* b,
                   const double* w, const double* h0, double* o, double* hT, int n_threads) {
    if (!q || !k || !v || !g || !b || !w) return -1;
    job_t J;
    memset(&J, 0, sizeof(J));
    J.N = N; J.H = H; J.dk = dk; J.dv = dv; J.cu = cu_seqlens; J.scale = scale;
    J.q = q; J.k = k; J.v = v; J.g = g; J.b = b; J.w = w; J.h0 = h0; J.o = o; J.hT = hT;
    J.want_bwd = 0;
    return run_job(&J, n_threads);
}

/* Forward + reverse-time adjoint.  dq, dk, dv, dg, db, dw are required; o, hT, dh0, h0, dhT may be NULL
 * (a NULL h0 / dhT means zero).  For GDN (b = w = beta) the caller adds d beta = db + dw. */
int gdn_oracle_bwd(int N, const int32_t* cu_seqlens, int H, int dk, int dv, double scale,
                   const double* q, const double* k, const double* v, const double* g, const double* b,
                   const double* w, const double* h0, const double* dO, const double* dhT,
                   double* o, double* hT, double* dq, double* dk_out, double* dv_out, double* dg, double* db,
                   double* dw, double* dh0, int n_threads) {
    if (!q || !k || !v || !g || !b || !w || !dO || !dq || !dk_out || !dv_out || !dg || !db || !dw) return -1;
    job_t J;
    memset(&J, 0, sizeof(J));
    J.N = N; J.H = H; J.dk = dk; J.dv = dv; J.cu = cu_seqlens; J.scale = scale;
    J.q = q; J.k = k; J.v = v; J.g = g; J.b = b; J.w = w; J.h0 = h0; J.dO = dO; J.dhT = dhT;
    J.o = o; J.hT = hT; J.dq = dq; J.dkk = dk_out; J.dvv = dv_out; J.dg = dg; J.db = db; J.dw = dw; J.dh0 = dh0;
    J.want_bwd = 1;
    return run_job(&J, n_threads);
}
