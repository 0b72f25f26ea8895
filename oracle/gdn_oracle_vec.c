/*
 * CPU fp64 oracle for the general gated-delta-rule recurrence with PER-CHANNEL gates and its gradient.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call this file.  It shares no code with
 * the CUDA path, and none with the scalar-gate oracle next to it either (whose arithmetic it leaves
 * untouched): the two are compared with each other by the tests.
 *
 * What it computes (paper Eq. 1 as printed: three gate vectors per (token, head); Table 2 lists the
 * named models as gate settings).  Per (sequence, head) chain, state h of shape d_k x d_v, log-decay
 * g_t in R^{d_k}, erase gate b_t in R^{d_k}, write gate w_t in R^{d_v}:
 *
 *     ht_t = Diag(exp(g_t)) h_{t-1}                  channel-wise decay (row r of h scaled by exp(g_t[r]))
 *     p_t  = ht_t^T (b_t . k_t)                      what the state predicts for the gated key
 *     u_t  = w_t . v_t - p_t                         delta-rule correction
 *     h_t  = ht_t + k_t u_t^T                        rank-one write
 *     o_t  = scale * h_t^T q_t                       read-out
 *
 * which is  h_t = (I - k_t (b_t . k_t)^T) Diag(exp(g_t)) h_{t-1} + k_t (w_t . v_t)^T  ("." = elementwise).
 * KDA is b_t = beta_t 1, w_t = beta_t 1 with a per-channel g; GLA is b = 0, w = 1.
 *
 * Gradient: for L = sum_t <dO_t, o_t> + <dh_T, h_T> the reverse-time adjoint of the five lines above,
 * walked from t = T down to 1 (Appendix A gives its shape: dS_t = Diag(e^{g_t}) dS_{t+1} + rank-one
 * correction).  dg, db are d_k-vectors per token, dw a d_v-vector; dg is w.r.t. the log-decay.
 *
 * Parity pins (tests, no GPU needed): central finite differences of every gradient, the T = 1 closed
 * form in matrix notation, b = w = beta against a plain matrix statement of the KDA row of Table 2 to
 * 1e-12, gates with equal entries against the scalar-gate oracle (outputs equal, gate gradients equal
 * to its channel sums), b = 0, w = 1 against gated linear attention with per-channel decay written as a
 * masked contraction, and equality with an independent chunked fp64 formulation.
 *
 * Memory layout (all host pointers, all double, row-major):
 *     q, k [Ttot, H, d_k]   v, o, dO [Ttot, H, d_v]   g, b, dg, db [Ttot, H, d_k]   w, dw [Ttot, H, d_v]
 *     h0, hT, dhT, dh0 [N, H, d_k, d_v]               cu_seqlens int32 [N + 1]
 * Return value: 0 on success, negative on argument error.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define VEC_SEG 64 /* forward states are kept every VEC_SEG tokens and re-materialised in between */

typedef struct {
    int N, H, dk, dv;
    const int32_t* cu;
    double scale;
    const double *q, *k, *v, *g, *b, *w, *h0, *dO, *dhT;
    double *o, *hT, *dq, *dkk, *dvv, *dg, *db, *dw, *dh0;
    int want_bwd;
    int next_chain;
    pthread_mutex_t mu;
    int failed;
} vjob_t;

/* One forward step in place.  Returns u_t in `u` and, when ht_out != NULL, the decayed state. */
static void vec_step(int dk, int dv, double* h, const double* kt, const double* vt, const double* gt,
                     const double* bt, const double* wt, double* u, double* ht_out) {
    for (int r = 0; r < dk; ++r) {
        const double a = exp(gt[r]);
        for (int c = 0; c < dv; ++c) h[r * dv + c] *= a;
    }
    if (ht_out) memcpy(ht_out, h, sizeof(double) * (size_t)dk * dv);
    for (int c = 0; c < dv; ++c) {
        double p = 0.0;
        for (int r = 0; r < dk; ++r) p += h[r * dv + c] * (bt[r] * kt[r]);
        u[c] = wt[c] * vt[c] - p;
    }
    for (int r = 0; r < dk; ++r)
        for (int c = 0; c < dv; ++c) h[r * dv + c] += kt[r] * u[c];
}

static int vec_chain(vjob_t* J, int n, int hd) {
    const int H = J->H, dk = J->dk, dv = J->dv;
    const int t0 = J->cu[n], t1 = J->cu[n + 1], len = t1 - t0;
    const size_t S = (size_t)dk * dv;
    const size_t soff = ((size_t)n * H + hd) * S;
    const int nseg = (len + VEC_SEG - 1) / VEC_SEG;

    double* h = (double*)malloc(sizeof(double) * S);
    double* u = (double*)malloc(sizeof(double) * dv);
    double* seg0 = J->want_bwd ? (double*)malloc(sizeof(double) * S * (size_t)(nseg > 0 ? nseg : 1)) : NULL;
    if (!h || !u || (J->want_bwd && !seg0)) { free(h); free(u); free(seg0); return -1; }
    if (J->h0) memcpy(h, J->h0 + soff, sizeof(double) * S); else memset(h, 0, sizeof(double) * S);

    /* ---- forward sweep ---- */
    for (int t = 0; t < len; ++t) {
        if (J->want_bwd && t % VEC_SEG == 0) memcpy(seg0 + (size_t)(t / VEC_SEG) * S, h, sizeof(double) * S);
        const size_t x = (size_t)(t0 + t) * H + hd;
        vec_step(dk, dv, h, J->k + x * dk, J->v + x * dv, J->g + x * dk, J->b + x * dk, J->w + x * dv, u, NULL);
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
    double* hs = (double*)malloc(sizeof(double) * S * VEC_SEG);  /* h_t of one segment */
    double* hts = (double*)malloc(sizeof(double) * S * VEC_SEG); /* ht_t (decayed, before the write) */
    double* us = (double*)malloc(sizeof(double) * (size_t)dv * VEC_SEG);
    double* du = (double*)malloc(sizeof(double) * dv);
    if (!dh || !hs || !hts || !us || !du) { free(h); free(u); free(seg0); free(dh); free(hs); free(hts); free(us); free(du); return -1; }
    if (J->dhT) memcpy(dh, J->dhT + soff, sizeof(double) * S); else memset(dh, 0, sizeof(double) * S);

    for (int sgm = nseg - 1; sgm >= 0; --sgm) {
        const int a0 = sgm * VEC_SEG;
        const int a1 = (a0 + VEC_SEG < len) ? a0 + VEC_SEG : len;
        memcpy(h, seg0 + (size_t)sgm * S, sizeof(double) * S);
        for (int t = a0; t < a1; ++t) {
            const size_t x = (size_t)(t0 + t) * H + hd;
            const int j = t - a0;
            vec_step(dk, dv, h, J->k + x * dk, J->v + x * dv, J->g + x * dk, J->b + x * dk, J->w + x * dv,
                     us + (size_t)j * dv, hts + (size_t)j * S);
            memcpy(hs + (size_t)j * S, h, sizeof(double) * S);
        }
        for (int t = a1 - 1; t >= a0; --t) {
            const size_t x = (size_t)(t0 + t) * H + hd;
            const int j = t - a0;
            const double *qt = J->q + x * dk, *kt = J->k + x * dk, *vt = J->v + x * dv, *dOt = J->dO + x * dv;
            const double *gt = J->g + x * dk, *bt = J->b + x * dk, *wt = J->w + x * dv;
            const double *ht_ = hts + (size_t)j * S, *h_ = hs + (size_t)j * S, *ut = us + (size_t)j * dv;
            const double sc = J->scale;
            double *dq = J->dq + x * dk, *dkt = J->dkk + x * dk, *dvt = J->dvv + x * dv;
            double *dgt = J->dg + x * dk, *dbt = J->db + x * dk, *dwt = J->dw + x * dv;

            /* o_t = scale h_t^T q_t */
            for (int r = 0; r < dk; ++r) {
                double s = 0.0;
                for (int c = 0; c < dv; ++c) { s += h_[r * dv + c] * dOt[c]; dh[r * dv + c] += sc * qt[r] * dOt[c]; }
                dq[r] = sc * s;
            }
            /* h_t = ht_t + k_t u_t^T  =>  du = dh^T k_t */
            for (int c = 0; c < dv; ++c) {
                double s = 0.0;
                for (int r = 0; r < dk; ++r) s += dh[r * dv + c] * kt[r];
                du[c] = s;
            }
            /* u_t = w_t . v_t - p_t */
            for (int c = 0; c < dv; ++c) {
                dvt[c] = wt[c] * du[c];
                dwt[c] = vt[c] * du[c];
            }
            /* p_t = ht_t^T (b_t . k_t), dp = -du:  gradient w.r.t. the gated key is -(ht_t du) */
            for (int r = 0; r < dk; ++r) {
                double s1 = 0.0, s2 = 0.0, dgr = 0.0;
                const double a = exp(gt[r]);
                for (int c = 0; c < dv; ++c) {
                    s1 += dh[r * dv + c] * ut[c];                 /* from the write k u^T      */
                    s2 += ht_[r * dv + c] * du[c];                /* (ht du)[r]                */
                    const double dht = dh[r * dv + c] - bt[r] * kt[r] * du[c]; /* grad w.r.t. ht_t */
                    dgr += dht * ht_[r * dv + c];                 /* d ht[r,:] / d g[r] = ht[r,:] */
                    dh[r * dv + c] = a * dht;                     /* grad w.r.t. h_{t-1}       */
                }
                dkt[r] = s1 - bt[r] * s2;
                dbt[r] = -kt[r] * s2;
                dgt[r] = dgr;
            }
        }
    }
    if (J->dh0) memcpy(J->dh0 + soff, dh, sizeof(double) * S);
    free(h); free(u); free(seg0); free(dh); free(hs); free(hts); free(us); free(du);
    return 0;
}

static void* vec_worker(void* arg) {
    vjob_t* J = (vjob_t*)arg;
    const int total = J->N * J->H;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        const int c = J->next_chain++;
        pthread_mutex_unlock(&J->mu);
        if (c >= total) break;
        if (vec_chain(J, c / J->H, c % J->H) != 0) {
            pthread_mutex_lock(&J->mu);
            J->failed = 1;
            pthread_mutex_unlock(&J->mu);
        }
    }
    return NULL;
}

static int vec_run(vjob_t* J, int n_threads) {
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
    for (int i = 1; i < n_threads; ++i)
        if (pthread_create(&th[started], NULL, vec_worker, J) == 0) ++started;
    vec_worker(J);
    for (int i = 0; i < started; ++i) pthread_join(th[i], NULL);
    pthread_mutex_destroy(&J->mu);
    return J->failed ? -3 : 0;
}

int gdn_oracle_vec_fwd(int N, const int32_t* cu_seqlens, int H, int dk, int dv, double scale,
                       const double* q, const double* k, const double* v, const double* g, const double* b,
                       const double* w, const double* h0, double* o, double* hT, int n_threads) {
    if (!q || !k || !v || !g || !b || !w) return -1;
    vjob_t J;
    memset(&J, 0, sizeof(J));
    J.N = N; J.H = H; J.dk = dk; J.dv = dv; J.cu = cu_seqlens; J.scale = scale;
    J.q = q; J.k = k; J.v = v; J.g = g; J.b = b; J.w = w; J.h0 = h0; J.o = o; J.hT = hT;
    J.want_bwd = 0;
    return vec_run(&J, n_threads);
}

int gdn_oracle_vec_bwd(int N, const int32_t* cu_seqlens, int H, int dk, int dv, double scale,
                       const double* q, const double* k, const double* v, const double* g, const double* b,
                       const double* w, const double* h0, const double* dO, const double* dhT,
                       double* o, double* hT, double* dq, double* dk_out, double* dv_out, double* dg, double* db,
                       double* dw, double* dh0, int n_threads) {
    if (!q || !k || !v || !g || !b || !w || !dO || !dq || !dk_out || !dv_out || !dg || !db || !dw) return -1;
    vjob_t J;
    memset(&J, 0, sizeof(J));
    J.N = N; J.H = H; J.dk = dk; J.dv = dv; J.cu = cu_seqlens; J.scale = scale;
    J.q = q; J.k = k; J.v = v; J.g = g; J.b = b; J.w = w; J.h0 = h0; J.dO = dO; J.dhT = dhT;
    J.o = o; J.hT = hT; J.dq = dq; J.dkk = dk_out; J.dvv = dv_out; J.dg = dg; J.db = db; J.dw = dw; J.dh0 = dh0;
    J.want_bwd = 1;
    return vec_run(&J, n_threads);
}
