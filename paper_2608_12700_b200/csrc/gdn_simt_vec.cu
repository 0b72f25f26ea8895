// fp32 FFMA kernels for the general recurrence with PER-CHANNEL gates (Eq. 1 of the paper as printed: log-decay
// g_t and erase gate b_t in R^{d_k}, write gate w_t in R^{d_v}; Table 2: KDA, GLA and the full GDN are gate settings).
//
// The channel-wise decay does not factor out of the chunk-local contractions as a token-token matrix; it folds inside
// them (Appendix A, last paragraph): every token-token quantity is a sum over the channel r that carries the factor
// exp(gam_i[r] - gam_j[r]), evaluated for j <= i only, so that no exponent is ever positive.  This family is the
// plain CUDA-core statement of that formulation (arithmetic in fp32 whatever the I/O dtype), stage by stage:
//   table  : chunk table from cu_seqlens (shared with the scalar-gate family)
//   vprep  : gam = cumsum(g) per channel;  A_ij = sum_r b_i k_i k_j e^{gam_i - gam_j} (j < i);  T = (I + A)^-1;
//            P_ij = sum_r q_i k_j e^{gam_i - gam_j} (j <= i);  W = T (Gam . b . K);  Ut = T (w . V)
//   vscan  : forward   h'  = Diag(Gam_e) h   + Kb^T (Ut - W h),   Kb_j = e^{gam_e - gam_j} . k_j   (stores h per chunk)
//            reverse   dh  = Diag(Gam_e) dh' + E - W^T (Kb dh')                                     (stores dh'; K#1)
//   veprep : E = scale (Gam . Q - P W)^T dO
//   vintra : every token gradient, including the VJP of the triangular solve from the stored T (K#2), the gate
//            gradients per channel, and dg by a reverse cumulative sum inside the chunk
// One CTA handles one (chunk, head) in the parallel stages and one (sequence, head) chain in the scans.  Every
// reduction has a fixed order: results are bit-identical from run to run.
// With bf16 I/O at d_k = d_v = 128 the whole path runs on the tensor cores instead (gdn_tc_cw.cu and tc_scan_cw in
// gdn_tc.cu); only the optional forward output is formed here, from the bf16 tile images those kernels leave.
#include "simt_common.cuh"
#include "tc_ptx.cuh"

namespace gdn {
namespace {

// acc[a][b] += sum_m fa(i0 + a, m) fb(j0 + b, m) exp(gam[i][m] - gam[j][m])  for j <= i - strict (else 0 is added)
template <int DK, class FA, class FB>
__device__ __forceinline__ void mac_decay(float (&acc)[4][4], int i0, int j0, int strict, const float* gam, FA fa, FB fb) {
    if (j0 > i0 + 3 - strict) return;
#pragma unroll 2
    for (int m = 0; m < DK; ++m) {
        float a[4], b[4], gi[4], gj[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            a[x] = fa(i0 + x, m); b[x] = fb(j0 + x, m);
            gi[x] = gam[(i0 + x) * (DK + 1) + m]; gj[x] = gam[(j0 + x) * (DK + 1) + m];
        }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y)
                if (j0 + y <= i0 + x - strict) acc[x][y] = fmaf(a[x] * b[y], expf(gi[x] - gj[y]), acc[x][y]);
    }
}

// Whether this launch has work: normally when no earlier stage has reported an error; a launch of the fall-back sequence
// only when the tensor-core route has refused the gates of this call (decided on the device, no host round trip).
__device__ __forceinline__ bool vec_go(const Problem& p) {
    const int st = reinterpret_cast<const WsHeader*>(p.ws)->status;
    return p.fallback ? st == GDN_ERR_DECAY_RANGE : st == GDN_OK;
}
__global__ void vec_clear_refusal_kernel(Problem p) {
    WsHeader* hdr = reinterpret_cast<WsHeader*>(p.ws);
    const bool refused = hdr->status == GDN_ERR_DECAY_RANGE;
    hdr->cw_fallback = refused ? 1 : 0;   // a backward on this workspace "fresh from the forward" must know whose data it holds
    if (refused) { hdr->status = GDN_OK; hdr->detail = 0; }
}

// Chunk-local cumulative log decay per channel into shared memory (pitch DK + 1); rows beyond the sequence repeat the
// last valid row (identity padding: g = 0 there).
template <int DK>
__device__ __forceinline__ void cumulate_gates(const Problem& p, const ChunkCtx& x, float* gam) {
    for (int r = threadIdx.x; r < DK; r += blockDim.x) {
        float s = 0.f;
        for (int i = 0; i < kC; ++i) {
            if (i < x.len) s += p.gv[((size_t)(x.tok0 + i) * p.d.H + x.hd) * DK + r];
            gam[i * (DK + 1) + r] = s;
        }
    }
}
template <int DK>
__device__ __forceinline__ void load_gamma(const float* wsG, float* gam) {
    for (int t = threadIdx.x; t < kC * DK; t += blockDim.x) gam[(t / DK) * (DK + 1) + t % DK] = wsG[t];
}

// ------------------------------------------------------------------------------------------------
// vprep
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) vprep_kernel(Problem p) {
    ChunkCtx x;
    if (!vec_go(p) || !chunk_ctx(p, x)) return;
    extern __shared__ __align__(16) float smf[];
    float* gam = smf;                                   // [64][DK + 1]
    float (*A)[kC + 1] = reinterpret_cast<float (*)[kC + 1]>(smf + kC * (DK + 1));
    float (*Ti)[kC + 1] = A + kC;
    const int H = p.d.H;
    const size_t base_k = ((size_t)x.tok0 * H + x.hd) * DK, base_v = ((size_t)x.tok0 * H + x.hd) * DV;
    const size_t rk = (size_t)H * DK, rv = (size_t)H * DV;
    const IO* qp = reinterpret_cast<const IO*>(p.q) + base_k;
    const IO* kp = reinterpret_cast<const IO*>(p.k) + base_k;
    const IO* vp = reinterpret_cast<const IO*>(p.v) + base_v;
    auto Qf = [&](int i, int m) -> float { return i < x.len ? ldf(qp + i * rk + m) : 0.f; };
    auto Kf = [&](int i, int m) -> float { return i < x.len ? ldf(kp + i * rk + m) : 0.f; };
    auto Vf = [&](int i, int m) -> float { return i < x.len ? ldf(vp + i * rv + m) : 0.f; };
    auto Bf = [&](int i, int m) -> float { return i < x.len ? p.bv[base_k + i * rk + m] : 0.f; };
    auto Wf = [&](int i, int m) -> float { return i < x.len ? p.wv[base_v + i * rv + m] : 0.f; };
    float* wsG = reinterpret_cast<float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC * DK;
    float* wsT = reinterpret_cast<float*>(p.ws + p.L.Tm) + (size_t)x.ch * kC * kC;
    float* wsP = reinterpret_cast<float*>(p.ws + p.L.Pm) + (size_t)x.ch * kC * kC;
    float* wsW = reinterpret_cast<float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    float* wsU = reinterpret_cast<float*>(p.ws + p.L.Ut) + (size_t)x.ch * kC * DV;

    cumulate_gates<DK>(p, x, gam);
    __syncthreads();
    for (int t = threadIdx.x; t < kC * DK; t += blockDim.x) wsG[t] = gam[(t / DK) * (DK + 1) + t % DK];
    // A (strictly lower) and P (lower, diagonal included): the decay sits inside the contraction over the channel
    tiles(kC, kC, [&](int i0, int j0) {
        float aa[4][4] = {}, pp[4][4] = {};
        mac_decay<DK>(aa, i0, j0, 1, gam, [&](int i, int m) { return Bf(i, m) * Kf(i, m); }, Kf);
        mac_decay<DK>(pp, i0, j0, 0, gam, Qf, Kf);
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                A[i0 + a][j0 + b] = aa[a][b];
                wsP[(i0 + a) * kC + j0 + b] = pp[a][b];
            }
    });
    __syncthreads();
    // T = (I + A)^-1: column j of T solves (I + A) x = e_j by forward substitution (one thread per column).
    if (threadIdx.x < kC) {
        const int j = threadIdx.x;
        for (int i = 0; i < kC; ++i) {
            float s = (i == j) ? 1.f : 0.f;
            for (int m = j; m < i; ++m) s = fmaf(-A[i][m], Ti[m][j], s);
            Ti[i][j] = (i >= j) ? s : 0.f;
        }
    }
    __syncthreads();
    for (int t = threadIdx.x; t < kC * kC; t += blockDim.x) wsT[t] = Ti[t / kC][t % kC];
    // W = T (Gam . b . K),  Ut = T (w . V)
    tiles(kC, DK, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return Ti[i][m]; },
            [&](int m, int j) { return expf(gam[m * (DK + 1) + j]) * Bf(m, j) * Kf(m, j); });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) wsW[(i0 + a) * DK + j0 + b] = acc[a][b];
    });
    tiles(kC, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return Ti[i][m]; }, [&](int m, int j) { return Wf(m, j) * Vf(m, j); });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) wsU[(i0 + a) * DV + j0 + b] = acc[a][b];
    });
}

// ------------------------------------------------------------------------------------------------
// veprep: E = scale (Gam . Q - P W)^T dO
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) veprep_kernel(Problem p) {
    ChunkCtx x;
    if (!vec_go(p) || !chunk_ctx(p, x)) return;
    const int H = p.d.H;
    const IO* qp = reinterpret_cast<const IO*>(p.q) + ((size_t)x.tok0 * H + x.hd) * DK;
    const IO* gp = reinterpret_cast<const IO*>(p.dO) + ((size_t)x.tok0 * H + x.hd) * DV;
    const size_t rk = (size_t)H * DK, rv = (size_t)H * DV;
    auto Qf = [&](int i, int m) -> float { return i < x.len ? ldf(qp + i * rk + m) : 0.f; };
    auto Of = [&](int i, int m) -> float { return i < x.len ? ldf(gp + i * rv + m) : 0.f; };
    const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC * DK;
    const float* wsP = reinterpret_cast<const float*>(p.ws + p.L.Pm) + (size_t)x.ch * kC * kC;
    const float* wsW = reinterpret_cast<const float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    float* wsE = reinterpret_cast<float*>(p.ws + p.L.E) + (size_t)x.ch * DK * DV;
    float* X = reinterpret_cast<float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * x.ch);  // [64, DK]
    tiles(kC, DK, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return wsP[i * kC + m]; }, [&](int m, int j) { return wsW[m * DK + j]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b)
                X[(i0 + a) * DK + j0 + b] = expf(wsG[(i0 + a) * DK + j0 + b]) * Qf(i0 + a, j0 + b) - acc[a][b];
    });
    __syncthreads();
    const float sc = p.d.scale;
    tiles(DK, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return X[m * DK + i]; }, Of);
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) wsE[(i0 + a) * DV + j0 + b] = sc * acc[a][b];
    });
}

// ------------------------------------------------------------------------------------------------
// Forward and reverse carries in low-rank form.  One CTA per (sequence, head); the fp32 state lives in shared memory.
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV, bool REVERSE>
__global__ void __launch_bounds__(kThreads) vscan_kernel(Problem p) {
    extern __shared__ __align__(16) float sm[];
    float* cur = sm;                  // [DK][DV]
    float* nxt = sm + DK * DV;
    float* Y = nxt + DK * DV;         // [64][DV]: U = Ut - W h (forward) or Kb dh' (reverse)
    const int H = p.d.H, n = blockIdx.x / H, hd = blockIdx.x % H;
    const int32_t* seq_first = reinterpret_cast<const int32_t*>(p.ws + p.L.seq_first);
    if (!vec_go(p)) return;
    const int c0 = seq_first[n], c1 = seq_first[n + 1];
    const size_t soff = ((size_t)n * H + hd) * DK * DV;
    const float* init = REVERSE ? p.dhT : p.h0;
    for (int t = threadIdx.x; t < DK * DV; t += blockDim.x) cur[t] = init ? init[soff + t] : 0.f;
    __syncthreads();
    const size_t rk = (size_t)H * DK;
    for (int s = 0; s < c1 - c0; ++s) {
        const int c = REVERSE ? (c1 - 1 - s) : (c0 + s);
        const size_t ch = (size_t)c * H + hd;
        const int tok0 = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0)[c];
        const int len = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len)[c];
        const IO* kp = reinterpret_cast<const IO*>(p.k) + ((size_t)tok0 * H + hd) * DK;
        const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + ch * kC * DK;
        const float* wsW = reinterpret_cast<const float*>(p.ws + p.L.W) + ch * kC * DK;
        const float* wsU = reinterpret_cast<const float*>(p.ws + p.L.Ut) + ch * kC * DV;
        const float* wsE = reinterpret_cast<const float*>(p.ws + p.L.E) + ch * DK * DV;
        float* keep = reinterpret_cast<float*>(p.ws + (REVERSE ? p.L.dhn : p.L.hc)) + ch * DK * DV;
        // Kb_j[r] = exp(gam_e[r] - gam_j[r]) k_j[r]
        auto Kb = [&](int j, int r) -> float {
            return j < len ? expf(wsG[(kC - 1) * DK + r] - wsG[j * DK + r]) * ldf(kp + j * rk + r) : 0.f;
        };
        for (int t = threadIdx.x; t < DK * DV; t += blockDim.x) keep[t] = cur[t];
        tiles(kC, DV, [&](int i0, int j0) {
            float acc[4][4] = {};
            if (REVERSE) mac(acc, i0, j0, DK, Kb, [&](int m, int j) { return cur[m * DV + j]; });
            else mac(acc, i0, j0, DK, [&](int i, int m) { return wsW[i * DK + m]; }, [&](int m, int j) { return cur[m * DV + j]; });
            for (int a = 0; a < 4; ++a)
                for (int b = 0; b < 4; ++b) {
                    const int t = (i0 + a) * DV + j0 + b;
                    Y[t] = REVERSE ? acc[a][b] : wsU[t] - acc[a][b];
                }
        });
        __syncthreads();
        tiles(DK, DV, [&](int i0, int j0) {
            float acc[4][4] = {};
            if (REVERSE) mac(acc, i0, j0, kC, [&](int i, int m) { return wsW[m * DK + i]; }, [&](int m, int j) { return Y[m * DV + j]; });
            else mac(acc, i0, j0, kC, [&](int i, int m) { return Kb(m, i); }, [&](int m, int j) { return Y[m * DV + j]; });
            for (int a = 0; a < 4; ++a)
                for (int b = 0; b < 4; ++b) {
                    const int t = (i0 + a) * DV + j0 + b;
                    const float Ge = expf(wsG[(kC - 1) * DK + i0 + a]);
                    nxt[t] = REVERSE ? Ge * cur[t] + wsE[t] - acc[a][b] : Ge * cur[t] + acc[a][b];
                }
        });
        __syncthreads();
        float* tmp = cur; cur = nxt; nxt = tmp;
    }
    float* fin = REVERSE ? p.dh0 : p.hT;
    if (fin) for (int t = threadIdx.x; t < DK * DV; t += blockDim.x) fin[soff + t] = cur[t];
}

// ------------------------------------------------------------------------------------------------
// Forward output (optional): o = scale ((Gam . Q) h + P (Ut - W h))
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) vout_kernel(Problem p) {
    ChunkCtx x;
    if (!vec_go(p) || !chunk_ctx(p, x)) return;
    const int H = p.d.H;
    const IO* qp = reinterpret_cast<const IO*>(p.q) + ((size_t)x.tok0 * H + x.hd) * DK;
    IO* op = reinterpret_cast<IO*>(p.o) + ((size_t)x.tok0 * H + x.hd) * DV;
    const size_t rk = (size_t)H * DK, rv = (size_t)H * DV;
    auto Qf = [&](int i, int m) -> float { return i < x.len ? ldf(qp + i * rk + m) : 0.f; };
    const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC * DK;
    const float* wsP = reinterpret_cast<const float*>(p.ws + p.L.Pm) + (size_t)x.ch * kC * kC;
    const float* wsW = reinterpret_cast<const float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    const float* wsU = reinterpret_cast<const float*>(p.ws + p.L.Ut) + (size_t)x.ch * kC * DV;
    const float* wsH = reinterpret_cast<const float*>(p.ws + p.L.hc) + (size_t)x.ch * DK * DV;
    auto Pf = [&](int i, int m) -> float { return wsP[i * kC + m]; };
    auto Wm = [&](int i, int m) -> float { return wsW[i * DK + m]; };
    auto Um = [&](int i, int j) -> float { return wsU[i * DV + j]; };
    auto Hf = [&](int m, int j) -> float { return wsH[m * DV + j]; };
    float* U = reinterpret_cast<float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * x.ch);  // [64, DV]
    tiles(kC, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, DK, Wm, Hf);
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) U[(i0 + a) * DV + j0 + b] = Um(i0 + a, j0 + b) - acc[a][b];
    });
    __syncthreads();
    const float sc = p.d.scale;
    tiles(kC, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, DK, [&](int i, int m) { return expf(wsG[i * DK + m]) * Qf(i, m); }, Hf);
        mac(acc, i0, j0, kC, Pf, [&](int m, int j) { return U[m * DV + j]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b)
                if (i0 + a < x.len) stf(op + (i0 + a) * rv + j0 + b, sc * acc[a][b]);
    });
}

// ------------------------------------------------------------------------------------------------
// vintra: token gradients of one (chunk, head).
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) vintra_kernel(Problem p) {
    ChunkCtx x;
    if (!vec_go(p) || !chunk_ctx(p, x)) return;
    extern __shared__ __align__(16) float smf[];
    float* gam = smf;                                                                       // [64][DK + 1]
    float (*dP)[kC + 1] = reinterpret_cast<float (*)[kC + 1]>(smf + kC * (DK + 1));         // scale tril(dO U^T)
    float (*dA)[kC + 1] = dP + kC;                                                          // -stril(dXk W^T + dXv Ut^T)
    const int H = p.d.H;
    const size_t base_k = ((size_t)x.tok0 * H + x.hd) * DK, base_v = ((size_t)x.tok0 * H + x.hd) * DV;
    const size_t rk = (size_t)H * DK, rv = (size_t)H * DV;
    const IO* qp = reinterpret_cast<const IO*>(p.q) + base_k;
    const IO* kp = reinterpret_cast<const IO*>(p.k) + base_k;
    const IO* vp = reinterpret_cast<const IO*>(p.v) + base_v;
    const IO* gp = reinterpret_cast<const IO*>(p.dO) + base_v;
    IO* dqp = reinterpret_cast<IO*>(p.dq) + base_k;
    IO* dkp = reinterpret_cast<IO*>(p.dk) + base_k;
    IO* dvp = reinterpret_cast<IO*>(p.dv) + base_v;
    auto Qf = [&](int i, int m) -> float { return i < x.len ? ldf(qp + i * rk + m) : 0.f; };
    auto Kf = [&](int i, int m) -> float { return i < x.len ? ldf(kp + i * rk + m) : 0.f; };
    auto Vf = [&](int i, int m) -> float { return i < x.len ? ldf(vp + i * rv + m) : 0.f; };
    auto Of = [&](int i, int m) -> float { return i < x.len ? ldf(gp + i * rv + m) : 0.f; };
    auto Bf = [&](int i, int m) -> float { return i < x.len ? p.bv[base_k + i * rk + m] : 0.f; };
    auto Wf = [&](int i, int m) -> float { return i < x.len ? p.wv[base_v + i * rv + m] : 0.f; };
    const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC * DK;
    const float* Tm = reinterpret_cast<const float*>(p.ws + p.L.Tm) + (size_t)x.ch * kC * kC;
    const float* Pm = reinterpret_cast<const float*>(p.ws + p.L.Pm) + (size_t)x.ch * kC * kC;
    const float* W = reinterpret_cast<const float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    const float* Ut = reinterpret_cast<const float*>(p.ws + p.L.Ut) + (size_t)x.ch * kC * DV;
    const float* hs = reinterpret_cast<const float*>(p.ws + p.L.hc) + (size_t)x.ch * DK * DV;     // per-chunk states, fp32
    const float* dhs = reinterpret_cast<const float*>(p.ws + p.L.dhn) + (size_t)x.ch * DK * DV;
    auto Hs = [&](int m, int j) -> float { return hs[m * DV + j]; };     // h[m][j]
    auto DHs = [&](int m, int j) -> float { return dhs[m * DV + j]; };   // dh'[m][j]
    float* scr = reinterpret_cast<float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * x.ch);
    float* U = scr;                    // [64, DV]
    float* dU = U + kC * DV;           // [64, DV]
    float* dXv = dU + kC * DV;         // [64, DV]
    float* dOh = dXv + kC * DV;        // [64, DK]  dO h^T
    float* dW = dOh + kC * DK;         // [64, DK]  later dgam
    float* dXk = dW + kC * DK;         // [64, DK]
    float* UdH = dXk + kC * DK;        // [64, DK]  U dh'^T
    const float sc = p.d.scale;
    auto G = [&](int i, int r) -> float { return gam[i * (DK + 1) + r]; };

    load_gamma<DK>(wsG, gam);
    // (1) U = Ut - W h ;  dU = scale P^T dO + Kb dh'
    tiles(kC, DV, [&](int i0, int j0) {
        float a0[4][4] = {}, a1[4][4] = {}, a2[4][4] = {};
        mac(a0, i0, j0, DK, [&](int i, int m) { return W[i * DK + m]; }, Hs);
        mac(a1, i0, j0, DK, [&](int i, int m) { return expf(wsG[(kC - 1) * DK + m] - wsG[i * DK + m]) * Kf(i, m); },
            DHs);
        mac(a2, i0, j0, kC, [&](int i, int m) { return Pm[m * kC + i]; }, Of);
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int t = (i0 + a) * DV + j0 + b;
                U[t] = Ut[t] - a0[a][b];
                dU[t] = sc * a2[a][b] + a1[a][b];
            }
    });
    __syncthreads();
    // (2) dP = scale tril(dO U^T) ;  dO h^T ;  dW = -dU h^T ;  U dh'^T
    tiles(kC, kC, [&](int i0, int j0) {
        float acc[4][4] = {};
        if (j0 <= i0 + 3) mac(acc, i0, j0, DV, Of, [&](int m, int j) { return U[j * DV + m]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) dP[i0 + a][j0 + b] = (j0 + b <= i0 + a) ? sc * acc[a][b] : 0.f;
    });
    tiles(kC, DK, [&](int i0, int j0) {
        float a1[4][4] = {}, a2[4][4] = {}, a3[4][4] = {};
        mac(a1, i0, j0, DV, Of, [&](int m, int j) { return Hs(j, m); });
        mac(a2, i0, j0, DV, [&](int i, int m) { return dU[i * DV + m]; }, [&](int m, int j) { return Hs(j, m); });
        mac(a3, i0, j0, DV, [&](int i, int m) { return U[i * DV + m]; }, [&](int m, int j) { return DHs(j, m); });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int t = (i0 + a) * DK + j0 + b;
                dOh[t] = a1[a][b];
                dW[t] = -a2[a][b];
                UdH[t] = a3[a][b];
            }
    });
    __syncthreads();
    // (3) dXk = T^T dW ;  dXv = T^T dU ;  dv = w . dXv ;  dw = v . dXv
    tiles(kC, DK, [&](int i0, int j0) {
        float ax[4][4] = {};
        mac(ax, i0, j0, kC, [&](int i, int m) { return Tm[m * kC + i]; }, [&](int m, int j) { return dW[m * DK + j]; });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) dXk[(i0 + a) * DK + j0 + b] = ax[a][b];
    });
    tiles(kC, DV, [&](int i0, int j0) {
        float ax[4][4] = {};
        mac(ax, i0, j0, kC, [&](int i, int m) { return Tm[m * kC + i]; }, [&](int m, int j) { return dU[m * DV + j]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                dXv[i * DV + j] = ax[a][b];
                if (i < x.len) {
                    stf(dvp + i * rv + j, Wf(i, j) * ax[a][b]);
                    p.dwv[base_v + i * rv + j] = Vf(i, j) * ax[a][b];
                }
            }
    });
    __syncthreads();
    // (4) dA = -stril(dXk W^T + dXv Ut^T)
    tiles(kC, kC, [&](int i0, int j0) {
        float acc[4][4] = {};
        if (j0 < i0 + 3) {
            mac(acc, i0, j0, DK, [&](int i, int m) { return dXk[i * DK + m]; }, [&](int m, int j) { return W[j * DK + m]; });
            mac(acc, i0, j0, DV, [&](int i, int m) { return dXv[i * DV + m]; }, [&](int m, int j) { return Ut[j * DV + m]; });
        }
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) dA[i0 + a][j0 + b] = (j0 + b < i0 + a) ? -acc[a][b] : 0.f;
    });
    __syncthreads();
    // (5) per (token i, channel r): the sums over the other token carry the decay of that channel
    float* dgam = dW;   // dW is dead
    for (int t = threadIdx.x; t < kC * DK; t += blockDim.x) {
        const int i = t / DK, r = t % DK;
        const float gi = G(i, r);
        float sq = 0.f, srow = 0.f, scol = 0.f;
        for (int j = 0; j <= i; ++j) {           // row role: e^{gam_i - gam_j}, j <= i
            const float e = expf(gi - G(j, r)), kj = Kf(j, r);
            sq = fmaf(dP[i][j] * e, kj, sq);
            srow = fmaf(dA[i][j] * e, kj, srow);                       // (dA_ii = 0)
        }
        for (int j = i; j < kC; ++j) {           // column role: e^{gam_j - gam_i}, j >= i
            const float e = expf(G(j, r) - gi);
            scol = fmaf(dP[j][i] * e, Qf(j, r), scol);
            scol = fmaf(dA[j][i] * e, Bf(j, r) * Kf(j, r), scol);      // (dA_ii = 0)
        }
        const float Gi = expf(gi), ei = expf(G(kC - 1, r) - gi);
        const float ki = Kf(i, r), qi = Qf(i, r), bi = Bf(i, r);
        const float dq = sc * Gi * dOh[t] + sq;
        const float row = srow + Gi * dXk[t];
        const float col = scol + ei * UdH[t];
        if (i < x.len) {
            stf(dqp + i * rk + r, dq);
            stf(dkp + i * rk + r, bi * row + col);
            p.dbv[base_k + i * rk + r] = ki * row;
        }
        dgam[t] = qi * dq + ki * bi * row - ki * col;
    }
    __syncthreads();
    // the last row collects what enters through Gam_e: sum_j k_j . e_j . (U dh'^T)_j and Gam_e . rowdot(dh', h);
    // then dg_j = sum_{i >= j} dgam_i, channel by channel
    for (int r = threadIdx.x; r < DK; r += blockDim.x) {
        float extra = 0.f, hh = 0.f;
        const float ge = G(kC - 1, r);
        for (int j = 0; j < kC; ++j) extra = fmaf(Kf(j, r) * expf(ge - G(j, r)), UdH[j * DK + r], extra);
        for (int c = 0; c < DV; ++c) hh = fmaf(DHs(r, c), Hs(r, c), hh);
        float run = extra + expf(ge) * hh;
        for (int i = kC - 1; i >= 0; --i) {
            run += dgam[i * DK + r];
            if (i < x.len) p.dgv[base_k + i * rk + r] = run;
        }
    }
}

// The FFMA sequences.  `q` is the problem as these kernels see it (fp32 factors and states); with q.fallback set the chunk
// table is not rebuilt (the tensor-core route has built it, and rebuilding would reset the status word the launches look at).
template <typename IO, int DK, int DV>
cudaError_t ffma_fwd(const Problem& q, cudaStream_t st) {
    const int CH = q.L.max_chunks * q.d.H, chains = q.d.N * q.d.H;
    if (!q.fallback) launch_table(q, st);
    const size_t smp = sizeof(float) * (kC * (DK + 1) + 2 * kC * (kC + 1));
    cudaError_t e = cudaFuncSetAttribute(vprep_kernel<IO, DK, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smp);
    if (e != cudaSuccess) return e;
    if (CH > 0) { StageScope t(q.fallback ? ST_FALLBACK : ST_PREP, st); vprep_kernel<IO, DK, DV><<<CH, kThreads, smp, st>>>(q); }
    const size_t sm = sizeof(float) * (2 * DK * DV + kC * DV);
    e = cudaFuncSetAttribute(vscan_kernel<IO, DK, DV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    if (chains > 0) { StageScope t(q.fallback ? ST_FALLBACK : ST_FSCAN, st); vscan_kernel<IO, DK, DV, false><<<chains, kThreads, sm, st>>>(q); }
    if (q.o && CH > 0) { StageScope t(q.fallback ? ST_FALLBACK : ST_OUT, st); vout_kernel<IO, DK, DV><<<CH, kThreads, 0, st>>>(q); }
    return cudaGetLastError();
}

template <typename IO, int DK, int DV>
cudaError_t ffma_bwd(const Problem& q, bool skip_recompute, cudaStream_t st) {
    cudaError_t e;
    if (!skip_recompute && (e = ffma_fwd<IO, DK, DV>(q, st)) != cudaSuccess) return e;
    const int CH = q.L.max_chunks * q.d.H, chains = q.d.N * q.d.H;
    if (CH > 0) { StageScope t(q.fallback ? ST_FALLBACK : ST_EPREP, st); veprep_kernel<IO, DK, DV><<<CH, kThreads, 0, st>>>(q); }
    const size_t sm = sizeof(float) * (2 * DK * DV + kC * DV);
    e = cudaFuncSetAttribute(vscan_kernel<IO, DK, DV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    if (chains > 0) { StageScope t(q.fallback ? ST_FALLBACK : ST_RSCAN, st); vscan_kernel<IO, DK, DV, true><<<chains, kThreads, sm, st>>>(q); }
    const size_t smi = sizeof(float) * (kC * (DK + 1) + 2 * kC * (kC + 1));
    e = cudaFuncSetAttribute(vintra_kernel<IO, DK, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smi);
    if (e != cudaSuccess) return e;
    if (CH > 0) { StageScope t(q.fallback ? ST_FALLBACK : ST_INTRA, st); vintra_kernel<IO, DK, DV><<<CH, kThreads, smi, st>>>(q); }
    return cudaGetLastError();
}

// bf16 I/O at d = 128 runs on the tensor cores (gdn_tc_cw.cu).  That route refuses gates whose chunk-cumulative log decay
// leaves its range, through the status word; the FFMA sequence is therefore enqueued behind it in fall-back mode: its
// launches return at once unless the status word says so, in which case they compute the call (with the decay inside the
// contractions there is no range limit) and clear the refusal.  No host round trip, the same launches every call.
template <typename IO, int DK, int DV>
cudaError_t ffma_fallback(const Problem& p, bool bwd, bool skip_recompute, cudaStream_t st) {
    Problem q = p;
    q.fallback = 1;
    q.L.tc_scans = 0;
    cudaError_t e = bwd ? ffma_bwd<IO, DK, DV>(q, skip_recompute, st) : ffma_fwd<IO, DK, DV>(q, st);
    if (e != cudaSuccess) return e;
    { StageScope t(ST_FALLBACK, st); vec_clear_refusal_kernel<<<1, 1, 0, st>>>(q); }
    return cudaGetLastError();
}

template <typename IO, int DK, int DV>
cudaError_t vlaunch_fwd_t(const Problem& p, cudaStream_t st) {
    if (!p.L.tc_scans) return ffma_fwd<IO, DK, DV>(p, st);
    const int CH = p.L.max_chunks * p.d.H;
    cudaError_t e = cw_tc_launch(p, /*bwd=*/false, false, st);
    if (e != cudaSuccess) return e;
    if (p.o && CH > 0 && (e = tc_launch_out_channelwise(p, st)) != cudaSuccess) return e;
    return ffma_fallback<IO, DK, DV>(p, false, false, st);
}

template <typename IO, int DK, int DV>
cudaError_t vlaunch_bwd_t(const Problem& p, bool skip_recompute, cudaStream_t st) {
    if (!p.L.tc_scans) return ffma_bwd<IO, DK, DV>(p, skip_recompute, st);
    const cudaError_t e = cw_tc_launch(p, /*bwd=*/true, skip_recompute, st);
    return e != cudaSuccess ? e : ffma_fallback<IO, DK, DV>(p, true, skip_recompute, st);
}

}  // namespace

size_t vec_scratch_per_chunkhead(const gdn_desc& d) { return sizeof(float) * kC * (4 * (size_t)d.d_k + 3 * (size_t)d.d_v); }

#define GDN_VDISPATCH(FN, ...)                                                                      \
    do {                                                                                            \
        const bool bf = p.d.dtype == GDN_BF16;                                                      \
        if (p.d.d_k == 64 && p.d.d_v == 64)                                                         \
            return bf ? FN<__nv_bfloat16, 64, 64>(__VA_ARGS__) : FN<float, 64, 64>(__VA_ARGS__);    \
        if (p.d.d_k == 128 && p.d.d_v == 128)                                                       \
            return bf ? FN<__nv_bfloat16, 128, 128>(__VA_ARGS__) : FN<float, 128, 128>(__VA_ARGS__); \
        if (p.d.d_k == 128 && p.d.d_v == 64)                                                        \
            return bf ? FN<__nv_bfloat16, 128, 64>(__VA_ARGS__) : FN<float, 128, 64>(__VA_ARGS__);  \
        if (p.d.d_k == 64 && p.d.d_v == 128)                                                        \
            return bf ? FN<__nv_bfloat16, 64, 128>(__VA_ARGS__) : FN<float, 64, 128>(__VA_ARGS__);  \
        return cudaErrorInvalidValue;                                                               \
    } while (0)

cudaError_t vec_launch_fwd(const Problem& p, cudaStream_t st) { GDN_VDISPATCH(vlaunch_fwd_t, p, st); }
cudaError_t vec_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st) { GDN_VDISPATCH(vlaunch_bwd_t, p, skip_recompute, st); }

}  // namespace gdn
