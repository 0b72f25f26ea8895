// fp32 FFMA kernels for the GDN backward: the arithmetic path of the fp32 dtype (tolerance 1e-4 rules
// out tf32/bf16 operands) and a plain-CUDA-core statement of every stage of the chunked method.
//
// Stage map (Section 4.2 of the paper; names follow the library header):
//   table  : chunk table from cu_seqlens
//   prep   : gamma = cumsum(g); A = stril(Diag(b)(K K^T . D)); T = (I + A)^-1 by forward substitution;
//            W = T Diag(b Gam) K; Ut = T Diag(w) V; Nm = Kb^T W; Bf = Kb^T Ut
//   fscan  : h' = Gam_e h - Nm h + Bf           (forward carry; stores the state entering each chunk)
//   eprep  : P = tril(Q K^T . D); E = scale (Diag(Gam) Q - P W)^T dO
//   rscan  : dh = Gam_e dh' - Nm^T dh' + E       (reverse carry, the paper's K#1; stores dh' per chunk)
//   intra  : all token gradients of a chunk, including the VJP of the triangular solve (the paper's K#2)
// One CTA handles one (chunk, head) in the parallel stages and one (sequence, head) chain in the scans.
// Every reduction has a fixed order: results are bit-identical from run to run.
#include "simt_common.cuh"

namespace gdn {
namespace {

// ------------------------------------------------------------------------------------------------
// Chunk table.  One block.  Validates cu_seqlens; on failure records the status and leaves no work.
// ------------------------------------------------------------------------------------------------
__global__ void table_kernel(Problem p) {
    WsHeader* hdr = reinterpret_cast<WsHeader*>(p.ws);
    int32_t* seq_first = reinterpret_cast<int32_t*>(p.ws + p.L.seq_first);
    int32_t* chunk_seq = reinterpret_cast<int32_t*>(p.ws + p.L.chunk_seq);
    int32_t* chunk_tok0 = reinterpret_cast<int32_t*>(p.ws + p.L.chunk_tok0);
    int32_t* chunk_len = reinterpret_cast<int32_t*>(p.ws + p.L.chunk_len);
    const int N = p.d.N;
    __shared__ int ok;
    auto cu = [&](int n) -> long long { return p.cu ? (long long)p.cu[n] : (long long)n * p.d.T; };
    if (threadIdx.x == 0) {
        int good = 1, bad_at = -1;
        if (cu(0) != 0) { good = 0; bad_at = 0; }
        int acc = 0;
        for (int n = 0; n < N && good; ++n) {
            const long long a = cu(n), e = cu(n + 1);
            if (e < a || e > p.Ttot) { good = 0; bad_at = n + 1; break; }
            seq_first[n] = acc;
            acc += (int)((e - a + kC - 1) / kC);
        }
        if (good && cu(N) != p.Ttot) { good = 0; bad_at = N; }
        if (good) {
            seq_first[N] = acc;
            hdr->status = GDN_OK;
            hdr->n_chunks = acc;
            hdr->detail = 0;
        } else {
            for (int n = 0; n <= N; ++n) seq_first[n] = 0;
            hdr->status = GDN_ERR_BAD_SEQLENS;
            hdr->n_chunks = 0;
            hdr->detail = bad_at;
        }
        ok = good;
    }
    __syncthreads();
    if (!ok) return;
    const int nch = seq_first[N];
    for (int c = threadIdx.x; c < nch; c += blockDim.x) {
        int lo = 0, hi = N - 1;  // last n with seq_first[n] <= c and a non-empty chunk range
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (seq_first[mid] <= c) lo = mid; else hi = mid - 1;
        }
        const int n = lo;
        const long long a = cu(n), e = cu(n + 1);
        const long long t0 = a + (long long)(c - seq_first[n]) * kC;
        chunk_seq[c] = n;
        chunk_tok0[c] = (int)t0;
        chunk_len[c] = (int)((e - t0) < kC ? (e - t0) : kC);
    }
}

// Loads the gate rows of a chunk: g (0 when padded), erase gate b, write gate w.
__device__ __forceinline__ void load_gates(const Problem& p, const ChunkCtx& x, int i, float& g, float& b, float& w) {
    g = 0.f; b = 0.f; w = 0.f;
    if (i < x.len) {
        const size_t idx = (size_t)(x.tok0 + i) * p.d.H + x.hd;
        g = p.g[idx];
        if (p.d.delta_rule) { b = p.beta[idx]; w = b; } else { b = 0.f; w = 1.f; }
    }
}

// ------------------------------------------------------------------------------------------------
// prep
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) prep_kernel(Problem p) {
    ChunkCtx x;
    if (!chunk_ctx(p, x)) return;
    __shared__ float gam[kC], Gam[kC], ee[kC], bb[kC], ww[kC];
    __shared__ float A[kC][kC + 1], Ti[kC][kC + 1];
    const int H = p.d.H;
    const IO* kp = reinterpret_cast<const IO*>(p.k) + ((size_t)x.tok0 * H + x.hd) * DK;
    const IO* vp = reinterpret_cast<const IO*>(p.v) + ((size_t)x.tok0 * H + x.hd) * DV;
    const size_t rk = (size_t)H * DK, rv = (size_t)H * DV;
    auto Kf = [&](int i, int m) -> float { return i < x.len ? ldf(kp + i * rk + m) : 0.f; };
    auto Vf = [&](int i, int m) -> float { return i < x.len ? ldf(vp + i * rv + m) : 0.f; };
    float* wsG = reinterpret_cast<float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC;
    float* wsT = reinterpret_cast<float*>(p.ws + p.L.Tm) + (size_t)x.ch * kC * kC;
    float* wsW = reinterpret_cast<float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    float* wsU = reinterpret_cast<float*>(p.ws + p.L.Ut) + (size_t)x.ch * kC * DV;
    float* wsN = reinterpret_cast<float*>(p.ws + p.L.Nm) + (size_t)x.ch * DK * DK;
    float* wsB = reinterpret_cast<float*>(p.ws + p.L.Bf) + (size_t)x.ch * DK * DV;

    if (threadIdx.x < kC) {
        float g, b, w;
        load_gates(p, x, threadIdx.x, g, b, w);
        gam[threadIdx.x] = g; bb[threadIdx.x] = b; ww[threadIdx.x] = w;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int i = 0; i < kC; ++i) { s += gam[i]; gam[i] = s; }
    }
    __syncthreads();
    if (threadIdx.x < kC) {
        const int i = threadIdx.x;
        Gam[i] = expf(gam[i]);
        ee[i] = expf(gam[kC - 1] - gam[i]);
        wsG[i] = gam[i];
    }
    // A = stril(Diag(b) (K K^T . D)); the decay exponent is only evaluated where j < i (non-positive).
    tiles(kC, kC, [&](int i0, int j0) {
        float acc[4][4] = {};
        if (j0 < i0 + 4) mac(acc, i0, j0, DK, Kf, [&](int m, int j) { return Kf(j, m); });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                A[i][j] = (j < i) ? bb[i] * acc[a][b] * expf(gam[i] - gam[j]) : 0.f;
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
    // W = T Diag(b Gam) K,  Ut = T Diag(w) V
    tiles(kC, DK, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return Ti[i][m]; }, [&](int m, int j) { return bb[m] * Gam[m] * Kf(m, j); });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) wsW[(i0 + a) * DK + j0 + b] = acc[a][b];
    });
    tiles(kC, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return Ti[i][m]; }, [&](int m, int j) { return ww[m] * Vf(m, j); });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) wsU[(i0 + a) * DV + j0 + b] = acc[a][b];
    });
    __syncthreads();
    // Nm = Kb^T W,  Bf = Kb^T Ut,  Kb = Diag(exp(gam_e - gam)) K
    tiles(DK, DK, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return ee[m] * Kf(m, i); }, [&](int m, int j) { return wsW[m * DK + j]; });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) wsN[(i0 + a) * DK + j0 + b] = acc[a][b];
    });
    tiles(DK, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return ee[m] * Kf(m, i); }, [&](int m, int j) { return wsU[m * DV + j]; });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) wsB[(i0 + a) * DV + j0 + b] = acc[a][b];
    });
}

// ------------------------------------------------------------------------------------------------
// eprep: E = scale (Diag(Gam) Q - P W)^T dO
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) eprep_kernel(Problem p) {
    ChunkCtx x;
    if (!chunk_ctx(p, x)) return;
    __shared__ float gam[kC];
    __shared__ float P[kC][kC + 1];
    const int H = p.d.H;
    const IO* qp = reinterpret_cast<const IO*>(p.q) + ((size_t)x.tok0 * H + x.hd) * DK;
    const IO* kp = reinterpret_cast<const IO*>(p.k) + ((size_t)x.tok0 * H + x.hd) * DK;
    const IO* gp = reinterpret_cast<const IO*>(p.dO) + ((size_t)x.tok0 * H + x.hd) * DV;
    const size_t rk = (size_t)H * DK, rv = (size_t)H * DV;
    auto Qf = [&](int i, int m) -> float { return i < x.len ? ldf(qp + i * rk + m) : 0.f; };
    auto Kf = [&](int i, int m) -> float { return i < x.len ? ldf(kp + i * rk + m) : 0.f; };
    auto Gf = [&](int i, int m) -> float { return i < x.len ? ldf(gp + i * rv + m) : 0.f; };
    const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC;
    const float* wsW = reinterpret_cast<const float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    float* wsE = reinterpret_cast<float*>(p.ws + p.L.E) + (size_t)x.ch * DK * DV;
    float* X = reinterpret_cast<float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * x.ch);  // [64, DK]
    if (threadIdx.x < kC) gam[threadIdx.x] = wsG[threadIdx.x];
    __syncthreads();
    tiles(kC, kC, [&](int i0, int j0) {
        float acc[4][4] = {};
        if (j0 <= i0 + 3) mac(acc, i0, j0, DK, Qf, [&](int m, int j) { return Kf(j, m); });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                P[i][j] = (j <= i) ? acc[a][b] * expf(gam[i] - gam[j]) : 0.f;
            }
    });
    __syncthreads();
    tiles(kC, DK, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return P[i][m]; }, [&](int m, int j) { return wsW[m * DK + j]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) X[(i0 + a) * DK + j0 + b] = expf(gam[i0 + a]) * Qf(i0 + a, j0 + b) - acc[a][b];
    });
    __syncthreads();
    const float sc = p.d.scale;
    tiles(DK, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return X[m * DK + i]; }, Gf);
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) wsE[(i0 + a) * DV + j0 + b] = sc * acc[a][b];
    });
}

// ------------------------------------------------------------------------------------------------
// Forward and reverse carries.  One CTA per (sequence, head); the fp32 state lives in shared memory.
// REVERSE = false:  h' = Gam_e h - Nm h + Bf, stores h entering each chunk, optional final state.
// REVERSE = true :  dh = Gam_e dh' - Nm^T dh' + E, stores dh' per chunk, optional dh0.
// ------------------------------------------------------------------------------------------------
template <int DK, int DV, bool REVERSE>
__global__ void __launch_bounds__(kThreads) scan_kernel(Problem p) {
    extern __shared__ float sm[];
    float* cur = sm;
    float* nxt = sm + DK * DV;
    const int n = blockIdx.x / p.d.H, hd = blockIdx.x % p.d.H;
    const int32_t* seq_first = reinterpret_cast<const int32_t*>(p.ws + p.L.seq_first);
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    if (hdr->status != GDN_OK) return;
    const int c0 = seq_first[n], c1 = seq_first[n + 1];
    const size_t soff = ((size_t)n * p.d.H + hd) * DK * DV;
    const float* init = REVERSE ? p.dhT : p.h0;
    for (int t = threadIdx.x; t < DK * DV; t += blockDim.x) cur[t] = init ? init[soff + t] : 0.f;
    __syncthreads();
    for (int s = 0; s < c1 - c0; ++s) {
        const int c = REVERSE ? (c1 - 1 - s) : (c0 + s);
        const size_t ch = (size_t)c * p.d.H + hd;
        const float* wsN = reinterpret_cast<const float*>(p.ws + p.L.Nm) + ch * DK * DK;
        const float* add = reinterpret_cast<const float*>(p.ws + (REVERSE ? p.L.E : p.L.Bf)) + ch * DK * DV;
        float* keep = reinterpret_cast<float*>(p.ws + (REVERSE ? p.L.dhn : p.L.hc)) + ch * DK * DV;
        const float Ge = expf(reinterpret_cast<const float*>(p.ws + p.L.gamma)[ch * kC + kC - 1]);
        for (int t = threadIdx.x; t < DK * DV; t += blockDim.x) keep[t] = cur[t];
        tiles(DK, DV, [&](int i0, int j0) {
            float acc[4][4] = {};
            mac(acc, i0, j0, DK, [&](int i, int m) { return REVERSE ? wsN[m * DK + i] : wsN[i * DK + m]; },
                [&](int m, int j) { return cur[m * DV + j]; });
            for (int a = 0; a < 4; ++a)
                for (int b = 0; b < 4; ++b) {
                    const int t = (i0 + a) * DV + j0 + b;
                    nxt[t] = Ge * cur[t] - acc[a][b] + add[t];
                }
        });
        __syncthreads();
        float* tmp = cur; cur = nxt; nxt = tmp;
    }
    float* fin = REVERSE ? p.dh0 : p.hT;
    if (fin) for (int t = threadIdx.x; t < DK * DV; t += blockDim.x) fin[soff + t] = cur[t];
}

// ------------------------------------------------------------------------------------------------
// Forward output (optional): o = scale (Diag(Gam) Q h + P (Ut - W h))
// ------------------------------------------------------------------------------------------------
template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) out_kernel(Problem p) {
    ChunkCtx x;
    if (!chunk_ctx(p, x)) return;
    __shared__ float gam[kC];
    __shared__ float P[kC][kC + 1];
    const int H = p.d.H;
    const IO* qp = reinterpret_cast<const IO*>(p.q) + ((size_t)x.tok0 * H + x.hd) * DK;
    const IO* kp = reinterpret_cast<const IO*>(p.k) + ((size_t)x.tok0 * H + x.hd) * DK;
    IO* op = reinterpret_cast<IO*>(p.o) + ((size_t)x.tok0 * H + x.hd) * DV;
    const size_t rk = (size_t)H * DK, rv = (size_t)H * DV;
    auto Qf = [&](int i, int m) -> float { return i < x.len ? ldf(qp + i * rk + m) : 0.f; };
    auto Kf = [&](int i, int m) -> float { return i < x.len ? ldf(kp + i * rk + m) : 0.f; };
    const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC;
    const float* wsW = reinterpret_cast<const float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    const float* wsU = reinterpret_cast<const float*>(p.ws + p.L.Ut) + (size_t)x.ch * kC * DV;
    const float* h = reinterpret_cast<const float*>(p.ws + p.L.hc) + (size_t)x.ch * DK * DV;
    float* U = reinterpret_cast<float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * x.ch);  // [64, DV]
    if (threadIdx.x < kC) gam[threadIdx.x] = wsG[threadIdx.x];
    __syncthreads();
    tiles(kC, kC, [&](int i0, int j0) {
        float acc[4][4] = {};
        if (j0 <= i0 + 3) mac(acc, i0, j0, DK, Qf, [&](int m, int j) { return Kf(j, m); });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                P[i][j] = (j <= i) ? acc[a][b] * expf(gam[i] - gam[j]) : 0.f;
            }
    });
    tiles(kC, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, DK, [&](int i, int m) { return wsW[i * DK + m]; }, [&](int m, int j) { return h[m * DV + j]; });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) U[(i0 + a) * DV + j0 + b] = wsU[(i0 + a) * DV + j0 + b] - acc[a][b];
    });
    __syncthreads();
    const float sc = p.d.scale;
    tiles(kC, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, DK, [&](int i, int m) { return expf(gam[i]) * Qf(i, m); }, [&](int m, int j) { return h[m * DV + j]; });
        mac(acc, i0, j0, kC, [&](int i, int m) { return P[i][m]; }, [&](int m, int j) { return U[m * DV + j]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b)
                if (i0 + a < x.len) stf(op + (i0 + a) * rv + j0 + b, sc * acc[a][b]);
    });
}

// ------------------------------------------------------------------------------------------------
// intra: token gradients of one (chunk, head).
// ------------------------------------------------------------------------------------------------
struct IntraSmem {
    float gam[kC], Gam[kC], ee[kC], bb[kC], ww[kC];
    float r[kC], rq[kC], xk[kC], xv[kC], dgam[kC];
    float red[kThreads / 32];
    float P[kC][kC + 1];    // tril(Q K^T . D)
    float KK[kC][kC + 1];   // K K^T, later Z = G . KK
    float dP[kC][kC + 1];   // scale tril(dO U^T)
    float G[kC][kC + 1];    // dA . D
};

template <typename IO, int DK, int DV>
__global__ void __launch_bounds__(kThreads) intra_kernel(Problem p) {
    ChunkCtx x;
    if (!chunk_ctx(p, x)) return;
    extern __shared__ __align__(16) unsigned char smraw[];
    IntraSmem& S = *reinterpret_cast<IntraSmem*>(smraw);
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
    const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC;
    const float* Tm = reinterpret_cast<const float*>(p.ws + p.L.Tm) + (size_t)x.ch * kC * kC;
    const float* W = reinterpret_cast<const float*>(p.ws + p.L.W) + (size_t)x.ch * kC * DK;
    const float* Ut = reinterpret_cast<const float*>(p.ws + p.L.Ut) + (size_t)x.ch * kC * DV;
    const float* h = reinterpret_cast<const float*>(p.ws + p.L.hc) + (size_t)x.ch * DK * DV;
    const float* dhn = reinterpret_cast<const float*>(p.ws + p.L.dhn) + (size_t)x.ch * DK * DV;
    float* scr = reinterpret_cast<float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * x.ch);
    float* U = scr;                    // [64, DV]
    float* dU = U + kC * DV;           // [64, DV]
    float* dXv = dU + kC * DV;         // [64, DV]  (first holds Kb dh')
    float* dOh = dXv + kC * DV;        // [64, DK]  dO h^T
    float* dW = dOh + kC * DK;         // [64, DK]
    float* dXk = dW + kC * DK;         // [64, DK]
    const float sc = p.d.scale;

    if (threadIdx.x < kC) {
        const int i = threadIdx.x;
        float g, b, w;
        load_gates(p, x, i, g, b, w);
        (void)g;
        S.bb[i] = b; S.ww[i] = w;
        S.gam[i] = wsG[i];
    }
    __syncthreads();
    if (threadIdx.x < kC) {
        const int i = threadIdx.x;
        S.Gam[i] = expf(S.gam[i]);
        S.ee[i] = expf(S.gam[kC - 1] - S.gam[i]);
    }
    // D_ij, only ever evaluated for j <= i so that the exponent is non-positive
    auto D = [&](int i, int j) -> float { return expf(S.gam[i] - S.gam[j]); };

    // (1) U = Ut - W h ;  K K^T ;  P
    tiles(kC, DV, [&](int i0, int j0) {
        float acc[4][4] = {};
        mac(acc, i0, j0, DK, [&](int i, int m) { return W[i * DK + m]; }, [&](int m, int j) { return h[m * DV + j]; });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) U[(i0 + a) * DV + j0 + b] = Ut[(i0 + a) * DV + j0 + b] - acc[a][b];
    });
    tiles(kC, kC, [&](int i0, int j0) {
        float kk[4][4] = {}, qk[4][4] = {};
        if (j0 <= i0 + 3) {
            mac(kk, i0, j0, DK, Kf, [&](int m, int j) { return Kf(j, m); });
            mac(qk, i0, j0, DK, Qf, [&](int m, int j) { return Kf(j, m); });
        }
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                S.KK[i][j] = (j < i) ? kk[a][b] : 0.f;
                S.P[i][j] = (j <= i) ? qk[a][b] * D(i, j) : 0.f;
            }
    });
    __syncthreads();
    // (2) Kb dh' -> dXv (temporarily) ;  dU = scale P^T dO + Kb dh'
    tiles(kC, DV, [&](int i0, int j0) {
        float a1[4][4] = {}, a2[4][4] = {};
        mac(a1, i0, j0, DK, [&](int i, int m) { return S.ee[i] * Kf(i, m); }, [&](int m, int j) { return dhn[m * DV + j]; });
        mac(a2, i0, j0, kC, [&](int i, int m) { return S.P[m][i]; }, Of);
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                dXv[(i0 + a) * DV + j0 + b] = a1[a][b];
                dU[(i0 + a) * DV + j0 + b] = sc * a2[a][b] + a1[a][b];
            }
    });
    __syncthreads();
    // (3) dP = scale tril(dO U^T) ;  dO h^T ;  dW = -dU h^T ;  r_i = <(Kb dh')_i, U_i>
    tiles(kC, kC, [&](int i0, int j0) {
        float acc[4][4] = {};
        if (j0 <= i0 + 3) mac(acc, i0, j0, DV, Of, [&](int m, int j) { return U[j * DV + m]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) S.dP[i0 + a][j0 + b] = (j0 + b <= i0 + a) ? sc * acc[a][b] : 0.f;
    });
    tiles(kC, DK, [&](int i0, int j0) {
        float a1[4][4] = {}, a2[4][4] = {};
        mac(a1, i0, j0, DV, Of, [&](int m, int j) { return h[j * DV + m]; });
        mac(a2, i0, j0, DV, [&](int i, int m) { return dU[i * DV + m]; }, [&](int m, int j) { return h[j * DV + m]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                dOh[(i0 + a) * DK + j0 + b] = a1[a][b];
                dW[(i0 + a) * DK + j0 + b] = -a2[a][b];
            }
    });
    row_reduce(S.r, DV, [&](int i, int j) { return dXv[i * DV + j] * U[i * DV + j]; });
    __syncthreads();
    // (4) dQ ;  dXk = T^T dW ;  dXv = T^T dU ;  rq_i = <Q_i, (dO h^T)_i>
    tiles(kC, DK, [&](int i0, int j0) {
        float acc[4][4] = {}, ax[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return m <= i ? S.dP[i][m] * D(i, m) : 0.f; }, Kf);
        mac(ax, i0, j0, kC, [&](int i, int m) { return Tm[m * kC + i]; }, [&](int m, int j) { return dW[m * DK + j]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                if (i < x.len) stf(dqp + i * rk + j, sc * S.Gam[i] * dOh[i * DK + j] + acc[a][b]);
                dXk[i * DK + j] = ax[a][b];
            }
    });
    tiles(kC, DV, [&](int i0, int j0) {
        float ax[4][4] = {};
        mac(ax, i0, j0, kC, [&](int i, int m) { return Tm[m * kC + i]; }, [&](int m, int j) { return dU[m * DV + j]; });
        for (int a = 0; a < 4; ++a) for (int b = 0; b < 4; ++b) dXv[(i0 + a) * DV + j0 + b] = ax[a][b];
    });
    row_reduce(S.rq, DK, [&](int i, int j) { return Qf(i, j) * dOh[i * DK + j]; });
    __syncthreads();
    // (5) dA = -stril(dXk W^T + dXv Ut^T) ;  G = dA . D ;  Z = G . KK ;  row dots of dXk.K and dXv.V
    tiles(kC, kC, [&](int i0, int j0) {
        float acc[4][4] = {};
        if (j0 < i0 + 3) {
            mac(acc, i0, j0, DK, [&](int i, int m) { return dXk[i * DK + m]; }, [&](int m, int j) { return W[j * DK + m]; });
            mac(acc, i0, j0, DV, [&](int i, int m) { return dXv[i * DV + m]; }, [&](int m, int j) { return Ut[j * DV + m]; });
        }
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                const float g_ = (j < i) ? -acc[a][b] * D(i, j) : 0.f;
                S.G[i][j] = g_;
                S.KK[i][j] = g_ * S.KK[i][j];
            }
    });
    row_reduce(S.xk, DK, [&](int i, int j) { return dXk[i * DK + j] * Kf(i, j); });
    row_reduce(S.xv, DV, [&](int i, int j) { return dXv[i * DV + j] * Vf(i, j); });
    __syncthreads();
    // (6) dK, dV, gate gradients
    tiles(kC, DK, [&](int i0, int j0) {
        float acc[4][4] = {}, a2[4][4] = {};
        mac(acc, i0, j0, kC, [&](int i, int m) { return m >= i ? S.dP[m][i] * D(m, i) : 0.f; }, Qf);
        mac(acc, i0, j0, kC, [&](int i, int m) { return S.bb[i] * S.G[i][m] + S.bb[m] * S.G[m][i]; }, Kf);
        mac(a2, i0, j0, DV, [&](int i, int m) { return U[i * DV + m]; }, [&](int m, int j) { return dhn[j * DV + m]; });
        for (int a = 0; a < 4; ++a)
            for (int b = 0; b < 4; ++b) {
                const int i = i0 + a, j = j0 + b;
                if (i < x.len) stf(dkp + i * rk + j, acc[a][b] + S.ee[i] * a2[a][b] + S.bb[i] * S.Gam[i] * dXk[i * DK + j]);
            }
    });
    for (int t = threadIdx.x; t < kC * DV; t += blockDim.x) {
        const int i = t / DV, j = t % DV;
        if (i < x.len) stf(dvp + i * rv + j, S.ww[i] * dXv[t]);
    }
    // <dh', h> over the whole state, fixed order
    float part = 0.f;
    for (int t = threadIdx.x; t < DK * DV; t += blockDim.x) part = fmaf(dhn[t], h[t], part);
    part = warp_sum(part);
    if ((threadIdx.x & 31) == 0) S.red[threadIdx.x >> 5] = part;
    if (threadIdx.x < kC) {
        const int i = threadIdx.x;
        float rowZ = 0.f, colZ = 0.f, rowPP = 0.f, colPP = 0.f;
        for (int j = 0; j < kC; ++j) {
            rowZ += S.KK[i][j];
            colZ += S.bb[j] * S.KK[j][i];
            rowPP += S.dP[i][j] * S.P[i][j];
            colPP += S.dP[j][i] * S.P[j][i];
        }
        const float db = rowZ + S.Gam[i] * S.xk[i];
        const float dw = S.xv[i];
        if (p.d.delta_rule && i < x.len) p.dbeta[(size_t)(x.tok0 + i) * H + x.hd] = db + dw;
        S.dgam[i] = S.bb[i] * rowZ - colZ + rowPP - colPP + S.bb[i] * S.Gam[i] * S.xk[i] + sc * S.Gam[i] * S.rq[i] - S.r[i];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float hh = 0.f, rs = 0.f;
        for (int w_ = 0; w_ < kThreads / 32; ++w_) hh += S.red[w_];
        for (int i = 0; i < kC; ++i) rs += S.r[i];
        S.dgam[kC - 1] += rs + S.Gam[kC - 1] * hh;
        // gam_i = sum_{j<=i} g_j  =>  dg_j = sum_{i>=j} dgam_i
        float run = 0.f;
        for (int i = kC - 1; i >= 0; --i) {
            run += S.dgam[i];
            if (i < x.len) p.dg[(size_t)(x.tok0 + i) * H + x.hd] = run;
        }
    }
}

template <typename IO, int DK, int DV>
cudaError_t launch_fwd_t(const Problem& p, cudaStream_t st) {
    const int CH = p.L.max_chunks * p.d.H, chains = p.d.N * p.d.H;
    launch_table(p, st);
    if (CH > 0) { StageScope t(ST_PREP, st); prep_kernel<IO, DK, DV><<<CH, kThreads, 0, st>>>(p); }
    const size_t sm = 2 * sizeof(float) * DK * DV;
    cudaError_t e = cudaFuncSetAttribute(scan_kernel<DK, DV, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    if (chains > 0) { StageScope t(ST_FSCAN, st); scan_kernel<DK, DV, false><<<chains, kThreads, sm, st>>>(p); }
    if (p.o && CH > 0) { StageScope t(ST_OUT, st); out_kernel<IO, DK, DV><<<CH, kThreads, 0, st>>>(p); }
    return cudaGetLastError();
}

template <typename IO, int DK, int DV>
cudaError_t launch_bwd_t(const Problem& p, bool skip_recompute, cudaStream_t st) {
    cudaError_t e;
    if (!skip_recompute) {
        e = launch_fwd_t<IO, DK, DV>(p, st);
        if (e != cudaSuccess) return e;
    }
    const int CH = p.L.max_chunks * p.d.H, chains = p.d.N * p.d.H;
    if (CH > 0) { StageScope t(ST_EPREP, st); eprep_kernel<IO, DK, DV><<<CH, kThreads, 0, st>>>(p); }
    const size_t sm = 2 * sizeof(float) * DK * DV;
    e = cudaFuncSetAttribute(scan_kernel<DK, DV, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
    if (e != cudaSuccess) return e;
    if (chains > 0) { StageScope t(ST_RSCAN, st); scan_kernel<DK, DV, true><<<chains, kThreads, sm, st>>>(p); }
    e = cudaFuncSetAttribute(intra_kernel<IO, DK, DV>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(IntraSmem));
    if (e != cudaSuccess) return e;
    if (CH > 0) { StageScope t(ST_INTRA, st); intra_kernel<IO, DK, DV><<<CH, kThreads, sizeof(IntraSmem), st>>>(p); }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_table(const Problem& p, cudaStream_t st) {
    StageScope t(ST_TABLE, st);
    table_kernel<<<1, 256, 0, st>>>(p);
    return cudaGetLastError();
}

size_t simt_scratch_per_chunkhead(const gdn_desc& d) { return sizeof(float) * kC * 3 * ((size_t)d.d_k + d.d_v); }

#define GDN_DISPATCH(FN, ...)                                                                       \
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

cudaError_t simt_launch_fwd(const Problem& p, cudaStream_t st) { GDN_DISPATCH(launch_fwd_t, p, st); }
cudaError_t simt_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st) { GDN_DISPATCH(launch_bwd_t, p, skip_recompute, st); }

}  // namespace gdn
