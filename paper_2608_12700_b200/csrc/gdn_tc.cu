// tcgen05 / TMEM / TMA kernels of the GDN backward for bf16 I/O, d_k = d_v = 128, chunk 64 (sm_100a).
//
// Three kernels follow the stage map of the chunked method (Section 4.2 of the paper):
//   tc_prep  (one CTA per chunk-head)  gamma, A, T = (I + A)^-1, W, U~, Nm = Kb^T W, Bf = Kb^T U~ and, for the
//                                      backward, E = scale (Diag(Gam) Q - P W)^T dO
//   tc_scan  (one CTA per chain, direction and 64-column slice of the state)
//                                      forward carry  h'  = Gam_e h  - Nm   h  + Bf   (stores h per chunk)
//                                      reverse carry  dh  = Gam_e dh' - Nm^T dh' + E   (the paper's K#1; stores dh')
//   tc_intra (one CTA per chunk-head)  every token gradient, including the VJP of the triangular solve (K#2)
//
// All dense products run on tcgen05.mma with fp32 accumulators in tensor memory; operands are bf16 tiles in
// shared memory in the "blocked-64, 128-byte swizzle" format of tc_ptx.cuh, brought in by TMA (inputs) or by
// contiguous bulk copies of tile images (workspace).  Accumulators are produced with the feature dimension
// (128) on the TMEM lanes and the 64 tokens of the chunk on the columns, i.e. transposed, so that M = 128.
// The carried states stay fp32 in registers for the whole scan; tensor memory holds accumulators only and is
// allocated once per CTA and released once.  Every wait is bounded; a wait that gives up records
// GDN_ERR_DEVICE_TIMEOUT in the workspace header and the CTA leaves through its normal teardown.
#include "gdn_internal.cuh"
#include "tc_ptx.cuh"
#include "tc_tmap.cuh"

namespace gdn {
namespace {

using namespace tc;

constexpr int D = 128;          // d_k = d_v
constexpr int kThreads = 256;   // 8 warps: lane quadrant = warp % 4, column half = warp / 4

struct TcParams {
    Problem p;
    CUtensorMap tm_q, tm_k, tm_v, tm_do;   // [T_total, H * 128] bf16, boxes of 64 rows x 64 columns
    int with_bwd;                          // prep: also produce E
};

__device__ __forceinline__ void report_timeout(char* ws, int where) {
    WsHeader* h = reinterpret_cast<WsHeader*>(ws);
    h->status = GDN_ERR_DEVICE_TIMEOUT;
    h->detail = where;
}

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
    return p + ((1024u - (smem_u32(p) & 1023u)) & 1023u);
}

// 8 fp32 -> one 16-byte chunk of bf16
__device__ __forceinline__ uint4 pack8(const float* v) {
    return make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
__device__ __forceinline__ void unpack8(const uint4& u, float* v) {
    v[0] = bf16_lo(u.x); v[1] = bf16_hi(u.x); v[2] = bf16_lo(u.y); v[3] = bf16_hi(u.y);
    v[4] = bf16_lo(u.z); v[5] = bf16_hi(u.z); v[6] = bf16_lo(u.w); v[7] = bf16_hi(u.w);
}
// Write 32 consecutive columns [c0, c0 + 32) of row r of a tile with R rows (c0 % 32 == 0).
__device__ __forceinline__ void tile_store32(unsigned char* tile, int R, int r, int c0, const float* v) {
#pragma unroll
    for (int c = 0; c < 4; ++c) *reinterpret_cast<uint4*>(tile + tile_chunk_off(R, r, (c0 >> 3) + c)) = pack8(v + 8 * c);
}
__device__ __forceinline__ void tile_load32(const unsigned char* tile, int R, int r, int c0, float* v) {
#pragma unroll
    for (int c = 0; c < 4; ++c) unpack8(*reinterpret_cast<const uint4*>(tile + tile_chunk_off(R, r, (c0 >> 3) + c)), v + 8 * c);
}
__device__ __forceinline__ float tile_get(const unsigned char* tile, int R, int r, int c) {
    return __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(tile + tile_off(R, r, c)));
}

// Zero rows [len, 64) of a [rows0 .. rows0 + 64) window of a tile with R rows and 128 columns.
__device__ __forceinline__ void zero_tail_rows(unsigned char* tile, int R, int row0, int len) {
    for (int t = threadIdx.x; t < (kC - len) * 16; t += blockDim.x) {
        const int r = row0 + len + t / 16, ch = t % 16;
        *reinterpret_cast<uint4*>(tile + tile_chunk_off(R, r, ch)) = make_uint4(0, 0, 0, 0);
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ------------------------------------------------------------------------------------------------
// tc_prep
// ------------------------------------------------------------------------------------------------
namespace prep {
constexpr uint32_t QK = 0;                    // [Q rows 0..63 ; K rows 64..127] x 128   32 KB (later: Nm image)
constexpr uint32_t VO = 32768;                // [V ; dO] x 128                           32 KB
constexpr uint32_t TT = 65536;                // T                      [64][64]           8 KB
constexpr uint32_t TP = TT + 8192;            // T Diag(b Gam)
constexpr uint32_t TPP = TP + 8192;           // T Diag(w)
constexpr uint32_t PT = TPP + 8192;           // P = tril(Q K^T . D)
constexpr uint32_t WT = PT + 8192;            // W^T   [128 dk][64 tokens]                16 KB
constexpr uint32_t WET = WT + 16384;          // (Diag(e) W)^T
constexpr uint32_t UTT = WET + 16384;         // U~^T  [128 dv][64]
constexpr uint32_t UET = UTT + 16384;         // (Diag(e) U~)^T
constexpr uint32_t X = UET + 16384;           // fp32 A and T during the inversion; later R = Diag(Gam) dO and (P^T dO)^T
constexpr uint32_t XA = X, XT = X + 16640;
constexpr uint32_t XR = X, XPDO = X + 16384;
constexpr uint32_t TILES_END = X + 34816;
constexpr uint32_t SMEM_BYTES = TILES_END + 1024 /* alignment slack */;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
// TMEM columns (512 allocated): accumulators at fixed offsets, allocated once, released once.
constexpr uint32_t C_S1 = 0, C_W = 64, C_U = 128, C_PDO = 192, C_NM = 256, C_BF = 384, C_E = 0;
}  // namespace prep

__global__ void __launch_bounds__(kThreads, 1) tc_prep_kernel(const __grid_constant__ TcParams P) {
    using namespace prep;
    const Problem& p = P.p;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    const int c = blockIdx.x / p.d.H, hd = blockIdx.x % p.d.H;
    if (c >= hdr->n_chunks) return;
    const int ch = blockIdx.x;
    const int tok0 = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0)[c];
    const int len = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len)[c];
    const int H = p.d.H;
    const bool bwd = P.with_bwd != 0;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ float gam[kC], Gam[kC], ee[kC], bb[kC], ww[kC];
    __shared__ uint64_t bar_qk, bar_vo, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, half = warp >> 2;

    if (threadIdx.x == 0) {
        mbar_init(&bar_qk, 1); mbar_init(&bar_vo, 1); mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    bool ok = true;
    uint32_t mma_phase = 0;

    if (threadIdx.x == 0) {
        mbar_expect_tx(&bar_qk, 32768);
        for (int cb = 0; cb < 2; ++cb) {
            tma_load_2d(sm + QK + cb * 16384, &P.tm_q, hd * D + cb * 64, tok0, &bar_qk);
            tma_load_2d(sm + QK + cb * 16384 + 8192, &P.tm_k, hd * D + cb * 64, tok0, &bar_qk);
        }
        mbar_expect_tx(&bar_vo, bwd ? 32768 : 16384);
        for (int cb = 0; cb < 2; ++cb) {
            tma_load_2d(sm + VO + cb * 16384, &P.tm_v, hd * D + cb * 64, tok0, &bar_vo);
            if (bwd) tma_load_2d(sm + VO + cb * 16384 + 8192, &P.tm_do, hd * D + cb * 64, tok0, &bar_vo);
        }
    }
    // gates: g (0 when padded), erase gate b, write gate w; chunk-local cumulative decay
    if (threadIdx.x < kC) {
        const int i = threadIdx.x;
        float g = 0.f, b = 0.f;
        if (i < len) {
            const size_t idx = (size_t)(tok0 + i) * H + hd;
            g = p.g[idx];
            b = p.beta[idx];
        }
        gam[i] = g; bb[i] = b; ww[i] = b;
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
        reinterpret_cast<float*>(p.ws + p.L.gamma)[(size_t)ch * kC + i] = gam[i];
    }
    ok = mbar_wait(&bar_qk, 0) && mbar_wait(&bar_vo, 0);
    if (!ok && threadIdx.x == 0) report_timeout(p.ws, 1);
    if (ok && len < kC) {   // identity padding of a ragged tail: rows beyond the sequence read as zero
        zero_tail_rows(sm + QK, 128, 0, len);
        zero_tail_rows(sm + QK, 128, 64, len);
        zero_tail_rows(sm + VO, 128, 0, len);
        if (bwd) zero_tail_rows(sm + VO, 128, 64, len);
        fence_async_smem();
    }
    __syncthreads();

    // ---- phase 1: S1 = [Q; K] K^T  (rows 0..63: Q K^T, rows 64..127: K K^T)
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + C_S1, op_k_major(sm + QK, 128, 0), op_k_major(sm + QK, 128, 64), 128, 64, 128, false);
        mma_commit(&bar_mma);
    }
    if (ok) { ok = mbar_wait(&bar_mma, mma_phase); mma_phase ^= 1; if (!ok && threadIdx.x == 0) report_timeout(p.ws, 2); }
    tc_fence_after();
    float* Af = reinterpret_cast<float*>(sm + XA);   // [64][65]
    float* Tf = reinterpret_cast<float*>(sm + XT);   // [64][65]
    if (ok) {
        float v[32];
        tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + C_S1 + half * 32, v);
        tmem_wait_ld();
        const int i = (q4 & 1) * 32 + lane;
        const int j0 = half * 32;
        if (q4 < 2) {   // P_ij = (q_i . k_j) exp(gam_i - gam_j), j <= i (mask before exponentiating)
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (j0 + j <= i) ? v[j] * expf(gam[i] - gam[j0 + j]) : 0.f;
            tile_store32(sm + PT, 64, i, j0, v);
        } else {        // A_ij = b_i (k_i . k_j) exp(gam_i - gam_j), j < i
#pragma unroll
            for (int j = 0; j < 32; ++j) Af[i * 65 + j0 + j] = (j0 + j < i) ? bb[i] * v[j] * expf(gam[i] - gam[j0 + j]) : 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    // ---- T = (I + A)^-1: column j solves (I + A) x = e_j by forward substitution
    if (threadIdx.x < kC) {
        const int j = threadIdx.x;
        for (int i = 0; i < kC; ++i) {
            float s = (i == j) ? 1.f : 0.f;
            for (int m = j; m < i; ++m) s = fmaf(-Af[i * 65 + m], Tf[m * 65 + j], s);
            Tf[i * 65 + j] = (i >= j) ? s : 0.f;
        }
    }
    __syncthreads();
    for (int t = threadIdx.x; t < kC * 8; t += blockDim.x) {
        const int i = t >> 3, cch = t & 7;
        float a[8], b[8], w8[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const int m = cch * 8 + x;
            a[x] = Tf[i * 65 + m];
            b[x] = a[x] * bb[m] * Gam[m];
            w8[x] = a[x] * ww[m];
        }
        *reinterpret_cast<uint4*>(sm + TT + tile_chunk_off(64, i, cch)) = pack8(a);
        *reinterpret_cast<uint4*>(sm + TP + tile_chunk_off(64, i, cch)) = pack8(b);
        *reinterpret_cast<uint4*>(sm + TPP + tile_chunk_off(64, i, cch)) = pack8(w8);
    }
    fence_async_smem();
    __syncthreads();

    // ---- phase 2: W^T = K^T (T Diag(b Gam))^T ; U~^T = V^T (T Diag(w))^T ; (P^T dO)^T = dO^T P
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + C_W, op_mn_major(sm + QK, 128, 64), op_k_major(sm + TP, 64), 128, 64, 64, false);
        mma_tile(tmem + C_U, op_mn_major(sm + VO, 128, 0), op_k_major(sm + TPP, 64), 128, 64, 64, false);
        if (bwd) mma_tile(tmem + C_PDO, op_mn_major(sm + VO, 128, 64), op_mn_major(sm + PT, 64), 128, 64, 64, false);
        mma_commit(&bar_mma);
        bulk_store(p.ws + p.L.Tm + (size_t)ch * 8192, sm + TT, 8192);
        bulk_commit();
    }
    // R = Diag(Gam) dO (token-major tile), while the MMAs run.  The fp32 A / T scratch is dead by now.
    if (bwd) {
        for (int t = threadIdx.x; t < kC * 16; t += blockDim.x) {
            const int i = t >> 4, cch = t & 15;
            float v[8];
            unpack8(*reinterpret_cast<const uint4*>(sm + VO + tile_chunk_off(128, 64 + i, cch)), v);
#pragma unroll
            for (int x = 0; x < 8; ++x) v[x] *= Gam[i];
            *reinterpret_cast<uint4*>(sm + XR + tile_chunk_off(64, i, cch)) = pack8(v);
        }
    }
    if (ok) { ok = mbar_wait(&bar_mma, mma_phase); mma_phase ^= 1; if (!ok && threadIdx.x == 0) report_timeout(p.ws, 3); }
    tc_fence_after();
    if (ok) {
        const int f = q4 * 32 + lane, i0 = half * 32;
        float v[32], ve[32];
        tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + C_W + i0, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) ve[i] = v[i] * ee[i0 + i];
        tile_store32(sm + WT, 128, f, i0, v);
        tile_store32(sm + WET, 128, f, i0, ve);
        tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + C_U + i0, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) ve[i] = v[i] * ee[i0 + i];
        tile_store32(sm + UTT, 128, f, i0, v);
        tile_store32(sm + UET, 128, f, i0, ve);
        if (bwd) {
            tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + C_PDO + i0, v);
            tmem_wait_ld();
            tile_store32(sm + XPDO, 128, f, i0, v);
        }
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();

    // ---- phase 3: Nm = K^T (Diag(e) W) ; Bf = K^T (Diag(e) U~) ; E = Q^T R - W^T (P^T dO)
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + C_NM, op_mn_major(sm + QK, 128, 64), op_k_major(sm + WET, 128), 128, 128, 64, false);
        mma_tile(tmem + C_BF, op_mn_major(sm + QK, 128, 64), op_k_major(sm + UET, 128), 128, 128, 64, false);
        if (bwd) {
            mma_tile(tmem + C_E, op_mn_major(sm + QK, 128, 0), op_mn_major(sm + XR, 64), 128, 128, 64, false);
            mma_tile(tmem + C_E, op_k_major(sm + WT, 128), op_k_major(sm + XPDO, 128), 128, 128, 64, true, /*neg_a=*/true);
        }
        mma_commit(&bar_mma);
        bulk_store(p.ws + p.L.W + (size_t)ch * 16384, sm + WT, 16384);
        bulk_store(p.ws + p.L.Ut + (size_t)ch * 16384, sm + UTT, 16384);
        bulk_commit();
    }
    if (ok) { ok = mbar_wait(&bar_mma, mma_phase); mma_phase ^= 1; if (!ok && threadIdx.x == 0) report_timeout(p.ws, 4); }
    tc_fence_after();
    if (ok) {
        const int r = q4 * 32 + lane, c0 = half * 64;
        float v[32];
        // Nm -> bf16 tile image (reuses the Q/K tile, which no MMA reads any more)
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + C_NM + c0 + part * 32, v);
            tmem_wait_ld();
            tile_store32(sm + QK, 128, r, c0 + part * 32, v);
        }
        // Bf and E -> fp32, column-chunk-major: float4 index (col / 4) * 128 + row
        float4* gB = reinterpret_cast<float4*>(p.ws + p.L.Bf + (size_t)ch * D * D * 4);
        float4* gE = reinterpret_cast<float4*>(p.ws + p.L.E + (size_t)ch * D * D * 4);
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + C_BF + c0 + part * 32, v);
            tmem_wait_ld();
#pragma unroll
            for (int x = 0; x < 8; ++x) gB[(size_t)((c0 + part * 32) / 4 + x) * D + r] = make_float4(v[4 * x], v[4 * x + 1], v[4 * x + 2], v[4 * x + 3]);
        }
        if (bwd) {
            const float sc = p.d.scale;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + C_E + c0 + part * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int x = 0; x < 8; ++x)
                    gE[(size_t)((c0 + part * 32) / 4 + x) * D + r] = make_float4(sc * v[4 * x], sc * v[4 * x + 1], sc * v[4 * x + 2], sc * v[4 * x + 3]);
            }
        }
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
        if (ok) {
            bulk_store(p.ws + p.L.Nm + (size_t)ch * 32768, sm + QK, 32768);
            bulk_commit();
        }
        bulk_wait_all<0>();   // shared memory must stay valid until every bulk store has read it
    }
    if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
bool tc_supported(const gdn_desc& d) {
    return d.dtype == GDN_BF16 && d.d_k == 128 && d.d_v == 128 && d.delta_rule == 1 && d.chunk == kC;
}

static bool fill_params(TcParams& P, const Problem& p, bool with_bwd) {
    P.p = p;
    P.with_bwd = with_bwd ? 1 : 0;
    const uint64_t rows = (uint64_t)p.Ttot, cols = (uint64_t)p.d.H * D, pitch = cols * 2;
    if (!tc::make_tmap_bf16_2d(&P.tm_q, p.q, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_k, p.k, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_v, p.v, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_do, with_bwd ? p.dO : p.v, rows, cols, pitch, 64)) return false;
    return true;
}

static cudaError_t launch_prep(const TcParams& P, cudaStream_t st) {
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(tc_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)prep::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    const int CH = P.p.L.max_chunks * P.p.d.H;
    if (CH > 0) {
        StageScope t(ST_PREP, st);
        tc_prep_kernel<<<CH, kThreads, prep::SMEM_BYTES, st>>>(P);
    }
    return cudaGetLastError();
}

cudaError_t tc_launch_fwd(const Problem& p, cudaStream_t st) {
    TcParams P;
    if (p.Ttot == 0) return cudaSuccess;
    if (!fill_params(P, p, false)) return cudaErrorUnknown;
    cudaError_t e = launch_table(p, st);
    if (e != cudaSuccess) return e;
    return launch_prep(P, st);
}

cudaError_t tc_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st) {
    TcParams P;
    if (p.Ttot == 0) return cudaSuccess;
    if (!fill_params(P, p, true)) return cudaErrorUnknown;
    cudaError_t e = launch_table(p, st);
    if (e != cudaSuccess) return e;
    (void)skip_recompute;
    return launch_prep(P, st);
}

}  // namespace gdn
