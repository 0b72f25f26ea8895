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
    int scan_dirs;                         // scan: 0 = forward carry only, 1 = reverse only, 2 = both
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

// ------------------------------------------------------------------------------------------------
// tc_scan: forward and reverse inter-chunk carries.
// blockIdx.x = ((chain * 2 + direction) * 2 + slice); a CTA owns 64 columns of the 128 x 128 state.
// Per chunk: the fp32 state (registers) is rounded to a bf16 tile, one tcgen05.mma forms Nm h (forward) or
// Nm^T dh (reverse), and the state is updated in fp32:  s <- Gam_e s - (Nm s) + add.  The bf16 tile that fed
// the MMA is also what the chunk's gradient stage needs, so it is bulk-stored to the workspace as it is.
// ------------------------------------------------------------------------------------------------
namespace scan {
constexpr int STAGES = 2;
constexpr uint32_t NM = 0;                       // ring of Nm tile images, 32 KB each
constexpr uint32_t HT = NM + STAGES * 32768;     // two state tiles [128 rows][64 columns], 16 KB each
constexpr uint32_t SMEM_BYTES = HT + 2 * 16384 + 1024;
}  // namespace scan

__global__ void __launch_bounds__(kThreads, 2) tc_scan_kernel(const __grid_constant__ TcParams P) {
    using namespace scan;
    const Problem& p = P.p;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    if (hdr->status != GDN_OK) return;
    const int slice = blockIdx.x & 1;
    const int reverse = P.scan_dirs == 2 ? ((blockIdx.x >> 1) & 1) : P.scan_dirs;
    const int chain = P.scan_dirs == 2 ? (blockIdx.x >> 2) : (blockIdx.x >> 1);
    const int n = chain / p.d.H, hd = chain % p.d.H;
    const int32_t* seq_first = reinterpret_cast<const int32_t*>(p.ws + p.L.seq_first);
    const int c0 = seq_first[n], c1 = seq_first[n + 1], nsteps = c1 - c0;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ uint64_t bar_full[STAGES], bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, hf = warp >> 2;
    const int r = q4 * 32 + lane;              // state row owned by this thread
    const int lc0 = hf * 32;                   // first of its 32 columns inside the CTA's slice
    const int gc0 = slice * 64 + lc0;          // ... and inside the full state

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&bar_full[s], 1);
        mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 64); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    auto chunk_of = [&](int s) { return reverse ? (c1 - 1 - s) : (c0 + s); };
    const char* nm_base = p.ws + p.L.Nm;
    const char* add_base = p.ws + (reverse ? p.L.E : p.L.Bf);
    char* keep_base = p.ws + (reverse ? p.L.dhn : p.L.hc);
    const float* gamma = reinterpret_cast<const float*>(p.ws + p.L.gamma);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES && s < nsteps; ++s) {
            mbar_expect_tx(&bar_full[s], 32768);
            bulk_load(sm + NM + s * 32768, nm_base + ((size_t)chunk_of(s) * p.d.H + hd) * 32768, 32768, &bar_full[s]);
        }
    }
    // initial state
    float st[32];
    {
        const float* init = reverse ? p.dhT : p.h0;
        const size_t soff = ((size_t)n * p.d.H + hd) * D * D + (size_t)r * D + gc0;
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            float4 v = init ? *reinterpret_cast<const float4*>(init + soff + 4 * x) : make_float4(0.f, 0.f, 0.f, 0.f);
            st[4 * x] = v.x; st[4 * x + 1] = v.y; st[4 * x + 2] = v.z; st[4 * x + 3] = v.w;
        }
    }
    bool ok = true;
    uint32_t mma_phase = 0;
    for (int s = 0; s < nsteps; ++s) {
        const size_t ch = (size_t)chunk_of(s) * p.d.H + hd;
        const int stage = s % STAGES, hb = s & 1;
        unsigned char* Ht = sm + HT + hb * 16384;
        const float Ge = expf(gamma[ch * kC + kC - 1]);
        float4 add[8];
        const float4* ga = reinterpret_cast<const float4*>(add_base + ch * D * D * 4);
#pragma unroll
        for (int x = 0; x < 8; ++x) add[x] = ga[(size_t)(gc0 / 4 + x) * D + r];
        tile_store32(Ht, 128, r, lc0, st);
        fence_async_smem();
        __syncthreads();
        if (threadIdx.x == 0) {
            ok = mbar_wait(&bar_full[stage], (s / STAGES) & 1);
            if (ok) {
                tc_fence_after();
                const Operand a = reverse ? op_mn_major(sm + NM + stage * 32768, 128) : op_k_major(sm + NM + stage * 32768, 128);
                mma_tile(tmem, a, op_mn_major(Ht, 128), 128, 64, 128, false);
            } else {
                report_timeout(p.ws, 10);
            }
            bulk_store(keep_base + ch * 32768 + slice * 16384, Ht, 16384);
            bulk_commit();
            bulk_wait_read<1>();   // the store issued one step ago has finished reading the other state tile
            mma_commit(&bar_mma);
        }
        ok = mbar_wait(&bar_mma, mma_phase);
        mma_phase ^= 1;
        if (!ok) { if (threadIdx.x == 0) report_timeout(p.ws, 11); break; }
        tc_fence_after();
        float dl[32];
        tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + lc0, dl);
        tmem_wait_ld();
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            st[4 * x + 0] = fmaf(Ge, st[4 * x + 0], add[x].x - dl[4 * x + 0]);
            st[4 * x + 1] = fmaf(Ge, st[4 * x + 1], add[x].y - dl[4 * x + 1]);
            st[4 * x + 2] = fmaf(Ge, st[4 * x + 2], add[x].z - dl[4 * x + 2]);
            st[4 * x + 3] = fmaf(Ge, st[4 * x + 3], add[x].w - dl[4 * x + 3]);
        }
        tc_fence_before();
        if (threadIdx.x == 0 && s + STAGES < nsteps) {   // the MMA that read this ring slot has completed
            mbar_expect_tx(&bar_full[stage], 32768);
            bulk_load(sm + NM + stage * 32768, nm_base + ((size_t)chunk_of(s + STAGES) * p.d.H + hd) * 32768, 32768, &bar_full[stage]);
        }
    }
    float* fin = reverse ? p.dh0 : p.hT;
    if (fin && ok) {
        const size_t soff = ((size_t)n * p.d.H + hd) * D * D + (size_t)r * D + gc0;
#pragma unroll
        for (int x = 0; x < 8; ++x) *reinterpret_cast<float4*>(fin + soff + 4 * x) = make_float4(st[4 * x], st[4 * x + 1], st[4 * x + 2], st[4 * x + 3]);
    }
    if (threadIdx.x == 0) bulk_wait_all<0>();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 64);
}

// ------------------------------------------------------------------------------------------------
// tc_intra: token gradients of one (chunk, head).
//
// Products (all on tcgen05, outputs transposed: features on TMEM lanes, tokens on columns, except the 64 x 64
// token-token matrices which use M = 64):
//   phase 1  S = Q K^T ; (W h)^T ; (K dh')^T                      -> P = tril(S . D)
//   phase 2  (P^T dO)^T                                            -> U = U~ - W h ; dU = scale P^T dO + Diag(e) K dh'
//   phase 3  dO U^T ; (dO h^T)^T ; -(dU h^T)^T                     -> dPD = scale tril(dO U^T) . D ; dW
//   phase 4  (dPD K)^T ; (T^T dW)^T ; (T^T dU)^T ; (dPD^T Q)^T ; (U dh'^T)^T
//                                                                  -> dq ; dXk ; dXv ; dv ; dw
//   phase 5  dXk W^T + dXv U~^T                                    -> G = -stril(.) . D ; Diag(b) G
//   phase 6  (G K)^T ; += ((Diag(b) G)^T K)^T                      -> dk ; db ; dgamma -> dg
// The decay gradient uses the identities  rowsum(dP.P) + scale Gam <q, dO h^T> = <q, dq>  and its analogues for
// k:  dgamma_i = <q_i, dq_i> + <k_i, dk_i^row> - <k_i, dk_i^col>, where dk^row = Diag(b)(G K + Diag(Gam) dXk)
// collects the terms in which k_i enters with exp(+gamma_i) and dk^col those with exp(-gamma_i); the last row
// of the chunk adds sum_j r_j + Gam_e <dh', h> (r_j = <(Kb dh')_j, U_j>).
// ------------------------------------------------------------------------------------------------
namespace intra {
constexpr uint32_t QK = 0;                 // [Q ; K] x 128                     32 KB
constexpr uint32_t VT = 32768;             // V  [64][128]                      16 KB
constexpr uint32_t DO = VT + 16384;        // dO [64][128]                      16 KB   later dW^T [128][64]
constexpr uint32_t WT = DO + 16384;        // W^T  [128][64]                    16 KB
constexpr uint32_t UTT = WT + 16384;       // U~^T [128][64]                    16 KB
constexpr uint32_t TT = UTT + 16384;       // T [64][64]                         8 KB
constexpr uint32_t HH = TT + 8192;         // h [128][128]                      32 KB   later dXk^T, dXv^T [128][64] each
constexpr uint32_t DH = HH + 32768;        // dh' [128][128]                    32 KB
constexpr uint32_t PT = DH + 32768;        // P [64][64]                         8 KB   later dPD
constexpr uint32_t UT = PT + 8192;         // U^T [128][64]                     16 KB   later G, Diag(b) G [64][64] each
constexpr uint32_t DUT = UT + 16384;       // dU^T [128][64]                    16 KB
constexpr uint32_t SMEM_BYTES = DUT + 16384 + 1024;
constexpr uint32_t DWT = DO, DXKT = HH, DXVT = HH + 16384, DPD = PT, GT = UT, BGT = UT + 8192;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
__host__ __device__ constexpr uint32_t slot(int k) { return 64u * k; }   // eight accumulators of 64 columns in 512 TMEM columns
}  // namespace intra

// Sum v[t] over the 32 lanes of a warp for 32 values at once; lane l ends with the total of index l in v[0].
__device__ __forceinline__ void butterfly32(float (&v)[32], int lane) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int k = 0; k < off; ++k) {
            const float send = up ? v[k] : v[k + off];
            const float keep = up ? v[k + off] : v[k];
            v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
}

__global__ void __launch_bounds__(kThreads, 1) tc_intra_kernel(const __grid_constant__ TcParams P) {
    using namespace intra;
    const Problem& p = P.p;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    const int c = blockIdx.x / p.d.H, hd = blockIdx.x % p.d.H;
    if (c >= hdr->n_chunks) return;
    const int ch = blockIdx.x;
    const int tok0 = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0)[c];
    const int len = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len)[c];
    const int H = p.d.H;
    const float sc = p.d.scale;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ float gam[kC], Gam[kC], ee[kC], bb[kC];
    __shared__ float red1[2][4][32], red2[2][4][32], red3[2][4][32];
    __shared__ float dws[kC], dgam[kC], scal[2][kThreads / 32];
    __shared__ uint64_t bar_in0, bar_in1, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, half = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;

    if (threadIdx.x == 0) {
        mbar_init(&bar_in0, 1); mbar_init(&bar_in1, 1); mbar_init(&bar_mma, 1);
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
        mbar_expect_tx(&bar_in0, 32768 + 16384 + 32768 + 32768);
        for (int cb = 0; cb < 2; ++cb) {
            tma_load_2d(sm + QK + cb * 16384, &P.tm_q, hd * D + cb * 64, tok0, &bar_in0);
            tma_load_2d(sm + QK + cb * 16384 + 8192, &P.tm_k, hd * D + cb * 64, tok0, &bar_in0);
        }
        bulk_load(sm + WT, p.ws + p.L.W + (size_t)ch * 16384, 16384, &bar_in0);
        bulk_load(sm + HH, p.ws + p.L.hc + (size_t)ch * 32768, 32768, &bar_in0);
        bulk_load(sm + DH, p.ws + p.L.dhn + (size_t)ch * 32768, 32768, &bar_in0);
        mbar_expect_tx(&bar_in1, 16384 + 16384 + 16384 + 8192);
        for (int cb = 0; cb < 2; ++cb) {
            tma_load_2d(sm + VT + cb * 8192, &P.tm_v, hd * D + cb * 64, tok0, &bar_in1);
            tma_load_2d(sm + DO + cb * 8192, &P.tm_do, hd * D + cb * 64, tok0, &bar_in1);
        }
        bulk_load(sm + UTT, p.ws + p.L.Ut + (size_t)ch * 16384, 16384, &bar_in1);
        bulk_load(sm + TT, p.ws + p.L.Tm + (size_t)ch * 8192, 8192, &bar_in1);
    }
    if (threadIdx.x < kC) {
        const int i = threadIdx.x;
        const float g = reinterpret_cast<const float*>(p.ws + p.L.gamma)[(size_t)ch * kC + i];
        gam[i] = g;
        Gam[i] = expf(g);
        bb[i] = (i < len) ? p.beta[(size_t)(tok0 + i) * H + hd] : 0.f;
    }
    __syncthreads();
    if (threadIdx.x < kC) ee[threadIdx.x] = expf(gam[kC - 1] - gam[threadIdx.x]);
    ok = mbar_wait(&bar_in0, 0) && mbar_wait(&bar_in1, 0);
    if (!ok && threadIdx.x == 0) report_timeout(p.ws, 20);
    if (ok && len < kC) {
        zero_tail_rows(sm + QK, 128, 0, len);
        zero_tail_rows(sm + QK, 128, 64, len);
        zero_tail_rows(sm + VT, 64, 0, len);
        zero_tail_rows(sm + DO, 64, 0, len);
        fence_async_smem();
    }
    __syncthreads();
    auto Dij = [&](int i, int j) -> float { return expf(gam[i] - gam[j]); };   // only for j <= i
#define GDN_WAIT_MMA(where)                                                                         \
    if (ok) {                                                                                       \
        ok = mbar_wait(&bar_mma, mma_phase);                                                        \
        mma_phase ^= 1;                                                                             \
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, where);                                   \
    }                                                                                               \
    tc_fence_after();

    // ---- phase 1
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + slot(0), op_k_major(sm + QK, 128, 0), op_k_major(sm + QK, 128, 64), 64, 64, 128, false);
        mma_tile(tmem + slot(1), op_mn_major(sm + HH, 128), op_mn_major(sm + WT, 128), 128, 64, 128, false);
        mma_tile(tmem + slot(2), op_mn_major(sm + DH, 128), op_k_major(sm + QK, 128, 64), 128, 64, 128, false);
        mma_commit(&bar_mma);
    }
    // <dh', h> over the whole state while the MMAs run (both tiles share one format, so offsets pair up)
    float hh = 0.f;
    for (int t = threadIdx.x; t < 2048; t += blockDim.x) {
        float a[8], b[8];
        unpack8(*reinterpret_cast<const uint4*>(sm + HH + t * 16), a);
        unpack8(*reinterpret_cast<const uint4*>(sm + DH + t * 16), b);
#pragma unroll
        for (int x = 0; x < 8; ++x) hh = fmaf(a[x], b[x], hh);
    }
    GDN_WAIT_MMA(21)
    if (ok) {   // P_ij = (q_i . k_j) D_ij for j <= i   (M = 64 accumulator: row i on lane (i % 16) + 32 (i / 16))
        float v[32];
        tmem_ld32(tmem + lane_base + slot(0) + half * 32, v);
        tmem_wait_ld();
        const int i = q4 * 16 + lane, j0 = half * 32;
        if (lane < 16) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (j0 + j <= i) ? v[j] * Dij(i, j0 + j) : 0.f;
            tile_store32(sm + PT, 64, i, j0, v);
        }
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();

    // ---- phase 2
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + slot(3), op_mn_major(sm + DO, 64), op_mn_major(sm + PT, 64), 128, 64, 64, false);
        mma_commit(&bar_mma);
    }
    GDN_WAIT_MMA(22)
    const int f = q4 * 32 + lane;      // feature (lane of the transposed accumulators)
    const int i0 = half * 32;          // first of this thread's 32 tokens
    float rs = 0.f;
    if (ok) {
        float u[32], t[32];
        tile_load32(sm + UTT, 128, f, i0, u);
        tmem_ld32(tmem + lane_base + slot(1) + i0, t);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) u[i] -= t[i];                       // U = U~ - W h
        tile_store32(sm + UT, 128, f, i0, u);
        float kb[32];
        tmem_ld32(tmem + lane_base + slot(2) + i0, kb);
        tmem_ld32(tmem + lane_base + slot(3) + i0, t);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float kbe = ee[i0 + i] * kb[i];
            rs = fmaf(kbe, u[i], rs);                                     // sum_j r_j
            t[i] = fmaf(sc, t[i], kbe);                                   // dU = scale P^T dO + Diag(e) K dh'
        }
        tile_store32(sm + DUT, 128, f, i0, t);
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();

    // ---- phase 3
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + slot(0), op_k_major(sm + DO, 64), op_mn_major(sm + UT, 128), 64, 64, 128, false);
        mma_tile(tmem + slot(4), op_k_major(sm + HH, 128), op_k_major(sm + DO, 64), 128, 64, 128, false);
        mma_tile(tmem + slot(5), op_k_major(sm + HH, 128), op_mn_major(sm + DUT, 128), 128, 64, 128, false, /*neg_a=*/true);
        mma_commit(&bar_mma);
    }
    GDN_WAIT_MMA(23)
    if (ok) {
        float v[32];
        tmem_ld32(tmem + lane_base + slot(0) + half * 32, v);
        tmem_wait_ld();
        const int i = q4 * 16 + lane, j0 = half * 32;
        if (lane < 16) {   // dPD = scale tril(dO U^T) . D
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (j0 + j <= i) ? sc * v[j] * Dij(i, j0 + j) : 0.f;
            tile_store32(sm + DPD, 64, i, j0, v);
        }
        tmem_ld32(tmem + lane_base + slot(5) + i0, v);
        tmem_wait_ld();
        tile_store32(sm + DWT, 128, f, i0, v);                            // dW^T = -(dU h^T)^T
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();

    // ---- phase 4
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + slot(1), op_mn_major(sm + QK, 128, 64), op_k_major(sm + DPD, 64), 128, 64, 64, false);
        mma_tile(tmem + slot(2), op_k_major(sm + DWT, 128), op_mn_major(sm + TT, 64), 128, 64, 64, false);
        mma_tile(tmem + slot(3), op_k_major(sm + DUT, 128), op_mn_major(sm + TT, 64), 128, 64, 64, false);
        mma_tile(tmem + slot(6), op_mn_major(sm + QK, 128, 0), op_mn_major(sm + DPD, 64), 128, 64, 64, false);
        mma_tile(tmem + slot(7), op_k_major(sm + DH, 128), op_mn_major(sm + UT, 128), 128, 64, 128, false);
        mma_commit(&bar_mma);
    }
    GDN_WAIT_MMA(24)
    float acc1[32];   // <q, dq> - <k, dk^col> per token, this thread's feature only
#pragma unroll
    for (int i = 0; i < 32; ++i) acc1[i] = 0.f;
    __nv_bfloat16* gdq = reinterpret_cast<__nv_bfloat16*>(p.dq) + ((size_t)tok0 * H + hd) * D + f;
    __nv_bfloat16* gdk = reinterpret_cast<__nv_bfloat16*>(p.dk) + ((size_t)tok0 * H + hd) * D + f;
    __nv_bfloat16* gdv = reinterpret_cast<__nv_bfloat16*>(p.dv) + ((size_t)tok0 * H + hd) * D + f;
    const size_t rowp = (size_t)H * D;
    if (ok) {
        float a[32], b[32];
        tmem_ld32(tmem + lane_base + slot(4) + i0, a);
        tmem_ld32(tmem + lane_base + slot(1) + i0, b);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float dq = fmaf(sc * Gam[i0 + i], a[i], b[i]);          // dq = scale Gam (dO h^T) + dPD K
            acc1[i] = tile_get(sm + QK, 128, i0 + i, f) * dq;
            if (i0 + i < len) gdq[(size_t)(i0 + i) * rowp] = __float2bfloat16_rn(dq);
        }
        tmem_ld32(tmem + lane_base + slot(2) + i0, a);
        tmem_ld32(tmem + lane_base + slot(3) + i0, b);
        tmem_wait_ld();
        tile_store32(sm + DXKT, 128, f, i0, a);
        tile_store32(sm + DXVT, 128, f, i0, b);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if (i0 + i < len) gdv[(size_t)(i0 + i) * rowp] = __float2bfloat16_rn(bb[i0 + i] * b[i]);   // dv = w dXv
            b[i] *= tile_get(sm + VT, 64, i0 + i, f);                                             // dw partial
        }
        butterfly32(b, lane);
        red1[half][q4][lane] = b[0];
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();
    if (threadIdx.x < kC) {
        const int hf = threadIdx.x >> 5, l = threadIdx.x & 31;
        dws[threadIdx.x] = (red1[hf][0][l] + red1[hf][1][l]) + (red1[hf][2][l] + red1[hf][3][l]);
    }

    // ---- phase 5
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + slot(0), op_mn_major(sm + DXKT, 128), op_mn_major(sm + WT, 128), 64, 64, 128, false);
        mma_tile(tmem + slot(0), op_mn_major(sm + DXVT, 128), op_mn_major(sm + UTT, 128), 64, 64, 128, true);
        mma_commit(&bar_mma);
    }
    GDN_WAIT_MMA(25)
    if (ok) {
        float v[32], w[32];
        tmem_ld32(tmem + lane_base + slot(0) + half * 32, v);
        tmem_wait_ld();
        const int i = q4 * 16 + lane, j0 = half * 32;
        if (lane < 16) {   // G = dA . D,  dA = -stril(dXk W^T + dXv U~^T)
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                v[j] = (j0 + j < i) ? -v[j] * Dij(i, j0 + j) : 0.f;
                w[j] = bb[i] * v[j];
            }
            tile_store32(sm + GT, 64, i, j0, v);
            tile_store32(sm + BGT, 64, i, j0, w);
        }
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();

    // ---- phase 6
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + slot(4), op_mn_major(sm + QK, 128, 64), op_k_major(sm + GT, 64), 128, 64, 64, false);
        mma_tile(tmem + slot(6), op_mn_major(sm + QK, 128, 64), op_mn_major(sm + BGT, 64), 128, 64, 64, true);
        mma_commit(&bar_mma);
    }
    GDN_WAIT_MMA(26)
    if (ok) {
        float y[32], t[32];
        tmem_ld32(tmem + lane_base + slot(4) + i0, y);
        tmem_ld32(tmem + lane_base + slot(2) + i0, t);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] = fmaf(Gam[i0 + i], t[i], y[i]);     // Y = G K + Diag(Gam) dXk ; dk^row = Diag(b) Y
        float c2[32];
        tmem_ld32(tmem + lane_base + slot(6) + i0, t);
        tmem_ld32(tmem + lane_base + slot(7) + i0, c2);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float kcol = fmaf(ee[i0 + i], c2[i], t[i]);                   // dk^col
            const float kk = tile_get(sm + QK, 128, 64 + i0 + i, f);
            if (i0 + i < len) gdk[(size_t)(i0 + i) * rowp] = __float2bfloat16_rn(fmaf(bb[i0 + i], y[i], kcol));
            acc1[i] = fmaf(-kk, kcol, acc1[i]);
            y[i] *= kk;                                                         // db partial
        }
        butterfly32(y, lane);
        butterfly32(acc1, lane);
        red2[half][q4][lane] = y[0];
        red3[half][q4][lane] = acc1[0];
    }
    // block totals of sum_j r_j and <dh', h>
    rs = warp_sum(rs);
    hh = warp_sum(hh);
    if (lane == 0) { scal[0][warp] = rs; scal[1][warp] = hh; }
    __syncthreads();
    if (threadIdx.x < kC) {
        const int i = threadIdx.x, hf = i >> 5, l = i & 31;
        const float db = (red2[hf][0][l] + red2[hf][1][l]) + (red2[hf][2][l] + red2[hf][3][l]);
        const float d1 = (red3[hf][0][l] + red3[hf][1][l]) + (red3[hf][2][l] + red3[hf][3][l]);
        if (i < len) p.dbeta[(size_t)(tok0 + i) * H + hd] = db + dws[i];
        dgam[i] = fmaf(bb[i], db, d1);
    }
    __syncthreads();
    if (threadIdx.x == 0 && ok) {
        float rsum = 0.f, hsum = 0.f;
        for (int w = 0; w < kThreads / 32; ++w) { rsum += scal[0][w]; hsum += scal[1][w]; }
        dgam[kC - 1] += rsum + Gam[kC - 1] * hsum;
        float run = 0.f;   // gam_i = sum_{j<=i} g_j  =>  dg_j = sum_{i>=j} dgam_i
        for (int i = kC - 1; i >= 0; --i) {
            run += dgam[i];
            if (i < len) p.dg[(size_t)(tok0 + i) * H + hd] = run;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
#undef GDN_WAIT_MMA
}

// ------------------------------------------------------------------------------------------------
// tc_out (optional forward output): o = scale (Diag(Gam) Q h + P (U~ - W h))
// ------------------------------------------------------------------------------------------------
namespace outk {
constexpr uint32_t QK = 0, WT = 32768, UTT = WT + 16384, HH = UTT + 16384, PT = HH + 32768, UT = PT + 8192;
constexpr uint32_t SMEM_BYTES = UT + 16384 + 1024;
}  // namespace outk

__global__ void __launch_bounds__(kThreads, 1) tc_out_kernel(const __grid_constant__ TcParams P) {
    using namespace outk;
    const Problem& p = P.p;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    const int c = blockIdx.x / p.d.H, hd = blockIdx.x % p.d.H;
    if (c >= hdr->n_chunks) return;
    const int ch = blockIdx.x;
    const int tok0 = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0)[c];
    const int len = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len)[c];
    const int H = p.d.H;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ float gam[kC];
    __shared__ uint64_t bar_in, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, half = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    if (threadIdx.x == 0) { mbar_init(&bar_in, 1); mbar_init(&bar_mma, 1); fence_mbar_init(); }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    if (threadIdx.x == 0) {
        mbar_expect_tx(&bar_in, 32768 + 16384 + 16384 + 32768);
        for (int cb = 0; cb < 2; ++cb) {
            tma_load_2d(sm + QK + cb * 16384, &P.tm_q, hd * D + cb * 64, tok0, &bar_in);
            tma_load_2d(sm + QK + cb * 16384 + 8192, &P.tm_k, hd * D + cb * 64, tok0, &bar_in);
        }
        bulk_load(sm + WT, p.ws + p.L.W + (size_t)ch * 16384, 16384, &bar_in);
        bulk_load(sm + UTT, p.ws + p.L.Ut + (size_t)ch * 16384, 16384, &bar_in);
        bulk_load(sm + HH, p.ws + p.L.hc + (size_t)ch * 32768, 32768, &bar_in);
    }
    if (threadIdx.x < kC) gam[threadIdx.x] = reinterpret_cast<const float*>(p.ws + p.L.gamma)[(size_t)ch * kC + threadIdx.x];
    bool ok = mbar_wait(&bar_in, 0);
    if (!ok && threadIdx.x == 0) report_timeout(p.ws, 30);
    if (ok && len < kC) {
        zero_tail_rows(sm + QK, 128, 0, len);
        zero_tail_rows(sm + QK, 128, 64, len);
        fence_async_smem();
    }
    __syncthreads();
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + 0, op_k_major(sm + QK, 128, 0), op_k_major(sm + QK, 128, 64), 64, 64, 128, false);
        mma_tile(tmem + 64, op_mn_major(sm + HH, 128), op_mn_major(sm + WT, 128), 128, 64, 128, false);
        mma_tile(tmem + 128, op_mn_major(sm + HH, 128), op_k_major(sm + QK, 128, 0), 128, 64, 128, false);
        mma_commit(&bar_mma);
    }
    if (ok) { ok = mbar_wait(&bar_mma, 0); if (!ok && threadIdx.x == 0) report_timeout(p.ws, 31); }
    tc_fence_after();
    const int f = q4 * 32 + lane, i0 = half * 32;
    if (ok) {
        float v[32], u[32];
        tmem_ld32(tmem + lane_base + 0 + half * 32, v);
        tmem_wait_ld();
        const int i = q4 * 16 + lane, j0 = half * 32;
        if (lane < 16) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (j0 + j <= i) ? v[j] * expf(gam[i] - gam[j0 + j]) : 0.f;
            tile_store32(sm + PT, 64, i, j0, v);
        }
        tile_load32(sm + UTT, 128, f, i0, u);
        tmem_ld32(tmem + lane_base + 64 + i0, v);
        tmem_wait_ld();
#pragma unroll
        for (int i2 = 0; i2 < 32; ++i2) u[i2] -= v[i2];
        tile_store32(sm + UT, 128, f, i0, u);
    }
    tc_fence_before();
    fence_async_smem();
    __syncthreads();
    if (ok && threadIdx.x == 0) {
        tc_fence_after();
        mma_tile(tmem + 192, op_k_major(sm + UT, 128), op_k_major(sm + PT, 64), 128, 64, 64, false);
        mma_commit(&bar_mma);
    }
    if (ok) { ok = mbar_wait(&bar_mma, 1); if (!ok && threadIdx.x == 0) report_timeout(p.ws, 32); }
    tc_fence_after();
    if (ok) {
        float a[32], b[32];
        tmem_ld32(tmem + lane_base + 128 + i0, a);
        tmem_ld32(tmem + lane_base + 192 + i0, b);
        tmem_wait_ld();
        __nv_bfloat16* go = reinterpret_cast<__nv_bfloat16*>(p.o) + ((size_t)tok0 * H + hd) * D + f;
        const float sc = p.d.scale;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i0 + i < len) go[(size_t)(i0 + i) * H * D] = __float2bfloat16_rn(sc * fmaf(expf(gam[i0 + i]), a[i], b[i]));
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
bool tc_supported(const gdn_desc& d) {
    return d.dtype == GDN_BF16 && d.d_k == 128 && d.d_v == 128 && d.delta_rule == 1 && d.chunk == kC;
}

static bool fill_params(TcParams& P, const Problem& p, bool with_bwd, int scan_dirs) {
    P.p = p;
    P.with_bwd = with_bwd ? 1 : 0;
    P.scan_dirs = scan_dirs;
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

// which: 0 = forward carry only, 1 = reverse only, 2 = both (one launch; forward and reverse CTAs interleave)
static cudaError_t launch_scan(const TcParams& P, cudaStream_t st) {
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(tc_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)scan::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    const int chains = P.p.d.N * P.p.d.H;
    if (chains > 0) {
        StageScope t(ST_SCANS, st);
        tc_scan_kernel<<<chains * (P.scan_dirs == 2 ? 4 : 2), kThreads, scan::SMEM_BYTES, st>>>(P);
    }
    return cudaGetLastError();
}

static cudaError_t launch_intra(const TcParams& P, cudaStream_t st) {
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(tc_intra_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)intra::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    const int CH = P.p.L.max_chunks * P.p.d.H;
    if (CH > 0) {
        StageScope t(ST_INTRA, st);
        tc_intra_kernel<<<CH, kThreads, intra::SMEM_BYTES, st>>>(P);
    }
    return cudaGetLastError();
}

static cudaError_t launch_out(const TcParams& P, cudaStream_t st) {
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(tc_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)outk::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    const int CH = P.p.L.max_chunks * P.p.d.H;
    if (CH > 0) {
        StageScope t(ST_OUT, st);
        tc_out_kernel<<<CH, kThreads, outk::SMEM_BYTES, st>>>(P);
    }
    return cudaGetLastError();
}

// A call with no tokens still owes the pass-through of the states.
static cudaError_t empty_call(const Problem& p, bool bwd, cudaStream_t st) {
    const size_t bytes = (size_t)p.d.N * p.d.H * D * D * sizeof(float);
    float* dst = bwd ? p.dh0 : p.hT;
    const float* src = bwd ? p.dhT : p.h0;
    if (!dst) return cudaSuccess;
    return src ? cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) : cudaMemsetAsync(dst, 0, bytes, st);
}

cudaError_t tc_launch_fwd(const Problem& p, cudaStream_t st) {
    TcParams P;
    cudaError_t e = launch_table(p, st);
    if (e != cudaSuccess) return e;
    if (p.Ttot == 0) return empty_call(p, false, st);
    if (!fill_params(P, p, false, 0)) return cudaErrorUnknown;
    if ((e = launch_prep(P, st)) != cudaSuccess) return e;
    if ((e = launch_scan(P, st)) != cudaSuccess) return e;
    return p.o ? launch_out(P, st) : cudaSuccess;
}

// With a workspace fresh from gdn_fwd_recompute the forward carry is not repeated; the chunk factors are
// rebuilt together with E, which needs dO.
cudaError_t tc_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st) {
    TcParams P;
    cudaError_t e = launch_table(p, st);
    if (e != cudaSuccess) return e;
    if (p.Ttot == 0) return empty_call(p, true, st);
    if (!fill_params(P, p, true, skip_recompute ? 1 : 2)) return cudaErrorUnknown;
    if ((e = launch_prep(P, st)) != cudaSuccess) return e;
    if ((e = launch_scan(P, st)) != cudaSuccess) return e;
    return launch_intra(P, st);
}

}  // namespace gdn
