// The chunk-local preparation of the tcgen05 d = 128 family as two small kernels (included by gdn_tc.cu).
//
//   tc_factors  needs k, v, g, beta only:  gamma, A, T = (I + A)^-1, W^T, U~^T      (the forward's share; Section 4.2)
//   tc_eprep    needs q, k, dO and W:      P = tril(Q K^T . D), E = scale (Diag(Gam) Q - P W)^T dO   (the backward's)
//
// Each holds about 105 KB of shared memory and 256 columns of tensor memory, so that two CTAs share an SM: a CTA works
// through the dependent phases of one chunk-head (product -> readout -> product ...) while its neighbour is in another
// phase of another chunk-head, which is what keeps the tensor pipe and the load/store path busy.  A trip's inputs are
// dead once its last product is done, so the next trip's are loaded right then, under the last readout and the stores
// (look-ahead without a second buffer).  A backward that consumes a workspace fresh from the
// forward runs tc_eprep alone (T, W, U~ are reused: no product, inversion or store of the forward is repeated).
// The fused tc_prep kernel remains for carries in operator form, which also need Nm and Bf.
#pragma once

namespace split {
constexpr int kT = 256;   // 8 warps: TMEM lane quadrant = warp % 4, column half = warp / 4
}

// ------------------------------------------------------------------------------------------------
// tc_factors
// ------------------------------------------------------------------------------------------------
namespace factors {
constexpr uint32_t KV = 0;                  // [K rows 0..63 ; V rows 64..127] x 128          32 KB
constexpr uint32_t XA = 32768;              // fp32 A [64][kLdi]; after the inversion the bf16 tiles T and T Diag(b Gam)
constexpr uint32_t XT = XA + 17408;         // fp32 T [64][kLdi]
constexpr uint32_t WU = XT + 17408;         // fp32 scratch of the inversion; later the staged images W^T | U~^T   32 KB
constexpr uint32_t TPP = WU + 32768;        // T Diag(w)                                       8 KB
constexpr uint32_t TT = XA, TP = XA + 8192;
constexpr uint32_t SMEM_BYTES = TPP + 8192 + 1024 /* alignment slack */;
constexpr uint32_t C_S1 = 0, C_W = 64, C_U = 128;   // TMEM columns (256 allocated)
static_assert(kLdi * kC * 4 == 17408 && 2 * 8192 <= 17408, "T tiles fit over the fp32 A block");
static_assert(2 * (SMEM_BYTES + 4096) <= 228 * 1024, "two CTAs per SM");
}  // namespace factors

__global__ void __launch_bounds__(split::kT, 2) tc_factors_kernel(const __grid_constant__ TcParams P) {
    using namespace factors;
    const Problem& p = P.p;
    const int H = p.d.H;
    init_header_if_untabled(p);
    const int n_items = n_chunks_of(p) * H;
    if ((int)blockIdx.x >= n_items) return;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ __align__(16) float gates[6][kC];   // gam log2e, Gam, e, b, w, b Gam
    __shared__ uint64_t bar_in, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, grp = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    if (threadIdx.x == 0) { mbar_init(&bar_in, 1); mbar_init(&bar_mma, 1); fence_mbar_init(); }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const float* gl = gates[0];
    const float* bb = gates[3];
    const float* ww = gates[4];
    const float* bgam = gates[5];
    float* Af = reinterpret_cast<float*>(sm + XA);
    float* Tf = reinterpret_cast<float*>(sm + XT);
    float* Sf = reinterpret_cast<float*>(sm + WU);
    bool ok = true, pending = false;
    uint32_t mma_phase = 0, in_phase = 0;
    // K and V of a trip are dead once its last product is done, so the next trip's are loaded right then, under the last
    // readout and the stores; the gate values of the next trip are fetched into registers at the same moment.
    auto issue_loads = [&](const ChunkInfo& c) {   // thread 0
        mbar_expect_tx(&bar_in, 32768);
        for (int cb = 0; cb < 2; ++cb) {
            tma_load_2d(sm + KV + cb * 16384, &P.tm_k, c.hd * D + cb * 64, c.tok0, &bar_in);
            tma_load_2d(sm + KV + cb * 16384 + 8192, &P.tm_v, c.hd * D + cb * 64, c.tok0, &bar_in);
        }
        pending = true;
    };
    float gg[2] = {0.f, 0.f}, gb[2] = {0.f, 0.f}, gw[2] = {0.f, 0.f};   // warp 0: log decay, erase gate, write gate of tokens lane, lane + 32
    auto fetch_gates = [&](const ChunkInfo& c) {   // warp 0
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = lane + 32 * h;
            gg[h] = gb[h] = gw[h] = 0.f;
            if (i < c.len) {
                const size_t idx = (size_t)(c.tok0 + i) * H + c.hd;
                gg[h] = p.g[idx];
                gb[h] = p.d.delta_rule ? p.beta[idx] : 0.f;   // delta rule off: erase 0, write 1
                gw[h] = p.d.delta_rule ? gb[h] : 1.f;
            }
        }
    };
    ChunkInfo x;
    chunk_entry(p, x, blockIdx.x);
    if (threadIdx.x == 0) issue_loads(x);
    if (warp == 0) fetch_gates(x);
#pragma unroll 1
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, in_phase ^= 1) {
        const bool has_next = item + (int)gridDim.x < n_items;
        ChunkInfo xn = x;
        if (has_next) chunk_entry(p, xn, item + gridDim.x);
        if (warp == 0) {   // gate arrays of the chunk from the values fetched a trip ahead
            float a = gg[0], b = gg[1];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float ua = __shfl_up_sync(0xffffffffu, a, o), ub = __shfl_up_sync(0xffffffffu, b, o);
                if (lane >= o) { a += ua; b += ub; }
            }
            b += __shfl_sync(0xffffffffu, a, 31);
            const float gend = __shfl_sync(0xffffffffu, b, 31);
            const float gc[2] = {a, b};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int i = lane + 32 * h;
                const float G = expf(gc[h]);
                gates[0][i] = gc[h] * kLog2e;
                gates[1][i] = G;
                gates[2][i] = expf(gend - gc[h]);
                gates[3][i] = gb[h];
                gates[4][i] = gw[h];
                gates[5][i] = gb[h] * G;
                reinterpret_cast<float*>(p.ws + p.L.gamma)[(size_t)x.ch * kC + i] = gc[h];
            }
        }
        if (ok) {
            ok = mbar_wait(&bar_in, in_phase);
            if (!ok && threadIdx.x == 0) report_timeout(p.ws, 21);
            if (ok && threadIdx.x == 0) pending = false;
        }
        if (ok && x.len < kC) {   // identity padding of a ragged tail
            zero_tail_rows(sm + KV, 128, 0, x.len, split::kT);
            zero_tail_rows(sm + KV, 128, 64, x.len, split::kT);
            fence_async_smem();
        }
        __syncthreads();
        // ---- phase 1: S1 = [K; V] K^T (rows 0..63: K K^T; the V rows ride along unused)
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 128>(tmem + C_S1, op_k_major(sm + KV, 128, 0), op_k_major(sm + KV, 128, 0), false);
            mma_commit(&bar_mma);
        }
        if (threadIdx.x == 0) bulk_wait_read<0>();   // the previous trip's stores have read their tiles (rewritten from here on)
        GDN_WAIT_MMA(22)
        __syncthreads();
        if (ok && q4 < 2) {   // A_ij = b_i (k_i . k_j) exp(gam_i - gam_j), j < i (mask before exponentiating)
            const int i = q4 * 32 + lane, j0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float v[8], g8[8];
                const int jb = j0 + part * 8;
                tmem_ld8(tmem + lane_base + C_S1 + jb, v);
                tmem_wait_ld();
                ld8s(gl + jb, g8);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = (jb + j < i) ? bb[i] * v[j] * ex2(gl[i] - g8[j]) : 0.f;
                *reinterpret_cast<float4*>(Af + i * kLdi + jb) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4*>(Af + i * kLdi + jb + 4) = make_float4(v[4], v[5], v[6], v[7]);
            }
        }
        tc_fence_before();
        __syncthreads();
        // ---- T = (I + A)^-1, blocked, fp32
        inv_diag8(Af, Tf);
        __syncthreads();
        inv_diag16(Af, Tf, Sf);
        __syncthreads();
        inv_premul<2>(Af, Tf, Sf);
        __syncthreads();
        inv_level<1, 1, 2>(Sf, Tf);
        __syncthreads();
        inv_level<2, 2, 2>(Sf, Tf);
        __syncthreads();
        inv_level<3, 4, 2>(Sf, Tf);
        __syncthreads();
        {   // T -> bf16 tiles T, T Diag(b Gam), T Diag(w): a thread scales two rows of one 8-column piece
            const int cch = threadIdx.x & 7;
            float gb8[8], gw8[8];
            ld8s(bgam + cch * 8, gb8);
            ld8s(ww + cch * 8, gw8);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int i = (threadIdx.x >> 3) + 32 * h;
                float a[8], b[8], w8[8];
                if ((cch >> 1) <= (i >> 4)) {   // blocks above the block diagonal are zero and were never written
                    ld8s(Tf + i * kLdi + cch * 8, a);
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) a[k] = 0.f;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) { b[k] = gb8[k] * a[k]; w8[k] = gw8[k] * a[k]; }
                chunk_store(sm + TT, 64, i, cch, a);
                chunk_store(sm + TP, 64, i, cch, b);
                chunk_store(sm + TPP, 64, i, cch, w8);
            }
        }
        fence_async_smem();
        __syncthreads();
        // ---- phase 2: W^T = K^T (T Diag(b Gam))^T ; U~^T = V^T (T Diag(w))^T
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 64>(tmem + C_W, op_mn_major(sm + KV, 128, 0), op_k_major(sm + TP, 64), false);
            mma_tile<128, 64, 64>(tmem + C_U, op_mn_major(sm + KV, 128, 64), op_k_major(sm + TPP, 64), false);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(23)
        if (ok && has_next) {   // K, V have been read for the last time
            if (threadIdx.x == 0) issue_loads(xn);
            if (warp == 0) fetch_gates(xn);
        }
        if (ok) {
            const int f = q4 * 32 + lane, i0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                const int ib = i0 + part * 8;
                float v[8];
                tmem_ld8(tmem + lane_base + C_W + ib, v);
                tmem_wait_ld();
                chunk_store(sm + WU, 128, f, ib >> 3, v);
                tmem_ld8(tmem + lane_base + C_U + ib, v);
                tmem_wait_ld();
                chunk_store(sm + WU + 16384, 128, f, ib >> 3, v);
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        if (ok && threadIdx.x == 0) {
            bulk_store(p.ws + p.L.Tm + (size_t)x.ch * 8192, sm + TT, 8192);
            bulk_store(p.ws + p.L.W + (size_t)x.ch * 16384, sm + WU, 16384);
            bulk_store(p.ws + p.L.Ut + (size_t)x.ch * 16384, sm + WU + 16384, 16384);
            bulk_commit();
        }
        if (!ok) break;
        x = xn;
    }
    if (threadIdx.x == 0) {
        bulk_wait_read<0>();
        if (pending) (void)mbar_wait(&bar_in, in_phase);   // after a timeout a load may still be in flight
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
}

// ------------------------------------------------------------------------------------------------
// tc_eprep
// ------------------------------------------------------------------------------------------------
namespace eprep {
constexpr uint32_t QK = 0;                  // [Q rows 0..63 ; K rows 64..127] x 128                            32 KB
constexpr uint32_t DOT = 32768;             // dO [64][128]                                    16 KB
constexpr uint32_t WT = DOT + 16384;        // W^T [128][64] (image from the workspace)         16 KB
constexpr uint32_t PT = WT + 16384;         // P = tril(Q K^T . D)                              8 KB
constexpr uint32_t RT = PT + 8192;          // R = Diag(Gam) dO [64][128]                       16 KB  (these two: finally
constexpr uint32_t PDOT = RT + 16384;       // (P^T dO)^T [128][64]                             16 KB   the staged E image)
static_assert(RT % 1024 == 0 && PDOT == RT + 16384, "the E image [128][128] is two column blocks of 16 KB");
constexpr uint32_t SMEM_BYTES = PDOT + 16384 + 1024 /* alignment slack */;
constexpr uint32_t C_S1 = 0, C_PDO = 64, C_E = 128;   // TMEM columns (256 allocated)
static_assert(2 * (SMEM_BYTES + 4096) <= 228 * 1024, "two CTAs per SM");
}  // namespace eprep

__global__ void __launch_bounds__(split::kT, 2) tc_eprep_kernel(const __grid_constant__ TcParams P) {
    using namespace eprep;
    const Problem& p = P.p;
    const int H = p.d.H;
    if (reinterpret_cast<const WsHeader*>(p.ws)->status != GDN_OK) return;
    const int n_items = n_chunks_of(p) * H;
    if ((int)blockIdx.x >= n_items) return;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ __align__(16) float gl[kC], Gam[kC];
    __shared__ uint64_t bar_in, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, grp = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    if (threadIdx.x == 0) { mbar_init(&bar_in, 1); mbar_init(&bar_mma, 1); fence_mbar_init(); }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const float sc = p.d.scale;
    bool ok = true, pending = false;
    uint32_t mma_phase = 0, in_phase = 0;
    // Q, K, dO and W of a trip are dead once its last product is done: the next trip's are loaded right then, under the
    // readout of E and its store (E is staged over R and (P^T dO)^T, which are dead by then too, not over an input).
    auto issue_loads = [&](const ChunkInfo& c) {   // thread 0
        mbar_expect_tx(&bar_in, 65536);
        for (int cb = 0; cb < 2; ++cb) {
            tma_load_2d(sm + QK + cb * 16384, &P.tm_q, c.hd * D + cb * 64, c.tok0, &bar_in);
            tma_load_2d(sm + QK + cb * 16384 + 8192, &P.tm_k, c.hd * D + cb * 64, c.tok0, &bar_in);
            tma_load_2d(sm + DOT + cb * 8192, &P.tm_do, c.hd * D + cb * 64, c.tok0, &bar_in);
        }
        bulk_load(sm + WT, p.ws + p.L.W + (size_t)c.ch * 16384, 16384, &bar_in);
        pending = true;
    };
    float gnext = 0.f;   // threads 0..63: cumulative decay of the next trip's chunk, fetched a trip ahead
    auto fetch_gamma = [&](const ChunkInfo& c) {
        if (threadIdx.x < kC) gnext = reinterpret_cast<const float*>(p.ws + p.L.gamma)[(size_t)c.ch * kC + threadIdx.x];
    };
    ChunkInfo x;
    chunk_entry(p, x, blockIdx.x);
    if (threadIdx.x == 0) issue_loads(x);
    fetch_gamma(x);
#pragma unroll 1
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, in_phase ^= 1) {
        const bool has_next = item + (int)gridDim.x < n_items;
        ChunkInfo xn = x;
        if (has_next) chunk_entry(p, xn, item + gridDim.x);
        if (threadIdx.x < kC) {   // chunk-local cumulative decay, left in the workspace by the factor stage
            gl[threadIdx.x] = gnext * kLog2e;
            Gam[threadIdx.x] = expf(gnext);
        }
        if (ok) {
            ok = mbar_wait(&bar_in, in_phase);
            if (!ok && threadIdx.x == 0) report_timeout(p.ws, 24);
            if (ok && threadIdx.x == 0) pending = false;
        }
        if (ok && x.len < kC) {   // identity padding of a ragged tail
            zero_tail_rows(sm + QK, 128, 0, x.len, split::kT);
            zero_tail_rows(sm + QK, 128, 64, x.len, split::kT);
            zero_tail_rows(sm + DOT, 64, 0, x.len, split::kT);
            fence_async_smem();
        }
        __syncthreads();
        // ---- phase 1: S1 = [Q; K] K^T (rows 0..63: Q K^T)
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 128>(tmem + C_S1, op_k_major(sm + QK, 128, 0), op_k_major(sm + QK, 128, 64), false);
            mma_commit(&bar_mma);
        }
        if (threadIdx.x == 0) bulk_wait_read<0>();   // the previous trip's stores have read P and the staged E image
        GDN_WAIT_MMA(25)
        __syncthreads();
        // R = Diag(Gam) dO: four 16-byte pieces per thread
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int i = (threadIdx.x >> 4) + 16 * it;
            float v[8];
            chunk_load(sm + DOT, 64, i, threadIdx.x & 15, v);
            const float G = Gam[i];
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] *= G;
            chunk_store(sm + RT, 64, i, threadIdx.x & 15, v);
        }
        if (ok && q4 < 2) {   // P_ij = (q_i . k_j) exp(gam_i - gam_j), j <= i (mask before exponentiating)
            const int i = q4 * 32 + lane, j0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float v[8], g8[8];
                const int jb = j0 + part * 8;
                tmem_ld8(tmem + lane_base + C_S1 + jb, v);
                tmem_wait_ld();
                ld8s(gl + jb, g8);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = (jb + j <= i) ? v[j] * ex2(gl[i] - g8[j]) : 0.f;
                chunk_store(sm + PT, 64, i, jb >> 3, v);
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        // ---- phase 2: (P^T dO)^T = dO^T P ; first half of E: Q^T R
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 64>(tmem + C_PDO, op_mn_major(sm + DOT, 64), op_mn_major(sm + PT, 64), false);
            mma_tile<128, 128, 64>(tmem + C_E, op_mn_major(sm + QK, 128, 0), op_mn_major(sm + RT, 64), false);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(26)
        if (ok) {
            const int f = q4 * 32 + lane, i0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                const int ib = i0 + part * 8;
                float v[8];
                tmem_ld8(tmem + lane_base + C_PDO + ib, v);
                tmem_wait_ld();
                chunk_store(sm + PDOT, 128, f, ib >> 3, v);
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        // ---- phase 3: E -= W^T (P^T dO)
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 128, 64>(tmem + C_E, op_k_major(sm + WT, 128), op_k_major(sm + PDOT, 128), true, /*neg_a=*/true);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(27)
        if (ok && has_next) {   // every input tile has been read for the last time
            if (threadIdx.x == 0) issue_loads(xn);
            fetch_gamma(xn);
        }
        if (ok) {   // E -> bf16 tile image over R and (P^T dO)^T, which no product reads any more
            const int r = q4 * 32 + lane, c0 = grp * 64;
#pragma unroll 1
            for (int part = 0; part < 8; ++part) {
                const int cb = c0 + part * 8;
                float v[8];
                tmem_ld8(tmem + lane_base + C_E + cb, v);
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 8; ++k) v[k] *= sc;
                chunk_store(sm + RT, 128, r, cb >> 3, v);
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        if (ok && threadIdx.x == 0) {
            bulk_store(p.ws + p.L.Pm + (size_t)x.ch * 8192, sm + PT, 8192);
            bulk_store(p.ws + p.L.E + (size_t)x.ch * 32768, sm + RT, 32768);
            bulk_commit();
        }
        if (!ok) break;
        x = xn;
    }
    if (threadIdx.x == 0) {
        bulk_wait_read<0>();
        if (pending) (void)mbar_wait(&bar_in, in_phase);   // after a timeout a load may still be in flight
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
}
