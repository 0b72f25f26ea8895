// tcgen05 / TMEM / TMA kernels of the GDN backward for bf16 I/O, d_k = d_v = 128, chunk 64 (sm_100a).
//
// Kernels follow the stage map of the chunked method (Section 4.2 of the paper):
//   tc_prep  (one CTA per chunk-head)  gamma, A, T = (I + A)^-1, W, U~, Nm = Kb^T W, Bf = Kb^T U~ and, for the
//                                      backward, E = scale (Diag(Gam) Q - P W)^T dO
//   tc_scan  (one CTA per chain and direction)
//                                      forward carry  h'  = Gam_e h  - Nm   h  + Bf   (stores h per chunk)
//                                      reverse carry  dh  = Gam_e dh' - Nm^T dh' + E   (the paper's K#1; stores dh')
//   tc_intra (one CTA per chunk-head)  every token gradient, including the VJP of the triangular solve (K#2)
//   tc_out   (optional)                forward output o
//
// All dense products run on tcgen05.mma with fp32 accumulators in tensor memory; operands are bf16 tiles in
// shared memory in the "blocked-64, 128-byte swizzle" format of tc_ptx.cuh, brought in by TMA (inputs) or by
// contiguous bulk copies of tile images (workspace).  Accumulators are produced with the feature dimension
// (128) on the TMEM lanes and the 64 tokens of the chunk on the columns, i.e. transposed, so that M = 128.
// The carried states stay fp32 in registers for the whole scan; tensor memory holds accumulators only and is
// allocated once per CTA and released once.  Every wait is bounded; a wait that gives up records
// GDN_ERR_DEVICE_TIMEOUT in the workspace header and the CTA leaves through its normal teardown.
// Loops over accumulator columns are kept rolled (8 columns per trip): the kernels run each piece of code once
// per chunk, so instruction-cache footprint matters more than loop overhead.
#include "tc_common.cuh"
#include "tc_inverse.cuh"

namespace gdn {


namespace {

constexpr int D = 128;          // d_k = d_v
constexpr int kThreads = 256;   // 8 warps: lane quadrant = warp % 4, column half = warp / 4 (scan, out)
// The chunk kernels run 16 readout warps: four warps share a TMEM lane quadrant and split the 64 token columns four
// ways, which shortens every thread's serial readout chain and gives the scheduler more warps to hide latencies with.
constexpr int kWideThreads = 512;
constexpr int kGroups = kWideThreads / 128;   // column groups
constexpr int kTG = kC / kGroups;             // token columns per group (16)
constexpr int kIntraThreads = kWideThreads + 32;   // ... plus one warp whose first lane only issues MMAs; the kernels are
                                                   // launched with one more warp on top (kIntraThreads + 32) that only
                                                   // issues bulk copies and takes no part in the named barrier
struct TcParams {
    Problem p;
    CUtensorMap tm_q, tm_k, tm_v, tm_do;   // [T_total, H * 128] bf16, boxes of 64 rows x 64 columns
    CUtensorMap tm_dq, tm_dk, tm_dv;       // same geometry, for the gradient stores of full chunks
    CUtensorMap tm_o;                      // same geometry, for the forward output (forward calls that want it)
    int with_bwd;                          // prep: also produce E
    int scan_dirs;                         // scan: 0 = forward carry only, 1 = reverse only, 2 = both
    int lowrank;                           // carries in low-rank form (tc_scan_lr): tc_prep makes no Nm, Bf
    int withhold;                          // debugging hook: tc_prep leaves out one of its first loads, so that the wait
                                           // for it runs out (exercises the time-out path without any fault)
};

// ------------------------------------------------------------------------------------------------
// tc_prep
// ------------------------------------------------------------------------------------------------
namespace prep {
// The input tiles are never reused within a trip, so the next trip's inputs are loaded into them as soon as the last
// product that reads them is done; the three output images are staged over tiles that are dead by then.
constexpr uint32_t QK = 0;                    // [Q rows 0..63 ; K rows 64..127] x 128   32 KB
constexpr uint32_t VO = 32768;                // [V ; dO] x 128                           32 KB
constexpr uint32_t TT = 65536;                // T                      [64][64]           8 KB  (these four: finally
constexpr uint32_t TP = TT + 8192;            // T Diag(b Gam)                                    the Nm image)
constexpr uint32_t TPP = TP + 8192;           // T Diag(w)
constexpr uint32_t PT = TPP + 8192;           // P = tril(Q K^T . D)
constexpr uint32_t WT = PT + 8192;            // W^T   [128 dk][64 tokens]                16 KB (before: fp32 scratch S)
constexpr uint32_t UTT = WT + 16384;          // U~^T  [128 dv][64]
constexpr uint32_t WET = UTT + 16384;         // (Diag(e) W)^T                                    (these two: finally
constexpr uint32_t UET = WET + 16384;         // (Diag(e) U~)^T                                   the Bf image)
constexpr uint32_t X = UET + 16384;           // fp32 A and T during the inversion; then R = Diag(Gam) dO and
constexpr uint32_t XA = X, XT = X + 17408;    // (P^T dO)^T; finally the E image
constexpr uint32_t XR = X, XPDO = X + 16384;
constexpr uint32_t NMS = TT, BFS = WET, ES = X;   // staging of the three output images
constexpr uint32_t TILES_END = X + 34816;
constexpr uint32_t SMEM_BYTES = TILES_END + 1024 /* alignment slack */;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
// TMEM columns (512 allocated): accumulators at fixed offsets, allocated once, released once.
constexpr uint32_t C_S1 = 0, C_W = 64, C_U = 128, C_PDO = 192, C_NM = 256, C_BF = 384, C_E = 0;
constexpr uint32_t C_E_LR = 256;   // low-rank mode (no Nm, Bf): E is started early, in columns of its own
}  // namespace prep

__global__ void __launch_bounds__(kIntraThreads + 32, 1) tc_prep_kernel(const __grid_constant__ TcParams P) {
    using namespace prep;
    const Problem& p = P.p;
    // Persistent: a CTA walks over chunk-heads blockIdx.x, blockIdx.x + gridDim.x, ...; the inputs of its next one
    // are loaded while it works on the current one.
    const int H = p.d.H;
    init_header_if_untabled(p);
    const int n_items = n_chunks_of(p) * H;
    if ((int)blockIdx.x >= n_items) return;
    const bool bwd = P.with_bwd != 0;
    const bool opform = P.lowrank == 0;   // the carries want the chunk operator Nm and the additive term Bf

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    // gate arrays, two sets: a trip's set is written during the trip before it
    __shared__ __align__(16) float gate_sets[2][6][kC];
    __shared__ uint64_t bar_qk, bar_vo, bar_ld0, bar_t, bar_vofree, bar_ld1, bar_st, bar_tfree, bar_free1, bar_free2, bar_free, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, grp = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    const bool worker = warp < 16;                       // warps 0..15 read accumulators and do the fp32 work
    const bool issuer = threadIdx.x == kWideThreads;     // first lane of warp 16 feeds the tensor pipe
    // Warp 17 only moves data: its first lane issues the bulk stores of a trip's results and the loads of the next
    // trip's inputs (each such instruction costs its issuer hundreds of cycles).  It follows the other warps through
    // mbarriers and shares no block-wide barrier with them inside the loop (they use a named barrier).
    const bool loader = warp == 17;

    if (threadIdx.x == 0) {
        mbar_init(&bar_qk, 1); mbar_init(&bar_vo, 1); mbar_init(&bar_ld0, 1); mbar_init(&bar_t, 1);
        mbar_init(&bar_vofree, 1); mbar_init(&bar_ld1, 1); mbar_init(&bar_st, 1); mbar_init(&bar_tfree, 1);
        mbar_init(&bar_free1, 1); mbar_init(&bar_free2, 1); mbar_init(&bar_free, 1); mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    bool ok = true;
    const uint32_t VO_BYTES = bwd ? 32768 : 16384;
    auto load_piece = [&](int piece, const ChunkInfo& c) {   // 0,1: Q  2,3: K  4,5: V  6,7: dO   (column halves)
        const int cb = piece & 1, xq = c.hd * D + cb * 64;
        switch (piece >> 1) {
            case 0: tma_load_2d(sm + QK + cb * 16384, &P.tm_q, xq, c.tok0, &bar_qk); break;
            case 1: tma_load_2d(sm + QK + cb * 16384 + 8192, &P.tm_k, xq, c.tok0, &bar_qk); break;
            case 2: tma_load_2d(sm + VO + cb * 16384, &P.tm_v, xq, c.tok0, &bar_vo); break;
            case 3: if (bwd) tma_load_2d(sm + VO + cb * 16384 + 8192, &P.tm_do, xq, c.tok0, &bar_vo); break;
            default: break;
        }
    };

    if (loader) {
        if (lane == 0) {
            uint32_t ph = 0;
            bool lok = true, pend_qk = false, pend_vo = false;
#pragma unroll 1
            for (int item = blockIdx.x; item < n_items && lok; item += gridDim.x, ph ^= 1) {
                ChunkInfo x, nx;
                chunk_entry(p, x, item);
                const bool has_next = item + (int)gridDim.x < n_items;
                if (has_next) chunk_entry(p, nx, item + gridDim.x);
                pend_qk = pend_vo = false;
                // the trip is under way: the inputs of the next one (loaded late in this trip) -> L2
                if (!(lok = mbar_wait(&bar_ld0, ph))) break;
                if (has_next) {
                    for (int cb = 0; cb < 2; ++cb) {
                        prefetch_l2_tma_2d(&P.tm_v, nx.hd * D + cb * 64, nx.tok0);
                        if (bwd) prefetch_l2_tma_2d(&P.tm_do, nx.hd * D + cb * 64, nx.tok0);
                    }
                    for (int cb = 0; cb < 2; ++cb) {
                        prefetch_l2_tma_2d(&P.tm_q, nx.hd * D + cb * 64, nx.tok0);
                        prefetch_l2_tma_2d(&P.tm_k, nx.hd * D + cb * 64, nx.tok0);
                    }
                }
                // T is staged
                if (!(lok = mbar_wait(&bar_t, ph))) break;
                bulk_store(p.ws + p.L.Tm + (size_t)x.ch * 8192, sm + TT, 8192);
                if (bwd) bulk_store(p.ws + p.L.Pm + (size_t)x.ch * 8192, sm + PT, 8192);   // the gradient stage reads P from here
                bulk_commit();
                if (!opform) {   // low-rank mode: Q, K are dead after phase 2, before W^T, U~^T are staged
                    if (!(lok = mbar_wait(&bar_ld1, ph))) break;
                    if (has_next) {
                        mbar_expect_tx(&bar_qk, 32768);
                        pend_qk = true;
#pragma unroll 1
                        for (int piece = 0; piece < 4; ++piece) load_piece(piece, nx);
                    }
                }
                // W^T, U~^T are staged and V, dO have been read for the last time
                if (!(lok = mbar_wait(&bar_vofree, ph))) break;
                bulk_wait_read<0>();
                mbar_arrive(&bar_tfree);   // the T tile may be overwritten (by the staged Nm image)
                if (has_next) {            // (the loads first: the next trip starts with them, the stores have time)
                    mbar_expect_tx(&bar_vo, VO_BYTES);
                    pend_vo = true;
#pragma unroll 1
                    for (int piece = 4; piece < 8; ++piece) load_piece(piece, nx);
                }
                bulk_store(p.ws + p.L.W + (size_t)x.ch * 16384, sm + WT, 16384);
                bulk_store(p.ws + p.L.Ut + (size_t)x.ch * 16384, sm + UTT, 16384);
                bulk_commit();
                // phase 3 is done: Q, K have been read for the last time
                if (opform && !(lok = mbar_wait(&bar_ld1, ph))) break;
                if (opform && has_next) {
                    mbar_expect_tx(&bar_qk, 32768);
                    pend_qk = true;
#pragma unroll 1
                    for (int piece = 0; piece < 4; ++piece) {
                        load_piece(piece, nx);
                    }
                }
                // the three images are staged.  All CTAs store at about the same time, so the 96 KB drain at the rate of
                // HBM (some 22 bytes per cycle and SM); they leave in the order in which the next trip rewrites their
                // tiles: first the bytes under the fp32 A block (head of the E image) and under P (tail of the Nm image),
                // then those under the fp32 T block (rest of E), last what the T tiles and the second readout overwrite
                if (!(lok = mbar_wait(&bar_st, ph))) break;
                constexpr uint32_t A_BYTES = XT - XA;
                if (bwd) bulk_store(p.ws + p.L.E + (size_t)x.ch * 32768, sm + ES, A_BYTES);
                if (opform) bulk_store(p.ws + p.L.Nm + (size_t)x.ch * 32768 + (PT - TT), sm + NMS + (PT - TT), 8192);
                bulk_commit();
                if (bwd) bulk_store(p.ws + p.L.E + (size_t)x.ch * 32768 + A_BYTES, sm + ES + A_BYTES, 32768 - A_BYTES);
                bulk_commit();
                bulk_wait_read<1>();       // (issuing a store takes hundreds of cycles: the first group has drained by now)
                mbar_arrive(&bar_free1);   // the fp32 A block and P may be written (and the scratch over W^T: its store is older)
                if (opform) {
                    bulk_store(p.ws + p.L.Nm + (size_t)x.ch * 32768, sm + NMS, PT - TT);
                    bulk_store(p.ws + p.L.Bf + (size_t)x.ch * 32768, sm + BFS, 32768);
                }
                bulk_commit();
                bulk_wait_read<1>();
                mbar_arrive(&bar_free2);   // the fp32 T block may be written
                bulk_wait_read<0>();
                mbar_arrive(&bar_free);    // every staging tile may be rewritten
            }
            bulk_wait_read<0>();
            if (!lok) {   // after a timeout a copy may still be in flight: wait for it before the CTA may retire
                if (pend_qk) (void)mbar_wait(&bar_qk, ph ^ 1);
                if (pend_vo) (void)mbar_wait(&bar_vo, ph ^ 1);
            }
        }
        return;
    }

    auto cta_sync = [] { asm volatile("bar.sync 1, %0;" ::"n"(kIntraThreads) : "memory"); };   // all warps but the loader
    uint32_t mma_phase = 0, in_phase = 0;
    // The chunk table entry and the gate values of a trip are fetched one trip ahead into registers: they are tiny, but
    // read at the top of a trip their DRAM latency would be fully exposed.
    ChunkInfo xn;
    chunk_entry(p, xn, blockIdx.x);
    // Warp 0 owns the gates: lane l holds g (0 when padded) and the erase gate b of tokens l and l + 32.
    float ng[2] = {0.f, 0.f}, nb[2] = {0.f, 0.f};
    auto fetch_gates = [&](const ChunkInfo& c) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = lane + 32 * h;
            ng[h] = nb[h] = 0.f;
            if (i < c.len) {
                const size_t idx = (size_t)(c.tok0 + i) * H + c.hd;
                ng[h] = p.g[idx];
                if (p.d.delta_rule) nb[h] = p.beta[idx];   // delta rule off: erase gate 0 (T = I, W = 0 fall out of the same products)
            }
        }
    };
    // Warp 0 turns the fetched values into the gate arrays of chunk-head `ch` (set `set`): erase gate b, write gate w,
    // chunk-local cumulative decay gam (inclusive prefix sum of the 64 log decays), in registers.
    auto make_gates = [&](int set, int ch) {
        float a = ng[0], b = ng[1];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float ua = __shfl_up_sync(0xffffffffu, a, o), ub = __shfl_up_sync(0xffffffffu, b, o);
            if (lane >= o) { a += ua; b += ub; }
        }
        b += __shfl_sync(0xffffffffu, a, 31);
        const float gend = __shfl_sync(0xffffffffu, b, 31);
        const float gc[2] = {a, b};
        float (*gs)[kC] = gate_sets[set];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = lane + 32 * h;
            const float G = expf(gc[h]);
            gs[0][i] = gc[h] * kLog2e;
            gs[1][i] = G;
            gs[2][i] = expf(gend - gc[h]);
            gs[3][i] = nb[h];
            gs[4][i] = p.d.delta_rule ? nb[h] : (i < xn.len ? 1.f : 0.f);   // write gate (delta rule off: 1)
            gs[5][i] = nb[h] * G;
            reinterpret_cast<float*>(p.ws + p.L.gamma)[(size_t)ch * kC + i] = gc[h];
        }
    };
    if (warp == 0) { fetch_gates(xn); make_gates(0, xn.ch); }
    // first trip: the inputs are loaded at once, one instruction per warp
    if (issuer) { mbar_expect_tx(&bar_qk, 32768); mbar_expect_tx(&bar_vo, VO_BYTES); }
    if (lane == 0 && warp < 8 && !(P.withhold && warp == 0)) load_piece(warp, xn);
#pragma unroll 1
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, in_phase ^= 1) {
    const ChunkInfo x = xn;
    const bool has_next = item + (int)gridDim.x < n_items;
    const bool first = item == (int)blockIdx.x;
    if (has_next) chunk_entry(p, xn, item + gridDim.x);

    // this trip's gate arrays (written by warp 0 during the previous trip; the barrier before phase 1 publishes them)
    const float* gl = gate_sets[in_phase][0];
    const float* Gam = gate_sets[in_phase][1];
    const float* ee = gate_sets[in_phase][2];
    const float* bb = gate_sets[in_phase][3];
    const float* ww = gate_sets[in_phase][4];
    const float* bgam = gate_sets[in_phase][5];
    if (ok) {
        ok = mbar_wait(&bar_vo, in_phase);
        ok = ok && mbar_wait(&bar_qk, in_phase);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 1);
    }
    if (ok && x.len < kC) {   // identity padding of a ragged tail: rows beyond the sequence read as zero
        zero_tail_rows(sm + QK, 128, 0, x.len, kIntraThreads);
        zero_tail_rows(sm + QK, 128, 64, x.len, kIntraThreads);
        zero_tail_rows(sm + VO, 128, 0, x.len, kIntraThreads);
        if (bwd) zero_tail_rows(sm + VO, 128, 64, x.len, kIntraThreads);
        fence_async_smem();
    }
    cta_sync();

    // ---- phase 1: S1 = [Q; K] K^T  (rows 0..63: Q K^T, rows 64..127: K K^T)
    if (ok && issuer) {
        tc_fence_after();
        mma_tile<128, 64, 128>(tmem + C_S1, op_k_major(sm + QK, 128, 0), op_k_major(sm + QK, 128, 64), false);
        mma_commit(&bar_mma);
    }
    if (threadIdx.x == 32) mbar_arrive(&bar_ld0);   // this trip's inputs have arrived
    float* Af = reinterpret_cast<float*>(sm + XA);   // [64][kLdi]  strictly lower part of I + A
    float* Tf = reinterpret_cast<float*>(sm + XT);   // [64][kLdi]  T
    float* Sf = reinterpret_cast<float*>(sm + WT);   // [64][kLdi]  scratch of the blocked inversion
    if (has_next && warp == 0) fetch_gates(xn);   // next trip's gates -> registers while the product runs
    // R = Diag(Gam) dO (token-major tile) while the product runs.  In low-rank mode the tiles of Diag(e) W and
    // Diag(e) U~ are never written, so R has a tile of its own from here on and Q^T R can run under the inversion.
    auto form_R = [&](unsigned char* dst) {   // the 512 worker threads, two 16-byte pieces each (both loads in flight)
        if (worker) {
            float v[2][8];
#pragma unroll
            for (int it = 0; it < 2; ++it) chunk_load(sm + VO, 128, 64 + (threadIdx.x >> 4) + 32 * it, threadIdx.x & 15, v[it]);
#pragma unroll
            for (int it = 0; it < 2; ++it) {
                const int i = (threadIdx.x >> 4) + 32 * it;
                const float G = Gam[i];
#pragma unroll
                for (int k = 0; k < 8; ++k) v[it][k] *= G;
                chunk_store(dst, 64, i, threadIdx.x & 15, v[it]);
            }
        }
    };
    if (bwd && !opform) form_R(sm + WET);
    GDN_WAIT_MMA(2)
    if (ok && !first) {   // the previous trip's stores have read what lies under the fp32 A block and under P
        ok = mbar_wait(&bar_free1, in_phase ^ 1);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 6);
    }
    if (ok && worker) {
        const int i = (q4 & 1) * 32 + lane, j0 = grp * kTG;
#pragma unroll 1
        for (int part = 0; part < kTG / 8; ++part) {
            float v[8];
            tmem_ld8(tmem + lane_base + C_S1 + j0 + part * 8, v);
            tmem_wait_ld();
            const int jb = j0 + part * 8;
            if (q4 < 2) {   // P_ij = (q_i . k_j) exp(gam_i - gam_j), j <= i (mask before exponentiating)
                float g8[8];
                ld8s(gl + jb, g8);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = (jb + j <= i) ? v[j] * ex2(gl[i] - g8[j]) : 0.f;
                chunk_store(sm + PT, 64, i, jb >> 3, v);
            } else {        // A_ij = b_i (k_i . k_j) exp(gam_i - gam_j), j < i
                float g8[8];
                ld8s(gl + jb, g8);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = (jb + j < i) ? bb[i] * v[j] * ex2(gl[i] - g8[j]) : 0.f;
                *reinterpret_cast<float4*>(Af + i * kLdi + jb) = make_float4(v[0], v[1], v[2], v[3]);
                *reinterpret_cast<float4*>(Af + i * kLdi + jb + 4) = make_float4(v[4], v[5], v[6], v[7]);
            }
        }
    }
    tc_fence_before();
    fence_async_smem();
    cta_sync();
    // (P^T dO)^T = dO^T P needs nothing of the inversion: it runs under it and is covered by phase 2's commit
    if (ok && issuer && bwd) {
        tc_fence_after();
        mma_tile<128, 64, 64>(tmem + C_PDO, op_mn_major(sm + VO, 128, 64), op_mn_major(sm + PT, 64), false);
        // low-rank mode: so does the first half of E = Q^T R - W^T (P^T dO), into columns no other product uses
        if (!opform) mma_tile<128, 128, 64>(tmem + C_E_LR, op_mn_major(sm + QK, 128, 0), op_mn_major(sm + WET, 64), false);
    }
    // ---- T = (I + A)^-1, blocked (see inv_diag8 ... inv_level).  All fp32.
    if (ok && !first) {   // ... and what lies under the fp32 T block
        ok = mbar_wait(&bar_free2, in_phase ^ 1);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 8);
    }
    inv_diag8(Af, Tf);
    cta_sync();
    inv_diag16(Af, Tf, Sf);
    cta_sync();
    inv_premul<2>(Af, Tf, Sf);   // Sf <- T_rr A_rk for every block below the diagonal
    cta_sync();
    inv_level<1, 1, 2>(Sf, Tf);
    cta_sync();
    inv_level<2, 2, 2>(Sf, Tf);
    cta_sync();
    inv_level<3, 4, 2>(Sf, Tf);
    cta_sync();
    if (ok && !first) {   // every store of the previous trip has read its tile (the T tiles and the second readout are next)
        ok = mbar_wait(&bar_free, in_phase ^ 1);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 5);
    }
    if (threadIdx.x < kC * 4) {   // T -> bf16 tiles T, T Diag(b Gam), T Diag(w): a thread scales two rows of one 8-column piece
        const int cch = threadIdx.x & 7;
        float gb[8], gw[8];
        *reinterpret_cast<float4*>(gb) = *reinterpret_cast<const float4*>(bgam + cch * 8);
        *reinterpret_cast<float4*>(gb + 4) = *reinterpret_cast<const float4*>(bgam + cch * 8 + 4);
        *reinterpret_cast<float4*>(gw) = *reinterpret_cast<const float4*>(ww + cch * 8);
        *reinterpret_cast<float4*>(gw + 4) = *reinterpret_cast<const float4*>(ww + cch * 8 + 4);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = (threadIdx.x >> 3) + 32 * h;
            float a[8], b[8], w8[8];
            if ((cch >> 1) <= (i >> 4)) {   // the blocks above the block diagonal are zero and were never written
                *reinterpret_cast<float4*>(a) = *reinterpret_cast<const float4*>(Tf + i * kLdi + cch * 8);
                *reinterpret_cast<float4*>(a + 4) = *reinterpret_cast<const float4*>(Tf + i * kLdi + cch * 8 + 4);
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) a[k] = 0.f;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) { b[k] = gb[k] * a[k]; w8[k] = gw[k] * a[k]; }
            chunk_store(sm + TT, 64, i, cch, a);
            chunk_store(sm + TP, 64, i, cch, b);
            chunk_store(sm + TPP, 64, i, cch, w8);
        }
    }
    fence_async_smem();
    cta_sync();

    // ---- phase 2: W^T = K^T (T Diag(b Gam))^T ; U~^T = V^T (T Diag(w))^T
    if (ok && issuer) {
        tc_fence_after();
        mma_tile<128, 64, 64>(tmem + C_W, op_mn_major(sm + QK, 128, 64), op_k_major(sm + TP, 64), false);
        mma_tile<128, 64, 64>(tmem + C_U, op_mn_major(sm + VO, 128, 0), op_k_major(sm + TPP, 64), false);
        mma_commit(&bar_mma);
        if (!opform) mma_commit(&bar_ld1);   // low-rank mode: Q, K have been read for the last time
    }
    if (threadIdx.x == 32) mbar_arrive(&bar_t);   // the loader stores the T tile
    // operator mode: R while the MMAs run, over the fp32 A / T scratch, which is dead by now
    if (bwd && opform) form_R(sm + XR);
    GDN_WAIT_MMA(3)
    if (ok && worker) {
        const int f = q4 * 32 + lane, i0 = grp * kTG;
#pragma unroll 1
        for (int part = 0; part < kTG / 8; ++part) {
            const int ib = i0 + part * 8;
            float v[8], ve[8];
            tmem_ld8(tmem + lane_base + C_W + ib, v);
            tmem_wait_ld();
            float e8[8];
            ld8s(ee + ib, e8);
#pragma unroll
            for (int i = 0; i < 8; ++i) ve[i] = v[i] * e8[i];
            chunk_store(sm + WT, 128, f, ib >> 3, v);
            if (opform) chunk_store(sm + WET, 128, f, ib >> 3, ve);
            tmem_ld8(tmem + lane_base + C_U + ib, v);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 8; ++i) ve[i] = v[i] * e8[i];
            chunk_store(sm + UTT, 128, f, ib >> 3, v);
            if (opform) chunk_store(sm + UET, 128, f, ib >> 3, ve);
            if (bwd) {
                tmem_ld8(tmem + lane_base + C_PDO + ib, v);
                tmem_wait_ld();
                chunk_store(sm + XPDO, 128, f, ib >> 3, v);
            }
        }
    }
    tc_fence_before();
    fence_async_smem();
    cta_sync();

    // ---- phase 3: Nm = K^T (Diag(e) W) ; Bf = K^T (Diag(e) U~) ; E = Q^T R - W^T (P^T dO)
    if (ok && issuer) {
        tc_fence_after();
        // Nm and Bf share the operand K^T; their other operands and their accumulators are neighbours: one N = 256 product
        static_assert(UET == WET + 16384 && C_BF == C_NM + 128, "Nm | Bf as one product");
        if (opform) mma_tile<128, 256, 64>(tmem + C_NM, op_mn_major(sm + QK, 128, 64), op_k_major(sm + WET, 128), false);
        if (bwd && opform) mma_tile<128, 128, 64>(tmem + C_E, op_mn_major(sm + QK, 128, 0), op_mn_major(sm + XR, 64), false);
        if (bwd) mma_tile<128, 128, 64>(tmem + (opform ? C_E : C_E_LR), op_k_major(sm + WT, 128), op_k_major(sm + XPDO, 128), true, /*neg_a=*/true);
        mma_commit(&bar_mma);
        if (opform) mma_commit(&bar_ld1);   // Q, K have been read for the last time
    } else if (threadIdx.x == 32) {
        mbar_arrive(&bar_vofree);   // W^T, U~^T are staged; V, dO were last read by phase 2 and the pass that formed R
    }
    if (has_next && warp == 0) make_gates(in_phase ^ 1, xn.ch);   // the next trip's gate arrays, while the products run
    GDN_WAIT_MMA(4)
    if (ok) {   // the T tile, part of the Nm staging area, has left through its store
        ok = mbar_wait(&bar_tfree, in_phase);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 7);
    }
    if (ok && worker) {   // Nm, Bf, E -> bf16 tile images staged over tiles that no MMA reads any more
        const int r = q4 * 32 + lane, c0 = grp * (D / kGroups);
        const float sc = p.d.scale;
#pragma unroll 1
        for (int part = 0; part < D / kGroups / 8; ++part) {
            const int cb = c0 + part * 8;
            float v[8];
            if (opform) {
                tmem_ld8(tmem + lane_base + C_NM + cb, v);
                tmem_wait_ld();
                chunk_store(sm + NMS, 128, r, cb >> 3, v);
                tmem_ld8(tmem + lane_base + C_BF + cb, v);
                tmem_wait_ld();
                chunk_store(sm + BFS, 128, r, cb >> 3, v);
            }
            if (bwd) {
                tmem_ld8(tmem + lane_base + (opform ? C_E : C_E_LR) + cb, v);
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 8; ++k) v[k] *= sc;
                chunk_store(sm + ES, 128, r, cb >> 3, v);
            }
        }
    }
    tc_fence_before();
    fence_async_smem();
    cta_sync();
    if (threadIdx.x == 32) mbar_arrive(&bar_st);   // the three images are staged: the loader stores them
    if (!ok) break;
    }
    if (warp == 0) tmem_dealloc(tmem, 512);
}

#include "tc_prep_split.cuh"

// ------------------------------------------------------------------------------------------------
// tc_scan: forward and reverse inter-chunk carries, one CTA per (chain, direction).
// Per chunk: the fp32 state (registers; thread = one row, 64 columns) is rounded to a bf16 tile, one tcgen05.mma
// forms Nm h (forward) or Nm^T dh (reverse), and the state is updated in fp32:  s <- Gam_e s - (Nm s) + add.
// The bf16 tile that fed the MMA is also what the chunk's gradient stage needs, so each thread writes its part
// of the tile image to the workspace as well.  Nm and the additive term (Bf or E) arrive through a two-stage
// ring of bulk copies; the chunk decays exp(gamma_e) are fetched once per chain.
// ------------------------------------------------------------------------------------------------
namespace scan {
constexpr int GE_CAP = 2048;                     // chunk decays cached per chain (longer chains read them from global)
constexpr uint32_t NM = 0, ADD = 32768;          // ring stage: Nm tile image (32 KB) + the CTA's columns of the additive image
// S = number of CTAs that share a chain, each carrying 128 / S state columns (the columns of the state evolve
// independently).  S = 2 is used when there are too few chains to fill the machine.
template <int S> struct Cfg {
    static constexpr int NS = D / S;                         // state columns of this CTA
    static constexpr int STAGES = S == 1 ? 2 : 3;
    static constexpr int PREFETCH_AHEAD = STAGES + 1;        // steps by which L2 prefetches run ahead of the ring loads
    static constexpr uint32_t ADD_BYTES = 32768 / S, STAGE_BYTES = 32768 + ADD_BYTES;
    static constexpr uint32_t HT = STAGES * STAGE_BYTES;     // two state tiles [128][NS] (one feeds the MMA and the bulk
    static constexpr uint32_t HT_BYTES = 32768 / S;          // store of this step while the next step's is being written)
    static constexpr uint32_t SMEM_BYTES = HT + 2 * HT_BYTES + 1024;
    static_assert(SMEM_BYTES + GE_CAP * 4 <= 227 * 1024, "shared memory budget");
};
}  // namespace scan

template <int S>
__global__ void __launch_bounds__(kThreads, 1) tc_scan_kernel(const __grid_constant__ TcParams P) {
    using namespace scan;
    using C = Cfg<S>;
    constexpr int NS = C::NS, NSH = NS / 2, STAGES = C::STAGES, PREFETCH_AHEAD = C::PREFETCH_AHEAD;
    constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES, ADD_BYTES = C::ADD_BYTES, HT = C::HT, HT_BYTES = C::HT_BYTES;
    const int part = (int)blockIdx.x % S, bid = (int)blockIdx.x / S;   // column block of the state, (chain, direction)
    const Problem& p = P.p;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    if (hdr->status != GDN_OK) return;
    const int reverse = P.scan_dirs == 2 ? (bid & 1) : P.scan_dirs;
    const int chain = P.scan_dirs == 2 ? (bid >> 1) : bid;
    const int n = chain / p.d.H, hd = chain % p.d.H;
    const int c0 = seq_first_chunk(p, n), c1 = seq_first_chunk(p, n + 1), nsteps = c1 - c0;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ float ge[GE_CAP];
    __shared__ uint64_t bar_full[STAGES], bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, hf = warp >> 2;
    const int r = q4 * 32 + lane;              // state row owned by this thread
    const int lc0 = hf * NSH;                  // first of its NSH columns inside the CTA's block
    const int gc0 = part * NS + lc0;           // ... and inside the state
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&bar_full[s], 1);
        mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, NS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    auto chunk_of = [&](int s) { return reverse ? (c1 - 1 - s) : (c0 + s); };
    const char* nm_base = p.ws + p.L.Nm;
    const char* add_base = p.ws + (reverse ? p.L.E : p.L.Bf) + part * ADD_BYTES;
    char* keep_base = p.ws + (reverse ? p.L.dhn : p.L.hc) + part * HT_BYTES;
    const float* gamma = reinterpret_cast<const float*>(p.ws + p.L.gamma);
    auto fill = [&](int s) {   // thread 0: bring chunk step s into ring slot s % STAGES
        const int stage = s % STAGES;
        const size_t ch = (size_t)chunk_of(s) * p.d.H + hd;
        mbar_expect_tx(&bar_full[stage], STAGE_BYTES);
        bulk_load(sm + stage * STAGE_BYTES + NM, nm_base + ch * 32768, 32768, &bar_full[stage]);
        bulk_load(sm + stage * STAGE_BYTES + ADD, add_base + ch * 32768, ADD_BYTES, &bar_full[stage]);
        // The ring gives a load one step of lead, less than an HBM round trip; pull the step after next into L2 now.
        if (s + PREFETCH_AHEAD < nsteps) {
            const size_t chn = (size_t)chunk_of(s + PREFETCH_AHEAD) * p.d.H + hd;
            prefetch_l2_bulk(nm_base + chn * 32768, 32768);
            prefetch_l2_bulk(add_base + chn * 32768, ADD_BYTES);
        }
    };
    if (threadIdx.x == 32) {
        for (int s = STAGES; s < STAGES + PREFETCH_AHEAD && s < nsteps; ++s) {
            const size_t chn = (size_t)chunk_of(s) * p.d.H + hd;
            prefetch_l2_bulk(nm_base + chn * 32768, 32768);
            prefetch_l2_bulk(add_base + chn * 32768, ADD_BYTES);
        }
        for (int s = 0; s < STAGES && s < nsteps; ++s) fill(s);
    }
    for (int s = threadIdx.x; s < nsteps && s < GE_CAP; s += blockDim.x)
        ge[s] = expf(gamma[((size_t)chunk_of(s) * p.d.H + hd) * kC + kC - 1]);
    // initial state
    float st[NSH];
    {
        const float* init = reverse ? p.dhT : p.h0;
        const size_t soff = ((size_t)n * p.d.H + hd) * D * D + (size_t)r * D + gc0;
#pragma unroll
        for (int k = 0; k < NSH / 4; ++k) {
            float4 v = init ? *reinterpret_cast<const float4*>(init + soff + 4 * k) : make_float4(0.f, 0.f, 0.f, 0.f);
            st[4 * k] = v.x; st[4 * k + 1] = v.y; st[4 * k + 2] = v.z; st[4 * k + 3] = v.w;
        }
    }
    __syncthreads();
    bool ok = true;
    uint32_t mma_phase = 0;
#pragma unroll 1
    for (int s = 0; s < nsteps; ++s) {
        unsigned char* Ht = sm + HT + (s & 1) * HT_BYTES;
        const size_t ch = (size_t)chunk_of(s) * p.d.H + hd;
        const int stage = s % STAGES;
        const unsigned char* ring = sm + stage * STAGE_BYTES;
        const float Ge = s < GE_CAP ? ge[s] : expf(gamma[ch * kC + kC - 1]);
        // state -> bf16: operand tile of the MMA; the same bytes are the per-chunk state the gradient stage reads
#pragma unroll
        for (int k = 0; k < NSH / 8; ++k) *reinterpret_cast<uint4*>(Ht + tile_chunk_off(128, r, (lc0 >> 3) + k)) = pack8(st + 8 * k);
        fence_async_smem();
        __syncthreads();
        if (threadIdx.x == 0) {
            ok = mbar_wait(&bar_full[stage], (s / STAGES) & 1);
            if (ok) {
                tc_fence_after();
                const Operand a = reverse ? op_mn_major(ring + NM, 128) : op_k_major(ring + NM, 128);
                mma_tile<128, NS, 128>(tmem, a, op_mn_major(Ht, 128), false);
            } else {
                report_timeout(p.ws, 10);
            }
            // The tile leaves through the async proxy: generic global stores here would stall the next step's proxy
            // fence until they drain.  Waiting for the previous step's store to have read its tile before committing the
            // MMA orders that read before the overwrite of the tile two steps later.
            bulk_store(keep_base + ch * 32768, Ht, HT_BYTES);
            bulk_commit();
            bulk_wait_read<1>();
            mma_commit(&bar_mma);
        } else if (threadIdx.x == 32) {
            // every thread has finished step s - 1, so its ring slot can take step s - 1 + STAGES.  Bulk copies are slow
            // to issue; a thread of another warp does it so that the MMA issue is not delayed.
            if (s >= 1 && s - 1 + STAGES < nsteps) fill(s - 1 + STAGES);
        }
        ok = mbar_wait(&bar_full[stage], (s / STAGES) & 1);   // the additive term of this step is in shared memory
        if (ok) ok = mbar_wait(&bar_mma, mma_phase);
        mma_phase ^= 1;
        if (!ok) { if (threadIdx.x == 0) report_timeout(p.ws, 11); break; }
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < NSH / 8; ++k) {
            float dl[8], ad[8];
            tmem_ld8(tmem + lane_base + lc0 + 8 * k, dl);
            chunk_load(ring + ADD, 128, r, (lc0 >> 3) + k, ad);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) st[8 * k + j] = fmaf(Ge, st[8 * k + j], ad[j] - dl[j]);
        }
        tc_fence_before();
    }
    float* fin = reverse ? p.dh0 : p.hT;
    if (fin && ok) {
        const size_t soff = ((size_t)n * p.d.H + hd) * D * D + (size_t)r * D + gc0;
#pragma unroll
        for (int k = 0; k < NSH / 4; ++k) *reinterpret_cast<float4*>(fin + soff + 4 * k) = make_float4(st[4 * k], st[4 * k + 1], st[4 * k + 2], st[4 * k + 3]);
    }
    if (threadIdx.x == 0) bulk_wait_read<0>();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, NS);
}

// ------------------------------------------------------------------------------------------------
// tc_scan_lr: the same carries without the d x d operator of a chunk, for shapes whose carries are bound by HBM
// bandwidth (one CTA per chain and direction fills the machine).  With e_j = exp(gam_e - gam_j):
//   forward   h'  = Gam_e h   + K^T Diag(e) (U~ - W h)
//   reverse   dh  = Gam_e dh' + E - W^T Diag(e) (K dh')
// Two dependent products per step instead of one, but tc_prep neither forms nor writes Nm and Bf (64 KB per
// chunk-head less to write and 16 KB less to read).  Per step a ring slot receives W^T, the K tile of the chunk and
// U~^T (forward) or E (reverse); the first product leaves (W h)^T or (K dh')^T with features on TMEM lanes and tokens
// on columns, the readout forms the scaled bf16 operand of the second product in the same orientation, the second
// product yields the d_k x d_v increment of the state, which lives in fp32 registers as in tc_scan.
// ------------------------------------------------------------------------------------------------
namespace scanlr {
constexpr int GE_CAP = 2048;
constexpr uint32_t WT = 0, KT = 16384, XT = 32768;   // ring slot: W^T | K | this CTA's part of U~^T (16 KB / S) or E (32 KB / S)
constexpr uint32_t C_D1 = 0, C_D2 = 64;              // TMEM columns: first product (64), second product (128 / S)
// S = number of CTAs that share a chain, each carrying 128 / S state columns (the columns of the state evolve
// independently; W and K are needed whole by every one of them).  S = 2 serves calls that run one direction only with so
// few chains that half of the SMs would idle (the forward, the backward on a fresh workspace): a step of a half is
// shorter, and a step's latency is what bounds those launches.
template <int S> struct Cfg {
    static constexpr int NS = D / S;                          // state columns of this CTA = rows of the first product
    static constexpr int NSH = NS / 2;                        // ... of one thread
    static constexpr int STAGES = S == 1 ? 2 : 3;
    static constexpr uint32_t STAGE_BYTES = 32768 + 32768 / S;
    static constexpr uint32_t HT = STAGES * STAGE_BYTES;      // two bf16 state tiles [128][NS]
    static constexpr uint32_t HT_BYTES = 32768 / S;
    static constexpr uint32_t GT = HT + 2 * HT_BYTES;         // operand of the second product, [NS features][64 tokens]
    static constexpr uint32_t SMEM_BYTES = GT + 16384 / S + 1024;
    static constexpr uint32_t TMEM_COLS = S == 1 ? 256 : 128;
    static_assert(SMEM_BYTES + GE_CAP * 4 + 2048 <= 227 * 1024, "shared memory budget");
};
}  // namespace scanlr

// One direction of one chain (the direction is a compile-time constant: the two differ in operands and readouts).
// CW = carries of the channel-wise path (per-channel gates): the decay of the state is a vector (one factor per state
// row, i.e. per thread), and the key tile arrives already scaled, Kb_j = exp(gam_e - gam_j) . k_j, as a tile image from the
// workspace together with images of W^T, U~^T and E (written by the channel-wise preparation kernels), so the readout of the
// first product applies no per-token factor.
template <bool reverse, bool CW, int S>
__device__ __forceinline__ void scan_lr_chain(const TcParams& P, int chain, int part, float* ge, float (*ee2)[kC], uint64_t* bar_full,
                                              uint64_t& bar_mma, uint32_t& tmem_slot) {
    using namespace scanlr;
    using C = Cfg<S>;
    constexpr int NS = C::NS, NSH = C::NSH, STAGES = C::STAGES;
    constexpr uint32_t STAGE_BYTES = C::STAGE_BYTES, HT = C::HT, HT_BYTES = C::HT_BYTES, GT = C::GT;
    const Problem& p = P.p;
    const int H = p.d.H, n = chain / H, hd = chain % H;
    const SeqGeom sg = seq_geom(p, n);
    const int c0 = sg.c0, nsteps = sg.n_chunks, c1 = c0 + nsteps;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, hf = warp >> 2;
    const int r = q4 * 32 + lane;              // TMEM lane of this thread: state row (d_k) or feature of the first product (d_v)
    const int lc0 = hf * NSH;                  // first of its NSH state columns inside the CTA's block
    const int tk0 = hf * 32;                   // first of its 32 tokens in the first product
    // The first product has NS rows.  With 128 of them a thread's TMEM lane is its feature; with 64 (M = 64) the rows sit
    // on lanes 0..15 of each quadrant and the other lanes of a warp have nothing to read out.
    const int r1 = S == 1 ? r : q4 * 16 + (lane & 15);
    const bool act1 = S == 1 || lane < 16;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&bar_full[s], 1);
        mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, C::TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    auto chunk_of = [&](int s) { return reverse ? (c1 - 1 - s) : (c0 + s); };
    const char* w_base = p.ws + (CW ? p.L.img_W : p.L.W);
    // this CTA's part of the additive image: rows part * NS.. of U~^T [d_v][tokens], column block `part` of E [d_k][d_v]
    const uint32_t x_chunk = reverse ? 32768u : 16384u, x_bytes = x_chunk / S;
    const char* x_base = p.ws + (reverse ? (CW ? p.L.img_E : p.L.E) : (CW ? p.L.img_U : p.L.Ut)) + part * x_bytes;
    char* keep_base = p.ws + (reverse ? p.L.dhn : p.L.hc) + part * HT_BYTES;
    const float* gamma = reinterpret_cast<const float*>(p.ws + p.L.gamma);
    // (L2 prefetches running ahead of the ring, as in tc_scan, made this kernel slower: 79.7 -> 78.5 us without)
    auto fill = [&](int s) {   // thread 32: bring chunk step s into ring slot s % STAGES
        const int stage = s % STAGES, c = chunk_of(s);
        const size_t ch = (size_t)c * H + hd;
        unsigned char* slot = sm + stage * STAGE_BYTES;
        mbar_expect_tx(&bar_full[stage], 32768 + x_bytes);
        bulk_load(slot + WT, w_base + ch * 16384, 16384, &bar_full[stage]);
        if constexpr (CW) {
            // forward: Kb = Gam_e . k- (second product); reverse: k- itself, against the state scaled by Gam_e (below)
            bulk_load(slot + KT, p.ws + (reverse ? p.L.img_Km : p.L.img_K) + ch * 16384, 16384, &bar_full[stage]);
        } else {
            tma_load_2d(slot + KT, &P.tm_k, hd * D, sg.chunk_tok0(c), &bar_full[stage]);
            tma_load_2d(slot + KT + 8192, &P.tm_k, hd * D + 64, sg.chunk_tok0(c), &bar_full[stage]);
        }
        bulk_load(slot + XT, x_base + ch * x_chunk, x_bytes, &bar_full[stage]);
    };
    if (threadIdx.x == 32) {
        for (int s = 0; s < STAGES && s < nsteps; ++s) fill(s);
    }
    if constexpr (!CW)
        for (int s = threadIdx.x; s < nsteps && s < GE_CAP; s += blockDim.x)
            ge[s] = expf(gamma[((size_t)chunk_of(s) * H + hd) * kC + kC - 1]);
    // e_j of the first step; the cumulative decays of the second are fetched now
    auto gate_row = [&](int s) { return gamma + ((size_t)chunk_of(s) * H + hd) * kC; };
    float gnext = 0.f, gend_next = 0.f;
    if (!CW && threadIdx.x < kC && nsteps > 0) {
        ee2[0][threadIdx.x] = expf(gate_row(0)[kC - 1] - gate_row(0)[threadIdx.x]);
        if (nsteps > 1) { gnext = gate_row(1)[threadIdx.x]; gend_next = gate_row(1)[kC - 1]; }
    }
    float st[NSH];
    {
        const float* init = reverse ? p.dhT : p.h0;
        const size_t soff = ((size_t)n * H + hd) * D * D + (size_t)r * D + part * NS + lc0;
#pragma unroll
        for (int k = 0; k < NSH / 4; ++k) {
            float4 v = init ? *reinterpret_cast<const float4*>(init + soff + 4 * k) : make_float4(0.f, 0.f, 0.f, 0.f);
            st[4 * k] = v.x; st[4 * k + 1] = v.y; st[4 * k + 2] = v.z; st[4 * k + 3] = v.w;
        }
    }
    __syncthreads();
    bool ok = true;
    uint32_t mma_phase = 0;
    float cw_gam = (CW && nsteps > 0) ? gamma[(((size_t)chunk_of(0) * H + hd) * kC + kC - 1) * D + r] : 0.f;
#pragma unroll 1
    for (int s = 0; s < nsteps; ++s) {
        unsigned char* Ht = sm + HT + (s & 1) * HT_BYTES;
        const int c = chunk_of(s), stage = s % STAGES, len = sg.chunk_len(c);
        const size_t ch = (size_t)c * H + hd;
        unsigned char* ring = sm + stage * STAGE_BYTES;
        const float* ee = ee2[s & 1];
        // decay of the state over the chunk: a scalar, or (channel-wise) the factor of this thread's state row, whose log
        // was fetched during the step before (the reverse chain needs it at the top of the step)
        const float Ge = CW ? expf(cw_gam) : (s < GE_CAP ? ge[s] : expf(gamma[ch * kC + kC - 1]));
        if (CW && s + 1 < nsteps) cw_gam = gamma[(((size_t)chunk_of(s + 1) * H + hd) * kC + kC - 1) * D + r];
        // state -> bf16: operand of the first product, and the per-chunk state the gradient stage reads.  Channel-wise,
        // reverse: stored as dh'' = Diag(Gam_e) dh', the form the gradient stage works with ((Kb dh') = k- dh'').
#pragma unroll
        for (int k = 0; k < NSH / 8; ++k) {
            if constexpr (CW && reverse) {
                float sc8[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) sc8[j] = Ge * st[8 * k + j];
                *reinterpret_cast<uint4*>(Ht + tile_chunk_off(128, r, (lc0 >> 3) + k)) = pack8(sc8);
            } else {
                *reinterpret_cast<uint4*>(Ht + tile_chunk_off(128, r, (lc0 >> 3) + k)) = pack8(st + 8 * k);
            }
        }
        if (!CW && len < kC) {   // ragged tail: the K rows beyond the sequence belong to somebody else
            ok = mbar_wait_inline(&bar_full[stage], (s / STAGES) & 1);
            if (!ok) { if (threadIdx.x == 0) report_timeout(p.ws, 12); break; }
            zero_tail_rows(ring + KT, 64, 0, len, kThreads);
        }
        fence_async_smem();
        __syncthreads();
        if (threadIdx.x == 0) {
            ok = mbar_wait_inline(&bar_full[stage], (s / STAGES) & 1);
            if (ok) {
                tc_fence_after();
                // forward (W h)^T = h^T W^T ; reverse (K dh')^T = dh'^T K^T : [d_v][tokens]
                const Operand b = reverse ? op_k_major(ring + KT, 64) : op_mn_major(ring + WT, 128);
                mma_tile<NS, 64, 128>(tmem + C_D1, op_mn_major(Ht, 128), b, false);
            } else {
                report_timeout(p.ws, 10);
            }
            bulk_store(keep_base + ch * 32768, Ht, HT_BYTES);
            bulk_commit();
            bulk_wait_read<1>();   // (the store of the step before has read its tile: it is rewritten in the next step)
            mma_commit(&bar_mma);
        } else if (threadIdx.x == 32) {
            if (s >= 1 && s - 1 + STAGES < nsteps) fill(s - 1 + STAGES);
        }
        ok = mbar_wait_inline(&bar_full[stage], (s / STAGES) & 1);
        if (ok) ok = mbar_wait_inline(&bar_mma, mma_phase);
        mma_phase ^= 1;
        if (!ok) { if (threadIdx.x == 0) report_timeout(p.ws, 11); break; }
        tc_fence_after();
        // operand of the second product: forward Diag(e)(U~ - W h), reverse Diag(e)(K dh'), transposed
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float d1[8], u[8], e8[8];
            if constexpr (S == 2) {
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] = 0.f;
            }
            tmem_ld8(tmem + lane_base + C_D1 + tk0 + 8 * k, d1);
            if (!reverse && act1) chunk_load(ring + XT, NS, r1, (tk0 >> 3) + k, u);
            ld8s(ee + tk0 + 8 * k, e8);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) d1[j] = (CW ? 1.f : e8[j]) * (reverse ? d1[j] : (u[j] - d1[j]));
            if (act1) chunk_store(sm + GT, NS, r1, (tk0 >> 3) + k, d1);
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        if (threadIdx.x == 0) {
            tc_fence_after();
            if (reverse) mma_tile<128, NS, 64>(tmem + C_D2, op_k_major(ring + WT, 128), op_k_major(sm + GT, NS), false, /*neg_a=*/true);
            else mma_tile<128, NS, 64>(tmem + C_D2, op_mn_major(ring + KT, 64), op_k_major(sm + GT, NS), false);
            mma_commit(&bar_mma);
        }
        if (!CW && threadIdx.x < kC && s + 1 < nsteps) {   // e_j of the next step, while the product runs
            ee2[(s + 1) & 1][threadIdx.x] = expf(gend_next - gnext);
            if (s + 2 < nsteps) { gnext = gate_row(s + 2)[threadIdx.x]; gend_next = gate_row(s + 2)[kC - 1]; }
        }
        ok = mbar_wait_inline(&bar_mma, mma_phase);
        mma_phase ^= 1;
        if (!ok) { if (threadIdx.x == 0) report_timeout(p.ws, 13); break; }
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < NSH / 8; ++k) {
            float d2[8], ad[8];
            tmem_ld8(tmem + lane_base + C_D2 + lc0 + 8 * k, d2);
            if (reverse) chunk_load(ring + XT, 128, r, (lc0 >> 3) + k, ad);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) st[8 * k + j] = fmaf(Ge, st[8 * k + j], reverse ? ad[j] + d2[j] : d2[j]);
        }
        tc_fence_before();
    }
    float* fin = reverse ? p.dh0 : p.hT;
    if (fin && ok) {
        const size_t soff = ((size_t)n * H + hd) * D * D + (size_t)r * D + part * NS + lc0;
#pragma unroll
        for (int k = 0; k < NSH / 4; ++k) *reinterpret_cast<float4*>(fin + soff + 4 * k) = make_float4(st[4 * k], st[4 * k + 1], st[4 * k + 2], st[4 * k + 3]);
    }
    if (threadIdx.x == 0) bulk_wait_read<0>();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, C::TMEM_COLS);
}

// Block index -> (chain, direction, column block): with both directions in one launch the direction is the low bit
// (S = 1 only); with S = 2 (one direction per launch) the low bit is the column block.
template <int S>
__global__ void __launch_bounds__(kThreads, 1) tc_scan_lr_kernel(const __grid_constant__ TcParams P) {
    using namespace scanlr;
    __shared__ float ge[GE_CAP];
    __shared__ __align__(16) float ee2[2][kC];   // e_j of a step, made during the step before it
    __shared__ uint64_t bar_full[Cfg<S>::STAGES], bar_mma;
    __shared__ uint32_t tmem_slot;
    const int bid = (int)blockIdx.x;
    if (reinterpret_cast<const WsHeader*>(P.p.ws)->status != GDN_OK) return;
    const int rev = (S == 1 && P.scan_dirs == 2) ? (bid & 1) : P.scan_dirs;
    const int chain = (S == 2 || P.scan_dirs == 2) ? (bid >> 1) : bid;
    const int part = S == 2 ? (bid & 1) : 0;
    if (rev) scan_lr_chain<true, false, S>(P, chain, part, ge, ee2, bar_full, bar_mma, tmem_slot);
    else scan_lr_chain<false, false, S>(P, chain, part, ge, ee2, bar_full, bar_mma, tmem_slot);
}

// The carries of the channel-wise path (per-channel gates, d_k = d_v = 128, bf16 I/O) on the same machinery.
template <int S>
__global__ void __launch_bounds__(kThreads, 1) tc_scan_cw_kernel(const __grid_constant__ TcParams P) {
    using namespace scanlr;
    __shared__ __align__(16) float ee2[2][kC];   // (unused: the key tile arrives scaled)
    __shared__ uint64_t bar_full[Cfg<S>::STAGES], bar_mma;
    __shared__ uint32_t tmem_slot;
    const int bid = (int)blockIdx.x;
    if (reinterpret_cast<const WsHeader*>(P.p.ws)->status != GDN_OK) return;
    const int rev = (S == 1 && P.scan_dirs == 2) ? (bid & 1) : P.scan_dirs;
    const int chain = (S == 2 || P.scan_dirs == 2) ? (bid >> 1) : bid;
    const int part = S == 2 ? (bid & 1) : 0;
    if (rev) scan_lr_chain<true, true, S>(P, chain, part, nullptr, ee2, bar_full, bar_mma, tmem_slot);
    else scan_lr_chain<false, true, S>(P, chain, part, nullptr, ee2, bar_full, bar_mma, tmem_slot);
}

// ------------------------------------------------------------------------------------------------
// tc_intra: token gradients of one (chunk, head).
//
// Products (all on tcgen05, outputs transposed: features on TMEM lanes, tokens on columns, except the 64 x 64
// token-token matrices which use M = 64):
//   phase 1  (W h)^T ; (K dh')^T          (P = tril(Q K^T . D) comes from tc_prep, which forms it anyway)
//   phase 2  (P^T dO)^T ; then, under the readout, dO h^T          -> U = U~ - W h ; dU = scale P^T dO + Diag(e) K dh'
//   phase 3  dO U^T ; T^T dU                                       -> dPD = scale tril(dO U^T) . D ; dXv ; dv ; dw
//   phase 4  dXv U^T ; dPD K ; -dXv h^T ; under the readout dPD^T Q ; U dh'^T
//                                                                  -> G = -stril(dXv U^T) . D ; Diag(b) G ; dq ; (dXk)
//   phase 5  G K ; += (Diag(b) G)^T K                               -> dk ; db ; dgamma -> dg
// The vector-Jacobian product of the triangular solve (K#2) is taken in a shorter form than its definition
// dW = -dU h^T, dXk = T^T dW, dXv = T^T dU, dA = -stril(dXk W^T + dXv U~^T):  T^T dW = -(T^T dU) h^T, so dXk = -dXv h^T,
// and with it dXk W^T + dXv U~^T = dXv (U~ - W h)^T = dXv U^T.  dW is never formed, dXv follows dU directly (beside dP,
// not after dW), and the sandwich is one product: a phase, a readout and twelve MMA instructions fewer per chunk-head.
// The decay gradient uses the identities  rowsum(dP.P) + scale Gam <q, dO h^T> = <q, dq>  and its analogues for
// k:  dgamma_i = <q_i, dq_i> + <k_i, dk_i^row> - <k_i, dk_i^col>, where dk^row = Diag(b)(G K + Diag(Gam) dXk)
// collects the terms in which k_i enters with exp(+gamma_i) and dk^col those with exp(-gamma_i); the last row
// of the chunk adds sum_j r_j + Gam_e <dh', h> (r_j = <(Kb dh')_j, U_j>).  Phases 1-2 produce transposed
// accumulators (features on TMEM lanes) because their results feed later products; from phase 3 on every
// accumulator that becomes a gradient is token-major.
// ------------------------------------------------------------------------------------------------
namespace intra {
constexpr uint32_t QK = 0;                 // [Q ; K] x 128                     32 KB
constexpr uint32_t VT = 32768;             // V  [64][128]                      16 KB   later staged dv
constexpr uint32_t DO = VT + 16384;        // dO [64][128]                      16 KB   later dXv [64][128], then G and Diag(b) G [64][64] each
constexpr uint32_t WT = DO + 16384;        // W^T  [128][64]                    16 KB
constexpr uint32_t UTT = WT + 16384;       // U~^T [128][64]                    16 KB
constexpr uint32_t TT = UTT + 16384;       // T [64][64]                         8 KB
constexpr uint32_t HH = TT + 8192;         // h [128][128]                      32 KB
constexpr uint32_t DH = HH + 32768;        // dh' [128][128]                    32 KB
constexpr uint32_t PT = DH + 32768;        // P [64][64]                         8 KB   later dPD
constexpr uint32_t UT = PT + 8192;         // U^T [128][64]                     16 KB   later staged dk
constexpr uint32_t DUT = UT + 16384;       // dU^T [128][64]                    16 KB   later staged dq
constexpr uint32_t SMEM_BYTES = DUT + 16384 + 1024;
constexpr uint32_t DXV = DO, DPD = PT, GT = DO, BGT = DO + 8192;
// token-major staging of dq (over dU^T, last read by phase 3), of dv (in place over V: a thread overwrites exactly the
// chunk it has just read) and of dk (over U^T, last read by the products of phase 4).  None of these is read by a later
// product or rewritten within the trip, and of the loads that run ahead only V targets one of them (after its store
// has read it), so the asynchronous stores need no wait on the critical path.
constexpr uint32_t STG_A = DUT, STG_B = VT, STG_K = UT;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory budget");
__host__ __device__ constexpr uint32_t slot(int k) { return 64u * k; }   // eight accumulators of 64 columns
}  // namespace intra

__global__ void __launch_bounds__(kIntraThreads + 32, 1) tc_intra_kernel(const __grid_constant__ TcParams P) {
    using namespace intra;
    const Problem& p = P.p;
    // Persistent: a CTA walks over chunk-heads blockIdx.x, blockIdx.x + gridDim.x, ...  While it works on one, the
    // tiles of its next one are loaded into the regions the current one has finished with.
    const int H = p.d.H;
    if (reinterpret_cast<const WsHeader*>(p.ws)->status != GDN_OK) return;   // an earlier stage gave up: nothing is written
    const int n_items = n_chunks_of(p) * H;
    if ((int)blockIdx.x >= n_items) return;
    const float sc = p.d.scale;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ __align__(16) float gate_sets[2][5][kC];   // two sets: a trip's gate arrays are written during the trip before
    __shared__ float red[4][kGroups][kC];       // four token-wise partial sums: [which][column group][token]
    __shared__ float dgam[kC], scal[2][kIntraThreads / 32];
    __shared__ uint64_t bar_k, bar_g1, bar_g2, bar_do, bar_ld0, bar_ldw, bar_ldh, bar_ld1, bar_ld2, bar_st1, bar_st2, bar_kfree, bar_free, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, grp = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    // Warps 0..15 read accumulators; the first lane of warp 16 only feeds the tensor pipe.  Because the issuer has no
    // readout duties, a phase can commit the products the next readout needs first and keep issuing the ones that
    // are only needed later while the readout already runs.
    const bool worker = warp < 16;
    const bool issuer = threadIdx.x == kWideThreads;
    // Warp 17 only moves data.  Its first lane issues every bulk / TMA instruction of the steady state (each costs its
    // issuer hundreds of cycles): the stores of the staged gradients, and the loads of the NEXT trip's tiles, each as
    // soon as the region it goes to has been read for the last time in this trip.  It shares no block-wide barrier
    // with the other warps inside the loop (they use a named barrier); it follows them through mbarriers.
    const bool loader = warp == 17;

    if (threadIdx.x == 0) {
        mbar_init(&bar_k, 1); mbar_init(&bar_g1, 1); mbar_init(&bar_g2, 1); mbar_init(&bar_do, 1);
        mbar_init(&bar_ld0, 1); mbar_init(&bar_ldw, 1); mbar_init(&bar_ldh, 1); mbar_init(&bar_ld1, 1); mbar_init(&bar_ld2, 1);
        mbar_init(&bar_st1, 1); mbar_init(&bar_st2, 1); mbar_init(&bar_kfree, 16); mbar_init(&bar_free, 1);
        mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    bool ok = true;

    // The tiles of a trip arrive in groups, one mbarrier each, loaded during the previous trip as their regions fall free:
    //   g1  W, U~^T              once the second readout is done             needed by phase 1
    //       h, dh', P            once the products of phase 4 are done
    //       Q                    once the readout of phase 4 is done
    //   do  dO;  g2  T, V        once the products of the last phase are done  needed from phase 2 / 3 on
    //                            (V goes where dv is staged: its store, or the flush of a ragged tail, must have read it)
    //   k   K                    once the last readout holds its K values    needed by phase 1
    constexpr uint32_t K_BYTES = 16384, G1_BYTES = 16384 + 16384 + 32768 + 32768 + 16384 + 8192, G2_BYTES = 8192 + 16384, DO_BYTES = 16384;
    auto load_piece = [&](int piece, const ChunkInfo& c) {
        const int cb = piece & 1, xq = c.hd * D + cb * 64;
        switch (piece) {
            case 0: case 1: tma_load_2d(sm + QK + cb * 16384 + 8192, &P.tm_k, xq, c.tok0, &bar_k); break;
            case 2: case 3: tma_load_2d(sm + QK + cb * 16384, &P.tm_q, xq, c.tok0, &bar_g1); break;
            case 4: bulk_load(sm + UTT, p.ws + p.L.Ut + (size_t)c.ch * 16384, 16384, &bar_g1); break;
            case 5: bulk_load(sm + DH, p.ws + p.L.dhn + (size_t)c.ch * 32768, 32768, &bar_g1); break;
            case 6: bulk_load(sm + HH, p.ws + p.L.hc + (size_t)c.ch * 32768, 32768, &bar_g1); break;
            case 7: bulk_load(sm + WT, p.ws + p.L.W + (size_t)c.ch * 16384, 16384, &bar_g1); break;
            case 8: case 9: tma_load_2d(sm + DO + cb * 8192, &P.tm_do, xq, c.tok0, &bar_do); break;
            case 10: case 11: tma_load_2d(sm + VT + cb * 8192, &P.tm_v, xq, c.tok0, &bar_g2); break;
            case 12: bulk_load(sm + TT, p.ws + p.L.Tm + (size_t)c.ch * 8192, 8192, &bar_g2); break;
            case 13: bulk_load(sm + PT, p.ws + p.L.Pm + (size_t)c.ch * 8192, 8192, &bar_g1); break;
            default: break;
        }
    };

    if (loader) {
        if (lane == 0) {
            uint32_t ph = 0;
            bool lok = true, pend_k = false, pend1 = false, pend2 = false, pend_do = false;
#pragma unroll 1
            for (int item = blockIdx.x; item < n_items && lok; item += gridDim.x, ph ^= 1) {
                ChunkInfo x, nx;
                chunk_entry(p, x, item);
                const bool has_next = item + (int)gridDim.x < n_items;
                if (has_next) chunk_entry(p, nx, item + gridDim.x);
                const bool full = x.len == kC;
                pend_k = pend1 = pend2 = pend_do = false;
                // the trip is under way (all its tiles have arrived): K of the next one, the only late load, -> L2
                if (!(lok = mbar_wait(&bar_ld0, ph))) break;
                if (has_next) {
                    prefetch_l2_tma_2d(&P.tm_k, nx.hd * D, nx.tok0);
                    prefetch_l2_tma_2d(&P.tm_k, nx.hd * D + 64, nx.tok0);
                }
                // (Early loads not in a CTA's first trip: there every CTA of the grid reaches these points at the same moment,
                // the loads come as one burst of 25 MB, and the instruction fetches of the last phases, which run for the
                // first time, queue behind it for microseconds.  The first trip loads at its end instead.)
                const bool early = item != (int)blockIdx.x;
                // the second readout is done: W^T and U~^T have been read for the last time
                if (!(lok = mbar_wait(&bar_ldw, ph))) break;
                if (has_next && early) {
                    mbar_expect_tx(&bar_g1, G1_BYTES);   // the first piece of the group announces all of it
                    pend1 = true;
                    load_piece(7, nx);
                    load_piece(4, nx);
                }
                // the products of phase 4 are done: h, dh' and dPD (over P) have been read for the last time
                if (!(lok = mbar_wait(&bar_ldh, ph))) break;
                if (has_next && early) {
                    load_piece(6, nx);
                    load_piece(5, nx);
                    load_piece(13, nx);
                }
                // dq, dv are staged
                if (!(lok = mbar_wait(&bar_st1, ph))) break;
                if (full) {
                    for (int cb = 0; cb < 2; ++cb) {
                        tma_store_2d(&P.tm_dq, x.hd * D + cb * 64, x.tok0, sm + STG_A + cb * 8192);
                        tma_store_2d(&P.tm_dv, x.hd * D + cb * 64, x.tok0, sm + STG_B + cb * 8192);
                    }
                    bulk_commit();
                }
                // the readout of phase 4 is done too: Q has been read for the last time
                if (!(lok = mbar_wait(&bar_ld1, ph))) break;
                if (has_next && early) {
                    load_piece(2, nx);
                    load_piece(3, nx);
                }
                // the last phase is done and its readout holds its K values in registers: K first, the next trip starts with
                // it; dO, T, V are not needed before its second phase (V goes where dv is staged, so that store must have
                // read its source)
                if (!(lok = mbar_wait(&bar_ld2, ph))) break;
                if (!(lok = mbar_wait(&bar_kfree, ph))) break;
                if (has_next && early) {
                    mbar_expect_tx(&bar_k, K_BYTES);
                    pend_k = true;
                    load_piece(0, nx);
                    load_piece(1, nx);
                    mbar_expect_tx(&bar_do, DO_BYTES);   // dO next: the second phase starts with it
                    pend_do = true;
                    load_piece(8, nx);
                    load_piece(9, nx);
                    bulk_wait_read<0>();
                    mbar_expect_tx(&bar_g2, G2_BYTES);
                    pend2 = true;
#pragma unroll 1
                    for (int piece = 10; piece <= 12; ++piece) load_piece(piece, nx);
                }
                // dk is staged
                if (!(lok = mbar_wait(&bar_st2, ph))) break;
                if (full) {
                    for (int cb = 0; cb < 2; ++cb) tma_store_2d(&P.tm_dk, x.hd * D + cb * 64, x.tok0, sm + STG_K + cb * 8192);
                    bulk_commit();
                }
                bulk_wait_read<0>();
                mbar_arrive(&bar_free);   // the staging regions may be rewritten
                if (has_next && !early) {
                    mbar_expect_tx(&bar_k, K_BYTES);
                    mbar_expect_tx(&bar_g1, G1_BYTES);
                    mbar_expect_tx(&bar_g2, G2_BYTES);
                    mbar_expect_tx(&bar_do, DO_BYTES);
                    pend_k = pend1 = pend2 = pend_do = true;
#pragma unroll 1
                    for (int piece = 0; piece <= 13; ++piece) load_piece(piece, nx);
                }
            }
            bulk_wait_read<0>();
            if (!lok) {   // after a timeout a copy may still be in flight: wait for it before the CTA may retire
                if (pend_k) (void)mbar_wait(&bar_k, ph ^ 1);
                if (pend1) (void)mbar_wait(&bar_g1, ph ^ 1);
                if (pend2) (void)mbar_wait(&bar_g2, ph ^ 1);
                if (pend_do) (void)mbar_wait(&bar_do, ph ^ 1);
            }
        }
        return;
    }

    auto cta_sync = [] { asm volatile("bar.sync 1, %0;" ::"n"(kIntraThreads) : "memory"); };   // all warps but the loader
    uint32_t mma_phase = 0, in_phase = 0;
    // chunk table entry and gates of a trip are fetched one trip ahead into registers (their latency would be exposed)
    ChunkInfo xn;
    chunk_entry(p, xn, blockIdx.x);
    float ng = 0.f, ngend = 0.f, nb = 0.f;
    auto fetch_gates = [&](const ChunkInfo& c) {   // cumulative log decay of this thread's token and of the chunk end, gate b
        const float* gsrc = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)c.ch * kC;
        ng = gsrc[threadIdx.x];
        ngend = gsrc[kC - 1];
        nb = ((int)threadIdx.x < c.len && p.d.delta_rule) ? p.beta[(size_t)(c.tok0 + (int)threadIdx.x) * H + c.hd] : 0.f;
    };
    auto make_gates = [&](int set) {   // threads 0..63: the fetched values -> gate arrays of set `set`
        const int i = threadIdx.x;
        gate_sets[set][0][i] = ng * kLog2e;
        gate_sets[set][1][i] = expf(ng);
        gate_sets[set][2][i] = expf(ngend - ng);
        gate_sets[set][3][i] = nb;                                                    // erase gate
        gate_sets[set][4][i] = p.d.delta_rule ? nb : (i < xn.len ? 1.f : 0.f);        // write gate (delta rule off: 0 and 1)
    };
    // dbeta and dg of the previous trip's chunk, from its token-wise partial sums (warps 0 and 1; see the trip's end)
    ChunkInfo xp = xn;
    bool have_prev = false;
    float bb_prev = 0.f, Gam_last_prev = 0.f;
    auto finish_gates = [&]() {
        const int i = threadIdx.x;
        auto tot = [&](int w) { return (red[w][0][i] + red[w][1][i]) + (red[w][2][i] + red[w][3][i]); };
        const float qdq = tot(0), dw = tot(1), db = tot(2), kcol = tot(3);
        if (i < xp.len && p.dbeta) p.dbeta[(size_t)(xp.tok0 + i) * H + xp.hd] = db + dw;
        dgam[i] = fmaf(bb_prev, db, qdq - kcol);
        asm volatile("bar.sync 2, 64;" ::: "memory");
        if (warp == 0) {
            constexpr int nw = kIntraThreads / 32;   // per-warp partial sums, one per lane
            const float rsum = warp_sum(lane < nw ? scal[0][lane] : 0.f), hsum = warp_sum(lane < nw ? scal[1][lane] : 0.f);
            write_dg_suffix(dgam, nullptr, rsum + Gam_last_prev * hsum, p.dg + (size_t)xp.tok0 * H + xp.hd, (size_t)H, xp.len, lane);
        }
    };
    // first trip: every group is loaded at once, one instruction per warp
    if (issuer) { mbar_expect_tx(&bar_k, K_BYTES); mbar_expect_tx(&bar_g1, G1_BYTES); mbar_expect_tx(&bar_g2, G2_BYTES); mbar_expect_tx(&bar_do, DO_BYTES); }
    if (lane == 0 && warp < 14) load_piece(warp, xn);
    if (threadIdx.x < kC) { fetch_gates(xn); make_gates(0); }
#pragma unroll 1
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, in_phase ^= 1) {
    const ChunkInfo x = xn;
    // this trip's gate arrays (the barrier before phase 1 publishes them)
    const float* gl = gate_sets[in_phase][0];
    const float* Gam = gate_sets[in_phase][1];
    const float* ee = gate_sets[in_phase][2];
    const float* bb = gate_sets[in_phase][3];
    const bool has_next = item + (int)gridDim.x < n_items;
    const bool first = item == (int)blockIdx.x;
    if (has_next) chunk_entry(p, xn, item + gridDim.x);

    if (ok) {
        ok = mbar_wait(&bar_g1, in_phase);
        ok = ok && mbar_wait(&bar_k, in_phase);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 20);
    }
    if (ok && x.len < kC) {
        zero_tail_rows(sm + QK, 128, 0, x.len, kIntraThreads);
        zero_tail_rows(sm + QK, 128, 64, x.len, kIntraThreads);
        fence_async_smem();
    }
    cta_sync();

    // ---- phase 1: (W h)^T and (K dh')^T.  P = tril(Q K^T . D) is not formed here: tc_prep made it and it arrived
    // with the first group of tiles.
    if (ok && issuer) {
        tc_fence_after();
        mma_tile<128, 64, 128>(tmem + slot(1), op_mn_major(sm + HH, 128), op_mn_major(sm + WT, 128), false);
        mma_tile<128, 64, 128>(tmem + slot(2), op_mn_major(sm + DH, 128), op_k_major(sm + QK, 128, 64), false);
    }
    if (ok) {
        ok = mbar_wait(&bar_do, in_phase);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 27);
    }
    if (ok && x.len < kC) {
        zero_tail_rows(sm + DO, 64, 0, x.len, kIntraThreads);
        fence_async_smem();
    }
    cta_sync();

    // ---- phase 2
    if (ok && issuer) {
        tc_fence_after();
        mma_tile<128, 64, 64>(tmem + slot(3), op_mn_major(sm + DO, 64), op_mn_major(sm + PT, 64), false);
        mma_commit(&bar_mma);
        // dO h^T (token-major, group A of columns 384..511) is first read after phase 4: it runs under the readout
        mma_tile<64, 128, 128>(tmem + 384, op_k_major(sm + DO, 64), op_k_major(sm + HH, 128), false);
    }
    if (threadIdx.x == 32) mbar_arrive(&bar_ld0);   // every tile of this trip has arrived
    if (has_next && threadIdx.x < kC) fetch_gates(xn);
    if (ok && have_prev && warp < 2) finish_gates();   // warps 0 and 1: the previous chunk's gate gradients
    GDN_WAIT_MMA(22)
    if (ok && !first) {   // U^T and dU^T held the previous trip's staged dk and dq: their stores must have read them
        ok = mbar_wait(&bar_free, in_phase ^ 1);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 28);
    }
    const int f = q4 * 32 + lane;      // feature (lane of the transposed accumulators)
    const int i0 = grp * kTG;          // first of this thread's 32 tokens
    float rs = 0.f;
    if (ok && worker) {
        float t2[2][8], kb2[2][8], pd2[2][8];
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            tmem_ld8(tmem + lane_base + slot(1) + i0 + part * 8, t2[part]);
            tmem_ld8(tmem + lane_base + slot(2) + i0 + part * 8, kb2[part]);
            tmem_ld8(tmem + lane_base + slot(3) + i0 + part * 8, pd2[part]);
        }
        tmem_wait_ld();
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            const int ib = i0 + part * 8;
            float u[8], e8[8];
            float (&t)[8] = t2[part], (&kb)[8] = kb2[part], (&pd)[8] = pd2[part];
            chunk_load(sm + UTT, 128, f, ib >> 3, u);
            ld8s(ee + ib, e8);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                u[i] -= t[i];                                       // U = U~ - W h
                const float kbe = e8[i] * kb[i];
                rs = fmaf(kbe, u[i], rs);                           // sum_j r_j
                pd[i] = fmaf(sc, pd[i], kbe);                       // dU = scale P^T dO + Diag(e) K dh'
            }
            chunk_store(sm + UT, 128, f, ib >> 3, u);
            chunk_store(sm + DUT, 128, f, ib >> 3, pd);
        }
    }
    if (ok) {   // T and V, the last tiles of this trip, are needed from phase 3 on
        ok = mbar_wait(&bar_g2, in_phase);
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, 31);
    }
    if (ok && x.len < kC) zero_tail_rows(sm + VT, 64, 0, x.len, kIntraThreads);
    tc_fence_before();
    fence_async_smem();
    cta_sync();
    if (threadIdx.x == 32) mbar_arrive(&bar_ldw);   // W^T (read by phase 1) and U~^T (read by the readout) are free

    // From here on the accumulators that become gradients are produced token-major (64 token rows x 128 features,
    // M = 64): a thread owns a token row, so row dots are thread-local and rows leave with 16-byte stores.  A 64-row
    // accumulator occupies lanes 0..15 of each quadrant ("group A"); a second one sits in lanes 16..31 of the same
    // columns ("group B", address + 16 lanes), and one tcgen05.ld serves both groups.
    //   columns   group A                               group B
    //   0..127    U dh'^T (ph 4)                        dP (ph 3, 64 cols)
    //   128..255  (dP.D) K (ph 4)                       dXv (ph 3)
    //   256..383  dk^col: (dP.D)^T Q (ph 4) += (bG)^T K  dXk = -dXv h^T (ph 4; read with dk^col, handed over by shuffle)
    //   384..511  dO h^T (ph 2) -> G K (ph 5)           dXv U^T (ph 4, 64 cols)
    constexpr uint32_t LB = 16u << 16;
    const bool ga = lane < 16;
    const int tr = q4 * 16 + (lane & 15);   // token row of this lane in token-major accumulators
    const int cb0 = grp * 32;               // first of this thread's 32 feature columns
    const int j0b = grp * kTG;              // first of its 16 columns in 64-column accumulators

    // ---- phase 3: dO U^T and dXv = T^T dU
    if (ok && issuer) {
        tc_fence_after();
        mma_tile<64, 64, 128>(tmem + 0 + LB, op_k_major(sm + DO, 64), op_mn_major(sm + UT, 128), false);           // dO U^T
        mma_tile<64, 128, 64>(tmem + 128 + LB, op_mn_major(sm + TT, 64), op_k_major(sm + DUT, 128), false);         // T^T dU
        mma_commit(&bar_mma);
    }
    if (has_next && threadIdx.x < kC) make_gates(in_phase ^ 1);   // the next trip's gate arrays, while the products run
    // <dh', h> over the whole state, while the products run (both tiles share one format, so offsets pair up)
    float hh = 0.f;
#pragma unroll 1
    for (int t = (int)threadIdx.x - 64; t >= 0 && t < 2048; t += kIntraThreads - 64) {
        float a[8], b[8];
        unpack8(*reinterpret_cast<const uint4*>(sm + HH + t * 16), a);
        unpack8(*reinterpret_cast<const uint4*>(sm + DH + t * 16), b);
#pragma unroll
        for (int k = 0; k < 8; ++k) hh = fmaf(a[k], b[k], hh);
    }
    GDN_WAIT_MMA(23)
    const bool full = x.len == kC;
    // (addresses of the ragged-tail flushes are formed where they are used: nothing of them lives across the phases)
    auto grad_rows = [&](void* base) { return reinterpret_cast<__nv_bfloat16*>(base) + ((size_t)x.tok0 * H + x.hd) * D; };
    if (ok && worker) {   // group B holds both accumulators (the loads are warp-wide instructions)
        float v2[2][8];
        tmem_ld8(tmem + lane_base + 0 + j0b, v2[0]);
        tmem_ld8(tmem + lane_base + 0 + j0b + 8, v2[1]);
        tmem_wait_ld();
        if (!ga) {   // dPD = scale tril(dO U^T) . D
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const int jb = j0b + part * 8;
                float (&v)[8] = v2[part];
                float g8[8];
                ld8s(gl + jb, g8);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = (jb + j <= tr) ? sc * v[j] * ex2(gl[tr] - g8[j]) : 0.f;
                chunk_store(sm + DPD, 64, tr, jb >> 3, v);
            }
        }
        // dXv -> operand tile (over dO, which every product has read) ; <v, dXv> (dw partial) ; dv = w dXv, staged over V
        float acc = 0.f;
        const float wg = gate_sets[in_phase][4][tr];
#pragma unroll
        for (int part = 0; part < 4; ++part) {
            const int cb = cb0 + part * 8;
            float b[8], t8[8];
            tmem_ld8(tmem + lane_base + 128 + cb, b);
            tmem_wait_ld();
            if (!ga) {
                unpack8(*reinterpret_cast<const uint4*>(sm + VT + tile_chunk_off(64, tr, cb >> 3)), t8);
                chunk_store(sm + DXV, 64, tr, cb >> 3, b);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    acc = fmaf(t8[j], b[j], acc);
                    b[j] *= wg;
                }
                chunk_store(sm + STG_B, 64, tr, cb >> 3, b);
            }
        }
        if (!ga) red[1][grp][tr] = acc;
    }
    tc_fence_before();
    fence_async_smem();
    cta_sync();

    // ---- phase 4: dA = -stril(dXv U^T) (= -stril(dXk W^T + dXv U~^T), since dXk = T^T dW = -dXv h^T and U = U~ - W h),
    // (dP.D) K, dXk = -dXv h^T; under the readout (dP.D)^T Q and U dh'^T
    if (ok && issuer) {
        tc_fence_after();
        mma_tile<64, 64, 128>(tmem + 384 + LB, op_k_major(sm + DXV, 64), op_mn_major(sm + UT, 128), false);         // dXv U^T
        mma_tile<64, 128, 64>(tmem + 128, op_k_major(sm + DPD, 64), op_mn_major(sm + QK, 128, 64), false);          // (dP.D) K
        mma_tile<64, 128, 128>(tmem + 256 + LB, op_k_major(sm + DXV, 64), op_k_major(sm + HH, 128), false, /*neg_a=*/true);   // dXk
        mma_commit(&bar_mma);   // the two dk^col products are first read after the last phase
        mma_tile<64, 128, 64>(tmem + 256, op_mn_major(sm + DPD, 64), op_mn_major(sm + QK, 128, 0), false);           // (dP.D)^T Q
        mma_tile<64, 128, 128>(tmem + 0, op_mn_major(sm + UT, 128), op_k_major(sm + DH, 128), false);                // U dh'^T
        mma_commit(&bar_ldh);   // h, dh' and dPD (over P) have been read for the last time
    }
    GDN_WAIT_MMA(24)
    if (ok && worker) {
        // group A: dq = scale Gam (dO h^T) + (dP.D) K, staged ; acc = <q, dq>
        float acc = 0.f;
        const float coef = sc * Gam[tr];
#pragma unroll
        for (int part = 0; part < 4; ++part) {
            const int cb = cb0 + part * 8;
            float a[8], b[8], t8[8];
            tmem_ld8(tmem + lane_base + 384 + cb, a);     // A: dO h^T
            tmem_ld8(tmem + lane_base + 128 + cb, b);     // A: (dP.D) K
            tmem_wait_ld();
            if (ga) {
                unpack8(*reinterpret_cast<const uint4*>(sm + QK + tile_chunk_off(128, tr, cb >> 3)), t8);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    b[j] = fmaf(coef, a[j], b[j]);
                    acc = fmaf(t8[j], b[j], acc);
                }
                chunk_store(sm + STG_A, 64, tr, cb >> 3, b);
            }
        }
        if (ga) red[0][grp][tr] = acc;
        // group B: G = dA . D and Diag(b) G (over dXv, which the products above have read)
        float v2[2][8];
        tmem_ld8(tmem + lane_base + 384 + j0b, v2[0]);
        tmem_ld8(tmem + lane_base + 384 + j0b + 8, v2[1]);
        tmem_wait_ld();
        if (!ga) {
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float (&v)[8] = v2[part];
                float w[8], g8[8];
                const int jb = j0b + part * 8;
                ld8s(gl + jb, g8);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    v[j] = (jb + j < tr) ? -v[j] * ex2(gl[tr] - g8[j]) : 0.f;
                    w[j] = bb[tr] * v[j];
                }
                chunk_store(sm + GT, 64, tr, jb >> 3, v);
                chunk_store(sm + BGT, 64, tr, jb >> 3, w);
            }
        }
    }
    tc_fence_before();
    fence_async_smem();
    cta_sync();
    if (threadIdx.x == 32) mbar_arrive(&bar_st1);   // dq, dv are staged: the loader stores them (async proxy)
    if (ok && !full) {   // ragged tail: rows beyond the sequence must not be written
        flush_rows(sm + STG_A, grad_rows(p.dq), (size_t)H * D, x.len, kIntraThreads);
        flush_rows(sm + STG_B, grad_rows(p.dv), (size_t)H * D, x.len, kIntraThreads);
    }

    // ---- phase 5: G K ; += (Diag(b) G)^T K
    if (ok && issuer) {
        tc_fence_after();
        mma_commit(&bar_ld1);   // Q has been read for the last time (by (dP.D)^T Q and by the readout before this phase)
        mma_tile<64, 128, 64>(tmem + 384, op_k_major(sm + GT, 64), op_mn_major(sm + QK, 128, 64), false);            // G K
        mma_tile<64, 128, 64>(tmem + 256, op_mn_major(sm + BGT, 64), op_mn_major(sm + QK, 128, 64), true);           // += (bG)^T K
        mma_commit(&bar_mma);
        mma_commit(&bar_ld2);   // G (over dXv, over dO) and T have been read for the last time
    }
    GDN_WAIT_MMA(26)
    if (worker) {   // this thread's K values leave shared memory now, so that the next trip's K can be loaded over them
        uint4 kraw[4];
#pragma unroll
        for (int part = 0; part < 4; ++part)
            kraw[part] = *reinterpret_cast<const uint4*>(sm + QK + tile_chunk_off(128, 64 + tr, (cb0 >> 3) + part));
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_kfree);
        // Group A assembles dk = Diag(b)(G K + Gam dXk) + dk^col and both row dots with k; the lanes of group B hold
        // nothing of this phase (Diag(b) G K is a row scaling of G K, so one product serves dk and db).
        float acc_col = 0.f, acc_db = 0.f;   // <k, dk^col> ; db = <k, G K + Gam dXk>
        const float e6 = ee[tr], G6 = Gam[tr], b6 = bb[tr];
        if (ok) {
#pragma unroll
        for (int part = 0; part < 4; ++part) {
            const int cb = cb0 + part * 8;
            float a[8], b[8], c8[8], d8[8], kk[8];
            tmem_ld8(tmem + lane_base + 384 + cb, a);     // A: G K
            tmem_ld8(tmem + lane_base + 256 + cb, c8);    // A: (dP.D)^T Q + (bG)^T K      B: dXk
            tmem_ld8(tmem + lane_base + 0 + cb, d8);      // A: U dh'^T
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) b[j] = __shfl_down_sync(0xffffffffu, c8[j], 16);   // dXk of this token row comes over from group B
            if (ga) {
                unpack8(kraw[part], kk);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float kcol = fmaf(e6, d8[j], c8[j]);       // dk^col
                    const float t = fmaf(G6, b[j], a[j]);            // G K + Gam dXk
                    acc_col = fmaf(kk[j], kcol, acc_col);
                    acc_db = fmaf(kk[j], t, acc_db);
                    a[j] = fmaf(b6, t, kcol);
                }
                chunk_store(sm + STG_K, 64, tr, cb >> 3, a);
            }
        }
        }
        if (ga) { red[2][grp][tr] = acc_db; red[3][grp][tr] = acc_col; }
    }
    // block totals of sum_j r_j and <dh', h>
    rs = warp_sum(rs);
    hh = warp_sum(hh);
    if (lane == 0) { scal[0][warp] = rs; scal[1][warp] = hh; }
    fence_async_smem();
    cta_sync();
    if (threadIdx.x == 32) mbar_arrive(&bar_st2);   // dk is staged: the loader stores it
    if (ok && !full) flush_rows(sm + STG_K, grad_rows(p.dk), (size_t)H * D, x.len, kIntraThreads);
    // The token-wise sums are complete; turning them into dbeta and dg is left to warps 0 and 1 during the next trip's
    // first products (finish_gates).  They keep what the next trip overwrites: this chunk's gates and place.
    if (threadIdx.x < kC) { bb_prev = bb[threadIdx.x]; Gam_last_prev = Gam[kC - 1]; }
    xp = x;
    have_prev = true;
    tc_fence_before();
    cta_sync();   // every reader of this trip's tiles and scratch is done
    if (!ok) break;
    }
    if (ok && have_prev && warp < 2) finish_gates();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------
// tc_out (optional forward output): o = scale (Diag(Gam) Q h + P (U~ - W h)),  P = tril(Q K^T . D)
//
// Persistent, two CTAs per SM (96 KB of shared memory, 256 TMEM columns each): a CTA walks through the dependent
// steps of one chunk-head while its neighbour is in another step of another one.  The tiles of the next trip are
// loaded as soon as the last product (or store) that reads their region is done.  Q h and P U are formed token-major
// (M = 64: a thread owns a token row), so the output tile is staged with 16-byte stores and leaves by TMA.
// CW: the channel-wise path.  Its preparation kernels leave Q~ = Gam.q, P = tril(Q~ K-^T), W^T, U~^T and the per-chunk
// states in the workspace as tile images, the decay is inside Q~ and P, so o = scale (Q~ h + P (U~ - W h)): no product
// Q K^T, no gates, and P U accumulates onto Q~ h.  P arrives in the half of the [Q ; K] tile that K would occupy.
// ------------------------------------------------------------------------------------------------
namespace outk {
constexpr uint32_t QK = 0;                  // [Q rows 0..63 ; K rows 64..127] x 128              32 KB
constexpr uint32_t WT = 32768;              // W^T [128][64]; after the first products: P [64][64]  16 KB
constexpr uint32_t UTT = WT + 16384;        // U~^T [128][64]; U^T in place                         16 KB
constexpr uint32_t HH = UTT + 16384;        // h [128][128]; after the first products: staged o     32 KB
constexpr uint32_t PT = WT, STG = HH;
constexpr uint32_t SMEM_BYTES = HH + 32768 + 1024 /* alignment slack */;
constexpr uint32_t C_P = 0, C_WH = 64, C_QH = 128, C_PU = 0;   // TMEM columns (256 allocated)
constexpr uint32_t PT_CW = QK + 8192;        // channel-wise: P, loaded, in rows 64..127 of the first column block of [Q ; K]
constexpr uint32_t IN_BYTES = 32768 + 16384 + 16384 + 32768, IN_BYTES_CW = 16384 + 8192 + 16384 + 16384 + 32768;
static_assert(2 * (SMEM_BYTES + 4096) <= 228 * 1024, "two CTAs per SM");
}  // namespace outk

template <bool CW>
__global__ void __launch_bounds__(kThreads, 2) tc_out_kernel(const __grid_constant__ TcParams P) {
    using namespace outk;
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
    const int q4 = warp & 3, half = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    if (threadIdx.x == 0) { mbar_init(&bar_in, 1); mbar_init(&bar_mma, 1); fence_mbar_init(); }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    bool ok = true, pending = false;
    uint32_t mma_phase = 0, in_phase = 0, pending_phase = 0;   // (pending_phase: the phase of bar_in the loads in flight belong to)
    // One mbarrier phase per trip collects all five tiles; they are issued in three pieces, each when its region is free.
    auto load_qk = [&](const ChunkInfo& c, uint32_t phase) {   // thread 0; first piece of a trip: announces the whole trip's bytes
        pending_phase = phase;
        mbar_expect_tx(&bar_in, CW ? IN_BYTES_CW : IN_BYTES);
        for (int cb = 0; cb < 2; ++cb) {
            if (CW) {
                bulk_load(sm + QK + cb * 16384, p.ws + p.L.img_QKp + (size_t)c.ch * 32768 + cb * 16384, 8192, &bar_in);
            } else {
                tma_load_2d(sm + QK + cb * 16384, &P.tm_q, c.hd * D + cb * 64, c.tok0, &bar_in);
                tma_load_2d(sm + QK + cb * 16384 + 8192, &P.tm_k, c.hd * D + cb * 64, c.tok0, &bar_in);
            }
        }
        pending = true;
    };
    auto load_wu = [&](const ChunkInfo& c) {   // (channel-wise: and P, whose place the second product reads)
        bulk_load(sm + WT, p.ws + (CW ? p.L.img_W : p.L.W) + (size_t)c.ch * 16384, 16384, &bar_in);
        bulk_load(sm + UTT, p.ws + (CW ? p.L.img_U : p.L.Ut) + (size_t)c.ch * 16384, 16384, &bar_in);
        if (CW) bulk_load(sm + PT_CW, p.ws + p.L.Pm + (size_t)c.ch * 8192, 8192, &bar_in);
    };
    auto load_h = [&](const ChunkInfo& c) { bulk_load(sm + HH, p.ws + p.L.hc + (size_t)c.ch * 32768, 32768, &bar_in); };
    auto fetch_gamma = [&](const ChunkInfo& c) {   // threads 0..63: cumulative log decay of their token
        return reinterpret_cast<const float*>(p.ws + p.L.gamma)[(size_t)c.ch * kC + threadIdx.x];
    };
    ChunkInfo x;
    chunk_entry(p, x, blockIdx.x);
    if (threadIdx.x == 0) { load_qk(x, 0); load_wu(x); load_h(x); }
    float gnext = (!CW && threadIdx.x < kC) ? fetch_gamma(x) : 0.f;
    const int f = q4 * 32 + lane;            // feature row of the transposed accumulator (W h)^T
    const int tr = q4 * 16 + (lane & 15);    // token row of the M = 64 accumulators (lanes 0..15 of a quadrant hold them)
    const bool ga = lane < 16;
    const float sc = p.d.scale;
#pragma unroll 1
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, in_phase ^= 1) {
        const bool has_next = item + (int)gridDim.x < n_items;
        ChunkInfo xn = x;
        if (has_next) chunk_entry(p, xn, item + gridDim.x);
        if (!CW && threadIdx.x < kC) {
            gl[threadIdx.x] = gnext * kLog2e;
            Gam[threadIdx.x] = expf(gnext);
        }
        if (ok) {
            ok = mbar_wait(&bar_in, in_phase);
            if (!ok && threadIdx.x == 0) report_timeout(p.ws, 30);
            if (ok && threadIdx.x == 0) pending = false;
        }
        if (!CW && ok && x.len < kC) {   // ragged tail: rows beyond the sequence belong to somebody else (the images are padded)
            zero_tail_rows(sm + QK, 128, 0, x.len);
            zero_tail_rows(sm + QK, 128, 64, x.len);
            fence_async_smem();
        }
        __syncthreads();
        // ---- step 1: Q K^T ; (W h)^T ; Q h
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            if (!CW) mma_tile<64, 64, 128>(tmem + C_P, op_k_major(sm + QK, 128, 0), op_k_major(sm + QK, 128, 64), false);
            mma_tile<128, 64, 128>(tmem + C_WH, op_mn_major(sm + HH, 128), op_mn_major(sm + WT, 128), false);
            mma_tile<64, 128, 128>(tmem + C_QH, op_k_major(sm + QK, 128, 0), op_mn_major(sm + HH, 128), false);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(31)
        if (ok && has_next) {   // Q and K have been read for the last time
            if (threadIdx.x == 0) load_qk(xn, in_phase ^ 1);
            if (!CW && threadIdx.x < kC) gnext = fetch_gamma(xn);
        }
        if (ok) {   // P = tril(Q K^T . D) over W^T (dead), U = U~ - W h in place
            const int i0 = half * 32, j0 = half * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float v[8], u[8], t[8];
                const int jb = j0 + part * 8, ib = i0 + part * 8;
                if (!CW) tmem_ld8(tmem + lane_base + C_P + jb, v);
                tmem_ld8(tmem + lane_base + C_WH + ib, t);
                chunk_load(sm + UTT, 128, f, ib >> 3, u);
                tmem_wait_ld();
                if (!CW && ga) {
                    float g8[8];
                    ld8s(gl + jb, g8);
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = (jb + j <= tr) ? v[j] * ex2(gl[tr] - g8[j]) : 0.f;
                    chunk_store(sm + PT, 64, tr, jb >> 3, v);
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) u[i] -= t[i];
                chunk_store(sm + UTT, 128, f, ib >> 3, u);
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        // ---- step 2: P U (token-major, over the columns of the first two accumulators)
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            if (CW) mma_tile<64, 128, 64>(tmem + C_QH, op_k_major(sm + PT_CW, 64), op_k_major(sm + UTT, 128), true);
            else mma_tile<64, 128, 64>(tmem + C_PU, op_k_major(sm + PT, 64), op_k_major(sm + UTT, 128), false);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(32)
        if (ok && has_next && threadIdx.x == 0) load_wu(xn);   // P (over W^T) and U^T have been read for the last time
        if (ok) {   // o = scale (Gam . (Q h) + P U): the sixteen low lanes of a warp own a token row and 64 columns each
            const float coef = CW ? sc : sc * Gam[tr];
#pragma unroll 1
            for (int part = 0; part < 8; ++part) {
                const int cb = half * 64 + part * 8;
                float a[8], b[8];
                tmem_ld8(tmem + lane_base + C_QH + cb, a);
                if (!CW) tmem_ld8(tmem + lane_base + C_PU + cb, b);
                tmem_wait_ld();
                if (ga) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) b[j] = CW ? coef * a[j] : fmaf(coef, a[j], sc * b[j]);
                    chunk_store(sm + STG, 64, tr, cb >> 3, b);
                }
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        if (ok) {
            if (x.len == kC) {
                if (threadIdx.x == 0) {
                    for (int cb = 0; cb < 2; ++cb) tma_store_2d(&P.tm_o, x.hd * D + cb * 64, x.tok0, sm + STG + cb * 8192);
                    bulk_commit();
                }
            } else {
                flush_rows(sm + STG, reinterpret_cast<__nv_bfloat16*>(p.o) + ((size_t)x.tok0 * H + x.hd) * D, (size_t)H * D, x.len);
                __syncthreads();
            }
            if (threadIdx.x == 0) {
                bulk_wait_read<0>();            // the store has read the staged tile: h of the next trip may land on it
                if (has_next) load_h(xn);
            }
        }
        if (!ok) break;
        x = xn;
    }
    if (threadIdx.x == 0) {
        bulk_wait_read<0>();
        if (pending) (void)mbar_wait(&bar_in, pending_phase);   // after a timeout a load may still be in flight
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
}

#undef GDN_WAIT_MMA

}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
bool tc_supported(const gdn_desc& d) {
    return d.dtype == GDN_BF16 && d.d_k == 128 && d.d_v == 128 && d.chunk == kC;
}

thread_local int g_inject_timeout = 0;   // set by gdn_debug_inject_timeout, consumed by the next gdn_bwd of this family

static int sm_count();
// When one CTA per (chain, direction) of the backward fills more than half of the SMs the carries are bound by HBM
// bandwidth, and the low-rank form moves less.  With fewer chains a step's latency counts, and the operator form needs one
// product per step.  The rule looks at the chains only, so the forward, the backward and a backward on a workspace fresh
// from the forward agree on the form (and on the workspace layout that follows from it).
bool tc_carries_lowrank(const gdn_desc& d) {
    if (g_force_carries) return g_force_carries == 2;
    return 4 * (long long)d.N * d.H > sm_count();
}
static bool fill_params(TcParams& P, const Problem& p, bool with_bwd, int scan_dirs) {
    P.p = p;
    P.with_bwd = with_bwd ? 1 : 0;
    P.scan_dirs = scan_dirs;
    P.lowrank = tc_carries_lowrank(p.d) ? 1 : 0;
    P.withhold = 0;
    const uint64_t rows = (uint64_t)p.Ttot, cols = (uint64_t)p.d.H * D, pitch = cols * 2;
    if (!tc::make_tmap_bf16_2d(&P.tm_q, p.q, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_k, p.k, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_v, p.v, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_do, with_bwd ? p.dO : p.v, rows, cols, pitch, 64)) return false;
    if (!with_bwd && p.o && !tc::make_tmap_bf16_2d(&P.tm_o, p.o, rows, cols, pitch, 64)) return false;
    if (with_bwd) {
        if (!tc::make_tmap_bf16_2d(&P.tm_dq, p.dq, rows, cols, pitch, 64)) return false;
        if (!tc::make_tmap_bf16_2d(&P.tm_dk, p.dk, rows, cols, pitch, 64)) return false;
        if (!tc::make_tmap_bf16_2d(&P.tm_dv, p.dv, rows, cols, pitch, 64)) return false;
    }
    return true;
}

template <class Kernel>
static cudaError_t launch_chunk_kernel(Kernel kernel, SmemLimitOnce& once, uint32_t smem, Stage stage, int grid, int threads,
                                       const TcParams& P, cudaStream_t st) {
    const cudaError_t e = once.ensure(kernel, smem);
    if (e != cudaSuccess) return e;
    if (grid > 0) {
        StageScope t(stage, st);
        kernel<<<grid, threads, smem, st>>>(P);
    }
    return cudaGetLastError();
}

static int sm_count();
static cudaError_t launch_prep(const TcParams& P, cudaStream_t st) {
    static SmemLimitOnce done;
    const int items = P.p.L.max_chunks * P.p.d.H, sms = sm_count();
    return launch_chunk_kernel(tc_prep_kernel, done, prep::SMEM_BYTES, ST_PREP, items < sms ? items : sms, kIntraThreads + 32, P, st);
}
// Number of SMs of the current device (persistent kernels launch one CTA per SM).
static int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        cached[dev] = (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
    }
    return cached[dev];
}

// The two small preparation kernels, two CTAs per SM.
static cudaError_t launch_factors(const TcParams& P, cudaStream_t st) {
    static SmemLimitOnce done;
    const int items = P.p.L.max_chunks * P.p.d.H, ctas = 2 * sm_count();
    return launch_chunk_kernel(tc_factors_kernel, done, factors::SMEM_BYTES, ST_PREP, items < ctas ? items : ctas, split::kT, P, st);
}
static cudaError_t launch_eprep(const TcParams& P, cudaStream_t st) {
    static SmemLimitOnce done;
    const int items = P.p.L.max_chunks * P.p.d.H, ctas = 2 * sm_count();
    return launch_chunk_kernel(tc_eprep_kernel, done, eprep::SMEM_BYTES, ST_EPREP, items < ctas ? items : ctas, split::kT, P, st);
}

static cudaError_t launch_scan(const TcParams& P, cudaStream_t st) {
    static SmemLimitOnce done;
    static SmemLimitOnce done2;
    const int ctas = P.p.d.N * P.p.d.H * (P.scan_dirs == 2 ? 2 : 1);
    if (P.lowrank) {
        static SmemLimitOnce done_lr, done_lr2;
        // the reverse carry alone (backward on a fresh workspace) with few chains: two CTAs per chain, each carrying half of
        // the state columns (measured on 64 chains of 32 chunks: reverse 64 -> 58 us; the forward carry alone became
        // slower that way, 62 -> 66 us, and keeps one CTA per chain)
        if (P.scan_dirs == 1 && 2 * ctas <= sm_count())
            return launch_chunk_kernel(tc_scan_lr_kernel<2>, done_lr2, scanlr::Cfg<2>::SMEM_BYTES, ST_SCANS, 2 * ctas, kThreads, P, st);
        return launch_chunk_kernel(tc_scan_lr_kernel<1>, done_lr, scanlr::Cfg<1>::SMEM_BYTES, ST_SCANS, ctas, kThreads, P, st);
    }
    // few chains: two CTAs per (chain, direction), each carrying half of the state columns
    if (2 * ctas <= sm_count())
        return launch_chunk_kernel(tc_scan_kernel<2>, done2, scan::Cfg<2>::SMEM_BYTES, ST_SCANS, 2 * ctas, kThreads, P, st);
    return launch_chunk_kernel(tc_scan_kernel<1>, done, scan::Cfg<1>::SMEM_BYTES, ST_SCANS, ctas, kThreads, P, st);
}
static cudaError_t launch_intra(const TcParams& P, cudaStream_t st) {
    static SmemLimitOnce done;
    const int items = P.p.L.max_chunks * P.p.d.H, sms = sm_count();
    return launch_chunk_kernel(tc_intra_kernel, done, intra::SMEM_BYTES, ST_INTRA, items < sms ? items : sms, kIntraThreads + 32, P, st);
}
static cudaError_t launch_out(const TcParams& P, cudaStream_t st) {
    static SmemLimitOnce done;
    const int items = P.p.L.max_chunks * P.p.d.H, ctas = 2 * sm_count();
    return launch_chunk_kernel(tc_out_kernel<false>, done, outk::SMEM_BYTES, ST_OUT, items < ctas ? items : ctas, kThreads, P, st);
}

// Forward output of the channel-wise path from the tile images its preparation kernels and carries left in the workspace.
cudaError_t tc_launch_out_channelwise(const Problem& p, cudaStream_t st) {
    static SmemLimitOnce done;
    TcParams P{};
    P.p = p;
    const uint64_t rows = (uint64_t)p.Ttot, cols = (uint64_t)p.d.H * D;
    if (!tc::make_tmap_bf16_2d(&P.tm_o, p.o, rows, cols, cols * 2, 64)) return cudaErrorUnknown;
    const int items = p.L.max_chunks * p.d.H, ctas = 2 * sm_count();
    return launch_chunk_kernel(tc_out_kernel<true>, done, outk::SMEM_BYTES, ST_OUT, items < ctas ? items : ctas, kThreads, P, st);
}

// Carries of the channel-wise path: dirs = 0 forward, 1 reverse, 2 both in one launch.  Needs the tile images the
// channel-wise preparation kernels leave in the workspace; no tensor map is used.
cudaError_t tc_launch_scan_channelwise(const Problem& p, int dirs, cudaStream_t st) {
    static SmemLimitOnce done;
    TcParams P{};
    P.p = p;
    P.scan_dirs = dirs;
    P.lowrank = 1;
    const int ctas = p.d.N * p.d.H * (dirs == 2 ? 2 : 1);
    static SmemLimitOnce done2;
    if (dirs != 2 && 2 * ctas <= sm_count())
        return launch_chunk_kernel(tc_scan_cw_kernel<2>, done2, scanlr::Cfg<2>::SMEM_BYTES, ST_SCANS, 2 * ctas, kThreads, P, st);
    return launch_chunk_kernel(tc_scan_cw_kernel<1>, done, scanlr::Cfg<1>::SMEM_BYTES, ST_SCANS, ctas, kThreads, P, st);
}

// A call with no tokens still owes the pass-through of the states.
static cudaError_t empty_call(const Problem& p, bool bwd, cudaStream_t st) {
    const size_t bytes = (size_t)p.d.N * p.d.H * D * D * sizeof(float);
    float* dst = bwd ? p.dh0 : p.hT;
    const float* src = bwd ? p.dhT : p.h0;
    if (!dst) return cudaSuccess;
    return src ? cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, st) : cudaMemsetAsync(dst, 0, bytes, st);
}

// The chunk table is needed for packed sequences only (and for an empty call, whose only kernel it is).
static cudaError_t launch_table_if_needed(const Problem& p, cudaStream_t st) {
    return (p.cu || p.Ttot == 0) ? launch_table(p, st) : cudaSuccess;
}

// Carries in low-rank form take the chunk factors from tc_factors; in operator form they also need Nm and Bf, which
// only the fused tc_prep makes.
cudaError_t tc_launch_fwd(const Problem& p, cudaStream_t st) {
    TcParams P;
    cudaError_t e = launch_table_if_needed(p, st);
    if (e != cudaSuccess) return e;
    if (p.Ttot == 0) return empty_call(p, false, st);
    if (!fill_params(P, p, false, 0)) return cudaErrorUnknown;
    if ((e = P.lowrank ? launch_factors(P, st) : launch_prep(P, st)) != cudaSuccess) return e;
    if ((e = launch_scan(P, st)) != cudaSuccess) return e;
    return p.o ? launch_out(P, st) : cudaSuccess;
}

// With a workspace fresh from gdn_fwd_recompute nothing of the forward is repeated: T, W, U~ and the per-chunk states
// are taken from it, and only what needs dO is built (P, E; tc_eprep), followed by the reverse carry and the
// gradient stage.
cudaError_t tc_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st) {
    TcParams P;
    cudaError_t e = launch_table_if_needed(p, st);
    if (e != cudaSuccess) return e;
    if (p.Ttot == 0) return empty_call(p, true, st);
    if (!fill_params(P, p, true, skip_recompute ? 1 : 2)) return cudaErrorUnknown;
    const bool inject = g_inject_timeout && !skip_recompute;
    if (inject) {   // debugging hook, this call only: a millisecond of patience, and tc_prep withholds one load
        const unsigned long long ns = 1000000ull;
        g_inject_timeout = 0;
        P.withhold = 1;
        if ((e = cudaMemcpyToSymbolAsync(g_wait_limit_ns, &ns, sizeof(ns), 0, cudaMemcpyHostToDevice, st)) != cudaSuccess) return e;
    }
    // (the closed arm keeps the fused kernel: it reads k once and never moves W through HBM on its way to E; measured on
    // B = 4, T = 2048, H = 16: fused 99 us, tc_factors + tc_eprep 62 + 45 us)
    if ((e = skip_recompute ? launch_eprep(P, st) : launch_prep(P, st)) != cudaSuccess) return e;
    if ((e = launch_scan(P, st)) != cudaSuccess) return e;
    e = launch_intra(P, st);
    if (inject) {
        const unsigned long long ns = 2000000000ull;
        const cudaError_t e2 = cudaMemcpyToSymbolAsync(g_wait_limit_ns, &ns, sizeof(ns), 0, cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = e2;
    }
    return e;
}

}  // namespace gdn

