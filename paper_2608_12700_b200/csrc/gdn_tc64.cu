// tcgen05 kernels for the scalar-gate linear recurrence (delta rule off: erase gate 0, write gate 1; the SSD-like
// row of Table 2 of the paper), bf16 I/O, d_k = d_v = 64, chunk 64.
//
// With the erase gate at zero the triangular solve vanishes (M = 0, T = I, W = 0, U~ = V; Section 4.1), so the
// carries lose their matrix operator:   h' = Gam_e h + Kb^T V,   dh = Gam_e dh' + scale (Diag(Gam) Q)^T dO.
// A chain step then costs one small product, and the whole backward fits two sequential passes per chain that
// move little more than the inputs and outputs themselves:
//   tc64_fwd  (one CTA per chain, chunks ascending)   h per chunk -> workspace (8 KB bf16 tile image per chunk)
//   tc64_bwd  (one CTA per chain, chunks descending)  dh' carried in registers; per chunk all of
//             P = tril(Q K^T . D), dP = scale tril(dO V^T), dv = scale P^T dO + Diag(e) K dh',
//             dq = scale Gam (dO h^T) + (dP.D) K,  dk = (dP.D)^T Q + Diag(e) V dh'^T,
//             dgamma_i = <q_i,dq_i> - <k_i,dk_i>,  dgamma_63 += sum_j r_j + Gam_e <dh',h>,  dg = reverse cumsum.
// Accumulators are 64 x 64 (M = 64: row i on TMEM lane i % 16 + 32 (i / 16)), token rows on lanes, so a thread owns
// a token row: row dots are thread-local and gradient rows leave with 16-byte stores.  Two CTAs share an SM.
#define GDN_INLINE_WAIT   // small kernels: the polling loops sit at the wait sites (see tc_ptx.cuh)
#include "tc_common.cuh"

namespace gdn {

namespace {

constexpr int D6 = 64;
constexpr int kThreads64 = 256;   // 8 warps: lane quadrant = warp % 4 (rows 16 q .. 16 q + 15 on lanes 0..15), column half = warp / 4

struct Tc64Params {
    Problem p;
    CUtensorMap tm_q, tm_k, tm_v, tm_do;   // [T_total, H * 64] bf16, boxes of 64 rows x 64 columns
    CUtensorMap tm_dq, tm_dk, tm_dv;       // same geometry, for the gradient stores of full chunks
};

// Chunk-local cumulative log decay.  A block takes one chunk and 32 heads: the [64 tokens][32 heads] patch of g is
// read token by token (128 contiguous bytes each), then each warp scans the tokens of four heads (lane l owns
// tokens l and l + 32).  First kernel of a call.
__global__ void __launch_bounds__(256) tc64_gamma_kernel(Problem p) {
    init_header_if_untabled(p);
    __shared__ float gs[kC][33];
    const int c = blockIdx.x, h0 = blockIdx.y * 32, H = p.d.H;
    if (c >= n_chunks_of(p)) return;
    const ChunkGeom cg = chunk_geom(p);
    const int tok0 = cg.chunk_tok0(c), len = cg.chunk_len(c);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = warp; i < kC; i += 8)
        gs[i][lane] = (i < len && h0 + lane < H) ? p.g[(size_t)(tok0 + i) * H + h0 + lane] : 0.f;
    __syncthreads();
    for (int hh = warp; hh < 32 && h0 + hh < H; hh += 8) {
        float a = gs[lane][hh], b = gs[lane + 32][hh];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float ua = __shfl_up_sync(0xffffffffu, a, o), ub = __shfl_up_sync(0xffffffffu, b, o);
            if (lane >= o) { a += ua; b += ub; }
        }
        b += __shfl_sync(0xffffffffu, a, 31);
        float* out = reinterpret_cast<float*>(p.ws + p.L.gamma) + ((size_t)c * H + h0 + hh) * kC;
        out[lane] = a;
        out[lane + 32] = b;
    }
}

__device__ __forceinline__ void zero_tail_rows64(unsigned char* tile, int len) {   // [64][64] tile; threads 0 .. kThreads64-1
    for (int t = threadIdx.x; t < (kC - len) * 8; t += kThreads64)
        *reinterpret_cast<uint4*>(tile + tile_chunk_off(64, len + t / 8, t % 8)) = make_uint4(0, 0, 0, 0);
}

// ------------------------------------------------------------------------------------------------
// forward pass
// ------------------------------------------------------------------------------------------------
namespace f64 {
constexpr int STAGES = 2;
constexpr uint32_t KT = 0, VT = 8192, QT = 16384, STAGE_BYTES = 24576;   // per stage: K, V (and Q when o is wanted)
constexpr uint32_t VE = STAGES * STAGE_BYTES;   // Diag(e) V
constexpr uint32_t HT = VE + 8192;              // bf16 state tile: leaves for the workspace by a bulk store; operand of Q h
constexpr uint32_t PT = HT + 8192;              // P (only when o is wanted)
constexpr uint32_t SMEM_BYTES = PT + 8192 + 1024;
}  // namespace f64

__global__ void __launch_bounds__(kThreads64, 2) tc64_fwd_kernel(const __grid_constant__ Tc64Params P) {
    using namespace f64;
    const Problem& p = P.p;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    if (hdr->status != GDN_OK) return;
    const int H = p.d.H;
    const int n = blockIdx.x / H, hd = blockIdx.x % H;
    const SeqGeom cg = seq_geom(p, n);
    const int c0 = cg.c0, nsteps = cg.n_chunks;
    const bool want_o = p.o != nullptr;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ __align__(16) float gl[kC], Gam[kC], ee[kC];
    __shared__ uint64_t bar_full[STAGES], bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, half = warp >> 2;
    const int r = q4 * 16 + (lane & 15);      // row of the 64 x 64 accumulators / of the state held by this lane
    const bool act = lane < 16;
    const int cb0 = half * 32;                // first of its 32 columns
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&bar_full[s], 1);
        mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    auto fill = [&](int s) {
        const int stage = s % STAGES, tok0 = cg.chunk_tok0(c0 + s);
        unsigned char* st = sm + stage * STAGE_BYTES;
        mbar_expect_tx(&bar_full[stage], want_o ? 24576 : 16384);
        tma_load_2d(st + KT, &P.tm_k, hd * D6, tok0, &bar_full[stage]);
        tma_load_2d(st + VT, &P.tm_v, hd * D6, tok0, &bar_full[stage]);
        if (want_o) tma_load_2d(st + QT, &P.tm_q, hd * D6, tok0, &bar_full[stage]);
    };
    if (threadIdx.x == 0)
        for (int s = 0; s < STAGES && s < nsteps; ++s) fill(s);

    float st[32];
    const size_t soff = ((size_t)n * H + hd) * D6 * D6 + (size_t)r * D6 + cb0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        float4 v = (p.h0 && act) ? *reinterpret_cast<const float4*>(p.h0 + soff + 4 * k) : make_float4(0.f, 0.f, 0.f, 0.f);
        st[4 * k] = v.x; st[4 * k + 1] = v.y; st[4 * k + 2] = v.z; st[4 * k + 3] = v.w;
    }
    const float* gamma = reinterpret_cast<const float*>(p.ws + p.L.gamma);
    float gnext = (threadIdx.x < kC && nsteps > 0) ? gamma[((size_t)c0 * H + hd) * kC + threadIdx.x] : 0.f;
    bool ok = true;
    uint32_t mma_phase = 0;
    int len_n = nsteps > 0 ? cg.chunk_len(c0) : 0;   // fetched a step ahead
#pragma unroll 1
    for (int s = 0; s < nsteps; ++s) {
        const int c = c0 + s, stage = s % STAGES, len = len_n;
        if (s + 1 < nsteps) len_n = cg.chunk_len(c + 1);
        const size_t ch = (size_t)c * H + hd;
        unsigned char* tiles = sm + stage * STAGE_BYTES;
        if (threadIdx.x == 32) bulk_wait_read<0>();   // the previous step's state tile has left shared memory
        if (threadIdx.x < kC) {
            gl[threadIdx.x] = gnext * kLog2e;
            Gam[threadIdx.x] = expf(gnext);
            if (s + 1 < nsteps) gnext = gamma[(ch + H) * kC + threadIdx.x];
        }
        __syncthreads();
        if (threadIdx.x < kC) ee[threadIdx.x] = ex2(gl[kC - 1] - gl[threadIdx.x]);
        ok = mbar_wait(&bar_full[stage], (s / STAGES) & 1);
        if (!ok) { if (threadIdx.x == 0) report_timeout(p.ws, 40); break; }
        if (len < kC) {
            zero_tail_rows64(tiles + KT, len);
            zero_tail_rows64(tiles + VT, len);
            if (want_o) zero_tail_rows64(tiles + QT, len);
        }
        __syncthreads();
        const float Ge = Gam[kC - 1];
        for (int t = threadIdx.x; t < kC * 8; t += blockDim.x) {   // Diag(e) V
            const int i = t >> 3, cch = t & 7;
            float v[8];
            chunk_load(tiles + VT, 64, i, cch, v);
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] *= ee[i];
            chunk_store(sm + VE, 64, i, cch, v);
        }
        if (act) {   // state entering the chunk -> bf16 tile: the workspace copy (and, for o, the MMA operand)
#pragma unroll
            for (int k = 0; k < 4; ++k)
                *reinterpret_cast<uint4*>(sm + HT + tile_chunk_off(64, r, (cb0 >> 3) + k)) = pack8(st + 8 * k);
        }
        fence_async_smem();
        __syncthreads();
        if (threadIdx.x == 32) {   // the tile leaves through the async proxy (generic global stores would stall the next proxy fence)
            bulk_store(p.ws + p.L.hc + ch * 8192, sm + HT, 8192);
            bulk_commit();
        }
        if (threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<64, 64, 64>(tmem + 0, op_mn_major(tiles + KT, 64), op_mn_major(sm + VE, 64), false);              // Kb^T V
            if (want_o) {
                mma_tile<64, 64, 64>(tmem + 64, op_k_major(tiles + QT, 64), op_k_major(tiles + KT, 64), false);         // Q K^T
                mma_tile<64, 64, 64>(tmem + 128, op_k_major(tiles + QT, 64), op_mn_major(sm + HT, 64), false);          // Q h
            }
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(41)
        if (!ok) break;
        // without o the stage's K and V have now been read for the last time: refill it while the state is updated
        if (!want_o && threadIdx.x == 32 && s + STAGES < nsteps) fill(s + STAGES);
        if (want_o) {   // o = scale (Gam_i (Q h)_i + (P V)_i)
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float v[8];
                const int jb = cb0 + part * 8;
                tmem_ld8(tmem + lane_base + 64 + jb, v);
                tmem_wait_ld();
                if (act) {
                    float g8[8];
                    ld8s(gl + jb, g8);
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = (jb + j <= r) ? v[j] * ex2(gl[r] - g8[j]) : 0.f;
                    chunk_store(sm + PT, 64, r, jb >> 3, v);
                }
            }
            tc_fence_before();
            fence_async_smem();
            __syncthreads();
            if (threadIdx.x == 0) {
                tc_fence_after();
                mma_tile<64, 64, 64>(tmem + 192, op_k_major(sm + PT, 64), op_mn_major(tiles + VT, 64), false);          // P V
                mma_commit(&bar_mma);
            }
            GDN_WAIT_MMA(42)
            if (!ok) break;
            __nv_bfloat16* go = reinterpret_cast<__nv_bfloat16*>(p.o) + ((size_t)(cg.chunk_tok0(c) + r) * H + hd) * D6;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float a[8], b[8];
                const int jb = cb0 + part * 8;
                tmem_ld8(tmem + lane_base + 128 + jb, a);
                tmem_ld8(tmem + lane_base + 192 + jb, b);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 8; ++j) a[j] = p.d.scale * fmaf(Gam[r], a[j], b[j]);
                if (act && r < len) *reinterpret_cast<uint4*>(go + jb) = pack8(a);
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {   // h' = Gam_e h + Kb^T V
            float bf[8];
            tmem_ld8(tmem + lane_base + 0 + cb0 + 8 * k, bf);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) st[8 * k + j] = fmaf(Ge, st[8 * k + j], bf[j]);
        }
        tc_fence_before();
        if (want_o) {
            __syncthreads();   // every reader of this stage's tiles is done
            if (threadIdx.x == 0 && s + STAGES < nsteps) fill(s + STAGES);
        }
    }
    if (threadIdx.x == 32) bulk_wait_read<0>();
    if (p.hT && ok && act) {
#pragma unroll
        for (int k = 0; k < 8; ++k) *reinterpret_cast<float4*>(p.hT + soff + 4 * k) = make_float4(st[4 * k], st[4 * k + 1], st[4 * k + 2], st[4 * k + 3]);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 256);
}

// ------------------------------------------------------------------------------------------------
// backward pass
// ------------------------------------------------------------------------------------------------
namespace b64 {
constexpr int STAGES = 2;
constexpr uint32_t QT = 0, KT = 8192, VT = 16384, OT = 24576, HT = 32768, STAGE_BYTES = 40960;   // Q, K, V, dO, h
constexpr uint32_t DH = STAGES * STAGE_BYTES;   // bf16 tile of the carried dh' during phase 1, then Diag(Gam) dO
constexpr uint32_t PX = DH + 8192;              // P
constexpr uint32_t DPD = PX + 8192;             // scale tril(dO V^T) . D
constexpr uint32_t SMEM_BYTES = DPD + 8192 + 1024;
static_assert(2 * (SMEM_BYTES + 4096) <= 227 * 1024, "two CTAs per SM");
// Tensor memory: 256 columns per CTA so that two CTAs share an SM.  A 64-row accumulator occupies lanes 0..15 of
// each 32-lane quadrant; a second one lives in lanes 16..31 of the same columns (address + 16 lanes).  Lanes 0..15
// of every warp ("group A") therefore read S, dO V^T, K dh', P^T dO and the state increment, lanes 16..31 ("group
// B") read dO h^T, (dP.D) K, V dh'^T and (dP.D)^T Q with the same load instructions.
constexpr uint32_t C0 = 0, C1 = 64, C2 = 128, C3 = 192, LB = 16u << 16;
}  // namespace b64

__global__ void __launch_bounds__(kThreads64 + 32, 2) tc64_bwd_kernel(const __grid_constant__ Tc64Params P) {
    using namespace b64;
    const Problem& p = P.p;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    if (hdr->status != GDN_OK) return;
    const int H = p.d.H;
    const int n = blockIdx.x / H, hd = blockIdx.x % H;
    const SeqGeom cg = seq_geom(p, n);
    const int c0 = cg.c0, nsteps = cg.n_chunks, c1 = c0 + nsteps;
    const float sc = p.d.scale;

    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ __align__(16) float gl2[2][kC], Gam2[2][kC], ee2[2][kC], dgp[2][kC], scal[2][kThreads64 / 32];
    __shared__ uint64_t bar_full[STAGES], bar_st, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, half = warp >> 2;
    const int r = q4 * 16 + (lane & 15);      // accumulator / state row of this lane
    const bool ga = lane < 16;                // group A: lanes 0..15, group B: lanes 16..31
    const int cb0 = half * 32;                // first of this thread's 32 columns
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;

    // Warp 8 only moves data: its first lane stores a step's staged gradients and then loads the tiles of the step
    // after next into the ring slot they came from.  It follows the other warps through an mbarrier and shares no
    // block-wide barrier with them inside the loop (they use a named barrier).
    const bool loader = warp == kThreads64 / 32;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) mbar_init(&bar_full[s], 1);
        mbar_init(&bar_st, 1);
        mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    auto fill = [&](int s) {   // step s handles chunk c1 - 1 - s
        const int stage = s % STAGES, c = c1 - 1 - s, tok0 = cg.chunk_tok0(c);
        unsigned char* st = sm + stage * STAGE_BYTES;
        mbar_expect_tx(&bar_full[stage], 40960);
        tma_load_2d(st + QT, &P.tm_q, hd * D6, tok0, &bar_full[stage]);
        tma_load_2d(st + KT, &P.tm_k, hd * D6, tok0, &bar_full[stage]);
        tma_load_2d(st + VT, &P.tm_v, hd * D6, tok0, &bar_full[stage]);
        tma_load_2d(st + OT, &P.tm_do, hd * D6, tok0, &bar_full[stage]);
        bulk_load(st + HT, p.ws + p.L.hc + ((size_t)c * H + hd) * 8192, 8192, &bar_full[stage]);
    };
    if (loader) {
        if (lane == 0) {
            for (int s = 0; s < STAGES && s < nsteps; ++s) fill(s);
#pragma unroll 1
            for (int s = 0; s < nsteps; ++s) {
                if (!mbar_wait(&bar_st, s & 1)) break;          // step s has staged its gradient rows (or flushed them)
                const int c = c1 - 1 - s;
                if (cg.chunk_len(c) == kC) {
                    const int tok0 = cg.chunk_tok0(c);
                    unsigned char* st = sm + (s % STAGES) * STAGE_BYTES;
                    tma_store_2d(&P.tm_dv, hd * D6, tok0, st + VT);
                    tma_store_2d(&P.tm_dk, hd * D6, tok0, st + KT);
                    tma_store_2d(&P.tm_dq, hd * D6, tok0, st + QT);
                    bulk_commit();
                    bulk_wait_read<0>();   // the ring slot is loaded over next
                }
                if (s + STAGES < nsteps) fill(s + STAGES);
            }
            bulk_wait_read<0>();
        }
        return;
    }
    auto cta_sync = [] { asm volatile("bar.sync 1, %0;" ::"n"(kThreads64) : "memory"); };   // all warps but the loader

    float st[32];   // group A: dh' row r, columns cb0 .. cb0 + 31 (gradient w.r.t. the state leaving the current chunk)
    const size_t soff = ((size_t)n * H + hd) * D6 * D6 + (size_t)r * D6 + cb0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        float4 v = (p.dhT && ga) ? *reinterpret_cast<const float4*>(p.dhT + soff + 4 * k) : make_float4(0.f, 0.f, 0.f, 0.f);
        st[4 * k] = v.x; st[4 * k + 1] = v.y; st[4 * k + 2] = v.z; st[4 * k + 3] = v.w;
    }
    // Gate arrays of a step (log2-scaled cumulative decay, Gam = exp(gam), e = exp(gam_end - gam)) are prepared one
    // step ahead, into the other of two sets, while the tensor pipe works; their inputs are fetched a step before that.
    const float* gamma = reinterpret_cast<const float*>(p.ws + p.L.gamma);
    auto gate_row = [&](int step) { return gamma + ((size_t)(c1 - 1 - step) * H + hd) * kC; };
    auto make_gates = [&](int set, float g, float gend) {
        gl2[set][threadIdx.x] = g * kLog2e;
        Gam2[set][threadIdx.x] = expf(g);
        ee2[set][threadIdx.x] = ex2((gend - g) * kLog2e);
    };
    float gnext = 0.f, gend_next = 0.f;
    if (threadIdx.x < kC && nsteps > 0) {
        make_gates(0, gate_row(0)[threadIdx.x], gate_row(0)[kC - 1]);
        if (nsteps > 1) { gnext = gate_row(1)[threadIdx.x]; gend_next = gate_row(1)[kC - 1]; }
    }
    bool ok = true;
    uint32_t mma_phase = 0;
    int len_n = nsteps > 0 ? cg.chunk_len(c1 - 1) : 0, tok0_n = nsteps > 0 ? cg.chunk_tok0(c1 - 1) : 0;   // fetched a step ahead
#pragma unroll 1
    for (int s = 0; s < nsteps; ++s) {
        const int c = c1 - 1 - s, stage = s % STAGES, len = len_n, tok0 = tok0_n;
        if (s + 1 < nsteps) { len_n = cg.chunk_len(c - 1); tok0_n = cg.chunk_tok0(c - 1); }
        unsigned char* tiles = sm + stage * STAGE_BYTES;
        const float *gl = gl2[s & 1], *Gam = Gam2[s & 1], *ee = ee2[s & 1];
        ok = mbar_wait(&bar_full[stage], (s / STAGES) & 1);
        if (!ok) { if (threadIdx.x == 0) report_timeout(p.ws, 50); break; }
        if (len < kC) {
            zero_tail_rows64(tiles + QT, len);
            zero_tail_rows64(tiles + KT, len);
            zero_tail_rows64(tiles + VT, len);
            zero_tail_rows64(tiles + OT, len);
        }
        float hh = 0.f;   // <dh', h> restricted to this thread's part of the state
        if (ga) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float hv[8];
                chunk_load(tiles + HT, 64, r, (cb0 >> 3) + k, hv);
#pragma unroll
                for (int j = 0; j < 8; ++j) hh = fmaf(st[8 * k + j], hv[j], hh);
                chunk_store(sm + DH, 64, r, (cb0 >> 3) + k, st + 8 * k);
            }
        }
        fence_async_smem();
        cta_sync();
        const float Ge = Gam[kC - 1];
        // ---- phase 1: S = Q K^T ; dO V^T ; K dh' (group A) | dO h^T ; V dh'^T (group B)
        if (threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<64, 64, 64>(tmem + C0, op_k_major(tiles + QT, 64), op_k_major(tiles + KT, 64), false);
            mma_tile<64, 64, 64>(tmem + C1, op_k_major(tiles + OT, 64), op_k_major(tiles + VT, 64), false);
            mma_tile<64, 64, 64>(tmem + C2, op_k_major(tiles + KT, 64), op_mn_major(sm + DH, 64), false);
            mma_tile<64, 64, 64>(tmem + C0 + LB, op_k_major(tiles + OT, 64), op_k_major(tiles + HT, 64), false);
            mma_tile<64, 64, 64>(tmem + C2 + LB, op_k_major(tiles + VT, 64), op_k_major(sm + DH, 64), false);
            mma_commit(&bar_mma);
        }
        if (threadIdx.x < kC && s + 1 < nsteps) {
            make_gates((s + 1) & 1, gnext, gend_next);
            if (s + 2 < nsteps) { gnext = gate_row(s + 2)[threadIdx.x]; gend_next = gate_row(s + 2)[kC - 1]; }
        }
        GDN_WAIT_MMA(51)
        if (!ok) break;
        for (int t = threadIdx.x; t < kC * 8; t += kThreads64) {   // Diag(Gam) dO over the dh' tile, which no MMA reads any more
            const int i = t >> 3, cch = t & 7;
            float v[8];
            chunk_load(tiles + OT, 64, i, cch, v);
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] *= Gam[i];
            chunk_store(sm + DH, 64, i, cch, v);
        }
        float rs = 0.f;   // sum_j r_j, r_j = e_j <(K dh')_j, V_j>
#pragma unroll 1
        for (int part = 0; part < 4; ++part) {
            float s8[8], p8[8], kd[8], vv[8];
            const int jb = cb0 + part * 8;
            tmem_ld8(tmem + lane_base + C0 + jb, s8);
            tmem_ld8(tmem + lane_base + C1 + jb, p8);
            tmem_ld8(tmem + lane_base + C2 + jb, kd);
            tmem_wait_ld();
            if (ga) {
                chunk_load(tiles + VT, 64, r, jb >> 3, vv);
                float g8[8];
                ld8s(gl + jb, g8);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float dcy = (jb + j <= r) ? ex2(gl[r] - g8[j]) : 0.f;   // masked first: the exponent is never positive
                    s8[j] *= dcy;                   // P
                    p8[j] *= sc * dcy;              // dP . D
                    rs = fmaf(kd[j], vv[j], rs);
                }
                chunk_store(sm + PX, 64, r, jb >> 3, s8);
                chunk_store(sm + DPD, 64, r, jb >> 3, p8);
            }
        }
        rs *= ee[r];
        tc_fence_before();
        fence_async_smem();
        cta_sync();
        // ---- phase 2: P^T dO ; (Diag(Gam) Q)^T dO (group A) | (dP.D) K ; (dP.D)^T Q (group B)
        if (threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<64, 64, 64>(tmem + C3, op_mn_major(sm + PX, 64), op_mn_major(tiles + OT, 64), false);
            mma_tile<64, 64, 64>(tmem + C0, op_mn_major(tiles + QT, 64), op_mn_major(sm + DH, 64), false);
            mma_tile<64, 64, 64>(tmem + C1 + LB, op_k_major(sm + DPD, 64), op_mn_major(tiles + KT, 64), false);
            mma_tile<64, 64, 64>(tmem + C3 + LB, op_mn_major(sm + DPD, 64), op_mn_major(tiles + QT, 64), false);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(52)
        if (!ok) break;
        float dot = 0.f;   // group B: <q_r, dq_r> - <k_r, dk_r> over this thread's columns
        // Gradient rows are staged token-major in place over this step's input tiles (dv over V, which was last read in
        // phase 1; dk over K and dq over Q, where a thread overwrites exactly the piece it has just read) and leave by TMA
        // stores; generic global stores here would be one 16-byte piece per row.
#pragma unroll 1
        for (int part = 0; part < 4; ++part) {
            float a[8], b[8], x[8];
            const int jb = cb0 + part * 8;
            tmem_ld8(tmem + lane_base + C3 + jb, a);     // A: P^T dO        B: (dP.D)^T Q
            tmem_ld8(tmem + lane_base + C2 + jb, b);     // A: K dh'         B: V dh'^T
            tmem_wait_ld();
            if (ga) {
#pragma unroll
                for (int j = 0; j < 8; ++j) a[j] = fmaf(sc, a[j], ee[r] * b[j]);      // dv = scale P^T dO + Diag(e) K dh'
                chunk_store(tiles + VT, 64, r, jb >> 3, a);
            } else {
                chunk_load(tiles + KT, 64, r, jb >> 3, x);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    a[j] = fmaf(ee[r], b[j], a[j]);                                    // dk = (dP.D)^T Q + Diag(e) V dh'^T
                    dot = fmaf(-x[j], a[j], dot);
                }
                chunk_store(tiles + KT, 64, r, jb >> 3, a);
            }
            tmem_ld8(tmem + lane_base + C0 + jb, a);     //                  B: dO h^T
            tmem_ld8(tmem + lane_base + C1 + jb, b);     //                  B: (dP.D) K
            tmem_wait_ld();
            if (!ga) {
                chunk_load(tiles + QT, 64, r, jb >> 3, x);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    a[j] = fmaf(sc * Gam[r], a[j], b[j]);                              // dq = scale Gam dO h^T + (dP.D) K
                    dot = fmaf(x[j], a[j], dot);
                }
                chunk_store(tiles + QT, 64, r, jb >> 3, a);
            }
        }
        if (!ga) dgp[half][r] = dot;
        // group A: dh = Gam_e dh' + scale (Diag(Gam) Q)^T dO
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float e8[8];
            tmem_ld8(tmem + lane_base + C0 + cb0 + 8 * k, e8);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 8; ++j) st[8 * k + j] = fmaf(Ge, st[8 * k + j], sc * e8[j]);
        }
        rs = warp_sum(ga ? rs : 0.f);
        hh = warp_sum(ga ? hh : 0.f);
        if (lane == 0) { scal[0][warp] = rs; scal[1][warp] = hh; }
        tc_fence_before();
        fence_async_smem();
        cta_sync();   // every reader of this stage's tiles is done; partial sums and staged rows are visible
        if (len < kC) {   // ragged tail: rows beyond the sequence must not be written
            const size_t gbase = ((size_t)tok0 * H + hd) * D6;
            for (int t = threadIdx.x; t < kC * 8; t += kThreads64) {
                const int i = t >> 3, chk = t & 7;
                if (i < len) {
                    const size_t o = gbase + (size_t)i * H * D6 + chk * 8;
                    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.dv) + o) = *reinterpret_cast<const uint4*>(tiles + VT + tile_chunk_off(64, i, chk));
                    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.dk) + o) = *reinterpret_cast<const uint4*>(tiles + KT + tile_chunk_off(64, i, chk));
                    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.dq) + o) = *reinterpret_cast<const uint4*>(tiles + QT + tile_chunk_off(64, i, chk));
                }
            }
            cta_sync();   // the ring slot is handed to the loader only after every row has been read
        }
        if (threadIdx.x == 32) mbar_arrive(&bar_st);
        if (warp == 0) {
            float rsum = 0.f, hsum = 0.f;
            for (int w = 0; w < kThreads64 / 32; ++w) { rsum += scal[0][w]; hsum += scal[1][w]; }
            write_dg_suffix(dgp[0], dgp[1], rsum + Ge * hsum, p.dg + (size_t)tok0 * H + hd, (size_t)H, len, lane);
        }
    }
    if (p.dh0 && ok && ga) {
#pragma unroll
        for (int k = 0; k < 8; ++k) *reinterpret_cast<float4*>(p.dh0 + soff + 4 * k) = make_float4(st[4 * k], st[4 * k + 1], st[4 * k + 2], st[4 * k + 3]);
    }
    tc_fence_before();
    cta_sync();
    if (warp == 0) tmem_dealloc(tmem, 256);
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
bool tc64_supported(const gdn_desc& d) {
    return d.dtype == GDN_BF16 && d.d_k == 64 && d.d_v == 64 && d.delta_rule == 0 && d.chunk == kC;
}

static bool fill_params64(Tc64Params& P, const Problem& p, bool with_bwd) {
    P.p = p;
    const uint64_t rows = (uint64_t)p.Ttot, cols = (uint64_t)p.d.H * D6, pitch = cols * 2;
    if (!tc::make_tmap_bf16_2d(&P.tm_q, p.q, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_k, p.k, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_v, p.v, rows, cols, pitch, 64)) return false;
    if (!tc::make_tmap_bf16_2d(&P.tm_do, with_bwd ? p.dO : p.v, rows, cols, pitch, 64)) return false;
    if (with_bwd) {
        if (!tc::make_tmap_bf16_2d(&P.tm_dq, p.dq, rows, cols, pitch, 64)) return false;
        if (!tc::make_tmap_bf16_2d(&P.tm_dk, p.dk, rows, cols, pitch, 64)) return false;
        if (!tc::make_tmap_bf16_2d(&P.tm_dv, p.dv, rows, cols, pitch, 64)) return false;
    }
    return true;
}

static cudaError_t tc64_prologue(const Problem& p, cudaStream_t st) {
    // the chunk table is needed for packed sequences only (and for an empty call, whose only kernel it is)
    if (p.cu || p.Ttot == 0) {
        const cudaError_t e = launch_table(p, st);
        if (e != cudaSuccess) return e;
    }
    if (p.L.max_chunks > 0 && p.Ttot > 0) {
        StageScope t(ST_PREP, st);
        tc64_gamma_kernel<<<dim3(p.L.max_chunks, (p.d.H + 31) / 32), 256, 0, st>>>(p);
    }
    return cudaGetLastError();
}

static cudaError_t tc64_fwd_pass(const Tc64Params& P, cudaStream_t st) {
    static SmemLimitOnce once;
    const cudaError_t e0 = once.ensure(tc64_fwd_kernel, f64::SMEM_BYTES);
    if (e0 != cudaSuccess) return e0;
    const int chains = P.p.d.N * P.p.d.H;
    if (chains > 0) {
        StageScope t(ST_FSCAN, st);
        tc64_fwd_kernel<<<chains, kThreads64, f64::SMEM_BYTES, st>>>(P);
    }
    return cudaGetLastError();
}

cudaError_t tc64_launch_fwd(const Problem& p, cudaStream_t st) {
    Tc64Params P;
    cudaError_t e = tc64_prologue(p, st);
    if (e != cudaSuccess) return e;
    if (p.Ttot == 0) {
        const size_t bytes = (size_t)p.d.N * p.d.H * D6 * D6 * sizeof(float);
        if (!p.hT) return cudaSuccess;
        return p.h0 ? cudaMemcpyAsync(p.hT, p.h0, bytes, cudaMemcpyDeviceToDevice, st) : cudaMemsetAsync(p.hT, 0, bytes, st);
    }
    if (!fill_params64(P, p, false)) return cudaErrorUnknown;
    return tc64_fwd_pass(P, st);
}

cudaError_t tc64_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st) {
    Tc64Params P;
    cudaError_t e = tc64_prologue(p, st);
    if (e != cudaSuccess) return e;
    if (p.Ttot == 0) {
        const size_t bytes = (size_t)p.d.N * p.d.H * D6 * D6 * sizeof(float);
        if (!p.dh0) return cudaSuccess;
        return p.dhT ? cudaMemcpyAsync(p.dh0, p.dhT, bytes, cudaMemcpyDeviceToDevice, st) : cudaMemsetAsync(p.dh0, 0, bytes, st);
    }
    if (!fill_params64(P, p, true)) return cudaErrorUnknown;
    if (!skip_recompute) {
        Tc64Params F = P;
        F.p.o = nullptr;   // the backward never asks for the forward outputs
        F.p.hT = nullptr;
        if ((e = tc64_fwd_pass(F, st)) != cudaSuccess) return e;
    }
    static SmemLimitOnce once;
    if ((e = once.ensure(tc64_bwd_kernel, b64::SMEM_BYTES)) != cudaSuccess) return e;
    const int chains = p.d.N * p.d.H;
    if (chains > 0) {
        StageScope t(ST_RSCAN, st);
        tc64_bwd_kernel<<<chains, kThreads64 + 32, b64::SMEM_BYTES, st>>>(P);
    }
    return cudaGetLastError();
}

}  // namespace gdn

