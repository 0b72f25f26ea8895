// tcgen05 / TMEM kernels of the channel-wise path (per-channel gates, Eq. 1 of the paper as printed) for bf16 I/O and
// d_k = d_v = 128.
//
// "The channel-wise path folds the per-channel decay Diag(e^{g_t}) inside those contractions" (Appendix A): with the
// chunk-local cumulative log decay gam_i in R^{d_k} (reference: the chunk start, so gam <= 0 for a decaying gate) every
// factor exp(gam_i - gam_j) of a token pair splits into a row part and a column part, and the keys and queries are
// scaled once, element by element, before any product:
//     q~_i = Gam_i . q_i      k+_i = Gam_i . b_i . k_i   (row role)      k-_j = k_j / Gam_j   (column role)
//     v~_i = w_i . v_i        Kb_j = Gam_e . k-_j        (carries)        dO'  = scale dO
// In these variables the chunk is a decay-free delta rule whose token-token matrices carry plain triangular masks:
//     A = stril(K+ K-^T)   P = tril(Q~ K-^T)   T = (I + A)^-1   W = T K+   U~ = T V~   E = (Q~ - P W)^T dO'
//     U = U~ - W h   dU = P^T dO' + K- dh''   (dh'' = Diag(Gam_e) dh')
//     dP = tril(dO' U^T)   dW = -dU h^T   dXk = T^T dW   dXv = T^T dU   dA = -stril(dXk W^T + dXv U~^T)
//     dQ~ = dO' h^T + dP K-     dK+ = dXk + dA K-     dK- = U dh''^T + dP^T Q~ + dA^T K+
// and the gradients of the caller's tensors follow element by element (cw_post).  Four kernels beside the carries
// (tc_scan_cw in gdn_tc.cu):
//   cw_scale  scaled operand tiles as bf16 tile images, gam; checks that |gam| stays below 80 (beyond that the split
//             would need reference points inside the chunk): otherwise it records GDN_ERR_DECAY_RANGE, the kernels below
//             stand down, and the FFMA sequence enqueued behind them computes the call (gdn_simt_vec.cu)
//   cw_prep   [Q~;K+] K-^T, fp32 blocked inversion, W^T, U~^T, (P^T dO')^T, E               (tcgen05)
//   cw_intra  the sixteen products of the gradient stage in five dependent steps (K#2 reuses T)   (tcgen05)
//   cw_post   dq, dk, dv, db, dw, and dg by a reverse cumulative sum per channel
// The tensor-core kernels are written straight-line (one CTA per SM walks over chunk-heads; one thread issues every
// product and copy; CTA-wide barriers between the steps): the plain statement of the channel-wise path on tcgen05,
// not a tuned one.  Accumulators live in one TMEM reservation at fixed column offsets; every wait is bounded.
#include "tc_common.cuh"
#include "tc_inverse.cuh"

namespace gdn {
namespace {

using namespace tc;

constexpr int D = 128;
constexpr int kT = 256;               // 8 warps: TMEM lane quadrant = warp % 4, column half = warp / 4
constexpr float kMaxDecay = 80.f;     // bound on |gam| inside a chunk (exp(80) is still a bf16 number)

// (chunk, head) of an elementwise CTA, from the chunk table (which these calls always build)
struct ChunkCtx { int hd, ch, tok0, len; };
__device__ __forceinline__ bool chunk_ctx(const Problem& p, ChunkCtx& x) {
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    const int c = blockIdx.x / p.d.H;
    if (c >= hdr->n_chunks) return false;
    x.hd = blockIdx.x % p.d.H;
    x.ch = blockIdx.x;
    x.tok0 = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0)[c];
    x.len = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len)[c];
    return true;
}

// Per chunk-head scratch between cw_intra and cw_post (fp32): dQ~, dK+, dK-, dXv [64][128] each, and per key channel
// rowdot(dh'', h + K-^T U) [128], the chunk-end part of the decay gradient.
constexpr size_t S_DQ = 0, S_DKP = 32768, S_DKM = 65536, S_DXV = 98304, S_HH = 131072, S_BYTES = 131584;

// ------------------------------------------------------------------------------------------------
// cw_scale
// ------------------------------------------------------------------------------------------------
// mode 0: the forward's images; 1: those and dO' (closed backward); 2: dO' alone, for a backward on a workspace fresh
// from the forward (every other image, gam and the factors are still there).  If that forward was computed by the
// fall-back kernels (its gates were refused; the header remembers), the workspace holds their fp32 data instead: the
// refusal is raised again and the fall-back sequence computes this call too.
__global__ void __launch_bounds__(kT) cw_scale_kernel(Problem p, int mode) {
    ChunkCtx x;
    if (!chunk_ctx(p, x)) return;
    extern __shared__ __align__(16) float gam[];   // [64][D + 1]
    __shared__ int bad;
    const int H = p.d.H;
    const size_t base = ((size_t)x.tok0 * H + x.hd) * D, rs = (size_t)H * D;
    const bool with_bwd = mode != 0;
    const __nv_bfloat16* op = with_bwd ? reinterpret_cast<const __nv_bfloat16*>(p.dO) + base : nullptr;
    if (mode == 2) {
        WsHeader* hdr = reinterpret_cast<WsHeader*>(p.ws);
        if (hdr->cw_fallback) {
            if (blockIdx.x == 0 && threadIdx.x == 0) { hdr->status = GDN_ERR_DECAY_RANGE; hdr->detail = -1; }
            return;
        }
        char* iDO = p.ws + p.L.img_dO + (size_t)x.ch * 16384;
        const float sc = p.d.scale;
        for (int t = threadIdx.x; t < kC * 16; t += kT) {
            const int i = t >> 4, ch = t & 15;
            float o8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) o8[j] = 0.f;
            if (i < x.len) unpack8(*reinterpret_cast<const uint4*>(op + i * rs + ch * 8), o8);
#pragma unroll
            for (int j = 0; j < 8; ++j) o8[j] *= sc;
            *reinterpret_cast<uint4*>(iDO + tile_chunk_off(64, i, ch)) = pack8(o8);
        }
        return;
    }
    const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(p.q) + base;
    const __nv_bfloat16* kp = reinterpret_cast<const __nv_bfloat16*>(p.k) + base;
    const __nv_bfloat16* vp = reinterpret_cast<const __nv_bfloat16*>(p.v) + base;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    if (threadIdx.x < D) {
        const int r = threadIdx.x;
        float s = 0.f, worst = 0.f;
#pragma unroll 1
        for (int i0 = 0; i0 < kC; i0 += 16) {   // sixteen loads in flight, then their running sum in token order
            float g16[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) g16[k] = (i0 + k < x.len) ? p.gv[base + (size_t)(i0 + k) * rs + r] : 0.f;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                s += g16[k];
                gam[(i0 + k) * (D + 1) + r] = s;
                worst = fmaxf(worst, fabsf(s));
            }
        }
        if (!(worst <= kMaxDecay)) bad = 1;   // (also catches a NaN gate: it cannot be scaled apart either)
    }
    __syncthreads();
    if (bad) {
        if (threadIdx.x == 0) {
            WsHeader* hdr = reinterpret_cast<WsHeader*>(p.ws);
            hdr->status = GDN_ERR_DECAY_RANGE;
            hdr->detail = x.ch;
        }
        return;
    }
    float* wsG = reinterpret_cast<float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC * D;
    for (int t = threadIdx.x; t < kC * D; t += kT) wsG[t] = gam[(t / D) * (D + 1) + t % D];
    char* iQKp = p.ws + p.L.img_QKp + (size_t)x.ch * 32768;
    char* iKm = p.ws + p.L.img_Km + (size_t)x.ch * 16384;
    char* iKb = p.ws + p.L.img_K + (size_t)x.ch * 16384;
    char* iVt = p.ws + p.L.img_Vt + (size_t)x.ch * 16384;
    char* iDO = p.ws + p.L.img_dO + (size_t)x.ch * 16384;
    const float sc = p.d.scale;
    for (int t = threadIdx.x; t < kC * 16; t += kT) {   // one 16-byte piece (8 features) of one token row
        const int i = t >> 4, ch = t & 15;
        float q8[8], k8[8], v8[8], o8[8], a[8], b[8], c[8], d8[8], b8[8], w8[8];
        const bool live = i < x.len;
#pragma unroll
        for (int j = 0; j < 8; ++j) { q8[j] = k8[j] = v8[j] = o8[j] = b8[j] = w8[j] = 0.f; }
        if (live) {
            unpack8(*reinterpret_cast<const uint4*>(qp + i * rs + ch * 8), q8);
            unpack8(*reinterpret_cast<const uint4*>(kp + i * rs + ch * 8), k8);
            unpack8(*reinterpret_cast<const uint4*>(vp + i * rs + ch * 8), v8);
            if (with_bwd) unpack8(*reinterpret_cast<const uint4*>(op + i * rs + ch * 8), o8);
            const float4* bp = reinterpret_cast<const float4*>(p.bv + base + i * rs + ch * 8);
            const float4* wp = reinterpret_cast<const float4*>(p.wv + base + i * rs + ch * 8);
            const float4 b0 = bp[0], b1 = bp[1], w0 = wp[0], w1 = wp[1];
            b8[0] = b0.x; b8[1] = b0.y; b8[2] = b0.z; b8[3] = b0.w; b8[4] = b1.x; b8[5] = b1.y; b8[6] = b1.z; b8[7] = b1.w;
            w8[0] = w0.x; w8[1] = w0.y; w8[2] = w0.z; w8[3] = w0.w; w8[4] = w1.x; w8[5] = w1.y; w8[6] = w1.z; w8[7] = w1.w;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int r = ch * 8 + j;
            const float g = gam[i * (D + 1) + r], ge = gam[(kC - 1) * (D + 1) + r];
            const float G = expf(g);
            const float bb = b8[j], ww = w8[j];
            a[j] = G * q8[j];                 // q~
            b[j] = G * bb * k8[j];            // k+
            c[j] = expf(-g) * k8[j];          // k-
            d8[j] = expf(ge - g) * k8[j];     // Kb
            v8[j] *= ww;                      // v~
            o8[j] *= sc;                      // dO'
        }
        *reinterpret_cast<uint4*>(iQKp + tile_chunk_off(128, i, ch)) = pack8(a);
        *reinterpret_cast<uint4*>(iQKp + tile_chunk_off(128, 64 + i, ch)) = pack8(b);
        *reinterpret_cast<uint4*>(iKm + tile_chunk_off(64, i, ch)) = pack8(c);
        *reinterpret_cast<uint4*>(iKb + tile_chunk_off(64, i, ch)) = pack8(d8);
        *reinterpret_cast<uint4*>(iVt + tile_chunk_off(64, i, ch)) = pack8(v8);
        if (with_bwd) *reinterpret_cast<uint4*>(iDO + tile_chunk_off(64, i, ch)) = pack8(o8);
    }
}

// ------------------------------------------------------------------------------------------------
// cw_prep
// ------------------------------------------------------------------------------------------------
namespace prepcw {
constexpr uint32_t QKP = 0;                 // [Q~ rows 0..63 ; K+ rows 64..127] x 128                               32 KB
constexpr uint32_t KM = 32768;              // K- [64][128]                                     16 KB
constexpr uint32_t VT = KM + 16384;         // V~ [64][128]                                     16 KB
constexpr uint32_t DOT = VT + 16384;        // dO' [64][128]                                    16 KB
constexpr uint32_t XA = DOT + 16384;        // fp32 A [64][kLdi]
constexpr uint32_t XT = XA + 17408;         // fp32 T
constexpr uint32_t SF = XT + 17408;         // fp32 scratch of the inversion
constexpr uint32_t TT = SF + 17408;         // T  bf16 [64][64]                                  8 KB
constexpr uint32_t PT = TT + 8192;          // P  bf16 [64][64]                                  8 KB
constexpr uint32_t WT = PT + 8192;          // W^T  [128][64]                                   16 KB
constexpr uint32_t UTT = WT + 16384;        // U~^T [128][64]                                   16 KB
constexpr uint32_t PDOT = UTT + 16384;      // (P^T dO')^T [128][64]                            16 KB
constexpr uint32_t EST = XA;                // staged E image [128][128] over the fp32 A and T blocks                       32 KB
constexpr uint32_t SMEM_BYTES = PDOT + 16384 + 1024;
constexpr uint32_t C_S1 = 0, C_W = 64, C_U = 128, C_PDO = 192, C_E = 256;   // TMEM columns (512 allocated)
static_assert(EST % 1024 == 0 && EST + 32768 <= SF + 17408, "the E image fits over the inversion's scratch");
static_assert(TT % 1024 == 0 && SMEM_BYTES <= 225 * 1024, "tile alignment and shared memory budget");
}  // namespace prepcw

// mode 0: the forward's share (P, A, T, W, U~); 1: that and E (closed backward); 2: E alone from the stored P and W^T
// (backward on a workspace fresh from the forward: no product, inversion or store of the forward is repeated).
__global__ void __launch_bounds__(kT, 1) cw_prep_kernel(Problem p, int mode) {
    using namespace prepcw;
    const int H = p.d.H;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    if (hdr->status != GDN_OK) return;
    const int n_items = hdr->n_chunks * H;
    if ((int)blockIdx.x >= n_items) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ uint64_t bar_in, bar_mma;
    __shared__ uint32_t tmem_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, grp = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    if (threadIdx.x == 0) { mbar_init(&bar_in, 1); mbar_init(&bar_mma, 1); fence_mbar_init(); }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    float* Af = reinterpret_cast<float*>(sm + XA);
    float* Tf = reinterpret_cast<float*>(sm + XT);
    float* Sf = reinterpret_cast<float*>(sm + SF);
    const bool bwd = mode != 0, fresh = mode == 2;
    bool ok = true, pending = false;
    uint32_t mma_phase = 0, in_phase = 0, pending_phase = 0;   // (pending_phase: the phase of bar_in the loads in flight belong to)
    // The tiles of a trip arrive in two pieces on one mbarrier phase, each issued during the trip before as soon as the
    // last product that reads its region is done (E is staged over the inversion's scratch, never over an input tile):
    //   closed / forward:  a = K-                     after step 1      b = [Q~; K+], V~, dO'     after step 2
    //   fresh workspace:   a = Q~, dO', stored P      after its first products      b = stored W^T   after step 3
    auto load_a = [&](size_t c, uint32_t phase) {   // thread 0; the first piece announces the whole trip's bytes
        pending_phase = phase;
        pending = true;
        if (fresh) {
            mbar_expect_tx(&bar_in, 16384 + 16384 + 8192 + 16384);
            for (int cb = 0; cb < 2; ++cb) bulk_load(sm + QKP + cb * 16384, p.ws + p.L.img_QKp + c * 32768 + cb * 16384, 8192, &bar_in);
            bulk_load(sm + DOT, p.ws + p.L.img_dO + c * 16384, 16384, &bar_in);
            bulk_load(sm + PT, p.ws + p.L.Pm + c * 8192, 8192, &bar_in);
        } else {
            mbar_expect_tx(&bar_in, 65536 + (bwd ? 16384 : 0));
            bulk_load(sm + KM, p.ws + p.L.img_Km + c * 16384, 16384, &bar_in);
        }
    };
    auto load_b = [&](size_t c) {
        if (fresh) {
            bulk_load(sm + WT, p.ws + p.L.img_W + c * 16384, 16384, &bar_in);
        } else {
            bulk_load(sm + QKP, p.ws + p.L.img_QKp + c * 32768, 32768, &bar_in);
            bulk_load(sm + VT, p.ws + p.L.img_Vt + c * 16384, 16384, &bar_in);
            if (bwd) bulk_load(sm + DOT, p.ws + p.L.img_dO + c * 16384, 16384, &bar_in);
        }
    };
    if (threadIdx.x == 0) { load_a(blockIdx.x, 0); load_b(blockIdx.x); }
#pragma unroll 1
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, in_phase ^= 1) {
        const size_t ch = (size_t)item, chn = ch + gridDim.x;
        const bool has_next = item + (int)gridDim.x < n_items;
        if (threadIdx.x == 0) bulk_wait_read<0>();   // the previous trip's stores have read their tiles (rewritten from here on)
        if (ok) {
            ok = mbar_wait(&bar_in, in_phase);
            if (!ok && threadIdx.x == 0) report_timeout(p.ws, 40);
            if (ok && threadIdx.x == 0) pending = false;
        }
        __syncthreads();
        if (fresh) {
            // (P^T dO')^T and Q~^T dO' from the loaded tiles; then E = Q~^T dO' - W^T (P^T dO') as in the closed arm
            if (ok && threadIdx.x == 0) {
                tc_fence_after();
                mma_tile<128, 64, 64>(tmem + C_PDO, op_mn_major(sm + DOT, 64), op_mn_major(sm + PT, 64), false);
                mma_tile<128, 128, 64>(tmem + C_E, op_mn_major(sm + QKP, 128, 0), op_mn_major(sm + DOT, 64), false);
                mma_commit(&bar_mma);
            }
            GDN_WAIT_MMA(45)
            if (ok && has_next && threadIdx.x == 0) load_a(chn, in_phase ^ 1);   // Q~, dO' and P have been read for the last time
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
        } else {
        // ---- step 1: S1 = [Q~; K+] K-^T  (rows 0..63: P before masking, rows 64..127: A)
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 128>(tmem + C_S1, op_k_major(sm + QKP, 128, 0), op_k_major(sm + KM, 64), false);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(41)
        if (ok && has_next && threadIdx.x == 0) load_a(chn, in_phase ^ 1);   // K- has been read for the last time
        if (ok) {
            const int i = (q4 & 1) * 32 + lane, j0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float v[8];
                const int jb = j0 + part * 8;
                tmem_ld8(tmem + lane_base + C_S1 + jb, v);
                tmem_wait_ld();
                if (q4 < 2) {   // P = tril(.), diagonal included
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = (jb + j <= i) ? v[j] : 0.f;
                    chunk_store(sm + PT, 64, i, jb >> 3, v);
                } else {        // A = stril(.)
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = (jb + j < i) ? v[j] : 0.f;
                    *reinterpret_cast<float4*>(Af + i * kLdi + jb) = make_float4(v[0], v[1], v[2], v[3]);
                    *reinterpret_cast<float4*>(Af + i * kLdi + jb + 4) = make_float4(v[4], v[5], v[6], v[7]);
                }
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        // (P^T dO')^T and Q~^T dO' need nothing of the inversion: they run under it, covered by the next commit
        if (ok && bwd && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 64>(tmem + C_PDO, op_mn_major(sm + DOT, 64), op_mn_major(sm + PT, 64), false);
            mma_tile<128, 128, 64>(tmem + C_E, op_mn_major(sm + QKP, 128, 0), op_mn_major(sm + DOT, 64), false);
        }
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
        {   // T -> bf16 tile: a thread converts two rows of one 8-column piece
            const int cch = threadIdx.x & 7;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int i = (threadIdx.x >> 3) + 32 * h;
                float a[8];
                if ((cch >> 1) <= (i >> 4)) {   // blocks above the block diagonal are zero and were never written
                    ld8s(Tf + i * kLdi + cch * 8, a);
                } else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) a[k] = 0.f;
                }
                chunk_store(sm + TT, 64, i, cch, a);
            }
        }
        fence_async_smem();
        __syncthreads();
        // ---- step 2: W^T = K+^T T^T ; U~^T = V~^T T^T
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 64>(tmem + C_W, op_mn_major(sm + QKP, 128, 64), op_k_major(sm + TT, 64), false);
            mma_tile<128, 64, 64>(tmem + C_U, op_mn_major(sm + VT, 64), op_k_major(sm + TT, 64), false);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(42)
        if (ok && has_next && threadIdx.x == 0) load_b(chn);   // [Q~; K+], V~ and dO' have been read for the last time
        if (ok) {
            const int f = q4 * 32 + lane, i0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                const int ib = i0 + part * 8;
                float v[8];
                tmem_ld8(tmem + lane_base + C_W + ib, v);
                tmem_wait_ld();
                chunk_store(sm + WT, 128, f, ib >> 3, v);
                tmem_ld8(tmem + lane_base + C_U + ib, v);
                tmem_wait_ld();
                chunk_store(sm + UTT, 128, f, ib >> 3, v);
                if (bwd) {
                    tmem_ld8(tmem + lane_base + C_PDO + ib, v);
                    tmem_wait_ld();
                    chunk_store(sm + PDOT, 128, f, ib >> 3, v);
                }
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        }   // (!fresh)
        // ---- step 3: E = Q~^T dO' - W^T (P^T dO')
        if (bwd) {
            if (ok && threadIdx.x == 0) {
                tc_fence_after();
                mma_tile<128, 128, 64>(tmem + C_E, op_k_major(sm + WT, 128), op_k_major(sm + PDOT, 128), true, /*neg_a=*/true);
                mma_commit(&bar_mma);
            }
            GDN_WAIT_MMA(43)
            if (ok && fresh && has_next && threadIdx.x == 0) load_b(chn);   // W^T has been read for the last time
            if (ok) {   // E -> bf16 tile image, staged over the scratch of the inversion (dead since T was converted)
                const int r = q4 * 32 + lane, c0 = grp * 64;
#pragma unroll 1
                for (int part = 0; part < 8; ++part) {
                    const int cb = c0 + part * 8;
                    float v[8];
                    tmem_ld8(tmem + lane_base + C_E + cb, v);
                    tmem_wait_ld();
                    chunk_store(sm + EST, 128, r, cb >> 3, v);
                }
            }
            tc_fence_before();
            fence_async_smem();
            __syncthreads();
        }
        if (ok && threadIdx.x == 0) {
            if (!fresh) {
                bulk_store(p.ws + p.L.Tm + ch * 8192, sm + TT, 8192);
                bulk_store(p.ws + p.L.Pm + ch * 8192, sm + PT, 8192);
                bulk_store(p.ws + p.L.img_W + ch * 16384, sm + WT, 16384);
                bulk_store(p.ws + p.L.img_U + ch * 16384, sm + UTT, 16384);
            }
            if (bwd) bulk_store(p.ws + p.L.img_E + ch * 32768, sm + EST, 32768);
            bulk_commit();
        }
        if (!ok) break;
    }
    if (threadIdx.x == 0) {
        bulk_wait_read<0>();
        if (pending) (void)mbar_wait(&bar_in, pending_phase);   // after a timeout a load may still be in flight
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------
// cw_intra
// ------------------------------------------------------------------------------------------------
namespace intracw {
constexpr uint32_t QKM = 0;                 // [Q~ rows 0..63 ; K- rows 64..127] x 128         32 KB
constexpr uint32_t KP = 32768;              // K+ [64][128]                                     16 KB
constexpr uint32_t DOT = KP + 16384;        // dO' [64][128]                                    16 KB
constexpr uint32_t WT = DOT + 16384;        // W^T  [128][64]                                   16 KB
constexpr uint32_t UTT = WT + 16384;        // U~^T [128][64]                                   16 KB
constexpr uint32_t TT = UTT + 16384;        // T [64][64]; later dA                              8 KB
constexpr uint32_t PT = TT + 8192;          // P [64][64]; later dP                              8 KB
constexpr uint32_t HH = PT + 8192;          // h [128][128]                                     32 KB
constexpr uint32_t DH = HH + 32768;         // dh'' = Diag(Gam_e) dh' [128][128]                32 KB
constexpr uint32_t UT = DH + 32768;         // U^T  [128][64]                                   16 KB
constexpr uint32_t DUT = UT + 16384;        // dU^T [128][64]; later dXv^T [128][64]            16 KB
constexpr uint32_t SMEM_BYTES = DUT + 16384 + 1024;
constexpr uint32_t DA = TT, DP = PT, DXVT = DUT;   // (dA over T, dP over P, dXv^T over dU^T, each after its last reader)
// TMEM columns (512 allocated, fixed offsets).  Accumulators with features on the lanes use all 128 lanes (M = 128);
// token-major ones (M = 64) occupy lanes 0..15 of each lane quadrant.
//   0..63     (W h)^T  -> dXv^T                    (M = 128)
//   64..191   (K- dh'')^T | (P^T dO')^T (M = 128) -> K-^T U (M = 128) -> dK+ = dXk + dA K-   (M = 64, 128 columns)
//   192..255  dP -> dA                              (M = 64)
//   256..383  dQ~ = dO' h^T + dP K-                 (M = 64)
//   384..511  dK- = U dh''^T + dP^T Q~ + dA^T K+    (M = 64)
constexpr uint32_t C_A = 0, C_B = 64, C_PDO = 128, C_KP = 64, C_PP = 192, C_DQ = 256, C_KM = 384;
constexpr uint32_t C_X = 64;   // K-^T U [128][128] over C_B | C_PDO (read by then), gone before dXk lands on C_KP
static_assert(SMEM_BYTES <= 220 * 1024, "shared memory budget");
}  // namespace intracw

__global__ void __launch_bounds__(kT, 1) cw_intra_kernel(Problem p) {
    using namespace intracw;
    const int H = p.d.H;
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    if (hdr->status != GDN_OK) return;
    const int n_items = hdr->n_chunks * H;
    if ((int)blockIdx.x >= n_items) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = align1024(smem_raw);
    __shared__ uint64_t bar_s, bar_a, bar_b, bar_k, bar_q, bar_mma;
    __shared__ uint32_t tmem_slot;
    __shared__ float end_sum[3][D];   // per key channel: rowdot(dh'', h) and the two halves of rowdot(dh'', K-^T U)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int q4 = warp & 3, grp = warp >> 2;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    if (threadIdx.x == 0) {
        mbar_init(&bar_s, 1); mbar_init(&bar_a, 1); mbar_init(&bar_b, 1); mbar_init(&bar_k, 1); mbar_init(&bar_q, 1);
        mbar_init(&bar_mma, 1);
        fence_mbar_init();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    const int f = q4 * 32 + lane;             // feature row of the M = 128 accumulators
    const int tr = q4 * 16 + (lane & 15);     // token row of the M = 64 accumulators (lanes 0..15 of the quadrant)
    const bool ga = lane < 16;
    bool ok = true;
    uint32_t mma_phase = 0, in_phase = 0;
    // The tiles of a trip arrive in five groups, each loaded during the previous trip as soon as the last product that
    // reads its region is done (look-ahead without a second buffer):
    //   b  W^T, U~^T       after the first readout       s  h, dh''          after step 3
    //   a  dO'             after step 2                  k  K-               after step 4
    //      P               after step 3                  q  Q~, K+, T        after step 4 (needed from step 2 on)
    bool pend_s = false, pend_a = false, pend_b = false, pend_k = false, pend_q = false;   // thread 0
    auto load_s = [&](size_t c) {
        mbar_expect_tx(&bar_s, 65536);
        bulk_load(sm + HH, p.ws + p.L.hc + c * 32768, 32768, &bar_s);
        bulk_load(sm + DH, p.ws + p.L.dhn + c * 32768, 32768, &bar_s);
        pend_s = true;
    };
    auto load_a = [&](size_t c) {
        mbar_expect_tx(&bar_a, 24576);
        bulk_load(sm + DOT, p.ws + p.L.img_dO + c * 16384, 16384, &bar_a);
        bulk_load(sm + PT, p.ws + p.L.Pm + c * 8192, 8192, &bar_a);
        pend_a = true;
    };
    auto load_b = [&](size_t c) {
        mbar_expect_tx(&bar_b, 32768);
        bulk_load(sm + WT, p.ws + p.L.img_W + c * 16384, 16384, &bar_b);
        bulk_load(sm + UTT, p.ws + p.L.img_U + c * 16384, 16384, &bar_b);
        pend_b = true;
    };
    auto load_kq = [&](size_t c) {
        const char* iQKp = p.ws + p.L.img_QKp + c * 32768;
        const char* iKm = p.ws + p.L.img_Km + c * 16384;
        mbar_expect_tx(&bar_k, 16384);
        for (int cb = 0; cb < 2; ++cb) bulk_load(sm + QKM + cb * 16384 + 8192, iKm + cb * 8192, 8192, &bar_k);      // K-
        pend_k = true;
        mbar_expect_tx(&bar_q, 40960);
        for (int cb = 0; cb < 2; ++cb) {
            bulk_load(sm + QKM + cb * 16384, iQKp + cb * 16384, 8192, &bar_q);                                        // Q~
            bulk_load(sm + KP + cb * 8192, iQKp + cb * 16384 + 8192, 8192, &bar_q);                                   // K+
        }
        bulk_load(sm + TT, p.ws + p.L.Tm + c * 8192, 8192, &bar_q);
        pend_q = true;
    };
    if (threadIdx.x == 0) { load_s(blockIdx.x); load_kq(blockIdx.x); load_b(blockIdx.x); load_a(blockIdx.x); }
#pragma unroll 1
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, in_phase ^= 1) {
        const size_t ch = (size_t)item;
        const bool has_next = item + (int)gridDim.x < n_items;
        const size_t chn = ch + gridDim.x;
        float* scr = reinterpret_cast<float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * ch);
        if (ok) {   // everything step 1 reads (the reverse carry left dh'' = Diag(Gam_e) dh', the form used here)
            ok = mbar_wait(&bar_s, in_phase) && mbar_wait(&bar_k, in_phase) && mbar_wait(&bar_b, in_phase) && mbar_wait(&bar_a, in_phase);
            if (!ok && threadIdx.x == 0) report_timeout(p.ws, 44);
            if (ok && threadIdx.x == 0) pend_s = pend_k = pend_a = pend_b = false;
        }
        __syncthreads();
        // ---- step 1: (W h)^T ; (K- dh'')^T ; (P^T dO')^T
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<128, 64, 128>(tmem + C_A, op_mn_major(sm + HH, 128), op_mn_major(sm + WT, 128), false);
            mma_tile<128, 64, 128>(tmem + C_B, op_mn_major(sm + DH, 128), op_k_major(sm + QKM, 128, 64), false);
            mma_tile<128, 64, 64>(tmem + C_PDO, op_mn_major(sm + DOT, 64), op_mn_major(sm + PT, 64), false);
            mma_commit(&bar_mma);
        }
        {   // rowdot(dh'', h) for the decay gradient of the chunk end, while the products run: two threads per state row
            const int r = threadIdx.x >> 1, half = threadIdx.x & 1;
            float hh = 0.f;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                float a[8], b[8];
                chunk_load(sm + DH, 128, r, half * 8 + k, a);
                chunk_load(sm + HH, 128, r, half * 8 + k, b);
#pragma unroll
                for (int j = 0; j < 8; ++j) hh = fmaf(a[j], b[j], hh);
            }
            hh += __shfl_xor_sync(0xffffffffu, hh, 1);
            if (half == 0) end_sum[0][r] = hh;
        }
        GDN_WAIT_MMA(45)
        if (ok) {   // U^T = U~^T - (W h)^T ; dU^T = (P^T dO')^T + (K- dh'')^T
            const int i0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                const int ib = i0 + part * 8;
                float t[8], kb[8], pd[8], u[8];
                tmem_ld8(tmem + lane_base + C_A + ib, t);
                tmem_ld8(tmem + lane_base + C_B + ib, kb);
                tmem_ld8(tmem + lane_base + C_PDO + ib, pd);
                tmem_wait_ld();
                chunk_load(sm + UTT, 128, f, ib >> 3, u);
#pragma unroll
                for (int j = 0; j < 8; ++j) { u[j] -= t[j]; pd[j] += kb[j]; }
                chunk_store(sm + UT, 128, f, ib >> 3, u);
                chunk_store(sm + DUT, 128, f, ib >> 3, pd);
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        if (ok && has_next && threadIdx.x == 0) load_b(chn);   // W^T (step 1) and U~^T (the readout) have been read for the last time
        // ---- step 2: dP = dO' U^T ; dXv^T = dU^T T ; dO' h^T ; K-^T U ; under the readout U dh''^T
        if (ok) {
            ok = mbar_wait(&bar_q, in_phase);   // T (and Q~, K+, needed from step 3 on)
            if (!ok && threadIdx.x == 0) report_timeout(p.ws, 51);
            if (ok && threadIdx.x == 0) pend_q = false;
        }
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<64, 64, 128>(tmem + C_PP, op_k_major(sm + DOT, 64), op_mn_major(sm + UT, 128), false);
            mma_tile<128, 64, 64>(tmem + C_A, op_k_major(sm + DUT, 128), op_mn_major(sm + TT, 64), false);
            mma_tile<64, 128, 128>(tmem + C_DQ, op_k_major(sm + DOT, 64), op_k_major(sm + HH, 128), false);
            // K-^T U: its row dots with dh'' are the part sum_j k-_j . (U dh''^T)_j of the decay gradient of the chunk end
            mma_tile<128, 128, 64>(tmem + C_X, op_mn_major(sm + QKM, 128, 64), op_k_major(sm + UT, 128), false);
            mma_commit(&bar_mma);
            // U dh''^T is only accumulated upon: it runs under the readout (its operands stay untouched until step 3's
            // products, whose commit covers it, are done)
            mma_tile<64, 128, 128>(tmem + C_KM, op_mn_major(sm + UT, 128), op_k_major(sm + DH, 128), false);
        }
        GDN_WAIT_MMA(46)
        if (ok && has_next && threadIdx.x == 0) {   // dO' has been read for the last time; P (by then dP) follows after step 3
            mbar_expect_tx(&bar_a, 24576);
            bulk_load(sm + DOT, p.ws + p.L.img_dO + chn * 16384, 16384, &bar_a);
            pend_a = true;
        }
        if (ok) {
            const int j0 = grp * 32, i0 = grp * 32, c0 = grp * 64;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float v[8], x8[8];
                const int ib = i0 + part * 8;
                tmem_ld8(tmem + lane_base + C_PP + j0 + part * 8, v);     // dP rows on lanes 0..15
                tmem_ld8(tmem + lane_base + C_A + ib, x8);                // dXv^T, all lanes
                tmem_wait_ld();
                if (ga) {   // dP = tril(dO' U^T)
                    const int jb = j0 + part * 8;
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = (jb + j <= tr) ? v[j] : 0.f;
                    chunk_store(sm + DP, 64, tr, jb >> 3, v);
                }
                // dXv^T: operand tile (over dU^T, which its product has read) and, in fp32, the input of dv and dw
                chunk_store(sm + DXVT, 128, f, ib >> 3, x8);
#pragma unroll
                for (int j = 0; j < 8; ++j) scr[S_DXV / 4 + (ib + j) * D + f] = x8[j];   // token-major: a warp writes 128 contiguous bytes
            }
            float xs = 0.f;   // rowdot(dh'', K-^T U): this thread's state row f, its half of the columns
#pragma unroll 1
            for (int part = 0; part < 8; ++part) {
                float v[8], d8[8];
                tmem_ld8(tmem + lane_base + C_X + c0 + part * 8, v);
                chunk_load(sm + DH, 128, f, (c0 >> 3) + part, d8);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 8; ++j) xs = fmaf(v[j], d8[j], xs);
            }
            end_sum[1 + grp][f] = xs;
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        if (ok && threadIdx.x < D) scr[S_HH / 4 + threadIdx.x] = end_sum[0][threadIdx.x] + end_sum[1][threadIdx.x] + end_sum[2][threadIdx.x];
        // ---- step 3 (K#2): dA = -stril(dXv U^T) (= -stril(dXk W^T + dXv U~^T): dXk = T^T dW = -dXv h^T, U = U~ - W h) ;
        // dK+ = dXk = -dXv h^T ; dQ~ += dP K- ; dK- += dP^T Q~
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<64, 64, 128>(tmem + C_PP, op_mn_major(sm + DXVT, 128), op_mn_major(sm + UT, 128), false);
            mma_tile<64, 128, 128>(tmem + C_KP, op_mn_major(sm + DXVT, 128), op_k_major(sm + HH, 128), false, /*neg_a=*/true);
            mma_tile<64, 128, 64>(tmem + C_DQ, op_k_major(sm + DP, 64), op_mn_major(sm + QKM, 128, 64), true);
            mma_tile<64, 128, 64>(tmem + C_KM, op_mn_major(sm + DP, 64), op_mn_major(sm + QKM, 128, 0), true);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(47)
        if (ok && has_next && threadIdx.x == 0) {   // h, dh'' (U dh''^T is done too) and dP (over P) have been read for the last time
            load_s(chn);
            bulk_load(sm + PT, p.ws + p.L.Pm + chn * 8192, 8192, &bar_a);   // (the second piece of group a)
        }
        if (ok) {   // dA = -stril(.)  (over T, which step 2 has read)
            const int j0 = grp * 32;
#pragma unroll 1
            for (int part = 0; part < 4; ++part) {
                float v[8];
                const int jb = j0 + part * 8;
                tmem_ld8(tmem + lane_base + C_PP + jb, v);
                tmem_wait_ld();
                if (ga) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = (jb + j < tr) ? -v[j] : 0.f;
                    chunk_store(sm + DA, 64, tr, jb >> 3, v);
                }
            }
        }
        tc_fence_before();
        fence_async_smem();
        __syncthreads();
        // ---- step 4: dK+ += dA K- ; dK- += dA^T K+
        if (ok && threadIdx.x == 0) {
            tc_fence_after();
            mma_tile<64, 128, 64>(tmem + C_KP, op_k_major(sm + DA, 64), op_mn_major(sm + QKM, 128, 64), true);
            mma_tile<64, 128, 64>(tmem + C_KM, op_mn_major(sm + DA, 64), op_mn_major(sm + KP, 64), true);
            mma_commit(&bar_mma);
        }
        GDN_WAIT_MMA(49)
        if (ok && has_next && threadIdx.x == 0) load_kq(chn);   // every tile of this trip has been read for the last time
        if (ok) {
            const int c0 = grp * 64;
#pragma unroll 1
            for (int part = 0; part < 8; ++part) {
                float a[8], b[8], c[8];
                tmem_ld8(tmem + lane_base + C_DQ + c0 + part * 8, a);
                tmem_ld8(tmem + lane_base + C_KP + c0 + part * 8, b);
                tmem_ld8(tmem + lane_base + C_KM + c0 + part * 8, c);
                tmem_wait_ld();
                if (ga) {
                    const int o = tr * D + c0 + part * 8;
                    *reinterpret_cast<float4*>(scr + S_DQ / 4 + o) = make_float4(a[0], a[1], a[2], a[3]);
                    *reinterpret_cast<float4*>(scr + S_DQ / 4 + o + 4) = make_float4(a[4], a[5], a[6], a[7]);
                    *reinterpret_cast<float4*>(scr + S_DKP / 4 + o) = make_float4(b[0], b[1], b[2], b[3]);
                    *reinterpret_cast<float4*>(scr + S_DKP / 4 + o + 4) = make_float4(b[4], b[5], b[6], b[7]);
                    *reinterpret_cast<float4*>(scr + S_DKM / 4 + o) = make_float4(c[0], c[1], c[2], c[3]);
                    *reinterpret_cast<float4*>(scr + S_DKM / 4 + o + 4) = make_float4(c[4], c[5], c[6], c[7]);
                }
            }
        }
        tc_fence_before();
        __syncthreads();   // every reader of this trip's tiles and accumulators is done
        if (!ok) break;
    }
    if (threadIdx.x == 0 && !ok) {   // after a timeout a load may still be in flight: wait for it (bounded) before the CTA retires
        // a group issued during the trip that gave up belongs to the next phase of its barrier; one pending since the top of
        // that trip to the current one.  Both parities are tried; the wrong one returns at once or after the bound.
        uint64_t* bars[5] = {&bar_s, &bar_a, &bar_b, &bar_k, &bar_q};
        const bool pend[5] = {pend_s, pend_a, pend_b, pend_k, pend_q};
        for (int i = 0; i < 5; ++i)
            if (pend[i]) { (void)mbar_wait(bars[i], in_phase); (void)mbar_wait(bars[i], in_phase ^ 1); }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------
// cw_post
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kT) cw_post_kernel(Problem p) {
    ChunkCtx x;
    if (!chunk_ctx(p, x)) return;
    if (reinterpret_cast<const WsHeader*>(p.ws)->status != GDN_OK) return;
    extern __shared__ __align__(16) float dgam[];   // [64][D]
    const int H = p.d.H;
    const size_t base = ((size_t)x.tok0 * H + x.hd) * D, rs = (size_t)H * D;
    const __nv_bfloat16* qp = reinterpret_cast<const __nv_bfloat16*>(p.q) + base;
    const __nv_bfloat16* kp = reinterpret_cast<const __nv_bfloat16*>(p.k) + base;
    const __nv_bfloat16* vp = reinterpret_cast<const __nv_bfloat16*>(p.v) + base;
    __nv_bfloat16* dqp = reinterpret_cast<__nv_bfloat16*>(p.dq) + base;
    __nv_bfloat16* dkp = reinterpret_cast<__nv_bfloat16*>(p.dk) + base;
    __nv_bfloat16* dvp = reinterpret_cast<__nv_bfloat16*>(p.dv) + base;
    const float* wsG = reinterpret_cast<const float*>(p.ws + p.L.gamma) + (size_t)x.ch * kC * D;
    const float* scr = reinterpret_cast<const float*>(p.ws + p.L.scratch + p.L.scratch_per_ch * x.ch);
    const float *dQ = scr + S_DQ / 4, *dKp = scr + S_DKP / 4, *dKm = scr + S_DKM / 4;
    const float *dXv = scr + S_DXV / 4, *hh = scr + S_HH / 4;
    // a thread owns four adjacent channels and every eighth token: 16-byte accesses, coalesced rows
    const int r4 = (threadIdx.x & 31) * 4;
#pragma unroll 2
    for (int i = threadIdx.x >> 5; i < kC; i += kT / 32) {
        const int t = i * D + r4;
        const bool live = i < x.len;
        const float4 g4 = *reinterpret_cast<const float4*>(wsG + t), a4 = *reinterpret_cast<const float4*>(dQ + t);
        const float4 p4 = *reinterpret_cast<const float4*>(dKp + t), m4 = *reinterpret_cast<const float4*>(dKm + t);
        const float4 x4 = *reinterpret_cast<const float4*>(dXv + t);
        float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f), w4 = b4;
        uint2 qr = make_uint2(0, 0), kr = qr, vr = qr;
        if (live) {
            b4 = *reinterpret_cast<const float4*>(p.bv + base + i * rs + r4);
            w4 = *reinterpret_cast<const float4*>(p.wv + base + i * rs + r4);
            qr = *reinterpret_cast<const uint2*>(qp + i * rs + r4);
            kr = *reinterpret_cast<const uint2*>(kp + i * rs + r4);
            vr = *reinterpret_cast<const uint2*>(vp + i * rs + r4);
        }
        const float g[4] = {g4.x, g4.y, g4.z, g4.w}, dqt[4] = {a4.x, a4.y, a4.z, a4.w}, dkp4[4] = {p4.x, p4.y, p4.z, p4.w};
        const float dkm4[4] = {m4.x, m4.y, m4.z, m4.w}, xv[4] = {x4.x, x4.y, x4.z, x4.w};
        const float bb[4] = {b4.x, b4.y, b4.z, b4.w}, ww[4] = {w4.x, w4.y, w4.z, w4.w};
        const float q[4] = {bf16_lo(qr.x), bf16_hi(qr.x), bf16_lo(qr.y), bf16_hi(qr.y)};
        const float k[4] = {bf16_lo(kr.x), bf16_hi(kr.x), bf16_lo(kr.y), bf16_hi(kr.y)};
        const float v[4] = {bf16_lo(vr.x), bf16_hi(vr.x), bf16_lo(vr.y), bf16_hi(vr.y)};
        float dq[4], dk[4], db[4], dv[4], dw[4], dgm[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float G = expf(g[j]), iG = expf(-g[j]);
            dq[j] = G * dqt[j];                       // dq = Gam . dQ~
            const float row = G * dkp4[j];            // what multiplies b . k in the row role
            const float col = iG * dkm4[j];           // column role
            dk[j] = fmaf(bb[j], row, col);
            db[j] = k[j] * row;
            dgm[j] = q[j] * dq[j] + k[j] * bb[j] * row - k[j] * col;
            dv[j] = ww[j] * xv[j];                    // dv = w . dXv
            dw[j] = v[j] * xv[j];                     // dw = v . dXv
        }
        *reinterpret_cast<float4*>(dgam + t) = make_float4(dgm[0], dgm[1], dgm[2], dgm[3]);
        if (live) {
            *reinterpret_cast<uint2*>(dqp + i * rs + r4) = make_uint2(pack_bf16(dq[0], dq[1]), pack_bf16(dq[2], dq[3]));
            *reinterpret_cast<uint2*>(dkp + i * rs + r4) = make_uint2(pack_bf16(dk[0], dk[1]), pack_bf16(dk[2], dk[3]));
            *reinterpret_cast<uint2*>(dvp + i * rs + r4) = make_uint2(pack_bf16(dv[0], dv[1]), pack_bf16(dv[2], dv[3]));
            *reinterpret_cast<float4*>(p.dbv + base + i * rs + r4) = make_float4(db[0], db[1], db[2], db[3]);
            *reinterpret_cast<float4*>(p.dwv + base + i * rs + r4) = make_float4(dw[0], dw[1], dw[2], dw[3]);
        }
    }
    __syncthreads();
    // the chunk end collects rowdot(dh'', h + K-^T U) (from cw_intra); then dg_j = sum_{i >= j} dgam_i per channel
    if (threadIdx.x < D) {
        const int r = threadIdx.x;
        float run = hh[r];
        for (int i = kC - 1; i >= 0; --i) {
            run += dgam[i * D + r];
            if (i < x.len) p.dgv[base + i * rs + r] = run;
        }
    }
}

}  // namespace

#undef GDN_WAIT_MMA

// Host side: the channel-wise calls on this route (bf16 I/O, d_k = d_v = 128).
size_t cw_tc_scratch_per_chunkhead() { return S_BYTES; }

cudaError_t cw_tc_launch(const Problem& p, bool bwd, bool skip_recompute, cudaStream_t st) {
    static SmemLimitOnce once_scale, once_prep, once_intra, once_post;
    const int CH = p.L.max_chunks * p.d.H, chains = p.d.N * p.d.H;
    cudaError_t e = launch_table(p, st);
    if (e != cudaSuccess) return e;
    if (CH > 0) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int grid = CH < sms ? CH : sms;
        const uint32_t sm_scale = sizeof(float) * kC * (D + 1);
        if ((e = once_scale.ensure(cw_scale_kernel, sm_scale)) != cudaSuccess) return e;
        if ((e = once_prep.ensure(cw_prep_kernel, prepcw::SMEM_BYTES)) != cudaSuccess) return e;
        const int mode = bwd ? (skip_recompute ? 2 : 1) : 0;
        { StageScope t(ST_SCALE, st); cw_scale_kernel<<<CH, kT, sm_scale, st>>>(p, mode); }
        { StageScope t(ST_PREP, st); cw_prep_kernel<<<grid, kT, prepcw::SMEM_BYTES, st>>>(p, mode); }
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (chains > 0 && (e = tc_launch_scan_channelwise(p, bwd ? (skip_recompute ? 1 : 2) : 0, st)) != cudaSuccess) return e;
    if (bwd && CH > 0) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int grid = CH < sms ? CH : sms;
        const uint32_t sm_post = sizeof(float) * kC * D;
        if ((e = once_intra.ensure(cw_intra_kernel, intracw::SMEM_BYTES)) != cudaSuccess) return e;
        if ((e = once_post.ensure(cw_post_kernel, sm_post)) != cudaSuccess) return e;
        { StageScope t(ST_INTRA, st); cw_intra_kernel<<<grid, kT, intracw::SMEM_BYTES, st>>>(p); }
        { StageScope t(ST_POST, st); cw_post_kernel<<<CH, kT, sm_post, st>>>(p); }
    }
    return cudaGetLastError();
}

}  // namespace gdn
