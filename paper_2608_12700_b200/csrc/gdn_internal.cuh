// Internal declarations shared by the host API and the kernel translation units.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "gdn.h"

namespace gdn {

constexpr int kC = 64;  // chunk length (Section 4.2: chunks of 64 steps)

// Workspace header, first 256 bytes of the workspace.
struct WsHeader {
    int32_t status;    // device-side gdn_status (0 = ok)
    int32_t n_chunks;  // chunks actually present (<= max_chunks)
    int32_t detail;    // where a bounded wait gave up / offending sequence index
    int32_t cw_fallback;   // channel-wise calls: 1 if the last call on this workspace was computed by the fall-back kernels
                           // (then the workspace holds their fp32 data, not tile images); kept across calls
    int32_t pad[60];
};
static_assert(sizeof(WsHeader) == 256, "header size");

// Byte offsets of every workspace region.  Chunk-head index = chunk * H + head.
struct WsLayout {
    int max_chunks;        // bound on the number of chunks: sum over sequences of ceil(len/64) <= ceil(T_total/64) + N
    size_t seq_first;      // int32 [N + 1]   first chunk index of each sequence
    size_t chunk_seq;      // int32 [max_chunks]
    size_t chunk_tok0;     // int32 [max_chunks]   global token index of the chunk's first row
    size_t chunk_len;      // int32 [max_chunks]   valid rows (1..64)
    size_t gamma;          // f32 [CH, 64]         chunk-local cumulative log decay
    size_t Tm;             // f32|bf16 [CH, 64, 64]    T = (I + A)^-1
    size_t W;              // [CH, 64, d_k]
    size_t Ut;             // [CH, 64, d_v]            U~ = T Diag(w) V
    size_t Nm;             // [CH, d_k, d_k]           Kb^T W        (these two only when the carries run in operator
    size_t Bf;             // [CH, d_k, d_v]           Kb^T U~        form: has_operator; otherwise they take no space)
    int has_operator;
    size_t hc;             // [CH, d_k, d_v]           state entering the chunk
    size_t fwd_end;        // bytes needed by the forward recompute
    size_t E;              // [CH, d_k, d_v]           scale (Gam Q - P W)^T dO
    size_t dhn;            // [CH, d_k, d_v]           gradient w.r.t. the state leaving the chunk
    size_t Pm;             // [CH, 64, 64]             P = tril(Q K^T . D) (tcgen05 d = 128 family: made once, by tc_prep)
    size_t img_W, img_U, img_K, img_E;   // channel-wise path on the tensor cores (bf16, d = 128): bf16 tile images of W^T,
                                         // U~^T, the scaled keys Kb (16 KB per chunk-head each) and E (32 KB); else unused
    size_t img_QKp, img_Km, img_Vt, img_dO;   // ... of [Q~; K+] (32 KB), K-, V~ and scale dO (16 KB each)
    int tc_scans;                        // ... and T, P, hc, dhn are bf16 tile images as well (8, 8, 32, 32 KB)
    size_t scratch;        // kernel-private staging, per chunk-head
    size_t scratch_per_ch; // bytes of scratch per chunk-head
    size_t total;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// elem = bytes per element of the chunk factors and stored states (T, W, U~, Nm, hc, dhn): 4 on the fp32
// path, 2 for the bf16 tile images of the tcgen05 path.  elem_add = bytes per element of Bf and E.
inline WsLayout make_layout(const gdn_desc& d, size_t elem, size_t elem_add, size_t scratch_per_ch, bool with_operator = true) {
    WsLayout L{};
    const size_t Ttot = (size_t)d.B * (size_t)d.T;
    L.max_chunks = (int)((Ttot + kC - 1) / kC + (size_t)d.N);
    const size_t CH = (size_t)L.max_chunks * d.H;
    size_t o = sizeof(WsHeader);
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
    L.seq_first = take(4 * ((size_t)d.N + 1));
    L.chunk_seq = take(4 * (size_t)L.max_chunks);
    L.chunk_tok0 = take(4 * (size_t)L.max_chunks);
    L.chunk_len = take(4 * (size_t)L.max_chunks);
    L.gamma = take(4 * CH * kC);
    L.Tm = take(elem * CH * kC * kC);
    L.W = take(elem * CH * kC * d.d_k);
    L.Ut = take(elem * CH * kC * d.d_v);
    L.has_operator = with_operator ? 1 : 0;
    L.Nm = take(with_operator ? elem * CH * d.d_k * d.d_k : 0);
    L.Bf = take(with_operator ? elem_add * CH * d.d_k * d.d_v : 0);
    L.hc = take(elem * CH * d.d_k * d.d_v);
    L.fwd_end = o;
    L.E = take(elem_add * CH * d.d_k * d.d_v);
    L.dhn = take(elem * CH * d.d_k * d.d_v);
    L.Pm = take(elem * CH * kC * kC);
    L.scratch_per_ch = scratch_per_ch;
    L.scratch = take(scratch_per_ch * CH);
    L.total = o;
    return L;
}

// Layout of the channel-wise FFMA family: everything fp32; gamma is per channel ([CH, 64, d_k]), no chunk operator.
inline bool vec_tc_scans(const gdn_desc& d) { return d.dtype == GDN_BF16 && d.d_k == 128 && d.d_v == 128; }
inline WsLayout make_layout_vec(const gdn_desc& d, size_t scratch_per_ch) {
    WsLayout L{};
    const size_t Ttot = (size_t)d.B * (size_t)d.T;
    L.max_chunks = (int)((Ttot + kC - 1) / kC + (size_t)d.N);
    const size_t CH = (size_t)L.max_chunks * d.H;
    size_t o = sizeof(WsHeader);
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
    L.tc_scans = vec_tc_scans(d) ? 1 : 0;
    L.seq_first = take(4 * ((size_t)d.N + 1));
    L.chunk_seq = take(4 * (size_t)L.max_chunks);
    L.chunk_tok0 = take(4 * (size_t)L.max_chunks);
    L.chunk_len = take(4 * (size_t)L.max_chunks);
    L.gamma = take(4 * CH * kC * d.d_k);
    L.Tm = take(4 * CH * kC * kC);
    L.W = take(4 * CH * kC * d.d_k);
    L.Ut = take(4 * CH * kC * d.d_v);
    L.Pm = take(4 * CH * kC * kC);
    L.Nm = L.Bf = o;
    L.img_W = take(L.tc_scans ? CH * 16384 : 0);
    L.img_U = take(L.tc_scans ? CH * 16384 : 0);
    L.img_K = take(L.tc_scans ? CH * 16384 : 0);
    L.img_QKp = take(L.tc_scans ? CH * 32768 : 0);
    L.img_Km = take(L.tc_scans ? CH * 16384 : 0);
    L.img_Vt = take(L.tc_scans ? CH * 16384 : 0);
    L.hc = take(4 * CH * d.d_k * d.d_v);   // (fp32, or a bf16 tile image in the first half of each slot)
    L.fwd_end = o;
    L.E = take(4 * CH * d.d_k * d.d_v);
    L.img_E = take(L.tc_scans ? CH * 32768 : 0);
    L.img_dO = take(L.tc_scans ? CH * 16384 : 0);
    L.dhn = take(4 * CH * d.d_k * d.d_v);
    L.scratch_per_ch = scratch_per_ch;
    L.scratch = take(scratch_per_ch * CH);
    L.total = o;
    return L;
}

// Everything a kernel needs to know about one call.
struct Problem {
    gdn_desc d;
    int Ttot;  // B * T
    const void *q, *k, *v, *dO;
    const float *g, *beta, *h0, *dhT;
    const int32_t* cu;
    void *o, *dq, *dk, *dv;
    float *hT, *dg, *dbeta, *dh0;
    // channel-wise entry points only: gate vectors g, b [.., d_k], w [.., d_v] and their gradients (g, dg above unused)
    const float *gv, *bv, *wv;
    float *dgv, *dbv, *dwv;
    int fallback;   // channel-wise FFMA kernels only: 1 = run only if the tensor-core route has refused the gates (status word)
    char* ws;
    WsLayout L;
};

// Launch bookkeeping: every kernel launch goes through stage_begin / stage_end so that launches can be
// counted and, when enabled, timed per stage with CUDA events on the launching stream.
enum Stage { ST_TABLE = 0, ST_PREP, ST_FSCAN, ST_OUT, ST_EPREP, ST_RSCAN, ST_INTRA, ST_SCANS, ST_SCALE, ST_POST, ST_FALLBACK, ST_COUNT };
void stage_begin(Stage s, cudaStream_t st);
void stage_end(Stage s, cudaStream_t st);
struct StageScope {
    Stage s; cudaStream_t st;
    StageScope(Stage s_, cudaStream_t st_) : s(s_), st(st_) { stage_begin(s, st); }
    ~StageScope() { stage_end(s, st); }
};

// Raising a kernel's dynamic shared-memory limit is a per-device function attribute: remember, per kernel, on which
// devices it has been done (a process may drive several GPUs).
struct SmemLimitOnce {
    bool done[64] = {};
    template <class Kernel>
    cudaError_t ensure(Kernel kernel, uint32_t bytes) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
        return e;
    }
};

gdn_status check_desc(const gdn_desc* d);                       // shape / dtype envelope
gdn_status check_seq(const gdn_desc& d, const int32_t* cu);     // B, N against cu_seqlens
void call_begin();                                              // stage-timing bookkeeping at the top of an entry point

// Host-side argument checks of gdn_bwd (everything that can be refused before a launch), shared with the entry point
// that brings its own workspace.
gdn_status check_bwd_args(const gdn_desc* desc, const void* q, const void* k, const void* v, const float* g, const float* beta,
                          const float* h0, const void* dO, const float* dhT, const int32_t* cu, void* dq, void* dk, void* dv,
                          float* dg, float* dbeta, float* dh0, const void* workspace, size_t workspace_bytes);

// Kernel families (each defined in its own translation unit).  They enqueue on `st` and return the
// first CUDA error seen.
cudaError_t launch_table(const Problem& p, cudaStream_t st);
cudaError_t simt_launch_fwd(const Problem& p, cudaStream_t st);
cudaError_t simt_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st);
size_t simt_scratch_per_chunkhead(const gdn_desc& d);

// FFMA family for per-channel gates (Eq. 1 with gate vectors).
cudaError_t vec_launch_fwd(const Problem& p, cudaStream_t st);
cudaError_t vec_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st);
size_t vec_scratch_per_chunkhead(const gdn_desc& d);
// ... and its tensor-core route (bf16 I/O, d_k = d_v = 128; gdn_tc_cw.cu): forward (bwd = false) or backward.
cudaError_t cw_tc_launch(const Problem& p, bool bwd, bool skip_recompute, cudaStream_t st);
size_t cw_tc_scratch_per_chunkhead();

// tcgen05 family (bf16 I/O, d_k = d_v = 128, delta rule on).
extern thread_local int g_force_carries;   // form of the inter-chunk carries: 0 = chosen by shape, 1 = operator form, 2 = low-rank
extern thread_local int g_inject_timeout;   // debugging hook: the next gdn_bwd of this family provokes a device-side time-out
bool tc_supported(const gdn_desc& d);
// Form of the carries for a descriptor: one rule for the forward, the backward and a backward that consumes a workspace
// fresh from the forward, so that the layout of a workspace does not depend on which call sized it.
bool tc_carries_lowrank(const gdn_desc& d);
cudaError_t tc_launch_scan_channelwise(const Problem& p, int dirs, cudaStream_t st);   // carries of the channel-wise path
cudaError_t tc_launch_out_channelwise(const Problem& p, cudaStream_t st);              // its forward output (p.o non-null)
cudaError_t tc_launch_fwd(const Problem& p, cudaStream_t st);
cudaError_t tc_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st);


// bf16 shapes with a head dimension of 64, zero-padded onto the d = 128 kernels (gdn_pad.cu); `channelwise`: the call has
// gate vectors, which are padded too, and the widened problem runs through vec_launch_fwd / vec_launch_bwd.
bool tc_padded_supported(const gdn_desc& d);
gdn_desc tc_padded_desc(const gdn_desc& d);          // the widened descriptor (d_k = d_v = 128)
size_t tc_padded_extra_bytes(const gdn_desc& d, bool channelwise);   // bytes of padded copies behind the widened problem's own workspace
cudaError_t tc_padded_launch(const Problem& p, const WsLayout& inner, bool bwd, bool skip_recompute, bool channelwise, cudaStream_t st);

// tcgen05 family for the scalar-gate recurrence (bf16 I/O, d_k = d_v = 64, delta rule off).
bool tc64_supported(const gdn_desc& d);
cudaError_t tc64_launch_fwd(const Problem& p, cudaStream_t st);
cudaError_t tc64_launch_bwd(const Problem& p, bool skip_recompute, cudaStream_t st);

}  // namespace gdn
