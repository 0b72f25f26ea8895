// Host side of the C ABI: argument validation, workspace layout, launch sequencing.
#include <stdint.h>
#include <string.h>

#include <atomic>
#include <vector>

#include "gdn_internal.cuh"

namespace gdn {

// ---- launch counting and optional per-stage event timing ----
namespace {
std::atomic<uint64_t> g_launches{0};
int g_period = 0;         // 0: no stage timing; n: the stages of every n-th call are bracketed by events
uint64_t g_calls = 0;     // calls since timing was switched on
bool g_timing = false;    // the stages of the call under way are timed
struct Rec { Stage s; cudaEvent_t a, b; };
std::vector<Rec> g_recs;          // recorded since the last read
std::vector<cudaEvent_t> g_pool;  // reusable events
cudaEvent_t g_open = nullptr;
const char* kStageNames[ST_COUNT] = {"table", "prep", "fscan", "out", "eprep", "rscan", "intra", "scans", "scale", "post", "fallback"};
cudaEvent_t take_event() {
    if (!g_pool.empty()) { cudaEvent_t e = g_pool.back(); g_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}
}  // namespace
void call_begin() { g_timing = g_period > 0 && (g_calls++ % (uint64_t)g_period) == 0; }

void stage_begin(Stage, cudaStream_t st) {
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!g_timing) return;
    g_open = take_event();
    cudaEventRecord(g_open, st);
}
void stage_end(Stage s, cudaStream_t st) {
    if (!g_timing || !g_open) return;
    cudaEvent_t b = take_event();
    cudaEventRecord(b, st);
    g_recs.push_back({s, g_open, b});
    g_open = nullptr;
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

enum class Path { None, SimtF32, SimtBf16, TcBf16, Tc64Bf16, TcBf16Padded };

// Debug overrides of the dispatch are per thread: a thread that forces a family cannot change the workspace size
// another thread is computing at that moment.
thread_local int g_force_family = 0;
}  // namespace
thread_local int g_force_carries = 0;   // tcgen05 d = 128 family: 0 = by shape, 1 = operator form (Nm, Bf), 2 = low-rank form
namespace {

Path pick_path(const gdn_desc& d) {
    if (d.dtype == GDN_F32) return Path::SimtF32;
    if (d.dtype == GDN_BF16) {
        if (g_force_family == 1) return Path::SimtBf16;
        if (tc_supported(d)) return Path::TcBf16;
        if (tc64_supported(d)) return Path::Tc64Bf16;
        if (tc_padded_supported(d)) return Path::TcBf16Padded;
        return Path::SimtBf16;
    }
    return Path::None;
}

WsLayout layout_for(const gdn_desc& d) {
    // tcgen05 path: every factor, state and additive term of the carries is a bf16 tile image.
    // The d = 128 family keeps the chunk operator Nm and the additive term Bf only when its carries use them.
    if (pick_path(d) == Path::TcBf16) return make_layout(d, 2, 2, 0, !tc_carries_lowrank(d));
    if (pick_path(d) == Path::Tc64Bf16) return make_layout(d, 2, 2, 0);
    if (pick_path(d) == Path::TcBf16Padded) {   // the widened problem's layout, then the padded copies; one size for both calls
        const gdn_desc w = tc_padded_desc(d);
        WsLayout L = make_layout(w, 2, 2, 0, !tc_carries_lowrank(w));
        L.scratch = align_up(L.total, 256);
        L.total = L.scratch + tc_padded_extra_bytes(d, false);
        L.fwd_end = L.total;
        return L;
    }
    // The SIMT kernels keep every factor in fp32, whatever the I/O dtype.
    return make_layout(d, sizeof(float), sizeof(float), simt_scratch_per_chunkhead(d));
}

// Channel-wise calls: the layout the kernels see (of the widened problem when a head dimension of 64 is zero-padded onto
// the d = 128 tensor-core route) and the sizes the caller is told (padded: one size for both calls).
struct VecPlan {
    bool padded;
    WsLayout inner;
    size_t fwd_bytes, total;
};
VecPlan vec_plan(const gdn_desc& d) {
    VecPlan v{};
    v.padded = tc_padded_supported(d) && g_force_family != 1;
    const gdn_desc w = v.padded ? tc_padded_desc(d) : d;
    v.inner = make_layout_vec(w, vec_scratch_per_chunkhead(w));
    if (g_force_family == 1) v.inner.tc_scans = 0;   // (debug override: the FFMA kernels; the image regions stay unused)
    v.total = v.padded ? align_up(v.inner.total, 256) + tc_padded_extra_bytes(d, true) : v.inner.total;
    v.fwd_bytes = v.padded ? v.total : v.inner.fwd_end;
    return v;
}

}  // namespace
}  // namespace gdn

namespace gdn {
gdn_status check_desc(const gdn_desc* d) {
    if (!d) return GDN_ERR_NULL_ARG;
    if (d->B <= 0 || d->T < 0 || d->H <= 0 || d->N <= 0 || d->d_k <= 0 || d->d_v <= 0) return GDN_ERR_BAD_SHAPE;
    if ((long long)d->B * d->T > 0x7fffffffLL - 64 * 1024) return GDN_ERR_BAD_SHAPE;
    if (d->chunk != kC) return GDN_ERR_UNSUPPORTED_SHAPE;
    if (!((d->d_k == 64 || d->d_k == 128) && (d->d_v == 64 || d->d_v == 128))) return GDN_ERR_UNSUPPORTED_SHAPE;
    if (d->dtype != GDN_F32 && d->dtype != GDN_BF16) return GDN_ERR_UNSUPPORTED_SHAPE;
    if (d->delta_rule != 0 && d->delta_rule != 1) return GDN_ERR_BAD_SHAPE;
    return GDN_OK;
}

// Sequences are described either by cu_seqlens (then B must be 1) or by B rows of T tokens (then N == B).
gdn_status check_seq(const gdn_desc& d, const int32_t* cu) {
    if (cu) { if (d.B != 1) return GDN_ERR_BAD_SHAPE; }
    else if (d.N != d.B) return GDN_ERR_BAD_SHAPE;
    return GDN_OK;
}

gdn_status check_bwd_args(const gdn_desc* desc, const void* q, const void* k, const void* v, const float* g, const float* beta,
                          const float* h0, const void* dO, const float* dhT, const int32_t* cu, void* dq, void* dk, void* dv,
                          float* dg, float* dbeta, float* dh0, const void* workspace, size_t workspace_bytes) {
    gdn_status s = check_desc(desc);
    if (s != GDN_OK) return s;
    if ((s = check_seq(*desc, cu)) != GDN_OK) return s;
    const bool empty = (long long)desc->B * desc->T == 0;   // no tokens: token tensors may be NULL
    if (!workspace) return GDN_ERR_NULL_ARG;
    if (!empty && (!q || !k || !v || !g || !dO || !dq || !dk || !dv || !dg)) return GDN_ERR_NULL_ARG;
    if (!empty && desc->delta_rule && (!beta || !dbeta)) return GDN_ERR_NULL_ARG;
    const void* ptrs[] = {q, k, v, g, beta, h0, dO, dhT, cu, dq, dk, dv, dg, dbeta, dh0, workspace};
    for (const void* p : ptrs) if (!aligned16(p)) return GDN_ERR_MISALIGNED;
    if (workspace_bytes < layout_for(*desc).total) return GDN_ERR_WORKSPACE_TOO_SMALL;
    return GDN_OK;
}
}  // namespace gdn

using namespace gdn;

extern "C" {

gdn_status gdn_workspace_bytes(const gdn_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes) {
    gdn_status s = check_desc(desc);
    if (s != GDN_OK) return s;
    const WsLayout L = layout_for(*desc);
    if (fwd_bytes) *fwd_bytes = L.fwd_end;
    if (bwd_bytes) *bwd_bytes = L.total;
    return GDN_OK;
}

gdn_status gdn_fwd_recompute(const gdn_desc* desc, const void* q, const void* k, const void* v, const float* g,
                             const float* beta, const float* h0, const int32_t* cu, void* o, float* hT,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
    call_begin();
    gdn_status s = check_desc(desc);
    if (s != GDN_OK) return s;
    if ((s = check_seq(*desc, cu)) != GDN_OK) return s;
    const bool empty = (long long)desc->B * desc->T == 0;   // no tokens: token tensors may be NULL
    if (!workspace) return GDN_ERR_NULL_ARG;
    if (!empty && (!q || !k || !v || !g)) return GDN_ERR_NULL_ARG;
    if (!empty && desc->delta_rule && !beta) return GDN_ERR_NULL_ARG;
    const void* ptrs[] = {q, k, v, g, beta, h0, cu, o, hT, workspace};
    for (const void* p : ptrs) if (!aligned16(p)) return GDN_ERR_MISALIGNED;
    Problem p{};
    p.d = *desc;
    p.Ttot = desc->B * desc->T;
    p.L = layout_for(*desc);
    if (workspace_bytes < p.L.fwd_end) return GDN_ERR_WORKSPACE_TOO_SMALL;
    p.q = q; p.k = k; p.v = v; p.g = g; p.beta = beta; p.h0 = h0; p.cu = cu; p.o = o; p.hT = hT;
    p.ws = static_cast<char*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Path path = pick_path(*desc);
    cudaError_t e;
    if (path == Path::TcBf16Padded) {
        const gdn_desc w = tc_padded_desc(*desc);
        e = tc_padded_launch(p, make_layout(w, 2, 2, 0, !tc_carries_lowrank(w)), false, false, false, st);
    } else {
        e = path == Path::TcBf16 ? tc_launch_fwd(p, st) : path == Path::Tc64Bf16 ? tc64_launch_fwd(p, st) : simt_launch_fwd(p, st);
    }
    return e == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

gdn_status gdn_bwd(const gdn_desc* desc, const void* q, const void* k, const void* v, const float* g, const float* beta,
                   const float* h0, const void* dO, const float* dhT, const int32_t* cu, void* dq, void* dk, void* dv,
                   float* dg, float* dbeta, float* dh0, void* workspace, size_t workspace_bytes,
                   int32_t workspace_is_fresh_from_fwd, void* cuda_stream) {
    call_begin();
    const gdn_status s = check_bwd_args(desc, q, k, v, g, beta, h0, dO, dhT, cu, dq, dk, dv, dg, dbeta, dh0, workspace, workspace_bytes);
    if (s != GDN_OK) return s;
    Problem p{};
    p.d = *desc;
    p.Ttot = desc->B * desc->T;
    p.L = layout_for(*desc);
    p.q = q; p.k = k; p.v = v; p.g = g; p.beta = beta; p.h0 = h0; p.dO = dO; p.dhT = dhT; p.cu = cu;
    p.dq = dq; p.dk = dk; p.dv = dv; p.dg = dg; p.dbeta = dbeta; p.dh0 = dh0;
    p.ws = static_cast<char*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const bool fresh = workspace_is_fresh_from_fwd != 0;
    const Path path = pick_path(*desc);
    cudaError_t e;
    if (path == Path::TcBf16Padded) {
        const gdn_desc w = tc_padded_desc(*desc);
        e = tc_padded_launch(p, make_layout(w, 2, 2, 0, !tc_carries_lowrank(w)), true, fresh, false, st);
    } else {
        e = path == Path::TcBf16 ? tc_launch_bwd(p, fresh, st)
            : path == Path::Tc64Bf16 ? tc64_launch_bwd(p, fresh, st) : simt_launch_bwd(p, fresh, st);
    }
    return e == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

// ---- channel-wise entry points: Eq. 1 with gate vectors (FFMA family) ----
gdn_status gdn_workspace_bytes_channelwise(const gdn_desc* desc, size_t* fwd_bytes, size_t* bwd_bytes) {
    gdn_status s = check_desc(desc);
    if (s != GDN_OK) return s;
    const VecPlan v = vec_plan(*desc);
    if (fwd_bytes) *fwd_bytes = v.fwd_bytes;
    if (bwd_bytes) *bwd_bytes = v.total;
    return GDN_OK;
}

gdn_status gdn_fwd_recompute_channelwise(const gdn_desc* desc, const void* q, const void* k, const void* v, const float* g,
                                         const float* b, const float* w, const float* h0, const int32_t* cu, void* o,
                                         float* hT, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    call_begin();
    gdn_status s = check_desc(desc);
    if (s != GDN_OK) return s;
    if ((s = check_seq(*desc, cu)) != GDN_OK) return s;
    const bool empty = (long long)desc->B * desc->T == 0;
    if (!workspace) return GDN_ERR_NULL_ARG;
    if (!empty && (!q || !k || !v || !g || !b || !w)) return GDN_ERR_NULL_ARG;
    const void* ptrs[] = {q, k, v, g, b, w, h0, cu, o, hT, workspace};
    for (const void* p : ptrs) if (!aligned16(p)) return GDN_ERR_MISALIGNED;
    Problem p{};
    p.d = *desc;
    p.Ttot = desc->B * desc->T;
    const VecPlan plan = vec_plan(*desc);
    p.L = plan.inner;
    if (workspace_bytes < plan.fwd_bytes) return GDN_ERR_WORKSPACE_TOO_SMALL;
    p.q = q; p.k = k; p.v = v; p.gv = g; p.bv = b; p.wv = w; p.h0 = h0; p.cu = cu; p.o = o; p.hT = hT;
    p.ws = static_cast<char*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const cudaError_t e = plan.padded ? tc_padded_launch(p, plan.inner, false, false, true, st) : vec_launch_fwd(p, st);
    return e == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

gdn_status gdn_bwd_channelwise(const gdn_desc* desc, const void* q, const void* k, const void* v, const float* g,
                               const float* b, const float* w, const float* h0, const void* dO, const float* dhT,
                               const int32_t* cu, void* dq, void* dk, void* dv, float* dg, float* db, float* dw, float* dh0,
                               void* workspace, size_t workspace_bytes, int32_t workspace_is_fresh_from_fwd, void* cuda_stream) {
    call_begin();
    gdn_status s = check_desc(desc);
    if (s != GDN_OK) return s;
    if ((s = check_seq(*desc, cu)) != GDN_OK) return s;
    const bool empty = (long long)desc->B * desc->T == 0;
    if (!workspace) return GDN_ERR_NULL_ARG;
    if (!empty && (!q || !k || !v || !g || !b || !w || !dO || !dq || !dk || !dv || !dg || !db || !dw)) return GDN_ERR_NULL_ARG;
    const void* ptrs[] = {q, k, v, g, b, w, h0, dO, dhT, cu, dq, dk, dv, dg, db, dw, dh0, workspace};
    for (const void* p : ptrs) if (!aligned16(p)) return GDN_ERR_MISALIGNED;
    Problem p{};
    p.d = *desc;
    p.Ttot = desc->B * desc->T;
    const VecPlan plan = vec_plan(*desc);
    p.L = plan.inner;
    if (workspace_bytes < plan.total) return GDN_ERR_WORKSPACE_TOO_SMALL;
    p.q = q; p.k = k; p.v = v; p.gv = g; p.bv = b; p.wv = w; p.h0 = h0; p.dO = dO; p.dhT = dhT; p.cu = cu;
    p.dq = dq; p.dk = dk; p.dv = dv; p.dgv = dg; p.dbv = db; p.dwv = dw; p.dh0 = dh0;
    p.ws = static_cast<char*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const bool fresh = workspace_is_fresh_from_fwd != 0;
    const cudaError_t e = plan.padded ? tc_padded_launch(p, plan.inner, true, fresh, true, st) : vec_launch_bwd(p, fresh, st);
    return e == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}

gdn_status gdn_last_device_status(const void* workspace, void* cuda_stream) {
    if (!workspace) return GDN_ERR_NULL_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return GDN_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return GDN_ERR_CUDA;
    if (word == GDN_OK || word == GDN_ERR_BAD_SEQLENS || word == GDN_ERR_DEVICE_TIMEOUT || word == GDN_ERR_DECAY_RANGE)
        return (gdn_status)word;
    return GDN_ERR_CUDA;
}

const char* gdn_status_string(gdn_status s) {
    switch (s) {
        case GDN_OK: return "ok";
        case GDN_ERR_NULL_ARG: return "a required pointer is NULL";
        case GDN_ERR_BAD_SHAPE: return "invalid shape or sequence description";
        case GDN_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (chunk must be 64, d_k and d_v in {64,128}, dtype f32 or bf16)";
        case GDN_ERR_MISALIGNED: return "a pointer is not 16-byte aligned";
        case GDN_ERR_BAD_SEQLENS: return "cu_seqlens is malformed (must start at 0, be non-decreasing and end at T)";
        case GDN_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case GDN_ERR_CUDA: return "a CUDA call failed";
        case GDN_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
        case GDN_ERR_DECAY_RANGE: return "cumulative log decay of a chunk outside [-80, 80] (channel-wise call on the tensor cores)";
    }
    return "unknown status";
}

gdn_status gdn_debug_force_family(int32_t family) {
    if (family < 0 || family > 3) return GDN_ERR_BAD_SHAPE;
    g_force_family = family == 1 ? 1 : 0;
    g_force_carries = family >= 2 ? family - 1 : 0;
    return GDN_OK;
}

gdn_status gdn_debug_inject_timeout(int32_t on) {
    g_inject_timeout = on ? 1 : 0;
    return GDN_OK;
}

gdn_status gdn_debug_read(const gdn_desc* desc, const void* workspace, const char* what, int32_t chunk, int32_t head,
                          float* host_out) {
    gdn_status s = check_desc(desc);
    if (s != GDN_OK) return s;
    if (!workspace || !what || !host_out) return GDN_ERR_NULL_ARG;
    const WsLayout L = layout_for(*desc);
    if (chunk < 0 || chunk >= L.max_chunks || head < 0 || head >= desc->H) return GDN_ERR_BAD_SHAPE;
    if (pick_path(*desc) == Path::TcBf16Padded) return GDN_ERR_UNSUPPORTED_SHAPE;   // (stored as the widened problem)
    const bool tcp = pick_path(*desc) == Path::TcBf16 || pick_path(*desc) == Path::Tc64Bf16;
    const size_t ch = (size_t)chunk * desc->H + head;
    const int dk = desc->d_k, dv = desc->d_v;
    struct Q { const char* name; size_t off; int rows, cols; int kind; };  // kind 0: fp32 row-major always
    // kind 1: factor (fp32 row-major | bf16 tile image [rows][cols]); kind 2: factor stored transposed as an image
    // [cols][rows] on the tcgen05 path
    const Q table[] = {{"gamma", L.gamma, 1, kC, 0}, {"T", L.Tm, kC, kC, 1},    {"W", L.W, kC, dk, 2},
                       {"Ut", L.Ut, kC, dv, 2},      {"Nm", L.Nm, dk, dk, 1},   {"Bf", L.Bf, dk, dv, 1},
                       {"hc", L.hc, dk, dv, 1},      {"E", L.E, dk, dv, 1},     {"dhn", L.dhn, dk, dv, 1}};
    const Q* q = nullptr;
    for (const Q& t : table) if (strcmp(t.name, what) == 0) q = &t;
    if (!q) return GDN_ERR_BAD_SHAPE;
    if (!L.has_operator && (q->off == L.Nm || q->off == L.Bf) && (strcmp(what, "Nm") == 0 || strcmp(what, "Bf") == 0))
        return GDN_ERR_BAD_SHAPE;   // not stored: the carries of this descriptor run in low-rank form
    if (cudaDeviceSynchronize() != cudaSuccess) return GDN_ERR_CUDA;
    const size_t n = (size_t)q->rows * q->cols;
    const char* base = static_cast<const char*>(workspace) + q->off;
    if (q->kind == 0 || !tcp) {
        return cudaMemcpy(host_out, base + ch * n * 4, n * 4, cudaMemcpyDeviceToHost) == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
    }
    std::vector<uint16_t> img(n);
    if (cudaMemcpy(img.data(), base + ch * n * 2, n * 2, cudaMemcpyDeviceToHost) != cudaSuccess) return GDN_ERR_CUDA;
    const int R = q->kind == 2 ? q->cols : q->rows;       // rows of the stored tile
    auto at = [&](int r, int c) -> float {                 // element (r, c) of the stored tile
        const size_t off = (size_t)(c >> 6) * R * 128 + (size_t)r * 128 + ((((c & 63) >> 3) ^ (r & 7)) << 4) + ((c & 7) << 1);
        const uint32_t bits = (uint32_t)img[off / 2] << 16;
        float f;
        memcpy(&f, &bits, 4);
        return f;
    };
    for (int r = 0; r < q->rows; ++r)
        for (int c = 0; c < q->cols; ++c) host_out[(size_t)r * q->cols + c] = q->kind == 2 ? at(c, r) : at(r, c);
    return GDN_OK;
}

uint64_t gdn_launch_count(void) { return g_launches.load(); }

gdn_status gdn_stage_timing_enable(int32_t on) {
    g_period = on > 0 ? on : 0;
    g_calls = 0;
    g_timing = false;
    return GDN_OK;
}

gdn_status gdn_stage_timing_read(int32_t max_stages, float* total_ms, int32_t* launches, const char** names,
                                 int32_t* n_stages) {
    if (!total_ms || !launches || !names || !n_stages) return GDN_ERR_NULL_ARG;
    float ms[ST_COUNT] = {};
    int32_t cnt[ST_COUNT] = {};
    gdn_status rc = GDN_OK;
    for (const Rec& r : g_recs) {
        float t = 0.f;
        if (cudaEventSynchronize(r.b) != cudaSuccess || cudaEventElapsedTime(&t, r.a, r.b) != cudaSuccess) rc = GDN_ERR_CUDA;
        ms[r.s] += t;
        cnt[r.s] += 1;
        g_pool.push_back(r.a);
        g_pool.push_back(r.b);
    }
    g_recs.clear();
    const int n = max_stages < (int)ST_COUNT ? max_stages : (int)ST_COUNT;
    for (int i = 0; i < n; ++i) { total_ms[i] = ms[i]; launches[i] = cnt[i]; names[i] = kStageNames[i]; }
    *n_stages = n;
    return rc;
}

const char* gdn_kernel_path_channelwise(const gdn_desc* desc) {
    if (check_desc(desc) != GDN_OK) return nullptr;
    if (g_force_family != 1 && tc_padded_supported(*desc)) return "tcgen05_bf16_channelwise_padded";
    if (g_force_family != 1 && vec_tc_scans(*desc)) return "tcgen05_bf16_channelwise";
    return desc->dtype == GDN_BF16 ? "simt_bf16_channelwise" : "simt_f32_channelwise";
}

const char* gdn_kernel_path(const gdn_desc* desc) {
    if (check_desc(desc) != GDN_OK) return nullptr;
    switch (pick_path(*desc)) {
        case Path::SimtF32: return "simt_f32";
        case Path::SimtBf16: return "simt_bf16";
        case Path::TcBf16: return "tcgen05_bf16";
        case Path::Tc64Bf16: return "tcgen05_bf16_scalar_gate";
        case Path::TcBf16Padded: return "tcgen05_bf16_padded";
        default: return nullptr;
    }
}

}  // extern "C"
