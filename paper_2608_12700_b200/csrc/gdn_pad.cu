// bf16 shapes with a head dimension of 64 on the tcgen05 d = 128 kernels (scalar gates and channel-wise calls alike): the narrow dimension is padded
// with zeros to 128.  The recurrence is exact under this padding: a zero key/query column adds nothing to any dot
// product and leaves its state row at zero; a zero value / dO column evolves independently of the others (state
// columns never mix) and yields zero gradients.  The padded copies live in the caller's workspace behind the
// kernels' own regions; small copy kernels widen the inputs before and narrow the outputs after the three main kernels.
#include "gdn_internal.cuh"

namespace gdn {
namespace {

// rows of 64 bf16 -> rows of 128 bf16 (upper half zero), 16 bytes per thread and step
__global__ void widen_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t rows) {
    for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < rows * 16; t += (size_t)gridDim.x * blockDim.x) {
        const size_t r = t >> 4;
        const int c = (int)(t & 15);
        dst[t] = c < 8 ? src[r * 8 + c] : make_uint4(0, 0, 0, 0);
    }
}
// rows of 128 bf16 -> their first 64
__global__ void narrow_rows_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t rows) {
    for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < rows * 8; t += (size_t)gridDim.x * blockDim.x)
        dst[t] = src[(t >> 3) * 16 + (t & 7)];
}
// fp32 states [n, dk, dv] <-> [n, 128, 128]
__global__ void widen_state_kernel(const float* __restrict__ src, float* __restrict__ dst, size_t n, int dk, int dv) {
    for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < n * 128 * 128; t += (size_t)gridDim.x * blockDim.x) {
        const size_t s = t >> 14;
        const int r = (int)((t >> 7) & 127), c = (int)(t & 127);
        dst[t] = (r < dk && c < dv) ? src[(s * dk + r) * dv + c] : 0.f;
    }
}
__global__ void narrow_state_kernel(const float* __restrict__ src, float* __restrict__ dst, size_t n, int dk, int dv) {
    for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < n * dk * dv; t += (size_t)gridDim.x * blockDim.x) {
        const size_t s = t / ((size_t)dk * dv);
        const int r = (int)((t / dv) % dk), c = (int)(t % dv);
        dst[t] = src[(s * 128 + r) * 128 + c];
    }
}

// gate vectors: rows of 64 fp32 <-> rows of 128 fp32 (upper half zero: log decay 0, erase gate 0, write gate 0)
__global__ void widen_rows_f32_kernel(const float4* __restrict__ src, float4* __restrict__ dst, size_t rows) {
    for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < rows * 32; t += (size_t)gridDim.x * blockDim.x) {
        const size_t r = t >> 5;
        const int c = (int)(t & 31);
        dst[t] = c < 16 ? src[r * 16 + c] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
}
__global__ void narrow_rows_f32_kernel(const float4* __restrict__ src, float4* __restrict__ dst, size_t rows) {
    for (size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x; t < rows * 16; t += (size_t)gridDim.x * blockDim.x)
        dst[t] = src[(t >> 4) * 32 + (t & 15)];
}

int grid_for(size_t items) {
    const size_t b = (items + 255) / 256;
    return (int)(b < 1 ? 1 : b > 4096 ? 4096 : b);
}

struct PadPlan {
    size_t q, k, v, dO, dq, dk, dv, o, h0, dhT, dh0, hT;   // byte offsets from the start of the pad region
    size_t g, b, w, dg, db, dw;                              // channel-wise calls only: the gate vectors and their gradients
    size_t end;
};
PadPlan plan_for(const gdn_desc& d, bool channelwise) {
    PadPlan P{};
    const size_t rows = (size_t)d.B * d.T * d.H, tok = align_up(rows * 128 * 2, 256), st = align_up((size_t)d.N * d.H * 128 * 128 * 4, 256);
    const size_t gate = channelwise ? align_up(rows * 128 * 4, 256) : 0;
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t r = o; o += bytes; return r; };
    P.q = take(d.d_k == 64 ? tok : 0); P.k = take(d.d_k == 64 ? tok : 0); P.dq = take(d.d_k == 64 ? tok : 0); P.dk = take(d.d_k == 64 ? tok : 0);
    P.v = take(d.d_v == 64 ? tok : 0); P.dO = take(d.d_v == 64 ? tok : 0); P.dv = take(d.d_v == 64 ? tok : 0); P.o = take(d.d_v == 64 ? tok : 0);
    P.h0 = take(st); P.dhT = take(st); P.dh0 = take(st); P.hT = take(st);
    P.g = take(d.d_k == 64 ? gate : 0); P.b = take(d.d_k == 64 ? gate : 0); P.dg = take(d.d_k == 64 ? gate : 0); P.db = take(d.d_k == 64 ? gate : 0);
    P.w = take(d.d_v == 64 ? gate : 0); P.dw = take(d.d_v == 64 ? gate : 0);
    P.end = o;
    return P;
}

}  // namespace

bool tc_padded_supported(const gdn_desc& d) {
    return d.dtype == GDN_BF16 && d.chunk == kC && (d.d_k == 64 || d.d_k == 128) && (d.d_v == 64 || d.d_v == 128) &&
           !(d.d_k == 128 && d.d_v == 128);
}
gdn_desc tc_padded_desc(const gdn_desc& d) {
    gdn_desc w = d;
    w.d_k = w.d_v = 128;
    return w;
}
size_t tc_padded_extra_bytes(const gdn_desc& d, bool channelwise) { return plan_for(d, channelwise).end; }

// `inner` is the layout of the widened problem; the pad region starts at inner.total.
// With `channelwise` the widened problem is a channel-wise call: its gate vectors are widened and their gradients
// narrowed as well (a padded key channel has decay 1 and erase gate 0, a padded value channel write gate 0; with zero
// keys, queries and values there, every product is what it was).
cudaError_t tc_padded_launch(const Problem& p, const WsLayout& inner, bool bwd, bool skip_recompute, bool channelwise, cudaStream_t st) {
    const gdn_desc& d = p.d;
    const PadPlan pl = plan_for(d, channelwise);
    char* pad = p.ws + align_up(inner.total, 256);
    const size_t rows = (size_t)p.Ttot * d.H, chains = (size_t)d.N * d.H;
    Problem w = p;
    w.d = tc_padded_desc(d);
    w.L = inner;
    auto widen = [&](const void* src, size_t off) -> const void* {
        if (!src || rows == 0) return src;
        StageScope t(ST_TABLE, st);
        widen_rows_kernel<<<grid_for(rows * 16), 256, 0, st>>>(static_cast<const uint4*>(src), reinterpret_cast<uint4*>(pad + off), rows);
        return pad + off;
    };
    auto widen_state = [&](const float* src, size_t off) -> const float* {
        if (!src) return nullptr;
        StageScope t(ST_TABLE, st);
        widen_state_kernel<<<grid_for(chains * 16384), 256, 0, st>>>(src, reinterpret_cast<float*>(pad + off), chains, d.d_k, d.d_v);
        return reinterpret_cast<const float*>(pad + off);
    };
    auto widen_gate = [&](const float* src, size_t off) -> const float* {
        if (!src || rows == 0) return src;
        StageScope t(ST_TABLE, st);
        widen_rows_f32_kernel<<<grid_for(rows * 32), 256, 0, st>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<float4*>(pad + off), rows);
        return reinterpret_cast<const float*>(pad + off);
    };
    const bool fresh = bwd && skip_recompute;   // the widened forward inputs are still in the workspace
    if (channelwise && d.d_k == 64) {
        if (!fresh) { w.gv = widen_gate(p.gv, pl.g); w.bv = widen_gate(p.bv, pl.b); }
        else { w.gv = reinterpret_cast<const float*>(pad + pl.g); w.bv = reinterpret_cast<const float*>(pad + pl.b); }
        if (bwd) { w.dgv = reinterpret_cast<float*>(pad + pl.dg); w.dbv = reinterpret_cast<float*>(pad + pl.db); }
    }
    if (channelwise && d.d_v == 64) {
        if (!fresh) w.wv = widen_gate(p.wv, pl.w); else w.wv = reinterpret_cast<const float*>(pad + pl.w);
        if (bwd) w.dwv = reinterpret_cast<float*>(pad + pl.dw);
    }
    if (d.d_k == 64) {
        if (!fresh) { w.q = widen(p.q, pl.q); w.k = widen(p.k, pl.k); } else { w.q = pad + pl.q; w.k = pad + pl.k; }
        if (bwd) { w.dq = pad + pl.dq; w.dk = pad + pl.dk; }
    }
    if (d.d_v == 64) {
        if (!fresh) w.v = widen(p.v, pl.v); else w.v = pad + pl.v;
        if (bwd) { w.dO = widen(p.dO, pl.dO); w.dv = pad + pl.dv; }
        if (!bwd && p.o) w.o = pad + pl.o;
    }
    if (!fresh) w.h0 = widen_state(p.h0, pl.h0);
    else w.h0 = p.h0 ? reinterpret_cast<const float*>(pad + pl.h0) : nullptr;
    if (bwd) {
        w.dhT = widen_state(p.dhT, pl.dhT);
        if (p.dh0) w.dh0 = reinterpret_cast<float*>(pad + pl.dh0);
    } else if (p.hT) {
        w.hT = reinterpret_cast<float*>(pad + pl.hT);
    }
    cudaError_t e = channelwise ? (bwd ? vec_launch_bwd(w, skip_recompute, st) : vec_launch_fwd(w, st))
                                : (bwd ? tc_launch_bwd(w, skip_recompute, st) : tc_launch_fwd(w, st));
    if (e != cudaSuccess) return e;
    auto narrow = [&](const void* src, void* dst) {
        if (!dst || rows == 0) return;
        StageScope t(ST_TABLE, st);
        narrow_rows_kernel<<<grid_for(rows * 8), 256, 0, st>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst), rows);
    };
    auto narrow_state = [&](const float* src, float* dst) {
        if (!dst) return;
        StageScope t(ST_TABLE, st);
        narrow_state_kernel<<<grid_for(chains * d.d_k * d.d_v), 256, 0, st>>>(src, dst, chains, d.d_k, d.d_v);
    };
    auto narrow_gate = [&](const float* src, float* dst) {
        if (!dst || rows == 0) return;
        StageScope t(ST_TABLE, st);
        narrow_rows_f32_kernel<<<grid_for(rows * 16), 256, 0, st>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<float4*>(dst), rows);
    };
    if (bwd) {
        if (d.d_k == 64) { narrow(w.dq, p.dq); narrow(w.dk, p.dk); }
        if (d.d_v == 64) narrow(w.dv, p.dv);
        if (channelwise && d.d_k == 64) { narrow_gate(w.dgv, p.dgv); narrow_gate(w.dbv, p.dbv); }
        if (channelwise && d.d_v == 64) narrow_gate(w.dwv, p.dwv);
        narrow_state(w.dh0, p.dh0);
    } else {
        if (d.d_v == 64) narrow(w.o, p.o);
        narrow_state(w.hT, p.hT);
    }
    return cudaGetLastError();
}

}  // namespace gdn
