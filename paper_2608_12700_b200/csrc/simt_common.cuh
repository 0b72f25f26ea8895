// Helpers shared by the fp32 FFMA kernel families: element access for either I/O dtype, register-tiled products fed
// through accessor lambdas, fixed-order reductions, and the (chunk, head) context of a CTA.
#pragma once
#include "gdn_internal.cuh"

namespace gdn {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float x) { *p = x; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// Visit every 4x4 tile of an M x N output once; body(i0, j0).
template <class Body>
__device__ __forceinline__ void tiles(int M, int N, Body body) {
    const int nt = N / 4;
    for (int t = threadIdx.x; t < (M / 4) * nt; t += blockDim.x) body((t / nt) * 4, (t % nt) * 4);
}

// acc[a][b] += sum_m fa(i0 + a, m) * fb(m, j0 + b)
template <class FA, class FB>
__device__ __forceinline__ void mac(float (&acc)[4][4], int i0, int j0, int K, FA fa, FB fb) {
#pragma unroll 4
    for (int m = 0; m < K; ++m) {
        float a[4], b[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) { a[x] = fa(i0 + x, m); b[x] = fb(m, j0 + x); }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
            for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
    }
}

// Sum over a warp in a fixed order.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// out[i] = sum_j f(i, j) for i < 64, one warp per row round-robin.
template <class F>
__device__ __forceinline__ void row_reduce(float* out, int ncols, F f) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    for (int i = warp; i < kC; i += nw) {
        float s = 0.f;
        for (int j = lane; j < ncols; j += 32) s += f(i, j);
        s = warp_sum(s);
        if (lane == 0) out[i] = s;
    }
}

struct ChunkCtx {
    int c, hd, ch, tok0, len;
};

__device__ __forceinline__ bool chunk_ctx(const Problem& p, ChunkCtx& x) {
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(p.ws);
    x.c = blockIdx.x / p.d.H;
    x.hd = blockIdx.x % p.d.H;
    if (x.c >= hdr->n_chunks) return false;
    x.ch = blockIdx.x;
    x.tok0 = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0)[x.c];
    x.len = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len)[x.c];
    return true;
}

}  // namespace
}  // namespace gdn
