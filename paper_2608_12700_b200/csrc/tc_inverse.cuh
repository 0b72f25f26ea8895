// fp32 blocked inversion of a unit lower triangular 64 x 64 matrix in shared memory (T = (I + A)^-1 of the chunk-local
// solve, Section 4.2), shared by the tcgen05 kernel families.  Thread indices are those of the calling CTA; every step
// uses at most its first 256 threads, and the caller separates the steps by CTA-wide barriers.
#pragma once
#include "tc_common.cuh"

namespace gdn {
namespace {

constexpr int kInvMaxThreads = 512;   // bound used by the static checks of the level passes

// Blocked inverse of I + A (unit lower triangular), fp32 in shared memory, rows of kLdi floats:
//   diagonal 8 x 8 blocks by forward substitution; the 8 x 8 block below the diagonal of every 16 x 16 diagonal block
//   from T10 = -T11 (A10 T00); then with 16 x 16 blocks  At_rk = T_rr A_rk (r > k)  and
//   T_rc = -sum_{k=c}^{r-1} At_rk T_kc, one block diagonal at a time.
// These steps are chains of dependent FMAs fed by shared-memory loads, so a thread produces four adjacent outputs of a
// row (one broadcast scalar and one 16-byte load feed four FMAs) and the longer sums are split over SPLIT adjacent
// lanes and combined by shuffles.
constexpr int kLdi = 68;   // row pitch: 16-byte aligned rows, conflict-free for the access patterns below
__device__ __forceinline__ void inv_diag8(const float* Af, float* Tf) {   // threads 0..63: column j of block b0
    if (threadIdx.x < kC) {   // t_i = [i == j] - sum_{m<i} A_im t_m
        const int b0 = (threadIdx.x >> 3) * 8, j = threadIdx.x & 7;
        float t[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float s = (i == j) ? 1.f : 0.f;
#pragma unroll
            for (int m = 0; m < i; ++m) s = fmaf(-Af[(b0 + i) * kLdi + b0 + m], t[m], s);
            t[i] = s;
            Tf[(b0 + i) * kLdi + b0 + j] = s;
        }
    }
}
__device__ __forceinline__ void inv_diag16(const float* Af, float* Tf, float* Xf) {   // threads 0..255: one entry each
    if (threadIdx.x < 256) {
        const int r0 = (threadIdx.x >> 6) * 16, i = (threadIdx.x >> 3) & 7, j = threadIdx.x & 7;
        float x = 0.f;   // X = A10 T00
#pragma unroll
        for (int m = 0; m < 8; ++m) x = fmaf(Af[(r0 + 8 + i) * kLdi + r0 + m], Tf[(r0 + m) * kLdi + r0 + j], x);
        Xf[(r0 + 8 + i) * kLdi + r0 + j] = x;
        asm volatile("bar.sync 4, 256;" ::: "memory");
        float s = 0.f;   // T10 = -T11 X
#pragma unroll
        for (int k = 0; k < 8; ++k) s = fmaf(Tf[(r0 + 8 + i) * kLdi + r0 + 8 + k], Xf[(r0 + 8 + k) * kLdi + r0 + j], s);
        Tf[(r0 + 8 + i) * kLdi + r0 + j] = -s;     // (disjoint from T00 and T11, which other threads still read)
        Tf[(r0 + i) * kLdi + r0 + 8 + j] = 0.f;    // the block above the diagonal
    }
}
// R rows of a block per thread: the 16-byte load of a row of A feeds R x 4 FMAs (these steps are bound by the number of
// shared-memory wavefronts, and a 16-byte load costs a warp four of them however many lanes share an address).
template <int R>
__device__ __forceinline__ void inv_premul(const float* Af, const float* Tf, float* Sf) {
    // six blocks below the diagonal: (1,0) (2,0) (2,1) (3,0) (3,1) (3,2); per block 16 / R row groups x 4 column groups
    constexpr int per_blk = (16 / R) * 4;
    if (threadIdx.x < 6 * per_blk) {
        const int o = threadIdx.x, blk = o / per_blk, ig = (o % per_blk) >> 2, j4 = (o & 3) * 4;
        const int rb = (blk == 0 ? 1 : blk < 3 ? 2 : 3) * 16, cb = (blk == 0 ? 0 : blk < 3 ? blk - 1 : blk - 3) * 16;
        float4 s[R];
#pragma unroll
        for (int q = 0; q < R; ++q) s[q] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int m = 0; m < 16; ++m) {   // T_rr is lower triangular: zeros above the diagonal
            const float4 v = *reinterpret_cast<const float4*>(Af + (rb + m) * kLdi + cb + j4);
#pragma unroll
            for (int q = 0; q < R; ++q) {   // rows ig, ig + 16 / R, ...: a warp's scalar loads fall into distinct banks
                const float a = Tf[(rb + ig + q * (16 / R)) * kLdi + rb + m];
                s[q].x = fmaf(a, v.x, s[q].x); s[q].y = fmaf(a, v.y, s[q].y); s[q].z = fmaf(a, v.z, s[q].z); s[q].w = fmaf(a, v.w, s[q].w);
            }
        }
#pragma unroll
        for (int q = 0; q < R; ++q) *reinterpret_cast<float4*>(Sf + (rb + ig + q * (16 / R)) * kLdi + cb + j4) = s[q];
    }
}
template <int DIST, int SPLIT, int R>
__device__ __forceinline__ void inv_level(const float* At, float* Tf) {
    constexpr int items = (4 - DIST) * (16 / R) * 4, len = 16 * DIST / SPLIT;
    static_assert(items * SPLIT <= kInvMaxThreads && (items * SPLIT) % 32 == 0, "one pass, whole warps");
    if (threadIdx.x < items * SPLIT) {
        // a warp serves 32 / SPLIT items; the lanes of a quarter-warp share `part`, so their 16-byte loads fall into one
        // row of T (no bank conflicts), and the partial sums of an item sit 32 / SPLIT lanes apart
        constexpr int G = 32 / SPLIT, per_blk = (16 / R) * 4;
        const int wl = threadIdx.x & 31, o = (threadIdx.x >> 5) * G + (wl % G), part = wl / G;
        const int cb = (o / per_blk) * 16, rb = cb + DIST * 16, ig = (o % per_blk) >> 2, j4 = (o & 3) * 4;
        float4 s[R];
#pragma unroll
        for (int q = 0; q < R; ++q) s[q] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int mm = 0; mm < len; ++mm) {
            const int m = part * len + mm;
            const float4 v = *reinterpret_cast<const float4*>(Tf + (cb + m) * kLdi + cb + j4);
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const float a = At[(rb + ig + q * (16 / R)) * kLdi + cb + m];
                s[q].x = fmaf(a, v.x, s[q].x); s[q].y = fmaf(a, v.y, s[q].y); s[q].z = fmaf(a, v.z, s[q].z); s[q].w = fmaf(a, v.w, s[q].w);
            }
        }
#pragma unroll
        for (int q = 0; q < R; ++q) {
#pragma unroll
            for (int d = G; d < 32; d <<= 1) {
                s[q].x += __shfl_xor_sync(0xffffffffu, s[q].x, d); s[q].y += __shfl_xor_sync(0xffffffffu, s[q].y, d);
                s[q].z += __shfl_xor_sync(0xffffffffu, s[q].z, d); s[q].w += __shfl_xor_sync(0xffffffffu, s[q].w, d);
            }
            if (part == 0)
                *reinterpret_cast<float4*>(Tf + (rb + ig + q * (16 / R)) * kLdi + cb + j4) = make_float4(-s[q].x, -s[q].y, -s[q].z, -s[q].w);
        }
    }
}


}  // namespace
}  // namespace gdn
