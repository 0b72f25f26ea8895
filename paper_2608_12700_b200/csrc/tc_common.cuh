// Device helpers shared by the tcgen05 kernel families: tile chunk access, fixed-order reductions, staged output
// stores, chunk bookkeeping and the bounded MMA wait.
#pragma once
#include "gdn_internal.cuh"
#include "tc_ptx.cuh"
#include "tc_tmap.cuh"

namespace gdn {
namespace {

using namespace tc;

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ void report_timeout(char* ws, int where) {
    WsHeader* h = reinterpret_cast<WsHeader*>(ws);
    h->status = GDN_ERR_DEVICE_TIMEOUT;
    h->detail = where;
}

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
    return p + ((1024u - (smem_u32(p) & 1023u)) & 1023u);
}

// 8 fp32 <-> one 16-byte chunk of bf16
__device__ __forceinline__ uint4 pack8(const float* v) {
    return make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
}
__device__ __forceinline__ void unpack8(const uint4& u, float* v) {
    v[0] = bf16_lo(u.x); v[1] = bf16_hi(u.x); v[2] = bf16_lo(u.y); v[3] = bf16_hi(u.y);
    v[4] = bf16_lo(u.z); v[5] = bf16_hi(u.z); v[6] = bf16_lo(u.w); v[7] = bf16_hi(u.w);
}
// Chunk `ch` (columns 8 ch .. 8 ch + 7) of row r of a tile with R rows.
__device__ __forceinline__ void chunk_store(unsigned char* tile, int R, int r, int ch, const float* v) {
    *reinterpret_cast<uint4*>(tile + tile_chunk_off(R, r, ch)) = pack8(v);
}
__device__ __forceinline__ void chunk_load(const unsigned char* tile, int R, int r, int ch, float* v) {
    unpack8(*reinterpret_cast<const uint4*>(tile + tile_chunk_off(R, r, ch)), v);
}
// Eight consecutive floats from a 16-byte aligned shared array (two vector loads instead of eight scalar ones).
__device__ __forceinline__ void ld8s(const float* p, float* v) {
    *reinterpret_cast<float4*>(v) = *reinterpret_cast<const float4*>(p);
    *reinterpret_cast<float4*>(v + 4) = *reinterpret_cast<const float4*>(p + 4);
}
__device__ __forceinline__ float tile_get(const unsigned char* tile, int R, int r, int c) {
    return __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(tile + tile_off(R, r, c)));
}
__device__ __forceinline__ void tile_put(unsigned char* tile, int R, int r, int c, float x) {
    *reinterpret_cast<__nv_bfloat16*>(tile + tile_off(R, r, c)) = __float2bfloat16_rn(x);
}

// Zero rows [row0 + len, row0 + 64) of a tile with R rows and 128 columns (threads 0 .. nthr-1 of the CTA take part).
__device__ __forceinline__ void zero_tail_rows(unsigned char* tile, int R, int row0, int len, int nthr) {
    for (int t = threadIdx.x; t < (kC - len) * 16; t += nthr) {
        const int r = row0 + len + t / 16, ch = t % 16;
        *reinterpret_cast<uint4*>(tile + tile_chunk_off(R, r, ch)) = make_uint4(0, 0, 0, 0);
    }
}
__device__ __forceinline__ void zero_tail_rows(unsigned char* tile, int R, int row0, int len) {
    zero_tail_rows(tile, R, row0, len, (int)blockDim.x);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Each lane holds 8 values (one per token of a group of 8); returns, on every lane, the sum over the 32 lanes of
// the value belonging to token (lane % 8).  Fixed order: bit-identical from run to run.
__device__ __forceinline__ float reduce8(float (&v)[8], int lane) {
    bool up = (lane & 4) != 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float send = up ? v[k] : v[k + 4], keep = up ? v[k + 4] : v[k];
        v[k] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    }
    up = (lane & 2) != 0;
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const float send = up ? v[k] : v[k + 2], keep = up ? v[k + 2] : v[k];
        v[k] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
    }
    up = (lane & 1) != 0;
    {
        const float send = up ? v[0] : v[1], keep = up ? v[1] : v[0];
        v[0] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
    }
    float r = v[0];
    r += __shfl_xor_sync(0xffffffffu, r, 8);
    r += __shfl_xor_sync(0xffffffffu, r, 16);
    return r;
}

// Copy a staged [64 tokens][128 features] bf16 tile to a [T, H, 128] tensor with 16-byte stores (rows < len only).
__device__ __forceinline__ void flush_rows(const unsigned char* tile, __nv_bfloat16* gbase, size_t row_pitch, int len, int nthr) {
    for (int t = threadIdx.x; t < kC * 16; t += nthr) {
        const int i = t >> 4, chk = t & 15;
        if (i < len) *reinterpret_cast<uint4*>(gbase + (size_t)i * row_pitch + chk * 8) = *reinterpret_cast<const uint4*>(tile + tile_chunk_off(64, i, chk));
    }
}
__device__ __forceinline__ void flush_rows(const unsigned char* tile, __nv_bfloat16* gbase, size_t row_pitch, int len) {
    flush_rows(tile, gbase, row_pitch, len, (int)blockDim.x);
}

// dg_j = sum_{i >= j} dgam_i inside a chunk (gam_i = sum_{j <= i} g_j), by one warp: lane l owns tokens l and l + 32.
// v0 + v1 (two partial arrays, v1 may be null) are the 64 values of dgam; `last_extra` is added to the last one.
__device__ __forceinline__ void write_dg_suffix(const float* v0, const float* v1, float last_extra, float* dg, size_t stride,
                                                int len, int lane) {
    float a = v0[lane] + (v1 ? v1[lane] : 0.f);
    float b = v0[lane + 32] + (v1 ? v1[lane + 32] : 0.f) + (lane == 31 ? last_extra : 0.f);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float ta = __shfl_down_sync(0xffffffffu, a, o), tb = __shfl_down_sync(0xffffffffu, b, o);
        if (lane + o < 32) { a += ta; b += tb; }
    }
    a += __shfl_sync(0xffffffffu, b, 0);
    if (lane < len) dg[(size_t)lane * stride] = a;
    if (lane + 32 < len) dg[(size_t)(lane + 32) * stride] = b;
}

// Chunk geometry.  With packed sequences (cu_seqlens given) it is read from the table the table kernel wrote into the
// workspace; with equal-length sequences it is plain arithmetic and that kernel is not launched at all (the first
// kernel of the call initialises the header instead, see init_header_if_untabled).
struct ChunkInfo { int c, hd, ch, tok0, len; };
__device__ __forceinline__ int chunks_per_sequence(const Problem& p) { return (p.d.T + kC - 1) / kC; }
__device__ __forceinline__ int n_chunks_of(const Problem& p) {
    return p.cu ? reinterpret_cast<const WsHeader*>(p.ws)->n_chunks : p.d.N * chunks_per_sequence(p);
}
__device__ __forceinline__ int seq_first_chunk(const Problem& p, int n) {
    return p.cu ? reinterpret_cast<const int32_t*>(p.ws + p.L.seq_first)[n] : n * chunks_per_sequence(p);
}
// Entry of an item known to exist: no header read and no branch on loaded data, so the two table loads can stay in
// flight until their values are used (the persistent kernels fetch the entry one trip ahead).
__device__ __forceinline__ void chunk_entry(const Problem& p, ChunkInfo& x, int item) {
    x.c = item / p.d.H;
    x.hd = item % p.d.H;
    x.ch = item;
    if (p.cu) {
        x.tok0 = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0)[x.c];
        x.len = reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len)[x.c];
    } else {
        const int cps = chunks_per_sequence(p), n = x.c / cps, pos = x.c - n * cps;
        x.tok0 = n * p.d.T + pos * kC;
        x.len = min(kC, p.d.T - pos * kC);
    }
}
// The same geometry for kernels that walk along whole sequences.
struct ChunkGeom {
    const int32_t *first, *tok0, *len;   // tables (packed sequences), else null
    int cps, T;                          // equal lengths: chunks per sequence, tokens per sequence
    __device__ __forceinline__ int seq_first(int n) const { return first ? first[n] : n * cps; }
    __device__ __forceinline__ int chunk_tok0(int c) const {
        if (tok0) return tok0[c];
        const int n = c / cps;
        return n * T + (c - n * cps) * kC;
    }
    __device__ __forceinline__ int chunk_len(int c) const { return len ? len[c] : min(kC, T - (c % cps) * kC); }
};
__device__ __forceinline__ ChunkGeom chunk_geom(const Problem& p) {
    ChunkGeom g;
    g.first = p.cu ? reinterpret_cast<const int32_t*>(p.ws + p.L.seq_first) : nullptr;
    g.tok0 = p.cu ? reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_tok0) : nullptr;
    g.len = p.cu ? reinterpret_cast<const int32_t*>(p.ws + p.L.chunk_len) : nullptr;
    g.cps = max(1, chunks_per_sequence(p));
    g.T = p.d.T;
    return g;
}
// One sequence, for the kernels that walk along it: its chunks are consecutive, each starts 64 tokens after the one
// before, only the last can be short.  (cu_seqlens has been validated by the table kernel by the time it is read here.)
struct SeqGeom {
    int c0, n_chunks, tok0, len;   // first chunk, number of chunks, first token, tokens
    __device__ __forceinline__ int chunk_tok0(int c) const { return tok0 + (c - c0) * kC; }
    __device__ __forceinline__ int chunk_len(int c) const { return min(kC, len - (c - c0) * kC); }
};
__device__ __forceinline__ SeqGeom seq_geom(const Problem& p, int n) {
    SeqGeom g;
    if (p.cu) {
        g.tok0 = p.cu[n];
        g.len = p.cu[n + 1] - g.tok0;
        g.c0 = reinterpret_cast<const int32_t*>(p.ws + p.L.seq_first)[n];
    } else {
        g.tok0 = n * p.d.T;
        g.len = p.d.T;
        g.c0 = n * chunks_per_sequence(p);
    }
    g.n_chunks = (g.len + kC - 1) / kC;
    return g;
}
__device__ __forceinline__ bool chunk_info(const Problem& p, ChunkInfo& x, int item) {
    if (item / p.d.H >= n_chunks_of(p)) return false;
    chunk_entry(p, x, item);
    return true;
}
__device__ __forceinline__ bool chunk_info(const Problem& p, ChunkInfo& x) { return chunk_info(p, x, (int)blockIdx.x); }
// Called at the top of the first kernel of a call: without the table kernel somebody has to reset the status word.
__device__ __forceinline__ void init_header_if_untabled(const Problem& p) {
    if (!p.cu && blockIdx.x == 0 && threadIdx.x == 0) {
        WsHeader* hdr = reinterpret_cast<WsHeader*>(p.ws);
        hdr->status = GDN_OK;
        hdr->n_chunks = n_chunks_of(p);
        hdr->detail = 0;
    }
}

// Wait for the MMAs committed to `bar`; on a timeout record it once.
#define GDN_WAIT_MMA(where)                                                    \
    if (ok) {                                                                  \
        ok = mbar_wait(&bar_mma, mma_phase);                                   \
        mma_phase ^= 1;                                                        \
        if (!ok && threadIdx.x == 0) report_timeout(p.ws, where);              \
    }                                                                          \
    tc_fence_after();

}  // namespace
}  // namespace gdn
