// Thin inline-PTX layer for sm_100a: mbarrier, bulk/TMA copies, tensor memory and tcgen05.mma.
// Everything here is a one-to-one wrapper of a PTX instruction plus the shared-memory tile format the
// kernels agree on.
//
// Tile format ("blocked-64, 128-byte swizzle"): a bf16 matrix of R rows and 64*nb columns is stored as
// nb column blocks of R rows x 64 columns; a block row is 128 bytes; the eight 16-byte chunks of a row are
// permuted by XOR with (row % 8).  Blocks are R*128 bytes apart and must start on 1024-byte boundaries.
// The same bytes serve tcgen05.mma as a K-major operand (contraction over columns) and as an MN-major
// operand (contraction over rows), so no explicit transposes are ever made.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace gdn {
namespace tc {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---------------------------------------------------------------- tile addressing
// Byte offset of element (r, c) inside a tile with R rows.
__device__ __forceinline__ uint32_t tile_off(int R, int r, int c) {
    return (uint32_t)((c >> 6) * R * 128 + r * 128 + ((((c & 63) >> 3) ^ (r & 7)) << 4) + ((c & 7) << 1));
}
// Byte offset of the 16-byte chunk holding columns [8*ch, 8*ch + 8) of row r.
__device__ __forceinline__ uint32_t tile_chunk_off(int R, int r, int ch) {
    return (uint32_t)((ch >> 3) * R * 128 + r * 128 + (((ch & 7) ^ (r & 7)) << 4));
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// How long a bounded wait polls before it gives up (one copy per translation unit; two seconds unless the host-side
// debugging hook that provokes a time-out has shortened it for one call).
static __device__ unsigned long long g_wait_limit_ns = 2000000000ull;
// Bounded wait: gives up after about two seconds and returns false; the caller records the failure and
// leaves through its normal teardown (no trap, no endless spin).  Only the first probe is inlined at a wait site: a
// kernel has dozens of them and the polling loop with its time-out would multiply the code size (the instruction
// cache is cold at every launch and each CTA's first trip pays for every byte of code).
static __device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > g_wait_limit_ns) return false;
    }
}
// The same wait with its polling loop at the wait site: no call, so nothing has to be saved around it.  For the small
// kernels (the carries, the scalar-gate passes), where code size does not matter and a step is short.
__device__ __forceinline__ bool mbar_wait_inline(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
#pragma unroll 1
    for (uint32_t i = 1;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 0) {
            const uint64_t t = global_ns();
            if (t0 == 0) t0 = t;
            else if (t - t0 > g_wait_limit_ns) return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
#ifdef GDN_INLINE_WAIT
    return mbar_wait_inline(bar, parity);
#else
    return mbar_try_wait(bar, parity) || mbar_wait_slow(bar, parity);
#endif
}

// ---------------------------------------------------------------- proxies and copies
// Make generic-proxy writes to shared memory visible to the async proxy (TMA, tcgen05.mma).
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// 2-D tiled TMA load: box lands at smem_dst, completion bytes are counted on bar.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
// 2-D tiled TMA store of one box from shared memory (tracked by the bulk async-group of the issuing thread).
__device__ __forceinline__ void tma_store_2d(const void* tmap, int x, int y, const void* smem_src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(tmap), "r"(x), "r"(y),
                 "r"(smem_u32(smem_src))
                 : "memory");
}
// Contiguous bulk copy global -> shared (both 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
// Hints that bring data into L2 ahead of the copies that will need it (no shared memory involved).
__device__ __forceinline__ void prefetch_l2_bulk(const void* gsrc, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(gsrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void prefetch_l2_tma_2d(const void* tmap, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tmap), "r"(x), "r"(y) : "memory");
}
// Contiguous bulk copy shared -> global, tracked by the bulk async-group of the issuing thread.
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Wait until at most N of this thread's bulk groups still read their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }

// ---------------------------------------------------------------- tensor memory
// One warp allocates `cols` (power of two >= 32) columns; the base address is written to *slot (shared).
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Each thread of a warp reads 32 consecutive fp32 columns of its own lane (lane = 32 * (warp % 4) + laneid).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Same for 8 consecutive columns.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// ---------------------------------------------------------------- tcgen05.mma (bf16 x bf16 -> fp32)
// Instruction descriptor: dense, fp32 accumulate, bf16 A and B.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool a_mn_major, bool b_mn_major, bool neg_a = false) {
    return (1u << 4)                          // D format: fp32
           | (1u << 7) | (1u << 10)           // A, B format: bf16
           | ((neg_a ? 1u : 0u) << 13)        // negate A
           | ((a_mn_major ? 1u : 0u) << 15)   // A major
           | ((b_mn_major ? 1u : 0u) << 16)   // B major
           | ((uint32_t)(N >> 3) << 17)       // N / 8
           | ((uint32_t)(M >> 4) << 24);      // M / 16
}

// Shared-memory matrix descriptor, 128-byte swizzle; lbo/sbo in bytes.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((saddr >> 4) & 0x3FFF) | ((uint64_t)((lbo >> 4) & 0x3FFF) << 16) | ((uint64_t)((sbo >> 4) & 0x3FFF) << 32) |
           (1ull << 46)   // descriptor version of this architecture
           | (2ull << 61);  // 128-byte swizzle
}

// Operand view of a tile (or of a row/column window of it).  The descriptor of the k-th K=16 slice is
// base + k * step + (k / 4) * jump in units of 16 bytes, so that issuing a product costs a few integer adds.
struct Operand {
    uint32_t lo, hi;   // descriptor of slice 0
    uint32_t step;     // added to lo per K=16 slice
    uint32_t jump;     // added to lo on top of that after every fourth slice
    bool mn_major;     // false: contraction runs over tile columns; true: over tile rows
};
// Window whose MN index runs over tile rows starting at row0 and whose K index runs over columns from col0
// (row0 % 8 == 0, col0 % 64 == 0).  16 columns = 32 bytes inside a 128-byte row; every fourth slice moves on to
// the next 64-column block, R * 128 bytes further.
__device__ __forceinline__ Operand op_k_major(const void* tile, int R, int row0 = 0, int col0 = 0) {
    const uint64_t d = make_desc(smem_u32(tile) + (uint32_t)((col0 >> 6) * R * 128 + row0 * 128), 16, 1024);
    return Operand{(uint32_t)d, (uint32_t)(d >> 32), 2u, (uint32_t)(R * 8 - 8), false};
}
// Window whose MN index runs over tile columns starting at col0 and whose K index runs over rows from row0.
// 16 rows = 2048 bytes; LBO = distance between 64-column blocks, SBO = distance between 8-row groups.
__device__ __forceinline__ Operand op_mn_major(const void* tile, int R, int row0 = 0, int col0 = 0) {
    const uint64_t d = make_desc(smem_u32(tile) + (uint32_t)((col0 >> 6) * R * 128 + row0 * 128), (uint32_t)R * 128, 1024);
    return Operand{(uint32_t)d, (uint32_t)(d >> 32), 128u, 0u, true};
}

__device__ __forceinline__ void mma_issue(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[M x N] (+)= A[M x Kt] * B[Kt x N]: one thread issues Kt / 16 instructions, fully unrolled so that each costs two
// integer adds besides the tcgen05.mma itself (the tensor pipe accepts one such instruction every ~50-60 cycles).
template <int M, int N, int Kt>
__device__ __forceinline__ void mma_tile(uint32_t tmem_d, const Operand& a, const Operand& b, bool accumulate, bool neg_a = false) {
    const uint32_t idesc = make_idesc(M, N, a.mn_major, b.mn_major, neg_a);
#pragma unroll
    for (int ks = 0; ks < Kt / 16; ++ks) {
        const uint32_t al = a.lo + ks * a.step + (ks >> 2) * a.jump, bl = b.lo + ks * b.step + (ks >> 2) * b.jump;
        mma_issue(tmem_d, ((uint64_t)a.hi << 32) | al, ((uint64_t)b.hi << 32) | bl, idesc, (accumulate || ks > 0) ? 1u : 0u);
    }
}
// Arrive on `bar` when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// ---------------------------------------------------------------- small conversions
// 2^x, hardware approximation (about 2 ulp); callers pass non-positive arguments only.
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

}  // namespace tc
}  // namespace gdn
