// sm_100a building blocks: mbarriers with bounded waits, TMA loads, tensor memory management,
// tcgen05.mma with shared-memory descriptors, tcgen05.ld/st.  Everything is inline PTX; nothing
// here depends on a particular kernel.
//
// Shared-memory operand layout used throughout: the canonical 128-byte-swizzled layout of 16-bit
// elements.  A "box" is R rows of 128 bytes (64 bf16); the 16-byte chunk c of row r is stored at
// chunk position c ^ (r & 7).  Boxes start on 1024-byte boundaries.
//   * K-major operand (contraction index contiguous): rows = M or N index, a box covers 64
//     contraction elements; 8-row groups are 1024 bytes apart (SBO).  One MMA (K = 16) reads 32
//     bytes of each row: the descriptor start address advances by 32 bytes per K step.
//   * MN-major operand (M or N index contiguous): rows = contraction index, a box covers 64 M/N
//     elements; 8-row groups 1024 bytes apart (SBO), further 64-element M/N groups LBO bytes
//     apart.  One MMA reads 16 rows: the start address advances by 2048 bytes per K step.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace umma {

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------------------------------------
// mbarrier
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

// Invalidates a barrier so that its shared-memory word may be initialised again.
__device__ __forceinline__ void mbar_inval(uint64_t* bar)
{
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
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

// Bounded wait: gives up after `limit_cycles` of polling (about two seconds by default), records
// `code` in the device status word and returns false.  Callers then skip the dependent work; nothing
// spins forever.  The result is made uniform across the warp so that warp-aligned instructions stay
// converged.
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* status, int code,
                                          long long limit_cycles = WAIT_LIMIT_CYCLES)
{
    bool done = mbar_try_wait(bar, parity);
    if (!done) {
        const long long t0 = clock64();
        uint32_t it = 0;
        while (!(done = mbar_try_wait(bar, parity))) {
            if ((++it & 1023u) == 0u) {
                if (clock64() - t0 > limit_cycles) break;
                if (status && *reinterpret_cast<volatile int*>(status) != 0) break;
            }
        }
        if (!done && status) atomicCAS(status, 0, code);
    }
    return __all_sync(0xffffffffu, done);
}

// ---------------------------------------------------------------------------------------------
// proxies and fences
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void fence_proxy_async()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// TMA
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* tmap, int x, int y, uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(tmap), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// Plain bulk copy global -> shared (both 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

// Plain bulk copy shared -> global, tracked by the issuing thread's bulk async-group.  The source
// must have been made visible to the async proxy (fence_proxy_async by the writers, then a barrier).
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
}
// TMA tile store shared -> global through a tensor map (bulk async-group of the issuing thread).
__device__ __forceinline__ void tma_store_2d(const void* tmap, int x, int y, const void* smem_src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(tmap), "r"(x), "r"(y), "r"(smem_u32(smem_src)) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all committed bulk stores of this thread have finished READING shared memory
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... and have completed
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// ... all but the N most recently committed groups of this thread have completed
template <int N> __device__ __forceinline__ void bulk_wait_all_but() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }

// Requests that only warm the L2 cache (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_2d(const void* tmap, int x, int y)
{
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tmap), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void bulk_prefetch(const void* gsrc, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(gsrc), "r"(bytes) : "memory");
}

// 4-byte asynchronous copy global -> shared by the calling thread (cp.async group of that thread);
// with valid == false nothing is read and the destination is filled with zero.
__device__ __forceinline__ void cp_async4_zfill(void* smem_dst, const void* gsrc, bool valid)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(valid ? 4 : 0)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void prefetch_tmap(const void* tmap)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}

// ---------------------------------------------------------------------------------------------
// tensor memory
// ---------------------------------------------------------------------------------------------
// Generic-proxy and async-proxy accesses to global memory are ordered by this fence (a tile written by
// bulk stores is published with a plain store; a tile found through a plain load is read by bulk copies).
__device__ __forceinline__ void fence_proxy_async_all()
{
    asm volatile("fence.proxy.async.global;" ::: "memory");
}
__device__ __forceinline__ int ld_acquire_gpu(const int* p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int* p, int v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Barrier over the first `nthreads` threads of the CTA (a multiple of 32), hardware barrier `id` (1..15).
__device__ __forceinline__ void named_sync(int id, int nthreads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// ... that also ANDs a predicate over the participating threads.
__device__ __forceinline__ bool named_sync_and(int id, int nthreads, bool pred)
{
    int out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %3, 0;\n\t"
        "bar.red.and.pred p, %1, %2, q;\n\tselp.s32 %0, 1, 0, p;\n\t}"
        : "=r"(out)
        : "r"(id), "r"(nthreads), "r"((int)pred)
        : "memory");
    return out != 0;
}

// One full warp allocates `ncols` (power of two >= 32) columns; the base address lands in *dst_smem.
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// ---------------------------------------------------------------------------------------------
// descriptors
// ---------------------------------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle.  Fields: start address >> 4 (bits 0-13),
// leading byte offset >> 4 (16-29), stride byte offset >> 4 (32-45), version 1 (46-47),
// layout type SWIZZLE_128B = 2 (61-63).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
__device__ __forceinline__ uint64_t desc_kmajor(const void* box) { return make_desc(smem_u32(box), 16, 1024); }
__device__ __forceinline__ uint64_t desc_mnmajor(const void* box, uint32_t lbo_bytes)
{
    return make_desc(smem_u32(box), lbo_bytes, 1024);
}
__device__ __forceinline__ uint64_t desc_advance(uint64_t d, uint32_t bytes) { return d + (bytes >> 4); }

// Instruction descriptor for kind::f16 with bf16 operands and fp32 accumulation.
constexpr uint32_t IDESC_A_NEG = 1u << 13;
constexpr uint32_t IDESC_A_MN = 1u << 15;
constexpr uint32_t IDESC_B_MN = 1u << 16;
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, uint32_t flags = 0)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | flags | (static_cast<uint32_t>(N >> 3) << 17) |
           (static_cast<uint32_t>(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]; issued by ONE thread.
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Makes `bar` complete once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}

// A sequence of K steps of one product.  a_step / b_step: descriptor advance per K = 16 step in
// bytes (32 for K-major, 2048 for MN-major).
__device__ __forceinline__ void mma_ksteps(uint32_t d_tmem, uint64_t a_desc, uint32_t a_step, uint64_t b_desc,
                                           uint32_t b_step, uint32_t idesc, int ksteps, bool accumulate_first)
{
    for (int s = 0; s < ksteps; ++s)
        mma_ss(d_tmem, desc_advance(a_desc, a_step * s), desc_advance(b_desc, b_step * s), idesc,
               (s > 0 || accumulate_first) ? 1u : 0u);
}

// ---------------------------------------------------------------------------------------------
// tensor memory <-> registers.  32x32b shape: thread t of the warp accesses lane (base + t),
// `N` consecutive 32-bit columns.  The warp may only touch its own lane quadrant (warp % 4).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t* r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(taddr)
                 : "memory");
}
// 16x32bx2 shape: two 16-lane accesses in one instruction.  Threads 0-15 of the warp read lanes
// base .. base + 15 at columns [col, col + 8), threads 16-31 read the SAME 16 lanes at columns
// [col + 8, col + 16).  A 64-row accumulator keeps its rows in lanes 0-15 of every lane quadrant, so this
// form reads 16 of its columns with all 32 threads busy (8 columns each).
__device__ __forceinline__ void tmem_ld_half8(uint32_t taddr, uint32_t* r)
{
    asm volatile("tcgen05.ld.sync.aligned.16x32bx2.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8], 8;"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// swizzled shared-memory addressing for thread-written operands
// ---------------------------------------------------------------------------------------------
// Byte offset inside a box of the 16-byte chunk holding elements [8*chunk, 8*chunk+8) of row r.
__device__ __forceinline__ uint32_t sw128_chunk(uint32_t r, uint32_t chunk)
{
    return r * 128u + ((chunk ^ (r & 7u)) << 4);
}
// Byte offset of element (r, c), c in [0, 64).
__device__ __forceinline__ uint32_t sw128_elem(uint32_t r, uint32_t c)
{
    return sw128_chunk(r, c >> 3) + ((c & 7u) << 1);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

}  // namespace umma
