// Thin inline-PTX wrappers for the sm_100a features the GEMM kernel uses:
// mbarrier, TMA (cp.async.bulk[.tensor]), tensor memory and tcgen05 MMA.
// Every wait is bounded; nothing here spins forever.
#pragma once

#include <cuda.h>
#include <stdint.h>

namespace gpusq {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ uint64_t globaltimer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool elect_one()
{
    uint32_t pred;
    asm volatile(
        "{\n"
        ".reg .pred P;\n"
        "elect.sync _|P, 0xffffffff;\n"
        "selp.u32 %0, 1, 0, P;\n"
        "}\n"
        : "=r"(pred));
    return pred != 0;
}

// ---- mbarrier ----
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
// One try: the hardware parks the thread for a short, implementation-defined time unless the
// phase has completed.
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred P;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2;\n"
        "selp.u32 %0, 1, 0, P;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Bounded wait: gives up after the time limit, or as soon as another thread of the CTA has raised
// *abort_flag.  The limit, in microseconds, is the word behind the flag (abort_flag[1]; 2 s unless the
// test hook shortens it).  Returns false on either; the
// caller that timed out raises the flag itself.  The common case (the phase
// is complete already) costs one try and one branch; the retry loop is kept
// out of line so that it does not bloat the callers' instruction streams.
// A retry parks the thread in hardware until the phase completes or the hint
// time has passed, so a waiting warp issues a few instructions per microsecond
// and wakes as soon as the barrier flips; the flag and the clock are looked at
// after every `kTriesPerCheck` expired tries.
constexpr uint32_t kDefaultWaitUs = 2000000u;      // 2 s
constexpr uint32_t kSuspendHintNs = 1000;
__device__ __forceinline__ bool mbar_try_wait_32(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred P, Q;\n"
        ".reg .u32 n;\n"
        "mov.u32 n, 32;\n"
        "TRY_AGAIN:\n"
        "mbarrier.try_wait.parity.shared::cta.b64 P, [%1], %2, %3;\n"
        "@P bra DONE;\n"
        "sub.u32 n, n, 1;\n"
        "setp.ne.u32 Q, n, 0;\n"
        "@Q bra TRY_AGAIN;\n"
        "DONE:\n"
        "selp.u32 %0, 1, 0, P;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok != 0;
}

// returns 0 = phase complete, 1 = abort flag seen, 2 = time limit reached
__device__ __noinline__ int mbar_wait_slow(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag)
{
    const uint64_t t0 = globaltimer_ns();
    for (;;) {
        if (mbar_try_wait_32(bar, parity)) return 0;
        if (*abort_flag) return 1;
        if (globaltimer_ns() - t0 > (uint64_t)abort_flag[1] * 1000ull) return 2;
    }
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity,
                                                  volatile uint32_t *abort_flag, bool &timed_out)
{
    timed_out = false;
    if (mbar_try_wait(bar, parity)) return true;
    const int r = mbar_wait_slow(bar, parity, abort_flag);
    timed_out = r == 2;
    return r == 0;
}

// ---- TMA ----
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *m)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, uint32_t src, int32_t c0, int32_t c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(src), "r"(c0), "r"(c1)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void tma_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void tma_store_wait_all()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
// ---- tensor memory ----
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// arrive on an mbarrier once every tcgen05 operation issued so far by this thread has completed
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp receives lane (base + i)
__device__ __forceinline__ void tmem_ld_32x32b_x16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// 16 lanes x 32 columns in the MMA accumulator-fragment arrangement: for column block i (8 columns),
// thread t holds lane t/4, columns 8i + 2(t%4), +1 in r[4i], r[4i+1] and lane t/4 + 8, same columns,
// in r[4i+2], r[4i+3].  The lane field of taddr is a multiple of 16.
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// four 8x8 b16 matrices, stored transposed: memory row i of matrix j (address from thread 8j + i)
// receives, as 8 contiguous b16, the elements the threads hold in column i of their fragment
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r0),
                 "r"(r1), "r"(r2), "r"(r3)
                 : "memory");
}
// four 16x8 matrices of bytes, stored transposed: matrix j takes one register per thread, whose bytes
// are elements (row t/4, columns 2(t%4), 2(t%4)+1) and (row t/4 + 8, the same columns) -- the
// arrangement of an accumulator fragment -- and lands as eight memory rows of 16 bytes (memory row =
// column of the matrix, byte = row of the matrix); the address of memory row i of matrix j comes from
// thread 8j + i.
__device__ __forceinline__ void stmatrix_x4_trans_b8(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    asm volatile("stmatrix.sync.aligned.m16n8.x4.trans.shared.b8 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r0),
                 "r"(r1), "r"(r2), "r"(r3)
                 : "memory");
}
// ---- CTA pairs (clusters of two) ----
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on an mbarrier of any CTA of the cluster (address from map_to_cta)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    // default semantics (release at CTA scope): a cluster-scope release would first drain this thread's
    // global and shared stores, which costs over a thousand cycles while the memory system is loaded
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t cluster_addr, uint32_t v)
{
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// Tiled load whose completion bytes may be counted on an mbarrier of the pair's other CTA
// (bar is a shared::cluster address); the destination is this CTA's own shared memory.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar,
                                                 int32_t c0, int32_t c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

// ---- tensor memory and MMA over a CTA pair (cta_group::2) ----
// Allocation, release of the permit and deallocation are executed by the same warp of both CTAs.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// arrive on the mbarrier at the same shared-memory offset in every CTA of cta_mask once all
// tcgen05 operations issued so far by this thread have completed
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t cta_mask)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(cta_mask)
                 : "memory");
}
// each CTA of the pair copies 128 lanes x 128 bits from its own shared memory into its own tensor memory
__device__ __forceinline__ void tc_cp_128x128b_pair(uint32_t taddr, uint64_t sdesc)
{
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// M = 256 over the pair: each CTA supplies 128 rows of A (and their metadata) and half of B's rows
__device__ __forceinline__ void tc_mma_i8_pair(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_mma_sp_i8_pair(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t meta_taddr,
                                                  uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.sp.cta_group::2.kind::i8 [%0], %1, %2, [%5], %3, p;\n"
        "}\n" ::"r"(d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(meta_taddr)
        : "memory");
}
// binary16 A and B (the same type, as kind::f16 requires), FP32 accumulators, A 2:4 sparse
__device__ __forceinline__ void tc_mma_sp_f16_pair(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t meta_taddr,
                                                   uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%5], %3, p;\n"
        "}\n" ::"r"(d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(meta_taddr)
        : "memory");
}
// Wait for this thread's tensor-memory loads; the registers are operands so that no use of them
// can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait_regs(uint32_t (&r)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :
                 : "memory");
}

// ---- programmatic dependent launch ----
// wait until the kernel this one depends on has completed and its writes are visible (returns at
// once when the launch carried no programmatic dependency)
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// let the next kernel of the stream be scheduled as soon as this grid's CTAs make room
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- descriptors ----
// Shared-memory matrix descriptor for a K-major operand tile whose rows are
// `swizzle_bytes` long (32/64/128-byte swizzle) or, with swizzle_bytes == 0,
// stored as 8-row x 16-byte core matrices.  sbo = byte distance between
// consecutive groups of eight rows.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t sbo, uint32_t swizzle_bytes)
{
    const uint64_t layout = swizzle_bytes == 128 ? 2ull : swizzle_bytes == 64 ? 4ull : swizzle_bytes == 32 ? 6ull : 0ull;
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                                   // leading-dimension offset: unused here
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;               // stride-dimension offset
    d |= (uint64_t)1 << 46;                                   // descriptor version of sm_100
    d |= layout << 61;
    return d;
}

// Instruction descriptor of kind::i8: signed 8-bit A and B, both K-major, INT32 accumulator.
__host__ __device__ constexpr uint32_t make_idesc_i8(int mma_m, int mma_n, bool sparse)
{
    return (sparse ? 1u << 2 : 0u)     // sparsity enabled
           | (2u << 4)                 // accumulator format: S32
           | (1u << 7)                 // A: signed 8-bit
           | (1u << 10)                // B: signed 8-bit
           | ((uint32_t)(mma_n >> 3) << 17) | ((uint32_t)(mma_m >> 4) << 24);
}

// kind::f16, 2:4 sparse A: binary16 A and B (format 0), FP32 accumulators (format 1), K-major operands
__host__ __device__ constexpr uint32_t make_idesc_f16_sparse(int mma_m, int mma_n)
{
    return (1u << 2) | (1u << 4) | ((uint32_t)(mma_n >> 3) << 17) | ((uint32_t)(mma_m >> 4) << 24);
}

}  // namespace ptx
}  // namespace gpusq
