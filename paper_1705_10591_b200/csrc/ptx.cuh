// Thin wrappers over the sm_100a PTX this library uses: mbarriers with bounded waits, bulk (TMA)
// copies, the async-proxy fence, tcgen05 tensor-memory allocation, MMA issue, commit and loads,
// and the shared-memory / instruction descriptors of tcgen05.mma.
#pragma once

#include <stdint.h>

namespace conv2d_b200 {
namespace ptx {

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}"
                 ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait: gives up after `max_polls` unsuccessful polls (each poll may itself suspend for a
// hardware-defined short time) or as soon as another thread has raised *abort_flag.
// Returns false on give-up; the caller must then stop issuing work and fall through to teardown.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                  uint32_t max_polls = (1u << 22))
{
    for (uint32_t i = 0; i < max_polls; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1u;
    return false;
}

// ---------------------------------------------------------------- thread-block clusters (distributed shared memory)
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in block `rank` of this cluster (shared::cluster window).
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, float a, float b, float c, float d)
{
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
// Arrives on a barrier of another block of the cluster; this thread's earlier writes into that block's shared
// memory are visible to whoever then waits on it with cluster-scope acquire.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_bar_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait on a barrier that threads of the peer block arrive on (see mbar_wait_bounded).
__device__ __forceinline__ bool mbar_wait_bounded_cluster(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                          uint32_t max_polls)
{
    for (uint32_t i = 0; i < max_polls; ++i) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1u;
    return false;
}
// Barrier over all threads of all blocks of the cluster (every thread must call it).
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// ---------------------------------------------------------------- programmatic dependent launch
// grid_dep_launch: the next kernel on the stream (if it was launched with programmatic stream
// serialization) may start to be scheduled now instead of when this grid has drained.
// grid_dep_wait: returns when the preceding grid has completed and its memory operations are visible;
// it must come before the first access to anything that grid may have written or may still be reading.
// Both do nothing in a kernel that was launched the ordinary way.
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- proxies and bulk copies
// Makes this thread's earlier shared-memory writes visible to the async proxy (TMA, tcgen05.mma).
__device__ __forceinline__ void fence_proxy_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// 1-D bulk copy global -> shared of `bytes` (multiple of 16; both addresses 16-byte aligned);
// completion is signalled on `bar` as transaction bytes.
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gmem_src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Tiled (tensor-map) TMA copies.  `map` points to a CUtensorMap in kernel-parameter (grid-constant) space.
// Loads signal `bar` with the box's byte count (out-of-range elements are written as zeros and still counted);
// the innermost coordinate times the element size must be a multiple of 16 bytes.
// (`bar`: shared-memory address of the barrier, as smem_u32 gives it)
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const void* map, int c0, int c1, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const void* map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const void* map, int c0, int c1, int c2, int c3, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar) : "memory");
}
// The same loads for a pair of blocks that run two-SM MMAs (cta_group::2): the box lands in this block's shared
// memory, the bytes are signalled on `cluster_bar`, a shared::cluster address that may name a barrier of the peer
// block (the block that issues the pair's MMAs waits for both blocks' boxes on one barrier).
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const void* map, int c0, int c1, uint32_t cluster_bar)
{
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(void* smem_dst, const void* map, int c0, int c1, int c2, uint32_t cluster_bar)
{
    asm volatile("cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(void* smem_dst, const void* map, int c0, int c1, int c2, int c3, uint32_t cluster_bar)
{
    asm volatile("cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(cluster_bar) : "memory");
}
// Store of one box shared -> global (elements outside the tensor are dropped); completion is tracked per thread
// in bulk groups.
__device__ __forceinline__ void tma_store_3d(const void* map, int c0, int c1, int c2, const void* smem_src)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(smem_src)) : "memory");
}
// The same with the box added to what global memory holds (element-wise, type as in the tensor map) instead of
// replacing it.
__device__ __forceinline__ void tma_reduce_add_3d(const void* map, int c0, int c1, int c2, const void* smem_src)
{
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(smem_src)) : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// all but the newest `N` groups of this thread have finished READING their shared-memory source
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
// all but the newest `N` groups of this thread are complete (their global writes are done)
template <int N>
__device__ __forceinline__ void bulk_wait_group() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void prefetch_tensormap(const void* map)
{
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t columns)   // whole warp; columns: power of 2 >= 32
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(smem_result)), "r"(columns) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t columns)      // whole warp
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(columns) : "memory");
}
// Two-SM form: the same warp of both blocks of the pair executes each of these; both blocks get the same columns.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t columns)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"(smem_u32(smem_result)), "r"(columns) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t columns)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(columns) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, TF32 operands, fp32 accumulate; one thread issues.
__device__ __forceinline__ void mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
// Same with 16-bit operands, bf16 or fp16 as the instruction descriptor says (kind::f16, K = 16 per instruction).
__device__ __forceinline__ void mma_b16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
// Arrives once on `bar` when all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void mma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}
// Two-SM MMAs, issued by one thread of the pair's first block.  D is 256 x N: rows 0-127 in the first block's tensor
// memory, rows 128-255 in the second's, N columns in both.  The descriptors are offsets that hold in both blocks:
// each block's shared memory holds its 128 rows of A and its half of B's N rows at the same addresses.
__device__ __forceinline__ void mma_tf32_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
__device__ __forceinline__ void mma_b16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
// Arrives once on `bar` of this block when all two-SM MMAs issued so far by this thread have completed ...
__device__ __forceinline__ void mma_commit_pair(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(smem_u32(bar)) : "memory");
}
// ... and on the barrier at the same offset in both blocks of the pair.
__device__ __forceinline__ void mma_commit_pair_both(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp receives lane (base lane + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
// 32 lanes x 32 consecutive columns
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld1(uint32_t taddr, uint32_t (&v)[1])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(v[0]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor, K-major, no swizzle.  The operand is stored as 8-row x 16-byte
// core matrices (8 rows of 4 fp32, 16 bytes apart); `k_step_bytes` is the distance between core
// matrices adjacent along K (leading byte offset), `row_group_bytes` the distance between groups
// of 8 rows (stride byte offset).  With row_group_bytes = 128 the rows of one K chunk are simply
// 16 bytes apart, so a descriptor may start at any row.
__device__ __forceinline__ uint64_t smem_desc_kmajor_noswizzle(uint32_t smem_addr, uint32_t k_step_bytes, uint32_t row_group_bytes)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu)
         | ((uint64_t)((k_step_bytes >> 4) & 0x3FFFu) << 16)
         | ((uint64_t)((row_group_bytes >> 4) & 0x3FFFu) << 32)
         | (1ull << 46);                       // descriptor version of sm_100
}
// Shared-memory matrix descriptor for a 128-byte-swizzled operand, as a tiled TMA copy with SWIZZLE_128B and a
// 128-byte inner box writes it: 1024-byte atoms of 8 rows x 128 bytes whose 16-byte chunks are XOR-ed with the row
// number (atoms must start on 1024 bytes).
//   K-major  (a row = one M/N index, 32 consecutive K elements of 4 bytes): `stride_bytes` = distance between
//            groups of 8 rows; a K step of 8 elements advances the start address by 32 bytes inside the row.
//   MN-major (a row = one K index, 32 consecutive M/N elements): `leading_bytes` = distance between atoms that are
//            adjacent along M/N, `stride_bytes` = distance between groups of 8 K rows.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr, uint32_t leading_bytes, uint32_t stride_bytes)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu)
         | ((uint64_t)((leading_bytes >> 4) & 0x3FFFu) << 16)
         | ((uint64_t)((stride_bytes >> 4) & 0x3FFFu) << 32)
         | (1ull << 46)                        // descriptor version of sm_100
         | (2ull << 61);                       // layout type: 128-byte swizzle
}
// MN-major operand of 4-byte elements (TF32): the one layout the tensor core takes for it swizzles 32-byte chunks
// inside 128-byte rows (chunk index XOR row number mod 4; tensor-map copies write it with SWIZZLE_128B_ATOM_32B).
// Atom = 4 K rows x 128 bytes (32 consecutive M/N elements per row).  `leading_bytes` = distance between atoms
// adjacent along M/N, `stride_bytes` = distance between groups of 4 K rows (an MMA of K = 8 reads two groups).
__device__ __forceinline__ uint64_t smem_desc_mn_sw128_32b(uint32_t smem_addr, uint32_t leading_bytes, uint32_t stride_bytes)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu)
         | ((uint64_t)((leading_bytes >> 4) & 0x3FFFu) << 16)
         | ((uint64_t)((stride_bytes >> 4) & 0x3FFFu) << 32)
         | (1ull << 46)                        // descriptor version of sm_100
         | (1ull << 61);                       // layout type: 128-byte swizzle with 32-byte atoms
}
// Bit of the instruction descriptor that declares the B operand MN-major (its M/N index contiguous in memory).
constexpr uint32_t kIdescBMajorMN = 1u << 16;

// Instruction descriptor: TF32 x TF32 -> fp32, both operands K-major, M x N tile.
__host__ __device__ constexpr uint32_t idesc_tf32(uint32_t m, uint32_t n)
{
    return (1u << 4)            // accumulator format fp32
         | (2u << 7)            // A format TF32
         | (2u << 10)           // B format TF32
         | ((n >> 3) << 17)
         | ((m >> 4) << 24);
}

// Instruction descriptor: 16-bit x 16-bit -> fp32 (operand format 0 = fp16, 1 = bf16), both operands K-major.
__host__ __device__ constexpr uint32_t idesc_b16(uint32_t m, uint32_t n, bool fp16)
{
    return (1u << 4)                    // accumulator format fp32
         | ((fp16 ? 0u : 1u) << 7)      // A format
         | ((fp16 ? 0u : 1u) << 10)     // B format
         | ((n >> 3) << 17)
         | ((m >> 4) << 24);
}

__device__ __forceinline__ float to_tf32_rna(float v)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(v));
    return __uint_as_float(r);
}

}  // namespace ptx
}  // namespace conv2d_b200
