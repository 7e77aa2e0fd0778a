// Fifth-generation tensor-core primitives (tcgen05) used by the integer distance kernels: tensor
// memory allocation, the shared-memory and instruction descriptors of an 8-bit integer MMA with
// 32-bit accumulators, issue, commit and accumulator read-back.  One CTA per MMA (cta_group::1).
#pragma once

#include "tma_pipeline.cuh"

namespace bz {

// ---- tensor memory -------------------------------------------------------------------------------
// Warp-collective.  The base address of the allocation is written to *slot (shared memory).
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t n_cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(n_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t base, uint32_t n_cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Writes made with ordinary stores become visible to the tensor core's reads of shared memory.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---- descriptors ---------------------------------------------------------------------------------
// Operand tile in shared memory, K-major, 128-byte swizzle: rows of 128 bytes, groups of 8 rows
// (1024 bytes, 1024-byte aligned), 16-byte chunk c of row r stored at chunk c ^ (r % 8).
__device__ __forceinline__ uint64_t smem_desc_k128(uint32_t smem_addr) {
    uint64_t desc = static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4);
    desc |= static_cast<uint64_t>(1) << 16;             // leading-dimension offset: unused for this layout
    desc |= static_cast<uint64_t>(1024 >> 4) << 32;     // stride between 8-row groups
    desc |= static_cast<uint64_t>(1) << 46;             // descriptor version of this architecture
    desc |= static_cast<uint64_t>(2) << 61;             // 128-byte swizzle
    return desc;
}
// Signed 8-bit A and B (both K-major), signed 32-bit accumulator, M x N tile; K = 32 per instruction.
constexpr uint32_t idesc_s8(int M, int N) {
    return (2u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

// ---- issue (one thread) --------------------------------------------------------------------------
__device__ __forceinline__ void mma_s8(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The barrier gets one arrival once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// ---- accumulator read-back (warp-collective; a warp reaches lanes 32*(warp % 4) .. +31) ------------
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, int32_t (&x)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]), "=r"(x[4]), "=r"(x[5]), "=r"(x[6]), "=r"(x[7])
                 : "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- shared memory by 32-bit address: the offsets of an unrolled loop fold into the instructions ----------
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }

// ---- bounded waits that give up early once another thread of the CTA has ---------------------------
// Each probe lets the hardware suspend the thread for up to `nap_ns` nanoseconds, so a warp that waits
// takes no issue slots from the warps that work.  At most `probes` probes.
__device__ __forceinline__ bool mbar_wait_live(uint64_t* bar, uint32_t parity, volatile int* dead, uint32_t nap_ns = 2000,
                                               uint32_t probes = 1u << 19) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t spin = 0; spin < probes; ++spin) {
        uint32_t done;
        asm volatile(
            "{\n"
            ".reg .pred p;\n"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
            "selp.u32 %0, 1, 0, p;\n"
            "}\n"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(nap_ns)
            : "memory");
        if (done) return true;
        if (*dead) return false;
    }
    *dead = 1;
    return false;
}

}  // namespace bz
