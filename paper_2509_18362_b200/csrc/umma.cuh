// Wrappers over the sm_100a tensor-core path: tensor memory (TMEM) allocation, tcgen05.mma with
// both operands in shared memory, its completion (tcgen05.commit onto an mbarrier), TMEM loads
// for the epilogue, and the descriptors the instruction takes.
#pragma once
#include "ptx.cuh"

namespace fmtp {

// ---- tensor memory ------------------------------------------------------------------------
// One full warp allocates `ncols` columns (a power of two, 32..512) of the SM's 512; the base
// address lands in the shared-memory word `slot`. The same warp must free it before the CTA exits.
__device__ __forceinline__ void tmem_alloc(uint32_t *slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Ordering of tcgen05 operations against other threads' synchronisation (mbarrier, bar.sync).
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- descriptors --------------------------------------------------------------------------
// Shared-memory operand, K-major, 128-byte swizzle: the tile is rows of 128 bytes (64 bf16 along
// K), row r at byte r*128 from a 1024-byte aligned base, its eight 16-byte chunks stored at
// chunk position (c ^ (r & 7)). Groups of eight rows are 1024 bytes apart (the stride offset).
// Stepping K by 16 elements inside the 128-byte row adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr) {
    return static_cast<uint64_t>((saddr & 0x3ffffu) >> 4)      // start address, 16-byte units
           | (static_cast<uint64_t>(1) << 16)                  // leading offset: unused with a swizzled K-major tile
           | (static_cast<uint64_t>(1024 >> 4) << 32)          // stride between 8-row groups
           | (static_cast<uint64_t>(1) << 46)                  // descriptor version of this architecture
           | (static_cast<uint64_t>(2) << 61);                 // 128-byte swizzle
}
// Instruction descriptor of kind::f16 with bf16 A and B (both K-major), fp32 accumulator, M = 128.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int n) {
    return (1u << 4)                      // D: fp32
           | (1u << 7) | (1u << 10)       // A, B: bf16
           | (static_cast<uint32_t>(n >> 3) << 17)
           | (static_cast<uint32_t>(128 >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem]^T, one K = 16 slice; issued by ONE thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate ? 1u : 0u)
        : "memory");
}
// `bar` receives one arrival when every tcgen05.mma this thread issued so far has completed.
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// ---- epilogue loads: warp w (w = warp index mod 4) reads TMEM lanes 32w..32w+31, one lane per
// thread, 32 consecutive fp32 columns starting at the column in `taddr`.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// The same load without the wait: several can be in flight; the registers hold the data after tmem_ld_wait().
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Copies 128 rows x 32 bytes of shared memory, described like an MMA operand (K-major, 128-byte swizzle: row r of
// the tile at r*128 bytes, this instruction's two 16-byte pieces selected by the start address), into tensor-memory
// lanes 0..127, eight 32-bit columns from the column in `taddr`. Asynchronous; issued by ONE thread and tracked by
// that thread's next tcgen05.commit.
__device__ __forceinline__ void tmem_cp_128x256b(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}

// 16-byte asynchronous copy with an immediate byte offset on the source and a source size of 16
// (copy) or 0 (write zeros, read nothing).
template <int OFF>
__device__ __forceinline__ void cp_async16_off(uint32_t dst_smem, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1+%2], 16, %3;" ::"r"(dst_smem), "l"(src), "n"(OFF), "r"(src_bytes)
                 : "memory");
}
// The same copies with an L2 eviction policy (see l2_evict_first): for data that is read once per step.
template <int OFF>
__device__ __forceinline__ void cp_async16_off_hint(uint32_t dst_smem, const void *src, uint32_t src_bytes, uint64_t policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1+%2], 16, %3, %4;" ::"r"(dst_smem), "l"(src), "n"(OFF),
                 "r"(src_bytes), "l"(policy) : "memory");
}
template <int OFF>
__device__ __forceinline__ void cp_async16_full_hint(uint32_t dst_smem, const void *src, uint64_t policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1+%2], 16, %3;" ::"r"(dst_smem), "l"(src), "n"(OFF), "l"(policy)
                 : "memory");
}
// Weights and cached K/V are streamed once per step: marked evict-first they do not push out of L2 what the step
// keeps re-reading (the activation operand every tile re-reads, partial sums, the kernels' own code).
__device__ __forceinline__ uint64_t l2_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait_group() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// ---- programmatic dependent launch: a kernel launched with launch_chained may start (be scheduled,
// run its set-up) while its predecessor in the stream still runs; chain_wait() returns once every
// earlier kernel has completed and its writes are visible, so everything after it sees what a plain
// stream-ordered launch would see. chain_release() lets the successor's launch begin.
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

}  // namespace fmtp
