// Building blocks shared by the tensor-core GEMM cores (one SM per tile, and the two-SM form): bounded mbarrier waits,
// TMA tile loads, shared-memory / instruction descriptors of tcgen05.mma, tensor-memory loads and stores.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sc {

constexpr long long kUWaitCycles = 1500000000LL;   // default clock limit of a device-side wait (about 0.8 s)
constexpr uint32_t kUSbo = 128;                    // bytes between consecutive 8-row groups of a K-major, unswizzled operand

__device__ __forceinline__ uint32_t u_smem(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void u_mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void u_mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void u_mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool u_mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded, abortable wait: false when the clock limit passes or another role has already given up.  The poll
// loop itself is only the try_wait (a barrier operation costs ~100 cycles, and every cycle added to a poll is
// added to the hand-over latency between roles); the abort flag and the clock are looked at every 64 polls.
__device__ __forceinline__ bool u_mbar_wait(uint32_t bar, uint32_t parity, volatile int32_t *abort_flag,
                                            long long limit_cycles = kUWaitCycles)
{
    long long t0 = 0;
    for (uint32_t spins = 1;; ++spins) {
        if (u_mbar_try(bar, parity)) return true;
        if ((spins & 63u) == 0u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_cycles) return false;
        }
    }
}
// One lane polls, the warp follows (keeps 31 lanes off the shared-memory pipe).
__device__ __forceinline__ bool u_mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int32_t *abort_flag, int lane)
{
    int ok = 1;
    if (lane == 0) ok = u_mbar_wait(bar, parity, abort_flag) ? 1 : 0;
    return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
}
__device__ __forceinline__ bool u_mbar_wait_warp_limit(uint32_t bar, uint32_t parity, volatile int32_t *abort_flag, int lane,
                                                       long long limit_cycles)
{
    int ok = 1;
    if (lane == 0) ok = u_mbar_wait(bar, parity, abort_flag, limit_cycles) ? 1 : 0;
    return __shfl_sync(0xFFFFFFFFu, ok, 0) != 0;
}
__device__ __forceinline__ void u_tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Shared-memory matrix descriptor, K-major, no swizzle: start address, leading-dimension byte offset (between
// 16-byte K chunks), stride-dimension byte offset (between 8-row groups), all in 16-byte units; version 1.
__device__ __forceinline__ uint64_t u_smem_desc(uint32_t addr, uint32_t lbo_bytes)
{
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((kUSbo >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// Instruction descriptor of kind::mxf4 (block scaled): e2m1 A and B, both K-major, ue8m0 scale factors, K = 64.
__device__ __forceinline__ constexpr uint32_t u_idesc_fp4(uint32_t m_rows, uint32_t n_cols)
{
    return (1u << 7) | (1u << 10) | ((n_cols >> 3) << 17) | (1u << 23) | ((m_rows >> 4) << 24);
}
// D[tmem] (+)= (A[tmem] x B[smem]) with per-block scale factors read from tensor memory
__device__ __forceinline__ void u_mma_fp4_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate, uint32_t sfa_tmem, uint32_t sfb_tmem)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], [%1], %2, %3, [%5], [%6], p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
                 : "memory");
}
__device__ __forceinline__ void u_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void u_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void u_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void u_tmem_ld32(uint32_t taddr, uint32_t v[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                   "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                   "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// 8 consecutive 32-bit columns of this thread's tensor-memory lane (the 32 K bytes of one row for one MMA step)
__device__ __forceinline__ void u_tmem_st8(uint32_t taddr, const uint32_t v[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}

}  // namespace sc
