// Peak measurements for the roofline denominators.
// Register-only instruction-mix loops measure the integer-pipe ceilings the ALU cores are bound by (POPC, LOP3, IADD3
// alone; the plain gate+popcount+add mix; the carry-save mix); a bare chain of tcgen05.mma kind::mxf4 instructions
// measures the issue-rate ceiling of the tensor-core core's instruction.
#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

constexpr int kMbThreads = 256;
constexpr int kMbChains = 16;      // independent dependency chains per thread

template <int kKind>
__global__ void __launch_bounds__(kMbThreads) microbench_kernel(int iters, uint32_t seed, uint32_t *sink)
{
    uint32_t x[kMbChains], acc[kMbChains];
    const uint32_t t = seed ^ (blockIdx.x * kMbThreads + threadIdx.x);
#pragma unroll
    for (int c = 0; c < kMbChains; ++c) { x[c] = t * 2654435761u + c * 40503u; acc[c] = c; }
    const uint32_t k1 = t | 0x01010101u, k2 = ~t;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int rep = 0; rep < 8; ++rep) {
#pragma unroll
            for (int c = 0; c < kMbChains; ++c) {
                if (kKind == 0) {                    // POPC only (result feeds the next POPC input)
                    x[c] = __popc(x[c]) + k1;
                    x[c] = __popc(x[c]) ^ k2;         // the add/xor are needed to keep values moving;
                } else if (kKind == 1) {             // LOP3 only: two three-input functions
                    x[c] = (x[c] & k1) ^ acc[c];
                    acc[c] = (acc[c] ^ x[c]) & (k1 | x[c]);
                } else if (kKind == 2) {             // gate + POPC + add: the plain core mix
                    acc[c] += __popc(x[c] ^ k1);
                    x[c] += k2;                       // stands in for operand change (1 IADD, like the core's IADD3 share)
                } else if (kKind == 3) {             // carry-save mix: 3 gates, 2 CSA ops, 2 POPC, 2 adds
                    const uint32_t a = x[c] ^ k1, b = x[c] ^ k2, d = x[c] ^ t;
                    const uint32_t s = a ^ b ^ d;
                    const uint32_t cy = (a & b) | (d & (a | b));
                    acc[c] += __popc(s) + 2 * __popc(cy);
                    x[c] = x[c] * 3u + acc[c];
                } else {                             // IADD3 only
                    x[c] = x[c] + acc[c] + k1;
                    acc[c] = acc[c] + x[c] + k2;
                }
            }
        }
    }
    uint32_t r = 0;
#pragma unroll
    for (int c = 0; c < kMbChains; ++c) r ^= x[c] + acc[c];
    if (r == 0x12345678u) sink[0] = r;               // keeps the loop alive without real stores
}

// Legacy warp-level tensor instructions: 1-bit XOR/AND-popcount tiles and int8 tiles, four independent
// accumulator sets per warp.  Measures whether sm_100a runs them natively or expands them.
template <int kKind>
__global__ void __launch_bounds__(kMbThreads) microbench_mma_kernel(int iters, uint32_t seed, uint32_t *sink)
{
    const uint32_t t = seed ^ (blockIdx.x * kMbThreads + threadIdx.x) * 2654435761u;
    uint32_t a[4] = {t, t ^ 0x9E3779B9u, t * 3u, ~t}, b[2] = {t * 5u, t ^ 0x7F4A7C15u};
    int32_t d[4][4];
#pragma unroll
    for (int s = 0; s < 4; ++s)
#pragma unroll
        for (int k = 0; k < 4; ++k) d[s][k] = s + k;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int rep = 0; rep < 4; ++rep) {
#pragma unroll
            for (int s = 0; s < 4; ++s) {
                if (kKind == 5)
                    asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc "
                                 "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                 : "+r"(d[s][0]), "+r"(d[s][1]), "+r"(d[s][2]), "+r"(d[s][3])
                                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
                else if (kKind == 6)
                    asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc "
                                 "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                 : "+r"(d[s][0]), "+r"(d[s][1]), "+r"(d[s][2]), "+r"(d[s][3])
                                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
                else
                    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 "
                                 "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                                 : "+r"(d[s][0]), "+r"(d[s][1]), "+r"(d[s][2]), "+r"(d[s][3])
                                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
            }
        }
    }
    int32_t r = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s)
#pragma unroll
        for (int k = 0; k < 4; ++k) r ^= d[s][k];
    if (r == 0x12345678) sink[0] = (uint32_t)r;
}

static double words_per_iteration(int kind)
{
    // operations of the NAMED kind per inner (rep, chain) body
    switch (kind) {
        case 0: return 2.0;   // POPCs
        case 1: return 2.0;   // LOP3-class ops (each line is one three-input function)
        case 2: return 1.0;   // gate evaluations (32 bit-ops each)
        case 3: return 3.0;   // gate evaluations
        case 4: return 2.0;   // IADD3s
        default: return 0.0;
    }
}

cudaError_t run_microbench(sc_ctx_impl *ctx, int kind, int iters, float *ms, double *words)
{
    const int blocks = ctx->sm_count * 8;
    uint32_t *sink = reinterpret_cast<uint32_t *>(ctx->scratch + 32);
    auto launch = [&](int n) {
        switch (kind) {
            case 5: microbench_mma_kernel<5><<<blocks, kMbThreads>>>(n, 1u, sink); break;
            case 6: microbench_mma_kernel<6><<<blocks, kMbThreads>>>(n, 1u, sink); break;
            case 7: microbench_mma_kernel<7><<<blocks, kMbThreads>>>(n, 1u, sink); break;
            case 0: microbench_kernel<0><<<blocks, kMbThreads>>>(n, 1u, sink); break;
            case 1: microbench_kernel<1><<<blocks, kMbThreads>>>(n, 1u, sink); break;
            case 2: microbench_kernel<2><<<blocks, kMbThreads>>>(n, 1u, sink); break;
            case 3: microbench_kernel<3><<<blocks, kMbThreads>>>(n, 1u, sink); break;
            default: microbench_kernel<4><<<blocks, kMbThreads>>>(n, 1u, sink); break;
        }
    };
    launch(iters / 8 + 1);                                 // warm-up
    cudaError_t e = cudaEventRecord(ctx->ev0);
    if (e != cudaSuccess) return e;
    launch(iters);
    e = cudaEventRecord(ctx->ev1);
    if (e != cudaSuccess) return e;
    e = cudaEventSynchronize(ctx->ev1);
    if (e != cudaSuccess) return e;
    e = cudaEventElapsedTime(ms, ctx->ev0, ctx->ev1);
    if (e != cudaSuccess) return e;
    if (kind >= 5) {
        // per warp and loop trip: 16 tile instructions; a 1-bit tile is 16 x 8 x 256 bit-ops = 1024 words,
        // an int8 tile 16 x 8 x 32 multiply-accumulates (reported as such)
        const double per_instr = kind == 7 ? 4096.0 : 1024.0;
        *words = per_instr * 16.0 * (double)iters * (double)(kMbThreads / 32) * (double)blocks;
    } else {
        *words = words_per_iteration(kind) * 8.0 * kMbChains * (double)iters * (double)kMbThreads * (double)blocks;
    }
    count_launches(2);
    return cudaGetLastError();
}


// ---- issue rate of the tensor-core core's instruction --------------------------------------------------------------
// One CTA per SM, one thread: a chain of `n_mma` block-scaled 4-bit MMAs (128 x n_cols x 64 each, A operand and scale
// factors in tensor memory, B operand in shared memory, fp32 accumulators in tensor memory) on zero-filled operands,
// eight per loop trip with precomputed descriptors, one commit at the end.  The elapsed SM clocks of the slowest SM
// give multiply-accumulates per clock per SM.  The wait for the commit is bounded.
__device__ __forceinline__ uint32_t mb_smem(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(128, 1) mxf4_rate_kernel(int n_mma, int n_cols, long long *cycles_out)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    __shared__ uint32_t s_tmem;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int kBytes = 8 * 256 * 32;                    // eight B tiles of up to 256 columns x 32 bytes of K
    for (int i = threadIdx.x; i < kBytes / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(smem)[i] = 0u;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(mb_smem(&bar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(mb_smem(&s_tmem)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;
    {   // scale factors (columns 480..511): every byte 2^0; A operand (columns 256..319): zeros
        uint32_t v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = 0x7F7F7F7Fu;
        const uint32_t lane_base = ((uint32_t)warp * 32u) << 16;
        for (uint32_t c = 480; c < 512; c += 8)
            asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                         ::"r"(tmem + c + lane_base), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
        for (uint32_t c = 256; c < 320; c += 8)
            asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1};" ::"r"(tmem + c + lane_base), "r"(0u) : "memory");
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 0 && lane == 0) {
        const uint32_t lbo = (uint32_t)n_cols * 16u;        // bytes between the two 16-byte K chunks of a tile
        uint64_t bd[8];
        uint32_t ad[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t addr = mb_smem(smem) + (uint32_t)k * (uint32_t)n_cols * 32u;
            bd[k] = (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo >> 4) & 0x3FFFu) << 16) |
                    ((uint64_t)(128u >> 4) << 32) | (1ull << 46);
            ad[k] = tmem + 256u + (uint32_t)k * 8u;
        }
        // kind::mxf4: e2m1 x e2m1, K-major, ue8m0 scale factors, M = 128
        const uint32_t idesc = (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | (1u << 23) | (8u << 24);
        const long long t0 = clock64();
        for (int g0 = 0; g0 < n_mma; g0 += 8) {
#pragma unroll
            for (int k = 0; k < 8; ++k)
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], [%1], %2, %3, [%5], [%6], p;\n\t}"
                             ::"r"(tmem), "r"(ad[k]), "l"(bd[k]), "r"(idesc), "r"((uint32_t)((g0 | k) != 0)), "r"(tmem + 480u),
                               "r"(tmem + 496u) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mb_smem(&bar)) : "memory");
        uint32_t ok = 0;
        const long long limit = t0 + 4000000000LL;
        while (!ok && clock64() < limit)
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(mb_smem(&bar)) : "memory");
        cycles_out[blockIdx.x] = ok ? (clock64() - t0) : -1;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
    }
}

// *mclk = SM clocks of the slowest SM / 1e6; *macs = multiply-accumulates per SM.
cudaError_t run_mxf4_rate(sc_ctx_impl *ctx, int n_cols, int iters, float *mclk, double *macs)
{
    iters = (iters + 7) / 8 * 8;
    long long *cyc = reinterpret_cast<long long *>(ctx->scratch + 1024);
    const size_t smem = 8 * 256 * 32;
    cudaError_t e = cudaFuncSetAttribute(mxf4_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaMemset(cyc, 0, sizeof(long long) * 256);
    if (e != cudaSuccess) return e;
    mxf4_rate_kernel<<<ctx->sm_count, 128, smem>>>(iters, n_cols, cyc);
    count_launches(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return e;
    long long host[256];
    e = cudaMemcpy(host, cyc, sizeof(long long) * 256, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return e;
    long long worst = 0;
    for (int i = 0; i < ctx->sm_count && i < 256; ++i) {
        if (host[i] <= 0) return cudaErrorLaunchTimeout;
        if (host[i] > worst) worst = host[i];
    }
    *mclk = (float)((double)worst / 1.0e6);
    *macs = 128.0 * n_cols * 64.0 * (double)iters;
    return cudaSuccess;
}

}  // namespace sc
