// Stream-length assignment (Sec. 4.4): group metric -> min-max normalisation -> length at a matched
// average budget (bisection on the slope of the dense ladder), and the explicit ladder/threshold rule.
// One CTA: the problem is a few thousand groups; 43 block-wide integer reductions dominate.
#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

constexpr int kAssignThreads = 1024;
constexpr int kQCacheMax = 40960;   // groups whose grid value is cached in shared memory (160 KB)

struct BlockReduce {
    // all threads receive the result
    template <typename T, typename Op>
    static __device__ T run(T v, Op op, T *smem /* >= 33 entries */)
    {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v = op(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
        __syncthreads();
        if (lane == 0) smem[warp] = v;
        __syncthreads();
        if (warp == 0) {
            T w = (lane < (int)(blockDim.x >> 5)) ? smem[lane] : smem[0];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) w = op(w, __shfl_xor_sync(0xFFFFFFFFu, w, o));
            if (lane == 0) smem[32] = w;
        }
        __syncthreads();
        return smem[32];
    }
};

__device__ __forceinline__ float group_metric(const float *g, int64_t M, int32_t group, int64_t gi, bool &bad)
{
    float m = -INFINITY;
    const int64_t i1 = min(M, (gi + 1) * (int64_t)group);
    for (int64_t i = gi * (int64_t)group; i < i1; ++i) {
        float x = __ldg(g + i);
        if (is_nonfinite(x)) { bad = true; x = 0.0f; }
        m = fmaxf(m, x);
    }
    return m;
}

__device__ __forceinline__ uint32_t grid_value(float G, float gmin, float gmax)
{
    float gt = __fdiv_rn(__fsub_rn(G, gmin), __fsub_rn(gmax, gmin));   // normalised metric in [0,1]
    int32_t q = __float2int_rn(__fmul_rn(gt, 65536.0f));
    return (uint32_t)min(max(q, 0), 65536);
}

__device__ __forceinline__ int64_t length_for(uint32_t q, uint64_t t, int32_t Lmin, int32_t Lmax)
{
    uint64_t l = ((uint64_t)q * t + (1ull << 31)) >> 32;
    l = l < (uint64_t)Lmin ? (uint64_t)Lmin : l;
    l = l > (uint64_t)Lmax ? (uint64_t)Lmax : l;
    return (int64_t)l;
}

__global__ void __launch_bounds__(kAssignThreads)
assign_lengths_kernel(const float *__restrict__ g, int64_t M, int32_t group, long long budget, int32_t uniform_len,
                      int32_t Lmin, int32_t Lmax, int32_t *__restrict__ L_out, int32_t *scratch)
{
    extern __shared__ uint32_t qcache[];
    __shared__ float red_f[33];
    __shared__ long long red_i[33];
    const int64_t ngroups = (M + group - 1) / group;
    const bool cached = ngroups <= kQCacheMax;
    int32_t *status = scratch + kSlotStatus;

    // group metrics, their range
    float lo_f = INFINITY, hi_f = -INFINITY;
    bool bad = false;
    for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
        float G = group_metric(g, M, group, gi, bad);
        lo_f = fminf(lo_f, G);
        hi_f = fmaxf(hi_f, G);
    }
    if (bad) report(status, SC_ERR_NONFINITE);
    const float gmin = BlockReduce::run(lo_f, [](float a, float b) { return fminf(a, b); }, red_f);
    const float gmax = BlockReduce::run(hi_f, [](float a, float b) { return fmaxf(a, b); }, red_f);

    int mode;                      // 0: all Lmin (infeasible), 1: all Lmax, 2: uniform, 3: slope search
    if ((long long)Lmin * M > budget) { mode = 0; if (threadIdx.x == 0) report(status, SC_ERR_BUDGET); }
    else if ((long long)Lmax * M <= budget) mode = 1;
    else if (gmax == gmin) mode = 2;
    else mode = 3;

    uint64_t slope = 0;
    if (mode == 3) {
        if (cached)
            for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
                bool b2 = false;
                qcache[gi] = grid_value(group_metric(g, M, group, gi, b2), gmin, gmax);
            }
        __syncthreads();
        auto total = [&](uint64_t t) -> long long {
            long long s = 0;
            for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
                bool b2 = false;
                uint32_t q = cached ? qcache[gi] : grid_value(group_metric(g, M, group, gi, b2), gmin, gmax);
                long long rows_here = min((int64_t)group, M - gi * group);
                s += rows_here * length_for(q, t, Lmin, Lmax);
            }
            return BlockReduce::run(s, [](long long a, long long b) { return a + b; }, red_i);
        };
        uint64_t lo = 0, hi = (1ull << 42) - 1;          // invariant: total(lo) <= budget < total(hi)
        if (total(hi) <= budget) {
            lo = hi;
        } else {
            while (hi - lo > 1) {
                uint64_t mid = lo + (hi - lo) / 2;
                if (total(mid) <= budget) lo = mid; else hi = mid;
            }
        }
        slope = lo;
    }

    long long sum = 0;
    for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
        int32_t L;
        if (mode == 0) L = Lmin;
        else if (mode == 1) L = Lmax;
        else if (mode == 2) L = uniform_len;
        else {
            bool b2 = false;
            uint32_t q = cached ? qcache[gi] : grid_value(group_metric(g, M, group, gi, b2), gmin, gmax);
            L = (int32_t)length_for(q, slope, Lmin, Lmax);
        }
        L_out[gi] = L;
        sum += (long long)L * min((int64_t)group, M - gi * group);
    }
    sum = BlockReduce::run(sum, [](long long a, long long b) { return a + b; }, red_i);
    if (threadIdx.x == 0) *reinterpret_cast<long long *>(scratch + kSlotRealizedTotal) = sum;
}

struct Ladder {
    int32_t levels;
    int32_t length[64];
    float tau[64];
};

__global__ void __launch_bounds__(kAssignThreads)
ladder_lengths_kernel(const float *__restrict__ g, int64_t M, int32_t group, Ladder ladder,
                      int32_t *__restrict__ L_out, int32_t *scratch)
{
    __shared__ float red_f[33];
    const int64_t ngroups = (M + group - 1) / group;
    float lo_f = INFINITY, hi_f = -INFINITY;
    bool bad = false;
    for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
        float G = group_metric(g, M, group, gi, bad);
        lo_f = fminf(lo_f, G);
        hi_f = fmaxf(hi_f, G);
    }
    if (bad) report(scratch + kSlotStatus, SC_ERR_NONFINITE);
    const float gmin = BlockReduce::run(lo_f, [](float a, float b) { return fminf(a, b); }, red_f);
    const float gmax = BlockReduce::run(hi_f, [](float a, float b) { return fmaxf(a, b); }, red_f);
    for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
        bool b2 = false;
        float G = group_metric(g, M, group, gi, b2);
        float gt = (gmax == gmin) ? 0.0f : __fdiv_rn(__fsub_rn(G, gmin), __fsub_rn(gmax, gmin));
        int level = ladder.levels - 1;
        for (int k = ladder.levels - 2; k >= 0; --k) if (gt >= ladder.tau[k]) level = k;   // first level reached
        L_out[gi] = ladder.length[level];
    }
}

cudaError_t launch_assign_lengths(const float *g, int64_t M, int32_t group, double avg_budget, int32_t Lmin,
                                  int32_t Lmax, int32_t *L_out, int32_t *scratch, cudaStream_t st)
{
    static bool attr_set = false;
    const size_t smem = sizeof(uint32_t) * kQCacheMax;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(assign_lengths_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    // a budget beyond Lmax per row means "every row at Lmax"; clamping first keeps the rounding in range for any
    // finite budget
    const double avg = fmin(avg_budget, (double)Lmax);
    long long budget = llround(avg * (double)M);
    long long u = (long long)floor(avg);
    u = u < Lmin ? Lmin : (u > Lmax ? Lmax : u);
    const int64_t ngroups = (M + group - 1) / group;
    const size_t use = ngroups <= kQCacheMax ? sizeof(uint32_t) * (size_t)ngroups : 0;
    assign_lengths_kernel<<<1, kAssignThreads, use, st>>>(g, M, group, budget, (int32_t)u, Lmin, Lmax, L_out, scratch);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_ladder_lengths(const float *g, int64_t M, int32_t group, const int32_t *ladder, const float *tau,
                                  int32_t levels, int32_t *L_out, int32_t *scratch, cudaStream_t st)
{
    Ladder lad;
    lad.levels = levels;
    for (int k = 0; k < 64; ++k) {
        lad.length[k] = k < levels ? ladder[k] : 0;
        lad.tau[k] = k < levels - 1 ? tau[k] : 0.0f;
    }
    ladder_lengths_kernel<<<1, kAssignThreads, 0, st>>>(g, M, group, lad, L_out, scratch);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace sc
