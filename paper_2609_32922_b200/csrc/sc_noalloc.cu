// sc_assign_lengths_static: the stream-length assignment for callers that may not allocate.
//
// Some users of this library run where device allocation is off limits: inside a serving loop whose
// memory pool is frozen after start-up, in a plugin that was handed fixed buffers by its host
// application, or under a tool that forbids cudaMalloc once the steady state begins.  sc_create (which
// allocates the context's scratch block) is not available to them.  This entry point needs no context:
// its scratch lives in a fixed array that is part of the loaded library image, so calling it never
// allocates anything -- no cudaMalloc / cudaFree, no allocating library routine.
//
// The array is shared by every call on a device and keeps whatever the previous call left there; the
// kernel rewrites every word it later reads, and the header words are cleared at the start of each
// call.  Two calls whose kernels overlap on the GPU (different streams, or different host threads)
// would race on it: issue calls on one stream, or otherwise order them.
#include <math.h>

#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

constexpr int kStaticThreads = 1024;
constexpr int kStaticHeaderWords = 64;                        // 256 bytes: word [0] is the status of the call, the rest is unused

// File-scope scratch: one grid value per group plus the header.  Every GPU that loads the library holds
// these SC_STATIC_MAX_GROUPS * 4 + 256 bytes (about 1 MB) until the process exits.
static __device__ __align__(256) uint32_t g_static_scratch[kStaticHeaderWords + SC_STATIC_MAX_GROUPS];

template <typename T, typename Op>
__device__ T block_all_reduce(T v, Op op, T *smem /* 33 entries */)
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

__device__ __forceinline__ float static_group_metric(const float *g, int64_t M, int32_t group, int64_t gi, bool &bad)
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

__device__ __forceinline__ long long static_length_for(uint32_t q, unsigned long long t, int32_t Lmin, int32_t Lmax)
{
    unsigned long long l = ((unsigned long long)q * t + (1ull << 31)) >> 32;
    l = l < (unsigned long long)Lmin ? (unsigned long long)Lmin : l;
    l = l > (unsigned long long)Lmax ? (unsigned long long)Lmax : l;
    return (long long)l;
}

// Same rule as the context-based kernel (Sec. 4.4 assignment); the per-group grid values are kept in the
// static global scratch instead of shared memory.  `scratch` is the DEVICE address of g_static_scratch.
__global__ void __launch_bounds__(kStaticThreads)
assign_lengths_static_kernel(const float *__restrict__ g, int64_t M, int32_t group, long long budget,
                             int32_t uniform_len, int32_t Lmin, int32_t Lmax, int32_t *__restrict__ L_out,
                             uint32_t *scratch, int32_t *status_out, long long *total_out)
{
    __shared__ float red_f[33];
    __shared__ long long red_i[33];
    uint32_t *q = scratch + kStaticHeaderWords;
    int32_t *status = reinterpret_cast<int32_t *>(scratch);
    const int64_t ngroups = (M + group - 1) / group;

    if (threadIdx.x == 0) scratch[0] = 0u;                   // the status word starts at zero
    __syncthreads();

    float lo_f = INFINITY, hi_f = -INFINITY;
    bool bad = false;
    for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
        const float G = static_group_metric(g, M, group, gi, bad);
        lo_f = fminf(lo_f, G);
        hi_f = fmaxf(hi_f, G);
    }
    if (bad) atomicMax(status, (int32_t)SC_ERR_NONFINITE);
    const float gmin = block_all_reduce(lo_f, [](float a, float b) { return fminf(a, b); }, red_f);
    const float gmax = block_all_reduce(hi_f, [](float a, float b) { return fmaxf(a, b); }, red_f);

    int mode;
    if ((long long)Lmin * M > budget) { mode = 0; if (threadIdx.x == 0) atomicMax(status, (int32_t)SC_ERR_BUDGET); }
    else if ((long long)Lmax * M <= budget) mode = 1;
    else if (gmax == gmin) mode = 2;
    else mode = 3;

    unsigned long long slope = 0;
    if (mode == 3) {
        for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x) {
            bool b2 = false;
            const float G = static_group_metric(g, M, group, gi, b2);
            const float gt = __fdiv_rn(__fsub_rn(G, gmin), __fsub_rn(gmax, gmin));
            const int32_t v = __float2int_rn(__fmul_rn(gt, 65536.0f));
            q[gi] = (uint32_t)min(max(v, 0), 65536);           // each thread re-reads only what it wrote
        }
        auto total = [&](unsigned long long t) -> long long {
            long long s = 0;
            for (int64_t gi = threadIdx.x; gi < ngroups; gi += blockDim.x)
                s += (long long)min((int64_t)group, M - gi * group) * static_length_for(q[gi], t, Lmin, Lmax);
            return block_all_reduce(s, [](long long a, long long b) { return a + b; }, red_i);
        };
        unsigned long long lo = 0, hi = (1ull << 42) - 1;
        if (total(hi) <= budget) {
            lo = hi;
        } else {
            while (hi - lo > 1) {
                const unsigned long long mid = lo + (hi - lo) / 2;
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
        else L = (int32_t)static_length_for(q[gi], slope, Lmin, Lmax);
        L_out[gi] = L;
        sum += (long long)L * min((int64_t)group, M - gi * group);
    }
    sum = block_all_reduce(sum, [](long long a, long long b) { return a + b; }, red_i);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (total_out) *total_out = sum;
        if (status_out) *status_out = *status;
    }
}

// Device address of the static array, looked up once per device (the symbol's name is only a host-side
// handle; kernels must be given the address cudaGetSymbolAddress returns on the current device).
static uint32_t *g_static_ptr[64] = {nullptr};

static cudaError_t static_scratch_address(uint32_t **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[dev] = static_cast<uint32_t *>(p);
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}

}  // namespace sc

using namespace sc;

extern "C" sc_status sc_assign_lengths_static(const float *g, int64_t M, int32_t group, double avg_budget,
                                              int32_t Lmin, int32_t Lmax, int32_t *L_out, int32_t *status_out,
                                              int64_t *total_out, void *stream)
{
    if (!g || !L_out || group < 1 || !(avg_budget >= 0.0) || !isfinite(avg_budget)) return SC_ERR_ARG;
    if (M <= 0 || M >= (1LL << 31)) return SC_ERR_SHAPE;
    if ((M + group - 1) / group > SC_STATIC_MAX_GROUPS) return SC_ERR_SHAPE;     // beyond the fixed scratch
    if (Lmin < 0 || Lmax < Lmin || Lmax > SC_L_CAP) return SC_ERR_LENGTH;
    uint32_t *scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess) return SC_ERR_CUDA;
    // a budget beyond Lmax per row means "every row at Lmax"; clamping first keeps the rounding in range for any
    // finite budget
    const double avg = fmin(avg_budget, (double)Lmax);
    const long long budget = llround(avg * (double)M);
    long long u = (long long)floor(avg);
    u = u < Lmin ? Lmin : (u > Lmax ? Lmax : u);
    assign_lengths_static_kernel<<<1, kStaticThreads, 0, (cudaStream_t)stream>>>(
        g, M, group, budget, (int32_t)u, Lmin, Lmax, L_out, scratch, status_out,
        reinterpret_cast<long long *>(total_out));
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}
