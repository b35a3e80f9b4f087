// Gaussian-perturbed surrogate of an SC product (Sec. 3.2, error tolerance): out_ij = Y_ij (1 + alpha(L_i) Z_ij),
// Z_ij independent standard normal, alpha(L) = coeff / L (the paper's table of alpha against L is coeff = 2.324 to
// its printed precision).  A cheap stand-in for the stochastic matmul in model-level sweeps: one pass over Y, HBM-bound.
//
// Z_ij comes from one Philox4x32-10 call per output cell (counter word 0 = 0x80000000, which no stream position
// uses; word 1 = stream_id << 1; words 2, 3 = the cell index i N + j; key = seed): two 24-bit uniforms
// u = ((x >> 8) + 1/2) 2^-24 and the Box-Muller transform sqrt(-2 ln u1) cos(2 pi u2), evaluated in binary64 so that
// the float result does not depend on the accuracy of single-precision log / cos.
#include <math.h>

#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

__device__ __forceinline__ double standard_normal(const PhiloxKeys &ks, uint32_t stream_word, uint64_t cell)
{
    uint32_t x[4];
    philox4x32_10(ks, 0x80000000u, stream_word, (uint32_t)cell, (uint32_t)(cell >> 32), x);
    const double u1 = ((double)(x[0] >> 8) + 0.5) * (1.0 / 16777216.0);
    const double u2 = ((double)(x[1] >> 8) + 0.5) * (1.0 / 16777216.0);
    return sqrt(-2.0 * log(u1)) * cospi(2.0 * u2);
}

__global__ void __launch_bounds__(256)
surrogate_kernel(const __grid_constant__ PhiloxKeys ks, const float *Y, int64_t M, int64_t N,
                 const int32_t *__restrict__ L, int32_t group, double coeff, uint32_t stream_word,
                 float *out, int32_t *status)
{
    // `out` may be the same buffer as `Y` (each thread reads a cell before it writes it): neither pointer is
    // declared restrict and Y is read with plain (coherent) loads.
    bool bad_value = false, bad_length = false;
    for (int64_t i = blockIdx.y; i < M; i += gridDim.y) {
        int32_t len = L ? __ldg(L + i / group) : 1;
        if (len < 0) { bad_length = true; len = 0; }
        const double alpha = len > 0 ? coeff / (double)len : 0.0;
        for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < N; j += (int64_t)gridDim.x * blockDim.x) {
            float y = Y[i * N + j];
            if (is_nonfinite(y)) { bad_value = true; y = 0.0f; }
            float r = 0.0f;
            if (len > 0) r = (float)((double)y * (1.0 + alpha * standard_normal(ks, stream_word, (uint64_t)(i * N + j))));
            out[i * N + j] = r;
        }
    }
    if (bad_value) report(status, SC_ERR_NONFINITE);
    if (bad_length) report(status, SC_ERR_LENGTH);
}

cudaError_t launch_surrogate(const float *Y, int64_t M, int64_t N, const int32_t *L, int32_t group, double coeff,
                             uint64_t seed, uint32_t stream_id, float *out, int32_t *status, cudaStream_t st)
{
    int64_t bx = (N + 255) / 256;
    if (bx > 64) bx = 64;
    const dim3 grid((unsigned)bx, (unsigned)(M < 32768 ? M : 32768));
    surrogate_kernel<<<grid, 256, 0, st>>>(philox_keys(seed), Y, M, N, L, group, coeff, stream_id << 1, out, status);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace sc
