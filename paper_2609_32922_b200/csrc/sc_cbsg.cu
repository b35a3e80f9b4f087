// Sobol-8 streams with conditional bitstream generation (Sec. 4.2 "cumulative-indicator" datapath, Appendix A.1),
// mapped onto the AND-popcount GEMM core.
//
// All elements share three 256-entry sequences of 8-bit draws: the activation stream of a value with boundary T is
// z_l = [sA_l < T]; the weight bit of a cycle comes from generator s1 on the cycles where the activation bit is 1 and
// from generator s0 where it is 0, each generator advancing only on its own cycles; the output bit is XNOR(zA, zW).
// Over L cycles the activation stream has n1 ones and n0 = L - n1 zeros, so the XNOR count of one (activation,
// weight) pair is
//     #{k < n1 : s1_k < Tw}  +  #{k < n0 : s0_k >= Tw}
//   = sum over generator steps k of [k < n1] [s1_k < Tw]  +  [k < n0] [s0_k >= Tw]:
// an AND-popcount of two codes, one that depends on the activation element only (two thermometers) and one that
// depends on the weight element only (its row of the indicator table of each generator: the table of Sec. 4.2, of
// which shorter streams use a prefix).  Only steps k < L can contribute, so with the two branches interleaved
// (position 2 k = ones branch, 2 k + 1 = zeros branch) a row of length L_i is a code of 2 L_i positions, and the
// product is the binary contraction the tensor-core core already runs, ragged lengths included: the cost follows
// the sum of the L_i as in Sec. 4.1.  The counts equal those of the cycle-by-cycle multiplier exactly.
//
// Sequences: sA = Sobol dimension 1 (base-2 radical inverse), s1 and s0 = Sobol dimension 2 (direction integers
// 1, 3, 5, 15, 17, 51, 85, 255), each XORed with a byte derived from (seed, stream_id) by one Philox call
// (counter word 0 = 0x80000001).
#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

constexpr int kKaWords = 257 * 8;            // activation indicator table: one 256-bit row per boundary
constexpr int kKwWords = 257 * 16;           // weight code table: one 512-bit row (two interleaved branches) per boundary

__device__ __forceinline__ uint32_t sobol8(int dim, uint32_t n)
{
    const uint32_t m2[8] = {1, 3, 5, 15, 17, 51, 85, 255};
    uint32_t x = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k)
        if ((n >> k) & 1u) x ^= (dim == 1 ? 1u : m2[k]) << (7 - k);
    return x & 255u;
}

// tables[0 .. 2056)      KA[T][w] : bit b = [sA_{32 w + b} < T]                           (activation stream, by cycle)
// tables[2056 .. 6168)   KW[T][w] : bit 2 j = [s1_{16 w + j} < T], bit 2 j + 1 = [s0_{16 w + j} >= T]
// Also turns the caller's lengths into the core's: a row of length L is a code of 2 L positions.
__global__ void __launch_bounds__(256)
cbsg_setup_kernel(const __grid_constant__ PhiloxKeys ks, uint32_t stream_word, uint32_t *__restrict__ tables,
                  const int32_t *__restrict__ L, int64_t n_groups, int32_t Lmax, int32_t *__restrict__ L_core,
                  int32_t *status)
{
    __shared__ uint8_t sA[256], s1[256], s0[256];
    bool bad = false;
    if (blockIdx.x == 0) {
        uint32_t x[4];
        philox4x32_10(ks, 0x80000001u, stream_word, 0u, 0u, x);
        const uint32_t scr_a = x[0] & 255u, scr_1 = (x[0] >> 8) & 255u, scr_0 = (x[0] >> 16) & 255u;
        const uint32_t k = threadIdx.x;
        sA[k] = (uint8_t)(sobol8(1, k) ^ scr_a);
        s1[k] = (uint8_t)(sobol8(2, k) ^ scr_1);
        s0[k] = (uint8_t)(sobol8(2, k) ^ scr_0);
        __syncthreads();
        for (int idx = threadIdx.x; idx < kKaWords; idx += blockDim.x) {
            const int T = idx >> 3, w = idx & 7;
            uint32_t ka = 0u;
            for (int b = 0; b < 32; ++b) ka |= (uint32_t)((int)sA[32 * w + b] < T) << b;
            tables[idx] = ka;
        }
        for (int idx = threadIdx.x; idx < kKwWords; idx += blockDim.x) {
            const int T = idx >> 4, w = idx & 15;
            uint32_t kw = 0u;
            for (int j = 0; j < 16; ++j) {
                kw |= (uint32_t)((int)s1[16 * w + j] < T) << (2 * j);
                kw |= (uint32_t)((int)s0[16 * w + j] >= T) << (2 * j + 1);
            }
            tables[kKaWords + idx] = kw;
        }
    }
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < n_groups; g += (int64_t)gridDim.x * blockDim.x) {
        int32_t v = L ? __ldg(L + g) : Lmax;
        if (v < 0 || v > Lmax) { bad = true; v = v < 0 ? 0 : Lmax; }
        L_core[g] = 2 * v;
    }
    if (bad) report(status, SC_ERR_LENGTH);
}

struct CbsgEncodeDev {
    const float *X;
    int64_t x_cols, stream_rows, depth, r_pad, n_row_groups;
    const int32_t *perm;           // A: sorted position -> source row; NULL for W
    const int32_t *l_sorted;       // A: code length per sorted position (longest first); NULL for W
    const int32_t *lmax_actual;    // device scalar: longest code of the call
    const int32_t *L;              // A: the caller's lengths per group (NULL = Lmax)
    const float *sigma;
    const uint32_t *tables;
    uint32_t *streams;
    int32_t *status;
    int32_t tensor_id, kw, group, Lmax, reverse_bytes, quant;
};

__device__ __forceinline__ uint32_t low_bits(int32_t n)      // n lowest bits set, n clamped to 0..32
{
    return n >= 32 ? 0xFFFFFFFFu : (n <= 0 ? 0u : ((1u << n) - 1u));
}

// One warp owns (8 stream rows, one depth word) and writes the code positions the core will read: lane = depth
// element while the codes are formed, lane = position after the 32 x 32 bit transpose (as in the Philox encode).
__global__ void __launch_bounds__(128)
cbsg_encode_kernel(const __grid_constant__ CbsgEncodeDev p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    const int32_t w = (int32_t)(warp % p.kw);
    const int64_t rg = warp / p.kw;
    if (rg >= p.n_row_groups) return;
    const int64_t r0 = rg * 8;
    // positions to write: up to the longest code of the call, for A only up to the longest row of this 128-row tile
    int32_t l_write = min(__ldg(p.lmax_actual), 2 * p.Lmax);
    if (p.l_sorted) l_write = min(l_write, __ldg(p.l_sorted + (r0 / kTileM) * kTileM));
    const int32_t n_blk = (l_write + 31) >> 5;
    if (n_blk == 0) return;
    const WarpTranspose transpose(lane);
    const int64_t d = (int64_t)w * 32 + (p.reverse_bytes ? w_bit_element(lane) : lane);
    const bool have_d = d < p.depth;

    // per row: A: the counts n1 (ones of the activation stream in its first L cycles) and n0 = L - n1; W: the boundary
    int32_t sel1[8], sel0[8];
    bool bad = false;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int64_t r = r0 + t;
        int64_t src = -1;
        if (r < p.r_pad) src = p.perm ? (int64_t)__ldg(p.perm + r) : (r < p.stream_rows ? r : -1);
        sel1[t] = p.tensor_id == 0 ? 0 : -1;                  // A: empty thermometers; W: no element
        sel0[t] = 0;
        if (src < 0 || !have_d) continue;
        float x = __ldg(p.X + (p.tensor_id == 0 ? src * p.x_cols + d : d * p.x_cols + src));
        if (is_nonfinite(x)) { bad = true; x = 0.0f; }
        const float v = normalise(x, __ldg(p.sigma + src));
        const int32_t T = p.quant ? boundary_bipolar_int8(v) : boundary_bipolar(v);
        if (p.tensor_id == 0) {
            int32_t len = p.L ? __ldg(p.L + src / p.group) : p.Lmax;
            len = min(max(len, 0), p.Lmax);
            int32_t n1 = 0;
#pragma unroll
            for (int wd = 0; wd < 8; ++wd) n1 += __popc(__ldg(p.tables + T * 8 + wd) & low_bits(len - 32 * wd));
            sel1[t] = n1;
            sel0[t] = len - n1;
        } else {
            sel1[t] = T;
        }
    }
    if (bad) report(p.status, SC_ERR_NONFINITE);

#pragma unroll 1
    for (int32_t blk = 0; blk < n_blk; ++blk) {               // positions 32 blk ..: generator steps 16 blk .. 16 blk + 15
        uint32_t out[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            uint32_t z;
            if (p.tensor_id == 0)      // [k < n1] at the even positions, [k < n0] at the odd ones
                z = (0x55555555u & low_bits(2 * (sel1[t] - 16 * blk))) | (0xAAAAAAAAu & low_bits(2 * (sel0[t] - 16 * blk)));
            else
                z = sel1[t] >= 0 ? __ldg(p.tables + kKaWords + sel1[t] * 16 + blk) : 0u;
            out[t] = transpose(z);
        }
        const int32_t l = blk * 32 + lane;
        if (l < l_write) {
            const int64_t plane = (int64_t)l * p.kw + w;
            uint4 *dst = reinterpret_cast<uint4 *>(p.streams + plane * p.r_pad + r0);
            dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
            dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
        }
    }
}

// Decode of Eq. (1) from the AND counts of the codes, which are the XNOR counts themselves:
// P = acc / 128, C = sA_i sW_j (2 P - K L_i) / L_i with the caller's L_i.
__global__ void __launch_bounds__(256)
cbsg_decode_kernel(const int32_t *acc, int64_t M, int64_t N, int32_t K, const int32_t *__restrict__ L, int32_t group,
                   int32_t Lmax, const float *__restrict__ sigma_a, const float *__restrict__ sigma_w, int32_t *P,
                   float *__restrict__ C)
{
    for (int64_t i = blockIdx.y; i < M; i += gridDim.y) {
        int32_t len = L ? __ldg(L + i / group) : Lmax;
        len = min(max(len, 0), Lmax);
        const float sa = __ldg(sigma_a + i);
        for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < N; j += (int64_t)gridDim.x * blockDim.x) {
            const int32_t count = acc[i * N + j];
            float c = 0.0f;
            if (len > 0)
                c = __fmul_rn(__fmul_rn(sa, __ldg(sigma_w + j)), __fdiv_rn((float)(2 * count - K * len), (float)len));
            if (P) P[i * N + j] = count;
            C[i * N + j] = c;
        }
    }
}

// Diagnostic (Appendix A.1): stochastic cross-correlation of the activation stream and the gated weight stream of n
// boundary pairs over L cycles, from the pair counts a, b, c, d = cycles with (zA, zW) = 11, 10, 01, 00.
// out[4 i .. 4 i + 3] = a, b, c, d; scc[i] = the normalised a d - b c.  One thread per pair, counts from the code tables.
__global__ void __launch_bounds__(256)
cbsg_scc_kernel(const uint32_t *__restrict__ tables, const int32_t *__restrict__ Ta, const int32_t *__restrict__ Tw,
                int64_t n, int32_t L, int32_t *__restrict__ counts, double *__restrict__ scc, int32_t *status)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    int32_t ta = __ldg(Ta + i), tw = __ldg(Tw + i);
    if (ta < 0 || ta > 256 || tw < 0 || tw > 256) { report(status, SC_ERR_ARG); ta = min(max(ta, 0), 256); tw = min(max(tw, 0), 256); }
    int32_t n1 = 0;
    for (int wd = 0; wd < 8; ++wd) n1 += __popc(__ldg(tables + ta * 8 + wd) & low_bits(L - 32 * wd));
    const int32_t n0 = L - n1;
    int32_t a = 0, d = 0;             // ones-branch steps k < n1 sit at even code positions, zeros-branch steps at odd ones
    for (int w = 0; w < 16; ++w) {
        const uint32_t code = __ldg(tables + kKaWords + tw * 16 + w);
        a += __popc(code & 0x55555555u & low_bits(2 * (n1 - 16 * w)));
        d += __popc(code & 0xAAAAAAAAu & low_bits(2 * (n0 - 16 * w)));
    }
    const int32_t b = n1 - a, c = n0 - d;
    if (counts) { counts[4 * i] = a; counts[4 * i + 1] = b; counts[4 * i + 2] = c; counts[4 * i + 3] = d; }
    const double num = (double)a * d - (double)b * c;
    double den;
    if (num > 0) den = (double)L * (double)min(a + b, a + c) - (double)(a + b) * (a + c);
    else den = (double)(a + b) * (a + c) - (double)L * (double)max(a - d, 0);
    scc[i] = den == 0.0 ? 0.0 : num / den;
}

cudaError_t launch_cbsg_scc(const uint32_t *tables, const int32_t *Ta, const int32_t *Tw, int64_t n, int32_t L,
                            int32_t *counts, double *scc, int32_t *status, cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    cbsg_scc_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(tables, Ta, Tw, n, L, counts, scc, status);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_cbsg_setup(uint64_t seed, uint32_t stream_id, uint32_t *tables, const int32_t *L, int64_t n_groups,
                              int32_t Lmax, int32_t *L_core, int32_t *status, cudaStream_t st)
{
    int64_t blocks = (n_groups + 255) / 256;
    if (blocks > 148 * 4) blocks = 148 * 4;
    if (blocks < 1) blocks = 1;
    cbsg_setup_kernel<<<(unsigned)blocks, 256, 0, st>>>(philox_keys(seed), stream_id << 1, tables, L, n_groups, Lmax,
                                                       L_core, status);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_cbsg_encode(const float *X, int64_t rows, int64_t cols, int tensor_id, int64_t r_pad,
                               const int32_t *perm, const int32_t *l_sorted, const int32_t *lmax_actual,
                               const int32_t *L, int32_t group, int32_t Lmax, const float *sigma,
                               const uint32_t *tables, uint32_t *streams, int reverse_bytes, int32_t *status,
                               cudaStream_t st, int quant)
{
    CbsgEncodeDev p;
    p.X = X; p.x_cols = cols;
    p.stream_rows = tensor_id == 0 ? rows : cols;
    p.depth = tensor_id == 0 ? cols : rows;
    p.r_pad = r_pad; p.n_row_groups = r_pad / 8;
    p.perm = perm; p.l_sorted = l_sorted; p.lmax_actual = lmax_actual; p.L = L; p.sigma = sigma; p.tables = tables; p.streams = streams; p.status = status;
    p.tensor_id = tensor_id; p.kw = (int32_t)((p.depth + 31) / 32); p.group = group; p.Lmax = Lmax;
    p.reverse_bytes = reverse_bytes;
    p.quant = quant;
    const int64_t warps = p.n_row_groups * p.kw;
    const int64_t blocks = (warps + 3) / 4;
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    cbsg_encode_kernel<<<(unsigned)blocks, 128, 0, st>>>(p);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_cbsg_decode(const int32_t *acc, int64_t M, int64_t N, int64_t K, const int32_t *L, int32_t group,
                               int32_t Lmax, const float *sigma_a, const float *sigma_w, int32_t *P, float *C,
                               cudaStream_t st)
{
    int64_t bx = (N + 255) / 256;
    if (bx > 64) bx = 64;
    const dim3 grid((unsigned)bx, (unsigned)(M < 32768 ? M : 32768));
    cbsg_decode_kernel<<<grid, 256, 0, st>>>(acc, M, N, (int32_t)K, L, group, Lmax, sigma_a, sigma_w, P, C);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace sc
