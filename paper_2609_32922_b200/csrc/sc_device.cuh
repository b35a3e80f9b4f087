// Device-side building blocks of the SNG: Philox4x32-10, the value -> boundary map, and the
// bit-plane comparator that evaluates 32 stream positions at once.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace sc {

#if defined(__CUDACC__)
#define SC_HD __host__ __device__ __forceinline__
#else
#define SC_HD inline
#endif

// ---- Philox4x32-10 -------------------------------------------------------------------------------
// The ten round keys depend on the seed only; callers build them once per thread.
struct PhiloxKeys {
    uint32_t k0[10], k1[10];
};

SC_HD PhiloxKeys philox_keys(uint64_t seed)
{
    PhiloxKeys ks;
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        ks.k0[r] = a;
        ks.k1[r] = b;
        a += 0x9E3779B9u;
        b += 0xBB67AE85u;
    }
    return ks;
}

SC_HD void mulhilo(uint32_t m, uint32_t x, uint32_t &hi, uint32_t &lo)
{
    const uint64_t p = (uint64_t)m * (uint64_t)x;        // one 32 x 32 -> 64 multiply
    lo = (uint32_t)p;
    hi = (uint32_t)(p >> 32);
}

SC_HD void philox4x32_10(const PhiloxKeys &ks, uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t out[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi_a, lo_a, hi_b, lo_b;
        mulhilo(0xD2511F53u, c0, hi_a, lo_a);
        mulhilo(0xCD9E8D57u, c2, hi_b, lo_b);
        c0 = hi_b ^ c1 ^ ks.k0[r];
        c2 = hi_a ^ c3 ^ ks.k1[r];
        c1 = lo_b;
        c3 = lo_a;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ---- bit-plane comparator ------------------------------------------------------------------------
// planes[k] holds bit k of 32 independent 8-bit draws (draw b in bit position b).  Returns the word
// whose bit b is [draw_b < T] for T in 0..256: a ripple from the least significant plane,
//   lt <- T_k ? (~r_k | lt) : (~r_k & lt),
// one three-input logic op per plane; T = 256 (bit 8 set) is above every draw.
SC_HD uint32_t draws_below(const uint32_t planes[8], int32_t T)
{
    uint32_t lt = 0u;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
#if defined(__CUDA_ARCH__)
        // bit k of T moved to the top of the low byte, then replicated over the word (byte permute, sign mode)
        uint32_t tk;
        asm("prmt.b32 %0, %1, 0, 0x8888;" : "=r"(tk) : "r"((uint32_t)T << (7 - k)));
#else
        uint32_t tk = ((T >> k) & 1) ? 0xFFFFFFFFu : 0u;
#endif
        uint32_t nr = ~planes[k];
        lt = (tk & (nr | lt)) | (~tk & (nr & lt));
    }
    return (T & 256) ? 0xFFFFFFFFu : lt;
}

// 32 stream positions (block `blk` = positions 32 blk .. 32 blk + 31) of element `elem`.
SC_HD uint32_t sng_word(const PhiloxKeys &ks, uint32_t stream_word, uint64_t elem, uint32_t blk, int32_t T)
{
    uint32_t planes[8];
    philox4x32_10(ks, 2u * blk, stream_word, (uint32_t)elem, (uint32_t)(elem >> 32), planes);
    philox4x32_10(ks, 2u * blk + 1u, stream_word, (uint32_t)elem, (uint32_t)(elem >> 32), planes + 4);
    return draws_below(planes, T);
}

// ---- operand layouts of the tensor-core core and the bit -> 4-bit float expansions -----------------
// Bipolar W planes: bit `lane` of a plane word holds depth element w_bit_element(lane) of the word's 32 elements (each
// group of four in reverse order).
SC_HD int w_bit_element(int lane) { return (lane & ~3) | (3 - (lane & 3)); }
// Unipolar W planes: the two planes of a position as two-bit (stream bit, stream bit AND sign) fields: nibble j of p0
// holds element 4 j at bits (2, 3) and element 4 j + 1 at bits (0, 1); p1 holds elements 4 j + 2 and 4 j + 3.
SC_HD void pack_w_fields(uint32_t z, uint32_t n, uint32_t &p0, uint32_t &p1)
{
    const uint32_t m = 0x11111111u;
    p0 = ((z >> 1) & m) | (((n >> 1) & m) << 1) | ((z & m) << 2) | ((n & m) << 3);
    p1 = ((z >> 3) & m) | (((n >> 3) & m) << 1) | (((z >> 2) & m) << 2) | (((n >> 2) & m) << 3);
}

// Expansion, 1 stream bit -> one 4-bit float (e2m1: bit 3 sign, bits 2..0 = 0.5 / 1 / 2 for a single set bit).
// 32 elements of a depth word become 32 nibbles = 4 words; nibble j of output word m <- element 4 j + m.
//
// Bipolar (0/1 operands).  The bits stay where they are up to one shift: the activation nibble is 0.5 / 1 / 2 / 2 for
// m = 0..3.  The weight planes were encoded with each group of four depth elements in reverse bit order, so element
// m sits at weight bit 3 - m and the same masks give 2 / 1 / 0.5 / 0.5: every product is exactly 1 and the fp32
// accumulators hold the AND count itself.
template <bool kHigh>
SC_HD void u_expand_bits(uint32_t src, uint32_t out[4])
{
    const uint32_t h = src >> 1;
    if (!kHigh) {
        out[0] = src & 0x11111111u;
        out[1] = src & 0x22222222u;
        out[2] = src & 0x44444444u;
        out[3] = h & 0x44444444u;
    } else {
        out[0] = h & 0x44444444u;
        out[1] = h & 0x22222222u;
        out[2] = h & 0x11111111u;
        out[3] = src & 0x11111111u;
    }
}
// Unipolar (sign-magnitude operands), activations: +-0.5 from the magnitude plane (value bit) and the negative plane
// (sign bit).  Activations without any negative stream bit in the call skip the sign.
SC_HD void u_expand_signed_a(uint32_t mag, uint32_t neg, uint32_t out[4], bool a_signed)
{
#if defined(__CUDA_ARCH__)
#pragma unroll
#endif
    for (int m = 0; m < 4; ++m) {
        out[m] = (mag >> m) & 0x11111111u;
        if (a_signed) out[m] |= (neg << (3 - m)) & 0x88888888u;
    }
}
// Unipolar weights: +-2.  The encode stored each position as two planes of two-bit (stream bit, stream bit AND sign)
// fields: nibble j of the first plane holds element 4 j at bits (2, 3) and element 4 j + 1 at bits (0, 1), the second
// plane elements 4 j + 2 and 4 j + 3: one shift and one mask per output word.  Every product is +-1.
SC_HD void u_expand_signed_w(uint32_t p0, uint32_t p1, uint32_t out[4])
{
    out[0] = p0 & 0xCCCCCCCCu;
    out[1] = (p0 << 2) & 0xCCCCCCCCu;
    out[2] = p1 & 0xCCCCCCCCu;
    out[3] = (p1 << 2) & 0xCCCCCCCCu;
}

#if defined(__CUDACC__)
// ---- value -> boundary (binary32, round-half-even; no contraction) --------------------------------
__device__ __forceinline__ float normalise(float x, float sigma)
{
    float v = __fdiv_rn(x, sigma);
    return fminf(fmaxf(v, -1.0f), 1.0f);
}

__device__ __forceinline__ int32_t boundary_bipolar(float v)
{
    float scaled = __fmul_rn(__fadd_rn(v, 1.0f), 128.0f);
    int32_t t = __float2int_rn(scaled);
    return min(max(t, 0), 256);
}

__device__ __forceinline__ int32_t boundary_unipolar(float v, uint32_t &negative)
{
    negative = (v < 0.0f) ? 1u : 0u;
    int32_t t = __float2int_rn(__fmul_rn(fabsf(v), 256.0f));
    return min(max(t, 0), 256);
}

// Two-step variant (Sec. 4.2): the int8 grid first (x_hat = round(127 v), binary32, round-half-even), then the nearest of
// the 257 boundaries in integer arithmetic (127 is odd: no grid point lies half-way between two boundaries).
__device__ __forceinline__ int32_t boundary_bipolar_int8(float v)
{
    int32_t q = __float2int_rn(__fmul_rn(v, 127.0f));
    q = min(max(q, -127), 127);
    return ((q + 127) * 256 + 127) / 254;
}

__device__ __forceinline__ int32_t boundary_unipolar_int8(float v, uint32_t &negative)
{
    negative = (v < 0.0f) ? 1u : 0u;
    int32_t q = __float2int_rn(__fmul_rn(fabsf(v), 127.0f));
    q = min(q, 127);
    return (q * 512 + 127) / 254;
}

__device__ __forceinline__ bool is_nonfinite(float x)
{
    return (__float_as_uint(x) & 0x7F800000u) == 0x7F800000u;
}

__device__ __forceinline__ void report(int32_t *status, int32_t code)
{
    atomicMax(status, code);
}

// Transposes the 32 x 32 bit matrix held one row per lane: afterwards bit d of lane b is what bit b of
// lane d was.  Stage j exchanges the off-diagonal j x j blocks with the lane j away: a lane keeps the bits
// selected by `keep[j]` and takes the others from the partner's word rotated by `rot[j]`.
struct WarpTranspose {
    uint32_t keep[5], rot[5];
    __device__ __forceinline__ explicit WarpTranspose(int lane)
    {
        const uint32_t low[5] = {0x0000FFFFu, 0x00FF00FFu, 0x0F0F0F0Fu, 0x33333333u, 0x55555555u};
#pragma unroll
        for (int s = 0; s < 5; ++s) {
            const int j = 16 >> s;
            const bool upper = (lane & j) != 0;
            keep[s] = upper ? ~low[s] : low[s];
            rot[s] = upper ? 32u - j : (uint32_t)j;
        }
    }
    __device__ __forceinline__ uint32_t operator()(uint32_t x) const
    {
#pragma unroll
        for (int s = 0; s < 5; ++s) {
            const uint32_t y = __shfl_xor_sync(0xFFFFFFFFu, x, 16 >> s);
            const uint32_t r = __funnelshift_l(y, y, rot[s]);
            x = (x & keep[s]) | (r & ~keep[s]);
        }
        return x;
    }
};
#endif

}  // namespace sc
