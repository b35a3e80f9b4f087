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
// Unipolar (sign-magnitude) operands of the tensor-core core: one magnitude plane per position (W in that same reversed
// order) plus, per (depth word, stream row), the signs of the 32 elements kept beside the planes -- a sign does not
// depend on the position -- already spread into the four nibble words the expansion produces (sign_nibble_words).
// Stream positions are stored in blocks: plane index of (position l, depth word w) with kw depth words and blocks of `block`
// positions (1 = position-major, the plain layout).  With block = 8 the eight planes of one operand stage of the core
// are eight positions of ONE depth word, so one set of sign words serves the whole stage.
SC_HD int64_t plane_index(int32_t l, int32_t w, int32_t kw, int32_t block)
{
    return (int64_t)(l / block) * kw * block + (int64_t)w * block + (l % block);
}
// the same for block = 2^shift, without a division
SC_HD int64_t plane_index_pow2(int32_t l, int32_t w, int32_t kw, int32_t shift)
{
    return ((((int64_t)(l >> shift) * kw + w)) << shift) + (l & ((1 << shift) - 1));
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
// Unipolar (sign-magnitude operands): the same powers of two with the sign in bit 3 of the nibble, so every product is
// +-1 and the accumulators hold the signed count.  s[m] has bit 3 of nibble j set iff element 4 j + m of the depth word
// is negative (`sign_word`: bit b = sign of the element that sits at bit b of the plane words; W planes hold element m
// of a nibble group at bit 3 - m, A planes at bit m).  A set sign on a zero magnitude is -0: harmless.
SC_HD void sign_nibble_words(uint32_t sign_word, bool reversed, uint32_t s[4])
{
#if defined(__CUDA_ARCH__)
#pragma unroll
#endif
    for (int m = 0; m < 4; ++m) s[m] = (sign_word << (reversed ? m : 3 - m)) & 0x88888888u;
}
template <bool kHigh>
SC_HD void u_expand_signed(uint32_t plane, const uint32_t s[4], uint32_t out[4])
{
    u_expand_bits<kHigh>(plane, out);
#if defined(__CUDA_ARCH__)
#pragma unroll
#endif
    for (int m = 0; m < 4; ++m) out[m] |= s[m];
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
