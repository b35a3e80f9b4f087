// Encode: fused scale -> boundary -> Philox SNG -> bit transpose -> packed stream planes
// (Sec. 3.1 Bitstream generation, Sec. 4.2 fused quantization).
//
// Packed layout ("depth-packed planes"): plane p is a row of r_pad 32-bit words, one per stream row;
// the word of stream row r in plane p = (l * kw + w) * ppq (+1 for the negative plane in unipolar
// mode) holds stream position l of the 32 elements d = 32 w .. 32 w + 31 of that row (bit d % 32).
// (The signed operands of the tensor-core core store the positions in blocks of 8, plane_index(l, w) * ppq, and
// its unipolar W operand keeps one sign word per (w, stream row) beside single magnitude planes.)
// The GEMM core then reduces over planes with whole-word XOR/AND + POPC, any integer length costs
// exactly l * kw planes (no padding to a multiple of 32 positions), and a tile of 128 stream rows x
// 16 planes is one 2-D TMA box.
//
// One warp owns (8 consecutive stream rows, one depth word w, a run of 32-position blocks): each lane
// evaluates 32 positions of its element with two Philox calls and the bit-plane comparator, a five-stage
// butterfly of warp shuffles transposes the 32 x 32 bit matrix of the warp (32 position-packed words ->
// 32 depth-packed words, lane b ends up with position b), and every lane stores its 8 rows as one
// 32-byte segment.
#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

// Everything the kernel needs besides the Philox round keys (both are passed by value: the keys then sit in
// the constant bank and cost no registers).
struct EncodeDev {
    const float *X;
    int64_t x_cols, stream_rows, depth, r_pad, n_row_groups;
    const int32_t *perm, *l_sorted, *lmax_actual;
    const float *sigma;
    uint32_t *streams;
    int32_t *status;
    int32_t tensor_id, kw, Lmax, n_chunks, chunk_blocks, reverse_bytes, vec_rows, quant;
    int32_t ppq, pos_shift;          // planes per position written (unipolar: 2, or 1 when the signs go to `signs`); log2 of the position block
    uint32_t *signs;                 // [kw][r_pad][4] nibble sign words of a unipolar operand (NULL: negative planes instead)
    uint32_t stream_word;
    // weight operand of a batched call: stream row r = b * batch_pad + j is output column j of product b, stored at
    // X[b][d][j] (or X[b][j][d] when transposed); batch_pad = 0 otherwise
    int64_t batch_pad, batch_real;
    int32_t w_transposed;
};

constexpr int kEncodeThreads = 128;

// One warp owns (8 consecutive stream rows, one depth word w, a run of 32-position blocks).  Phase 1 turns
// the warp's 8 x 32 values into boundaries once; phase 2 walks the blocks: two Philox calls and the bit-plane
// comparator per element and block, the 32 x 32 bit transpose, one 32-byte store per lane.
// (four CTAs = 16 warps per SM: at most 128 registers; the unipolar form would otherwise take 163 and run 4 % slower)
template <int kMode>
__global__ void __launch_bounds__(kEncodeThreads, 4)
encode_kernel(const __grid_constant__ PhiloxKeys ks, const __grid_constant__ EncodeDev p)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * (kEncodeThreads / 32) + (threadIdx.x >> 5);
    // warp index -> (row group, block run, depth word); depth word fastest so that neighbouring warps read
    // neighbouring 128-byte segments of a row of A
    const int32_t w = (int32_t)(warp % p.kw);
    const int64_t rest = warp / p.kw;
    const int32_t chunk = (int32_t)(rest % p.n_chunks);
    const int64_t rg = rest / p.n_chunks;
    if (rg >= p.n_row_groups) return;

    const int32_t l_call = p.lmax_actual ? min(__ldg(p.lmax_actual), p.Lmax) : p.Lmax;
    const int64_t r0 = rg * 8;
    // Rows are sorted by decreasing length when a permutation is given; the GEMM cores never read a tile of
    // 128 rows beyond its first (longest) row, so nothing past that needs to be written.
    int32_t l_write = l_call;
    if (p.perm && p.l_sorted) l_write = min(l_write, __ldg(p.l_sorted + (r0 / kTileM) * kTileM));
    const int32_t blk0 = chunk * p.chunk_blocks;
    const int32_t blk1 = min(blk0 + p.chunk_blocks, (l_write + 31) >> 5);
    if (blk0 >= blk1) return;

    const WarpTranspose transpose(lane);
    // Bit `lane` of an output word holds depth element d.  With reverse_bytes == 1 the elements of each group of
    // four are stored in reverse bit order (the tensor-core core pairs bit m of an activation nibble with bit
    // 3 - m of the weight nibble, so that every product of its power-of-two codes has the same weight).
    const int64_t d = (int64_t)w * 32 + (p.reverse_bytes == 1 ? w_bit_element(lane) : lane);
    const bool have_d = d < p.depth;

    // ---- phase 1: boundaries of the warp's 8 x 32 elements ----
    // Element (stream row t, depth d) sits at X[base[t] + d * d_stride]; that flat index also names its stream.
    int32_t info[8];            // boundary T (bits 0-8) | row length (bits 10-20); rows that do not exist: 0
    uint32_t neg_mask[8];       // unipolar: sign of the 32 depth elements of the row
    uint64_t elem[8];
    float x[8], sg[8];
    int64_t base[8], sig_idx[8];
    bool bad = false, any_negative = false;
    const bool row_major_streams = p.tensor_id == 0 || p.w_transposed;       // a stream row is a row of X
    const int64_t d_stride = row_major_streams ? 1 : p.x_cols;
    const int64_t per_batch = p.batch_pad ? p.batch_pad : p.r_pad;
    const int64_t b_idx = r0 / per_batch;                                    // the 8 rows share one product
    const int64_t j0 = r0 - b_idx * per_batch;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        const int64_t r = r0 + t;
        base[t] = -1;
        sig_idx[t] = 0;
        int32_t row_len = 0;
        if (r < p.r_pad) {
            if (p.perm) {
                // with a permutation the per-position arrays cover the padded range; source rows number all products
                const int64_t src = (int64_t)__ldg(p.perm + r);
                if (src >= 0) { base[t] = src * p.x_cols; sig_idx[t] = src; }
            } else if (p.batch_pad == 0) {
                if (r < p.stream_rows) { base[t] = row_major_streams ? r * p.x_cols : r; sig_idx[t] = r; }
            } else if (j0 + t < p.batch_real) {
                const int64_t j = j0 + t;
                sig_idx[t] = b_idx * p.batch_real + j;
                base[t] = p.w_transposed ? sig_idx[t] * p.x_cols : b_idx * p.depth * p.x_cols + j;
            }
            if (base[t] >= 0) row_len = p.l_sorted ? __ldg(p.l_sorted + r) : p.Lmax;
        }
        info[t] = row_len << 10;
        x[t] = 0.0f;
        sg[t] = 1.0f;
    }
    if (!row_major_streams && p.vec_rows && base[0] >= 0 && base[7] >= 0) {
        // W: the 8 stream rows are 8 consecutive floats of one row of X
        if (have_d) {
            const float4 *q = reinterpret_cast<const float4 *>(p.X + base[0] + d * d_stride);
            const float4 a = __ldg(q), b = __ldg(q + 1);
            x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
        }
#pragma unroll
        for (int t = 0; t < 8; ++t) sg[t] = __ldg(p.sigma + sig_idx[t]);
    } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            if (base[t] < 0) continue;
            if (have_d) x[t] = __ldg(p.X + base[t] + d * d_stride);
            sg[t] = __ldg(p.sigma + sig_idx[t]);
        }
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        uint32_t neg = 0u;
        int32_t T = 0;
        elem[t] = 0;
        if (base[t] >= 0 && have_d) {
            float xv = x[t];
            if (is_nonfinite(xv)) { bad = true; xv = 0.0f; }
            const float v = normalise(xv, sg[t]);
            if (kMode == SC_BIPOLAR_XNOR) T = p.quant ? boundary_bipolar_int8(v) : boundary_bipolar(v);
            else T = p.quant ? boundary_unipolar_int8(v, neg) : boundary_unipolar(v, neg);
            elem[t] = (uint64_t)(base[t] + d * d_stride);
        }
        info[t] |= T;
        neg_mask[t] = 0u;
        if (kMode == SC_UNIPOLAR_AND) {
            neg_mask[t] = __ballot_sync(0xFFFFFFFFu, neg);
            any_negative |= __ballot_sync(0xFFFFFFFFu, neg && T > 0) != 0u;
        }
    }
    if (bad) report(p.status, SC_ERR_NONFINITE);
    // activations without a single negative stream bit (post-ReLU / GELU outputs, attention probabilities) let the
    // tensor-core core expand them with the cheap unsigned rule
    if (kMode == SC_UNIPOLAR_AND && p.tensor_id == 0 && any_negative && lane == 0) atomicOr(p.status + kSlotAnyNegA, 1);

    // The tensor-core core takes the signs of a unipolar operand beside single magnitude planes: per (depth word, stream
    // row) the four nibble sign words of the row's 32 elements.  The warp that owns the first run of blocks writes them
    // (lane t the words of row t).
    if (kMode == SC_UNIPOLAR_AND && p.signs && chunk == 0 && lane < 8) {
        uint32_t sn[4];
        uint32_t mine = neg_mask[0];
#pragma unroll
        for (int t = 1; t < 8; ++t) mine = lane == t ? neg_mask[t] : mine;
        sign_nibble_words(mine, p.reverse_bytes == 1, sn);
        reinterpret_cast<uint4 *>(p.signs)[(int64_t)w * p.r_pad + r0 + lane] = make_uint4(sn[0], sn[1], sn[2], sn[3]);
    }

    // ---- phase 2: the blocks ----
    // (as far as the longest of the warp's eight rows reaches: groups of rows that do not exist -- the padding of a batched
    // product -- or that have all ended write zeros below without drawing anything)
    int32_t live_len = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) live_len = max(live_len, info[t] >> 10);
    const int32_t blk_live = min(blk1, (live_len + 31) >> 5);
#pragma unroll 1
    for (int32_t blk = blk0; blk < blk1; ++blk) {
        if (blk >= blk_live) {                                         // warp-uniform
            const int32_t l = blk * 32 + lane;
            if (l < l_write) {
                const int64_t plane = plane_index_pow2(l, w, p.kw, p.pos_shift) * p.ppq;
                uint4 *dst = reinterpret_cast<uint4 *>(p.streams + plane * p.r_pad + r0);
                dst[0] = make_uint4(0u, 0u, 0u, 0u);
                dst[1] = make_uint4(0u, 0u, 0u, 0u);
                if (kMode == SC_UNIPOLAR_AND && p.ppq == 2) {
                    uint4 *dn = reinterpret_cast<uint4 *>(p.streams + (plane + 1) * p.r_pad + r0);
                    dn[0] = make_uint4(0u, 0u, 0u, 0u);
                    dn[1] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            continue;
        }
        uint32_t out_pos[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) {
            // (no branch per row: the eight rows' Philox chains and shuffle butterflies are independent and interleave;
            // a row that has ended -- rows of a group are neighbours in the order of lengths -- is computed and dropped)
            const uint32_t z = sng_word(ks, p.stream_word, elem[t], (uint32_t)blk, info[t] & 0x1FF);
            // 32 x 32 bit transpose across the warp: lane b receives position b of the 32 depth elements
            const uint32_t zt = transpose(z);
            out_pos[t] = blk * 32 < (info[t] >> 10) ? zt : 0u;
        }
        const int32_t l = blk * 32 + lane;                             // the position this lane holds
        if (l < l_write) {
            const int64_t plane = plane_index_pow2(l, w, p.kw, p.pos_shift) * p.ppq;
            uint4 *dst = reinterpret_cast<uint4 *>(p.streams + plane * p.r_pad + r0);
            dst[0] = make_uint4(out_pos[0], out_pos[1], out_pos[2], out_pos[3]);
            dst[1] = make_uint4(out_pos[4], out_pos[5], out_pos[6], out_pos[7]);
            if (kMode == SC_UNIPOLAR_AND && p.ppq == 2) {
                // the negative plane: stream bit AND sign
                uint4 *dn = reinterpret_cast<uint4 *>(p.streams + (plane + 1) * p.r_pad + r0);
                dn[0] = make_uint4(out_pos[0] & neg_mask[0], out_pos[1] & neg_mask[1], out_pos[2] & neg_mask[2],
                                   out_pos[3] & neg_mask[3]);
                dn[1] = make_uint4(out_pos[4] & neg_mask[4], out_pos[5] & neg_mask[5], out_pos[6] & neg_mask[6],
                                   out_pos[7] & neg_mask[7]);
            }
        }
    }
}

cudaError_t launch_encode(const EncodeArgs &a, cudaStream_t st)
{
    EncodeDev p;
    p.X = a.X; p.x_cols = a.cols; p.stream_rows = a.stream_rows; p.depth = a.depth; p.r_pad = a.r_pad;
    p.n_row_groups = a.r_pad / 8;
    p.perm = a.perm; p.l_sorted = a.l_sorted; p.lmax_actual = a.lmax_actual; p.sigma = a.sigma;
    p.streams = a.streams; p.status = a.status;
    p.tensor_id = a.tensor_id; p.kw = (int32_t)a.kw; p.Lmax = a.Lmax; p.reverse_bytes = a.reverse_bytes;
    p.quant = a.quant;
    p.pos_shift = a.pos_block == kPosBlockSigned ? 3 : 0; p.signs = a.signs;
    if (a.pos_block != 1 && a.pos_block != kPosBlockSigned) return cudaErrorInvalidValue;
    p.ppq = (a.mode == SC_UNIPOLAR_AND && !a.signs) ? 2 : 1;
    p.stream_word = ((uint32_t)a.tensor_id & 1u) | (a.stream_id << 1);
    p.batch_pad = a.batch_pad; p.batch_real = a.batch_real; p.w_transposed = a.w_transposed;
    // W read as two 16-byte vectors per lane when its rows keep them aligned
    p.vec_rows = (a.tensor_id == 1 && !a.w_transposed && a.cols % 4 == 0 && (reinterpret_cast<uintptr_t>(a.X) & 15u) == 0) ? 1 : 0;
    // A warp walks a run of 32-position blocks with its boundaries held in registers.  Longer runs amortise
    // the boundary computation; shorter runs make more warps: keep about two waves of 16 warps per SM (measured:
    // on the ViT-B/16 fc1 weights a four-block run beats two runs of two blocks by 8 %).
    const int32_t n_blocks = (a.Lmax + 31) / 32;
    const int64_t base_warps = p.n_row_groups * a.kw;
    int32_t chunk_blocks = n_blocks;
    constexpr int64_t kMinWarps = 148LL * 16 * 2;
    while (chunk_blocks > 2 && base_warps * ((n_blocks + chunk_blocks - 1) / chunk_blocks) < kMinWarps)
        chunk_blocks = (chunk_blocks + 1) / 2;
    p.chunk_blocks = chunk_blocks;
    p.n_chunks = (n_blocks + chunk_blocks - 1) / chunk_blocks;
    const int64_t warps = base_warps * p.n_chunks;
    const int64_t blocks = (warps + kEncodeThreads / 32 - 1) / (kEncodeThreads / 32);
    if (blocks <= 0) return cudaSuccess;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const PhiloxKeys ks = philox_keys(a.seed);
    if (a.mode == SC_BIPOLAR_XNOR) encode_kernel<SC_BIPOLAR_XNOR><<<(unsigned)blocks, kEncodeThreads, 0, st>>>(ks, p);
    else encode_kernel<SC_UNIPOLAR_AND><<<(unsigned)blocks, kEncodeThreads, 0, st>>>(ks, p);
    count_launches(1);
    return cudaGetLastError();
}

// ---- test helper: packed planes -> one byte per stream bit ------------------------------------------
__global__ void unpack_kernel(const uint32_t *__restrict__ streams, int64_t stream_rows, int64_t depth, int32_t Lmax,
                              int32_t kw, int64_t r_pad, int ppq, uint8_t *__restrict__ bits,
                              uint8_t *__restrict__ neg)
{
    const int64_t total = stream_rows * depth * Lmax;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t l = (int32_t)(i % Lmax);
        const int64_t rd = i / Lmax;
        const int64_t d = rd % depth, r = rd / depth;
        const int64_t plane = ((int64_t)l * kw + d / 32) * ppq;
        bits[i] = (uint8_t)((streams[plane * r_pad + r] >> (d & 31)) & 1u);
        if (neg) neg[i] = ppq == 2 ? (uint8_t)((streams[(plane + 1) * r_pad + r] >> (d & 31)) & 1u) : 0;
    }
}

cudaError_t launch_unpack(const uint32_t *streams, int64_t stream_rows, int64_t depth, int32_t Lmax, int mode,
                          uint8_t *bits, uint8_t *neg, cudaStream_t st)
{
    const int64_t kw = (depth + 31) / 32, r_pad = round_up(stream_rows, kTileM);
    const int64_t total = stream_rows * depth * Lmax;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    if (blocks < 1) return cudaSuccess;
    unpack_kernel<<<(unsigned)blocks, 256, 0, st>>>(streams, stream_rows, depth, Lmax, (int32_t)kw, r_pad,
                                                    planes_per_step(mode), bits, neg);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace sc
