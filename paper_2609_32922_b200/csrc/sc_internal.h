// Internal declarations shared by the translation units of the SC-GEMM library (host side).
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/sc_gemm.h"

namespace sc {

constexpr int kTileM = 128;          // rows of A per CTA tile (sorted order)
constexpr int kTileN = 128;          // output columns per CTA tile (ALU cores)
constexpr int kTileNUmma = 192;      // output columns per CTA tile (tensor-core core)
constexpr int kColPad = 384;         // W stream rows are padded to a multiple of both tile widths
// Column tile of the one-SM tensor-core core for N output columns: the columns are spread evenly over the tiles a width of
// kTileNUmma needs, in multiples of 32 (tiles then start on 128-byte boundaries of the plane rows; with multiples of 16 --
// N = 1024 as six tiles of 176 -- the weight boxes straddle one more line each and the core ran 6 - 19 % slower than with
// 192), so that narrow products cost less (N = 64: one tile of 64; N = 257: two of 160 instead of 192).
inline int umma_tile_cols(int64_t N)
{
    const int64_t tiles = (N + kTileNUmma - 1) / kTileNUmma;
    const int64_t w = ((N + tiles - 1) / tiles + 31) / 32 * 32;
    return (int)(w < kTileNUmma ? w : kTileNUmma);
}
constexpr int kStagePlanes = 16;     // stream planes per pipeline stage
// Selection between the two tensor-core kernels (sc_plan.cu states the rule): a piece boundary of the two-SM core costs
// about kPairDrainUnits stage units, one of the one-SM core kPieceChargeUnits; on long pieces the two-SM core needs
// 100 / kPairAdvantagePct of the one-SM core's time per multiply-accumulate (break-even near 16 units per piece on unpadded
// shapes).  kPieceChargeUnits is also what the prefix sums charge every (row tile, column tile) of the one-SM core; measured:
// 0 / 4 / 8 / 12 units give 0.120 / 0.117 / 0.117 / 0.121 ms on the per-row mixed ViT-B/16 qkv configuration and
// 2.03 / 1.94 / 1.96 / 1.99 ms on the grouped DiT-like one.
constexpr long long kPairDrainUnits = 14;
constexpr long long kPairAdvantagePct = 150;
constexpr int kPieceChargeUnits = 4;
constexpr int kStages = 4;           // TMA pipeline depth
constexpr int kScratchBytes = 64 * 1024;

// Layout of the context's device scratch block (int32 slots).
enum ScratchSlot : int {
    kSlotStatus = 0,        // device status word (max of sc_status codes seen)
    kSlotTicket = 1,        // work-item ticket counter of the GEMM core
    kSlotLmaxActual = 2,    // largest stream length of the current call
    kSlotTensorMaxA = 3,    // bit pattern of max|A| (per-tensor scale)
    kSlotTensorMaxW = 4,    // bit pattern of max|W|
    kSlotRealizedTotal = 6, // int64 (slots 6,7): total assigned length
    kSlotTimeoutSite = 8,   // slots 8-10: where the first bounded wait of the tensor-core core ran out
    kSlotAnyNegA = 11,      // unipolar: set by the encode of A when any stream bit carries a negative sign
    kSlotPairSelected = 12, // the plan of the current call selected the two-SM tensor-core kernel
    kSlotCount = 16
};

struct sc_ctx_impl {
    int device;
    int sm_count;
    int32_t *scratch;       // device, kScratchBytes
    cudaEvent_t ev0, ev1;
    bool profiling;
    bool profile_valid;
    cudaEvent_t phase_ev[SC_PROFILE_PHASES];
    // the W-side work of a call (scales, encode, popcount tables) runs on a side stream beside the A-side work
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_plan, ev_join, ev_a_done, ev_rows_done;
    bool overlap;
};

// kernels launched by this library in this process (every launcher adds its launches)
void count_launches(int n);
long long launches_so_far();

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline int planes_per_step(int mode) { return mode == SC_UNIPOLAR_AND ? 2 : 1; }
// Stream positions are stored in blocks of this many (plane_index in sc_device.cuh).  The signed (unipolar) operands of
// the tensor-core core use blocks of 8, everything else the plain position-major order.
constexpr int kPosBlockSigned = 8;
inline int pos_block_for(int mode, bool umma) { return (umma && mode == SC_UNIPOLAR_AND) ? kPosBlockSigned : 1; }
// planes per position as written for a core family: the tensor-core core keeps the signs of unipolar operands beside
// single magnitude planes, the ALU cores read a magnitude and a negative plane
inline int planes_per_step_for(int mode, bool umma) { return (umma || mode != SC_UNIPOLAR_AND) ? 1 : 2; }

// Work plan written by the plan kernel and read by the core (device memory, int32 fields).
struct PlanHeader {
    int32_t total_items;
    int32_t chunk_planes;   // planes per work item (multiple of kStagePlanes)
    int32_t n_row_tiles;
    int32_t n_col_tiles;
    int32_t lmax_actual;
    int32_t pad[3];         // pad[0]: 1 = the two-SM tensor-core core runs the call, 0 = the one-SM core
    // followed by int32 prefix[n_row_tiles + 1] and int32 tile_planes[n_row_tiles]
};

// B independent products in one call: the rows of all A_b are stacked (row b*M + i), the output columns of all
// W_b too (column b*N + j); each product is padded to the tile sizes on its own, so that a row tile and a
// column tile never straddle products.  B = 1 is the plain product.
struct BatchGeom {
    int64_t B, M, N;            // products; rows of A / columns of W per product
    int64_t m_pad, n_pad;       // per product, padded (kTileM / kColPad)
    int32_t tiles_m;            // row tiles per product
    int32_t w_transposed;       // W stored as [B][N][K] (output columns as rows) instead of [B][K][N]
};

// Workspace offsets (bytes) of one sc_matmul call.
struct Workspace {
    size_t sigma_a, sigma_w, l_rows, perm, l_sorted, plan, acc, pop_a, pop_w, a_streams, w_streams, w_sign, a_sign, total;
    int64_t m_pad, n_pad, kw, a_planes, w_planes;      // plane counts as allocated (unipolar: lengths rounded up to 8, two planes
                                                       // per position for either core family)
};
// with_w = false leaves out everything derived from W alone (prepared weights carry it).
Workspace layout_workspace(int64_t M, int64_t K, int64_t N, int32_t Lmax, int mode, bool need_acc, bool with_w = true,
                           int64_t B = 1, int64_t col_pad = kColPad);

// Prepared weights: all that sc_matmul derives from W alone, kept in a caller-owned device buffer.
struct WeightsLayout {
    size_t sigma_w, pop_w, w_streams, w_sign, total;
    int64_t n_pad, kw, w_planes;
};
WeightsLayout layout_weights(int64_t K, int64_t N, int32_t Lmax, int mode);

struct sc_weights_impl {
    uint32_t magic;
    int device;
    int64_t K, N;
    int32_t Lmax;
    int mode, scale_w, quant;
    uint64_t seed;
    uint32_t stream_id;
    bool umma;               // laid out for the tensor-core core (else for the ALU cores)
    const float *sigma_w;
    const int32_t *pop_w;    // NULL unless umma && bipolar
    const uint32_t *w_streams;
    const uint32_t *w_sign;  // NULL unless umma && unipolar
};
constexpr uint32_t kWeightsMagic = 0x53435754u;

// ---- kernel launchers (each enqueues on `st` and returns the launch status) -----------------------
cudaError_t launch_row_absmax(const float *X, int64_t rows, int64_t cols, float *g, float *sigma,
                              int32_t *status, cudaStream_t st);
// per output column of each of `batch` consecutive [rows x cols] tensors; sigma has batch * cols entries
cudaError_t launch_col_absmax(const float *X, int64_t rows, int64_t cols, float *sigma, int32_t *status,
                              cudaStream_t st, int64_t batch = 1);
cudaError_t launch_tensor_absmax(const float *X, int64_t count, int32_t *slot_bits, int32_t *status,
                                 cudaStream_t st);
cudaError_t launch_fill_sigma(float *sigma, int64_t n, const int32_t *slot_bits_or_null, cudaStream_t st);

cudaError_t launch_assign_lengths(const float *g, int64_t M, int32_t group, double avg_budget, int32_t Lmin,
                                  int32_t Lmax, int32_t *L_out, int32_t *scratch, cudaStream_t st);
cudaError_t launch_ladder_lengths(const float *g, int64_t M, int32_t group, const int32_t *ladder,
                                  const float *tau, int32_t levels, int32_t *L_out, int32_t *scratch,
                                  cudaStream_t st);

// target_items > 0: cut tiles into chunks so that about that many items exist (ALU cores, dynamic tickets).
// wave_ctas > 0: pick the chunk count that minimises rounds x (chunk + epilogue cost) for a static
// round-robin over wave_ctas persistent CTAs (tensor-core core).
// M, m_pad: per product; `batch` products are planned (rows sorted inside each product).
cudaError_t launch_plan(const int32_t *L, int64_t M, int32_t group, int32_t Lmax, int64_t kw, int ppq,
                        int64_t m_pad, int64_t n_col_tiles, int32_t target_items, int32_t wave_ctas,
                        int32_t *l_rows, int32_t *perm, int32_t *l_sorted, PlanHeader *plan, int32_t *scratch,
                        cudaStream_t st, int64_t batch = 1, int32_t pos_block = 1, int32_t pair_col_tiles = 0,
                        int32_t pair_clusters = 0, int32_t pair_force = 0, int32_t single_tile_cols = kTileNUmma);

struct EncodeArgs {
    const float *X;
    int64_t rows, cols;          // shape of X
    int tensor_id;               // 0: stream row = row of X; 1: stream row = column of X
    int mode;
    int64_t stream_rows, depth, kw, r_pad;
    const int32_t *perm;         // sorted position -> stream row (NULL = identity)
    const int32_t *l_sorted;     // length per sorted position (NULL = Lmax)
    const int32_t *lmax_actual;  // device scalar: skip blocks beyond it (NULL = Lmax)
    int32_t Lmax;
    const float *sigma;          // per stream row (never NULL)
    uint64_t seed;
    uint32_t stream_id;
    uint32_t *streams;
    int32_t *status;
    int reverse_bytes;           // W operand of the tensor-core core: 1 = each group of 4 depth elements in reverse bit
                                 // order; 0 = plain
    int pos_block = 1;           // stream positions stored in blocks of this many (plane_index)
    uint32_t *signs = nullptr;   // unipolar operand of the tensor-core core: [kw][r_pad][4] nibble sign words written here
                                 // and only the magnitude planes (one per position) into `streams`
    // W operand of a batched call (tensor_id 1): stream row r = b * batch_pad + j is output column j of product b
    int64_t batch_pad = 0;       // padded stream rows per product (0: not batched, rows = stream rows)
    int64_t batch_real = 0;      // real stream rows per product
    int w_transposed = 0;        // X stored [B][N][K] instead of [B][K][N]
    int quant = 0;               // SC_QUANT_*: value -> boundary rule
};
cudaError_t launch_encode(const EncodeArgs &a, cudaStream_t st);
cudaError_t launch_unpack(const uint32_t *streams, int64_t stream_rows, int64_t depth, int32_t Lmax, int mode,
                          uint8_t *bits, uint8_t *neg, cudaStream_t st);

struct CoreArgs {
    const uint32_t *a_streams, *w_streams;
    int64_t m_pad, n_pad, a_planes, w_planes;
    int64_t M, N;
    int mode, variant;
    const int32_t *perm, *l_sorted;
    const PlanHeader *plan;
    int32_t kw, ppq;
    int32_t *acc;                // [M x N] accumulators (zeroed)
    int32_t *scratch;
    int sm_count;
    int32_t Lmax;
    int32_t tiles_m = 1;         // row tiles per product and ...
    int64_t w_batch_cols = 0;    // ... padded W stream rows per product: the W tile of an item starts at
                                 // (row tile / tiles_m) * w_batch_cols + column tile * tile width
    const uint32_t *w_sign = nullptr;   // unipolar tensor-core core: [kw][n_pad][4] nibble sign words of W ...
    const uint32_t *a_sign = nullptr;   // ... and [kw][m_pad][4] of A (sorted row order)
    int32_t pos_block = 1;       // block size of the stream positions in both operands' planes
    int32_t tile_n = kTileNUmma; // one-SM tensor-core core: output columns per tile (umma_tile_cols)
    int32_t *pop_a;              // [M] ones of each row of A below its own end (tensor-core core, bipolar)
    const int32_t *pop_w;        // [(Lmax + 1) x n_pad] prefix ones of each W column (tensor-core core, bipolar)
};
cudaError_t launch_core(const CoreArgs &a, cudaStream_t st);
cudaError_t launch_core_umma(const CoreArgs &a, cudaStream_t st);
// Two-SM tensor-core core (sc_core_umma2.cu): runs when the plan selected it (PlanHeader.pad[0]) or when forced; the one-SM
// core returns at once in that case.  `clusters` = CTA pairs to launch (pair_core_clusters).
cudaError_t launch_core_umma_pair(const CoreArgs &a, int clusters, bool force, cudaStream_t st);
cudaError_t pair_core_clusters(int mode, int sm_count, int *clusters);
int pair_core_tile_cols();
int pair_core_max_row_tiles();
cudaError_t launch_row_corrections(const CoreArgs &a, cudaStream_t st);
cudaError_t launch_col_corrections(const uint32_t *w_streams, int64_t n_pad, int32_t kw, int32_t Lmax,
                                   const int32_t *lmax_actual, int32_t *pop_w, cudaStream_t st);
// Decode launchers: M = stacked rows (B * rows_per_batch); column tables are indexed per product
// (sigma_w[b * N + j], pop_w[l * n_pad + b * w_batch_cols + j]).
cudaError_t launch_decode_and(const int32_t *acc, int64_t M, int64_t N, int64_t K, int64_t n_pad,
                              const int32_t *l_rows, const int32_t *pop_a, const int32_t *pop_w,
                              const float *sigma_a, const float *sigma_w, int32_t *P, float *C, cudaStream_t st,
                              int64_t rows_per_batch = 0, int64_t w_batch_cols = 0);

cudaError_t launch_decode(int mode, const int32_t *acc, int64_t M, int64_t N, int64_t K, const int32_t *l_rows,
                          const float *sigma_a, const float *sigma_w, int32_t *P, float *C,
                          cudaStream_t st, int64_t rows_per_batch = 0);

// Sobol-8 / conditional-generation streams (sc_cbsg.cu): a row of length L is a code of 2 L positions
constexpr size_t kCbsgTableBytes = (257 * 8 + 257 * 16) * sizeof(uint32_t);
cudaError_t launch_cbsg_setup(uint64_t seed, uint32_t stream_id, uint32_t *tables, const int32_t *L, int64_t n_groups,
                              int32_t Lmax, int32_t *L_core, int32_t *status, cudaStream_t st);
cudaError_t launch_cbsg_encode(const float *X, int64_t rows, int64_t cols, int tensor_id, int64_t r_pad,
                               const int32_t *perm, const int32_t *l_sorted, const int32_t *lmax_actual,
                               const int32_t *L, int32_t group, int32_t Lmax, const float *sigma,
                               const uint32_t *tables, uint32_t *streams, int reverse_bytes, int32_t *status,
                               cudaStream_t st, int quant = 0);
cudaError_t launch_cbsg_scc(const uint32_t *tables, const int32_t *Ta, const int32_t *Tw, int64_t n, int32_t L,
                            int32_t *counts, double *scc, int32_t *status, cudaStream_t st);
cudaError_t launch_cbsg_decode(const int32_t *acc, int64_t M, int64_t N, int64_t K, const int32_t *L, int32_t group,
                               int32_t Lmax, const float *sigma_a, const float *sigma_w, int32_t *P, float *C,
                               cudaStream_t st);

cudaError_t launch_surrogate(const float *Y, int64_t M, int64_t N, const int32_t *L, int32_t group, double coeff,
                             uint64_t seed, uint32_t stream_id, float *out, int32_t *status, cudaStream_t st);

cudaError_t run_microbench(sc_ctx_impl *ctx, int kind, int iters, float *ms, double *words);
cudaError_t run_bounded_wait_selftest(sc_ctx_impl *ctx, long long limit_cycles, int32_t site_out[3], long long cycles_out[2]);
cudaError_t run_mxf4_rate(sc_ctx_impl *ctx, int n_cols, int iters, float *mclk, double *macs_per_sm);

}  // namespace sc
