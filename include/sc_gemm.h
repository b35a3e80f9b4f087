/*
 * sc_gemm.h -- C ABI of the B200 stochastic-computing GEMM (SC-GEMM) emulation library.
 *
 * The library evaluates the paper's SC matrix multiplication C ~= A W on one GPU:
 *   scales (Sec. 3.1)  ->  fused quantise + SNG encode (Sec. 3.1, Sec. 4.2)  ->  XNOR / AND gate with
 *   popcount accumulation over the stream positions and the inner dimension (Eq. (1)), one stream
 *   length per output row or row group (Sec. 4.2: a row ends at its own length)  ->  decode (Eq. (1)),
 * plus the per-row stream-length assignment of Sec. 4.4.
 *
 * Conventions for every call
 *   - Tensor pointers are DEVICE pointers owned by the caller, dense row-major, 16-byte aligned
 *     (A[M x K], W[K x N], C[M x N] float; P[M x N], L[...] int32).  Nothing is retained after a call.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Every call only
 *     enqueues work on it and returns; nothing synchronises unless stated.
 *   - The library allocates no device memory in these calls: scratch comes from the caller's
 *     workspace `ws` (size from sc_workspace_bytes; 256-byte aligned); sc_create allocates a few KB once.
 *   - The return value reports what the host can check (arguments, shapes, workspace size, CUDA launch
 *     errors).  Conditions only visible on the device -- a non-finite input, a stream length outside
 *     [0, Lmax], a bounded wait that ran out -- never trap: the kernels record the first-priority code
 *     in a device status word that sc_device_status reads, and the offending value is clamped / treated
 *     as zero so that the call still terminates.
 *   - No exceptions, no C++ or framework types cross this boundary.
 */
#ifndef SC_GEMM_H
#define SC_GEMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sc_ctx sc_ctx;   /* opaque: device ordinal, a small device scratch block, SM count */

typedef enum {
    SC_OK = 0,
    SC_ERR_ARG = 1,        /* NULL pointer, bad enum, bad group, misaligned pointer            */
    SC_ERR_SHAPE = 2,      /* non-positive or too large dimension                              */
    SC_ERR_LENGTH = 3,     /* stream length outside [0, Lmax] or Lmax outside [1, SC_L_CAP]    */
    SC_ERR_NONFINITE = 4,  /* NaN / Inf met in an input tensor (device-detected)               */
    SC_ERR_BUDGET = 5,     /* average budget below the minimum length (device-detected)        */
    SC_ERR_WORKSPACE = 6,  /* workspace missing, misaligned or too small                       */
    SC_ERR_CUDA = 7,       /* a CUDA runtime / driver call failed                              */
    SC_ERR_TIMEOUT = 8     /* a bounded device-side wait ran out (device-detected)             */
} sc_status;

typedef enum { SC_BIPOLAR_XNOR = 0,   /* Pr[z=1] = (v+1)/2, XNOR gate (Sec. 3.1, Eq. (1))                */
               SC_UNIPOLAR_AND = 1    /* sign + magnitude, Pr[z=1] = |v|, AND gate (Fig. 1b)             */
} sc_mode;

typedef enum { SC_SCALE_NONE = 0,       /* sigma = 1, values are clamped to [-1, 1]                        */
               SC_SCALE_PER_ROW = 1,    /* A: sigma_i = max_d |A_id|;  W: sigma_j = max_d |W_dj| (Sec. 3.1) */
               SC_SCALE_PER_TENSOR = 2  /* sigma = max |x| over the tensor                                 */
} sc_scale;

/* GEMM core variants (sc_params.core).  0 lets the library pick the measured-fastest one. */
enum { SC_CORE_AUTO = 0, SC_CORE_POPC = 1,   /* LOP3 + POPC on the integer pipes                          */
       SC_CORE_CSA = 2,                      /* carry-save: 3 planes -> 2 POPC                             */
       SC_CORE_SIMPLE = 3,                   /* one thread per output, no staging (debug reference)        */
       SC_CORE_UMMA = 4,                     /* tcgen05 tensor cores (4-bit floats) on bits expanded on chip,
                                                one SM per 128 x 192 tile                                  */
       SC_CORE_UMMA_PAIR = 5 };              /* the same on pairs of SMs (tcgen05 cta_group::2, 256 x 256 tiles); AUTO
                                                picks between the two per call from the stream lengths (long work
                                                pieces: pairs); batched calls always run on single SMs     */

/* Value -> comparator boundary (sc_params.quant).  Sec. 4.2 maps operands to the int8 grid (q_max = 127) and then to
 * one of 257 comparison boundaries; how a grid point becomes a boundary is not printed. */
enum { SC_QUANT_DIRECT257 = 0,       /* default: v = x / sigma straight onto the boundary grid, T = round((v + 1) 128)
                                        (unipolar: round(|v| 256)): one rounding, E[decoded stream] = T / 128 - 1     */
       SC_QUANT_INT8_THEN_257 = 1 }; /* the two steps of Sec. 4.2: x_hat = round(127 v) in -127..127, then the boundary
                                        nearest to its stream probability (x_hat + 127) / 254 (Sec. 3.1) on the 0..256
                                        scale, T = round((x_hat + 127) 128 / 127); unipolar: round(|x_hat| 256 / 127) */

#define SC_L_CAP 1024           /* largest stream length accepted                                 */

typedef struct {
    int32_t  mode;        /* sc_mode                                                             */
    int32_t  scale_a;     /* sc_scale for A                                                      */
    int32_t  scale_w;     /* sc_scale for W                                                      */
    int32_t  group;       /* rows of A per entry of L (>= 1); the last group may be short        */
    uint64_t seed;        /* Philox key                                                          */
    uint32_t stream_id;   /* distinguishes calls that must not share streams (< 2^31)            */
    uint32_t core;        /* SC_CORE_*                                                           */
    int32_t  quant;       /* SC_QUANT_*                                                          */
    int32_t  reserved;    /* must be 0                                                           */
} sc_params;

/* ---- context ------------------------------------------------------------------------------- */
/* Creates a context on CUDA device `device` (allocates a 64 KB device scratch block; the only
 * allocation the library ever makes).  sc_destroy frees it.  A context is not thread-safe.          */
sc_status sc_create(sc_ctx **ctx_out, int device);
sc_status sc_destroy(sc_ctx *ctx);
const char *sc_status_string(sc_status s);

/* Synchronises the device of the context, returns the highest-priority code the kernels recorded
 * since the last call (SC_OK if none) in *code_host, and clears it.                                 */
sc_status sc_device_status(sc_ctx *ctx, int32_t *code_host);

/* ---- Sec. 4.4: row metric and stream-length assignment ----------------------------------------- */
/* g[i] = ||A_i||_inf, the row metric of the linear layers (also the per-row scale of Sec. 3.1).
 * A: device [M x K]; g: device [M].                                                                 */
sc_status sc_row_stats(sc_ctx *ctx, const float *A, int64_t M, int64_t K, float *g, void *stream);

/* Stream lengths from row metrics at a matched average budget (Sec. 4.4): the metric of a group is
 * the largest of its rows', metrics are min-max normalised over the call, and a group receives
 * L = clamp(round(g~ * slope), Lmin, Lmax) -- the first level of the dense ladder Lmax > ... > Lmin
 * whose threshold it reaches -- with the slope the largest one whose total length over the M rows
 * stays within round(avg_budget * M).  All metrics equal -> floor(avg_budget) clamped.
 * g: device [M]; L_out: device [ceil(M / group)].  If realized_avg (HOST pointer) is non-NULL the call
 * synchronises the stream and stores the realised average length over rows.  An infeasible budget
 * (Lmin * M above it) is reported through sc_device_status as SC_ERR_BUDGET and gives all-Lmin.      */
sc_status sc_assign_lengths(sc_ctx *ctx, const float *g, int64_t M, int32_t group, double avg_budget,
                            int32_t Lmin, int32_t Lmax, int32_t *L_out, double *realized_avg, void *stream);

/* Sec. 4.4 inference rule with an explicit ladder: level k*(i) = min{k : g~_i >= tau_k}, else the last.
 * ladder: HOST [levels] (L_1 > ... > L_K), tau: HOST [levels-1] (non-increasing), levels <= 64.      */
sc_status sc_ladder_lengths(sc_ctx *ctx, const float *g, int64_t M, int32_t group, const int32_t *ladder,
                            const float *tau, int32_t levels, int32_t *L_out, void *stream);

/* ---- Sec. 3.1 / Sec. 4.2: encode ----------------------------------------------------------------- */
/* Bytes of a packed stream buffer for `stream_rows` rows of `depth` elements at lengths up to Lmax. */
size_t sc_stream_bytes(int64_t stream_rows, int64_t depth, int32_t Lmax, int32_t mode);

/* Fused scale + quantise + SNG + pack of one operand (Sec. 4.2 "fused quantization", Sec. 3.1 SNG).
 * tensor_id 0: X = A[rows x cols], one stream row per row of A, depth = cols, scale = params->scale_a.
 * tensor_id 1: X = W[rows x cols], one stream row per COLUMN of W, depth = rows, scale = params->scale_w.
 * Element (r, c) of X draws from the Philox stream (seed; stream_id, tensor_id; r * cols + c) and bit l
 * of its stream is [draw_l < T], T its boundary in 0..256.  L_or_null: device, one length per stream
 * row (NULL = Lmax for all); positions l >= L of a row are left unwritten.
 * streams_out: device, sc_stream_bytes(...) bytes, layout private (see sc_debug_unpack);
 * scales_out: device [stream rows] (sigma used for each stream row).                                */
sc_status sc_encode(sc_ctx *ctx, const float *X, int64_t rows, int64_t cols, int32_t tensor_id,
                    const int32_t *L_or_null, int32_t Lmax, const sc_params *params,
                    void *streams_out, float *scales_out, void *stream);

/* Test helper: expands a packed buffer to one byte per bit, bits_out[(r * depth + d) * Lmax + l] in {0,1}.
 * neg_out (may be NULL; unipolar only) receives bit AND sign, same shape.                            */
sc_status sc_debug_unpack(sc_ctx *ctx, const void *streams, int64_t stream_rows, int64_t depth, int32_t Lmax,
                          int32_t mode, uint8_t *bits_out, uint8_t *neg_out, void *stream);

/* ---- Eq. (1): the SC matrix multiplication ---------------------------------------------------- */
size_t sc_workspace_bytes(int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params);

/* C = decode( sum_d sum_{l < L_i} gate(zA_{id,l}, zW_{dj,l}) ), the whole path of Eq. (1) in one call:
 * scales, row ordering by length, encode of A and W, the bit-serial GEMM core, decode.
 *   L    : device [ceil(M / group)] stream length of each row group, each in [0, Lmax]; NULL = all Lmax.
 *   Lmax : upper bound of the lengths, 1..SC_L_CAP (sizes the workspace).
 *   P    : device [M x N] or NULL; bipolar: the XNOR count P_ij; unipolar: the signed AND count S_ij.
 *   C    : device [M x N]; bipolar sigmaA_i sigmaW_j (2 P_ij - K L_i) / L_i, unipolar sigmaA_i sigmaW_j S_ij / L_i;
 *          rows with L_i = 0 give 0.
 * K and N are unrestricted (internally padded); M, N < 2^24, K <= 2^20.
 * Everything is enqueued without host synchronisation.  The weight-side work (scales, encode of W, its popcount
 * tables) runs on a stream owned by the context, forked from `stream` and joined back into it by events before the
 * GEMM core: to the caller the call behaves as if enqueued on `stream` alone, and it can be captured into a CUDA graph.
 * A context serves one call sequence at a time (its scratch block, side stream and events are shared).        */
sc_status sc_matmul(sc_ctx *ctx, const float *A, const float *W, int64_t M, int64_t K, int64_t N,
                    const int32_t *L, int32_t Lmax, const sc_params *params,
                    int32_t *P, float *C, void *ws, size_t ws_bytes, void *stream);

/* ---- batched products (Sec. 4.4: the attention matmuls qk and av run per head) ------------------ */
/* B independent products in one call, C_b = A_b W_b for b < B: the attention score product (A_b = the
 * queries of one head, W_b = its keys given as rows: w_transposed = 1) and the attention output product
 * (A_b = the attention probabilities, non-negative -> unipolar mode is natural, W_b = the values).
 *   A : device [B][M][K];  W : device [B][K][N], or [B][N][K] when w_transposed = 1;
 *   L : device, one entry per `group` consecutive rows of the stacked [B*M] rows (NULL = all Lmax);
 *   P, C : device [B][M][N] (P may be NULL).
 * Semantics are those of sc_matmul applied to each product, with the rows of all A_b and the output columns
 * of all W_b treated as one stacked operand each: per-row / per-column scales are per stacked row / column,
 * a per-tensor scale is the maximum over the whole [B][..][..] tensor, and the stream of an element is
 * keyed by its flat position in the caller's tensor as stored (so product 0 of an untransposed call equals
 * sc_matmul on A_0, W_0).  Row metrics for the length policy (Sec. 4.4: max |Q_i| for qk, the peak
 * probability for av) come from sc_row_stats on the stacked [B*M x K] operand.
 * 1 <= B <= 65535; B * round_up(M, 128) and B * round_up(N, 384) below 2^24.
 * Workspace: sc_workspace_bytes_batched(B, M, K, N, Lmax, params).                                  */
size_t sc_workspace_bytes_batched(int64_t B, int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params);
sc_status sc_matmul_batched(sc_ctx *ctx, const float *A, const float *W, int64_t B, int64_t M, int64_t K, int64_t N,
                            int32_t w_transposed, const int32_t *L, int32_t Lmax, const sc_params *params,
                            int32_t *P, float *C, void *ws, size_t ws_bytes, void *stream);

/* ---- prepared weights (Sec. 4.2: what depends on the layer alone is built once and kept) --------- */
/* For a static weight matrix everything sc_matmul derives from W alone -- its scales, its streams up to
 * Lmax (Sec. 3.1; stream bits never depend on the length they are cut at, so one buffer serves every
 * shorter call) and, for the tensor-core core, the prefix popcounts of its columns -- can be computed once.
 * sc_weights_prepare writes them into `wbuf`, a DEVICE buffer of at least sc_weights_bytes(K, N, Lmax,
 * params) bytes, 256-byte aligned, owned by the caller and left alone by the library afterwards; it
 * enqueues on `stream` and returns a small HOST record in *out that names the buffer and the parameters it
 * was built with.  The record does not own the buffer: sc_weights_release frees the record only; the
 * caller keeps the buffer alive, unchanged, while any call using the record is pending, and prepares again
 * after W changes (the record cannot see that).
 *
 * sc_matmul_prepared is sc_matmul with the W-side work left out; results are identical bit for bit.
 * K and N come from the record.  params must repeat the mode, scale_w, quant, seed and stream_id used at
 * preparation (SC_ERR_ARG otherwise), Lmax may be anything up to the prepared one (SC_ERR_LENGTH beyond).
 * The buffer is laid out for the core chosen at preparation (params->core there, SC_CORE_AUTO rule on the
 * prepared Lmax): a later SC_CORE_AUTO follows it; an explicit core of the other family (tensor-core vs
 * the ALU cores) is SC_ERR_ARG.  Workspace: sc_workspace_bytes_prepared(M, K, N, Lmax, params).
 * Calls that are enqueued after sc_weights_prepare on another stream must be ordered after it by the
 * caller (an event), as with any producer of a device buffer.                                        */
typedef struct sc_weights sc_weights;
size_t sc_weights_bytes(int64_t K, int64_t N, int32_t Lmax, const sc_params *params);
sc_status sc_weights_prepare(sc_ctx *ctx, const float *W, int64_t K, int64_t N, int32_t Lmax,
                             const sc_params *params, void *wbuf, size_t wbuf_bytes, void *stream,
                             sc_weights **out);
sc_status sc_weights_release(sc_weights *weights);
size_t sc_workspace_bytes_prepared(int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params);
sc_status sc_matmul_prepared(sc_ctx *ctx, const float *A, const sc_weights *weights, int64_t M,
                             const int32_t *L, int32_t Lmax, const sc_params *params,
                             int32_t *P, float *C, void *ws, size_t ws_bytes, void *stream);

/* ---- Sec. 4.2 / Appendix A.1: the paper's own generator ------------------------------------------- */
/* sc_matmul with deterministic Sobol-8 streams shared by all elements and conditional bitstream generation
 * instead of one Philox stream per element: the activation stream of a value is its row of the indicator table
 * over a 256-entry Sobol sequence (prefixes for shorter streams), and the weight-side generator is gated by the
 * activation stream (one weight generator advances on the cycles where the activation bit is 1, a second one
 * where it is 0; output bit = XNOR).  Error falls like 1/L instead of 1/sqrt(L); at L = 256 an 8-bit operand is
 * recovered exactly.  The paper leaves open which Sobol dimensions, scrambling and gating order its kernel uses:
 * here activation = dimension 1, weight generators = dimension 2, each XORed with a byte derived from
 * (seed, stream_id); comparator z = [r < T], boundaries as in sc_matmul (bipolar).
 * Arguments as sc_matmul, with: mode must be SC_BIPOLAR_XNOR, core SC_CORE_AUTO, SC_CORE_UMMA or SC_CORE_UMMA_PAIR (the product
 * runs on the tensor-core core as a binary contraction of codes of 2 L_i positions per element of row i, so
 * its cost follows the sum of the lengths), 1 <= Lmax <= 256, 2 K Lmax <= 2^24.  P receives the XNOR counts of
 * the cycle-by-cycle multiplier.  Workspace: sc_workspace_bytes_cbsg(M, K, N, Lmax, params).            */
size_t sc_workspace_bytes_cbsg(int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params);
sc_status sc_matmul_cbsg(sc_ctx *ctx, const float *A, const float *W, int64_t M, int64_t K, int64_t N,
                         const int32_t *L, int32_t Lmax, const sc_params *params,
                         int32_t *P, float *C, void *ws, size_t ws_bytes, void *stream);

/* Diagnostic of Appendix A.1: for n pairs of boundaries (Ta[i], Tw[i]) in 0..256 (device arrays) and a stream length
 * L <= 256, the cycles on which (activation bit, gated weight bit) = 11, 10, 01, 00 -- counts[4 i .. 4 i + 3], device,
 * may be NULL -- and their stochastic cross-correlation scc[i] (device, double): the normalised a d - b c, which
 * vanishes when the weight bit is independent of the activation bit.  Same generator as sc_matmul_cbsg for
 * (seed, stream_id).  ws: device, 256-byte aligned, at least SC_CBSG_SCC_WS_BYTES.                              */
#define SC_CBSG_SCC_WS_BYTES 32768
sc_status sc_cbsg_scc(sc_ctx *ctx, const int32_t *Ta, const int32_t *Tw, int64_t n, int32_t L, uint64_t seed,
                      uint32_t stream_id, int32_t *counts, double *scc, void *ws, size_t ws_bytes, void *stream);

/* ---- Sec. 3.2: Gaussian surrogate of an SC product -------------------------------------------- */
/* out_ij = Y_ij (1 + alpha(L_i) Z_ij), Z_ij independent standard normal, alpha(L) = coeff / L: the cheap
 * stand-in the paper uses to sweep model-level tolerance without running the stochastic matmul.
 * SC_SURROGATE_COEFF reproduces the paper's printed table of alpha against L.  Y and out are device
 * [M x N] (out may alias Y); L as in sc_matmul (device, one entry per `group` rows; NULL = no noise scale
 * division, alpha = coeff); rows with L = 0 give 0.  Z_ij is a function of (seed, stream_id, i N + j) only
 * (one Philox4x32-10 call per cell, Box-Muller), so the perturbation is reproducible and independent of
 * the launch shape.  Non-finite Y and negative L are reported through sc_device_status.             */
#define SC_SURROGATE_COEFF 2.324
sc_status sc_surrogate_noise(sc_ctx *ctx, const float *Y, int64_t M, int64_t N, const int32_t *L, int32_t group,
                             double coeff, uint64_t seed, uint32_t stream_id, float *out, void *stream);

/* ---- allocation-free variant (the paper has no counterpart: this serves callers, not the method) -- */
/* sc_assign_lengths for callers that cannot allocate device memory at all -- a serving loop whose pool
 * is frozen after start-up, a plugin that only gets fixed buffers from its host application -- and so
 * cannot call sc_create.  It needs no context: its scratch is a fixed array inside the library image
 * (SC_STATIC_MAX_GROUPS * 4 + 256 bytes, about 1 MB, held by every GPU that loads the library until the
 * process exits).  The call never allocates or frees anything.
 *   g, L_out            : as in sc_assign_lengths (device pointers).
 *   status_out          : device int32 or NULL; receives SC_OK, SC_ERR_NONFINITE or SC_ERR_BUDGET.
 *   total_out           : device int64 or NULL; receives the total assigned length over the M rows.
 * Limits and rules: ceil(M / group) <= SC_STATIC_MAX_GROUPS, otherwise SC_ERR_SHAPE and nothing runs.
 * The first call on each device looks up the device address of the array (with that device current);
 * make that first call outside any stream capture.  All calls on a device share the array, which keeps
 * the previous call's contents (the kernel clears the words that must start at zero): calls that overlap
 * on the GPU race -- keep them on one stream or order them yourself.  Results equal sc_assign_lengths'. */
#define SC_STATIC_MAX_GROUPS 262144
sc_status sc_assign_lengths_static(const float *g, int64_t M, int32_t group, double avg_budget, int32_t Lmin,
                                   int32_t Lmax, int32_t *L_out, int32_t *status_out, int64_t *total_out,
                                   void *stream);

/* ---- tracing ------------------------------------------------------------------------------------ */
/* With profiling on, sc_matmul records CUDA events on the caller's stream between its phases.
 * sc_profile_read synchronises on the last one and returns the milliseconds of the most recent
 * sc_matmul per phase: ms_out[0] scales, [1] row ordering + work list + accumulator clear, [2] encode A,
 * [3] encode W, [4] GEMM core, [5] decode, [6] total, [7] reserved.  Off by default (no events).      */
#define SC_PROFILE_PHASES 8
sc_status sc_profile_enable(sc_ctx *ctx, int32_t on);
sc_status sc_profile_read(sc_ctx *ctx, float *ms_out /* HOST [SC_PROFILE_PHASES] */);

/* Number of kernels this library has launched through `ctx` since sc_create (memsets not counted). */
sc_status sc_launch_count(sc_ctx *ctx, int64_t *count_host);

/* Which tensor-core kernel the most recent sc_matmul / sc_matmul_prepared / sc_matmul_cbsg call through `ctx` selected
 * (the choice is made on the device from the stream lengths): *pair_host = 1 the two-SM kernel (SC_CORE_UMMA_PAIR),
 * 0 the one-SM kernel or a call that ran on the integer cores.  Synchronises on the device.  `pair_host`: HOST.       */
sc_status sc_last_core_selected(sc_ctx *ctx, int32_t *pair_host);

/* ---- host-side self checks and device micro-benchmarks ---------------------------------------- */
/* Exhaustive host check of the bit-plane comparator used by the encode kernel against r < T for all
 * 257 boundaries and 256 draws; returns the number of mismatches (0 = correct).  Runs on the CPU.   */
int32_t sc_selftest_comparator(void);

/* Exhaustive-plus-random host check of the tensor-core core's operand encodings: bit planes in the layouts the encode
 * writes, expanded to 4-bit floats (e2m1) by the same routines the kernel uses, must give exactly the AND count (bipolar)
 * and the signed count (unipolar) of the 32 depth elements of a word as the sum of the nibble products; returns the
 * number of mismatches (0 = correct).  Runs on the CPU.                                                            */
int32_t sc_selftest_expansion(void);

/* Device check of the failure-detection path: every wait of the tensor-core core on an mbarrier is bounded (a clock
 * limit and an abort flag shared by the roles of a CTA); a wait that runs out records SC_ERR_TIMEOUT in the device
 * status word and where it happened beside it, raises the abort flag, and the kernel returns normally.  This call
 * makes that happen in a kernel of one small CTA that does nothing else: one warp waits, with the core's own wait
 * routine and a limit of `limit_cycles` SM clocks (1 .. 2e9), on a barrier that is never signalled; a second warp
 * waits with the default limit and must leave through the abort flag.  Synchronises.  site_host (HOST, 3 ints)
 * receives the recorded site word (site 99 | warp << 8 | CTA << 16) and its two counters; cycles_host (HOST, 2
 * int64) the SM clocks each warp waited (-1 if its wait was satisfied, which cannot happen).  The status word
 * stays set: the next sc_device_status returns SC_ERR_TIMEOUT and clears it.  Nothing else is disturbed.       */
sc_status sc_selftest_bounded_wait(sc_ctx *ctx, int64_t limit_cycles, int32_t *site_host, int64_t *cycles_host);

/* Device micro-benchmarks of the units the GEMM cores are bound by (the measured denominators of the reported roofline
 * fractions).  Every loop and every wait in them is bounded; they allocate nothing and touch only the context's
 * scratch block.
 *
 * kind 0..7 -- register-only instruction-mix loops, `iters` trips per thread on every SM.  0 POPC only,
 *   1 LOP3 only, 2 LOP3+POPC+IADD (the plain core mix), 3 carry-save mix (3 words -> 2 POPC), 4 IADD3 only,
 *   5 / 6 warp-level 1-bit XOR / AND popcount tensor tiles (m16n8k256), 7 warp-level int8 tensor tiles
 *   (m16n8k32).  *ms_out = elapsed milliseconds (CUDA events; synchronises); *words_out = 32-bit word
 *   operations of the named kind executed on the whole GPU (mixes: gate evaluations of 32 stream bit-ops
 *   each; kind 7: multiply-accumulates).
 *
 * kind 8, 9 -- issue-rate ceiling of the tensor-core core's instruction: one thread per SM issues `iters` (rounded up
 *   to a multiple of 8, at most 2^22) block-scaled 4-bit MMAs, 128 x N x 64 with N = 192 (kind 8, the core's tile) or 256
 *   (kind 9), A operand and scale factors in tensor memory, B operand in shared memory, back to back on zero-filled
 *   operands, and waits (bounded) for the last one.  *ms_out = SM CLOCKS / 1e6 of the slowest SM (not milliseconds),
 *   *words_out = multiply-accumulates PER SM; their ratio / 1e6 is multiply-accumulates per clock per SM.        */
sc_status sc_microbench(sc_ctx *ctx, int32_t kind, int32_t iters, float *ms_out, double *words_out);

#ifdef __cplusplus
}
#endif
#endif /* SC_GEMM_H */
