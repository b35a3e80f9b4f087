// extern "C" entry points of the SC-GEMM library: argument checks, workspace carving, kernel sequencing.
// No computation of the method happens on the host.
#include <math.h>
#include <new>
#include <string.h>

#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static long long g_launches = 0;
void count_launches(int n) { g_launches += n; }
long long launches_so_far() { return g_launches; }

Workspace layout_workspace(int64_t M, int64_t K, int64_t N, int32_t Lmax, int mode, bool need_acc, bool with_w, int64_t B,
                           int64_t col_pad)
{
    Workspace w;
    memset(&w, 0, sizeof(w));
    const int ppq = planes_per_step(mode);
    // B products are stacked, each padded on its own; the sizes below are totals
    w.m_pad = B * round_up(M, kTileM);
    w.n_pad = B * round_up(N, col_pad);
    M *= B;
    N *= B;
    w.kw = (K + 31) / 32;
    // unipolar: the tensor-core core stores the positions in blocks (lengths rounded up to whole blocks); the planes are
    // sized so that either core family fits (two planes per position; the tensor-core core's W uses one of them)
    const int64_t l_alloc = mode == SC_UNIPOLAR_AND ? round_up(Lmax, kPosBlockSigned) : Lmax;
    w.a_planes = l_alloc * w.kw * ppq;
    w.w_planes = w.a_planes;
    const int64_t n_row_tiles = w.m_pad / kTileM;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    w.sigma_a = take(sizeof(float) * (size_t)M);
    w.sigma_w = take(with_w ? sizeof(float) * (size_t)N : 0);
    w.l_rows = take(sizeof(int32_t) * (size_t)M);
    w.perm = take(sizeof(int32_t) * (size_t)w.m_pad);
    w.l_sorted = take(sizeof(int32_t) * (size_t)w.m_pad);
    w.plan = take(sizeof(PlanHeader) + sizeof(int32_t) * (size_t)(2 * n_row_tiles + 2));
    w.acc = take(need_acc ? sizeof(int32_t) * (size_t)M * (size_t)(N / B) : 0);
    w.pop_a = take(sizeof(int32_t) * (size_t)M);
    w.pop_w = take(with_w ? sizeof(int32_t) * (size_t)(Lmax + 1) * (size_t)w.n_pad : 0);
    w.a_streams = take(sizeof(uint32_t) * (size_t)w.a_planes * (size_t)w.m_pad);
    w.w_streams = take(with_w ? sizeof(uint32_t) * (size_t)w.w_planes * (size_t)w.n_pad : 0);
    w.w_sign = take(with_w && mode == SC_UNIPOLAR_AND ? 4 * sizeof(uint32_t) * (size_t)w.kw * (size_t)w.n_pad : 0);
    w.a_sign = take(mode == SC_UNIPOLAR_AND ? 4 * sizeof(uint32_t) * (size_t)w.kw * (size_t)w.m_pad : 0);
    w.total = off;
    return w;
}

WeightsLayout layout_weights(int64_t K, int64_t N, int32_t Lmax, int mode)
{
    WeightsLayout w;
    memset(&w, 0, sizeof(w));
    w.n_pad = round_up(N, kColPad);
    w.kw = (K + 31) / 32;
    const int64_t l_alloc = mode == SC_UNIPOLAR_AND ? round_up(Lmax, kPosBlockSigned) : Lmax;
    w.w_planes = l_alloc * w.kw * planes_per_step(mode);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    w.sigma_w = take(sizeof(float) * (size_t)N);
    w.pop_w = take(sizeof(int32_t) * (size_t)(Lmax + 1) * (size_t)w.n_pad);
    w.w_streams = take(sizeof(uint32_t) * (size_t)w.w_planes * (size_t)w.n_pad);
    w.w_sign = take(mode == SC_UNIPOLAR_AND ? 4 * sizeof(uint32_t) * (size_t)w.kw * (size_t)w.n_pad : 0);
    w.total = off;
    return w;
}

// The GEMM core a call runs: the tensor-core core is the measured fastest; its fp32 accumulators are exact
// integers up to 2^24, so it needs K * Lmax <= 2^24.  Beyond that, and for explicit requests that do not fit,
// the carry-save ALU core runs.
static int pick_variant(const sc_params *p, int64_t K, int32_t Lmax)
{
    const bool umma_fits = (int64_t)K * Lmax <= (1LL << 24);
    int variant = p->core == SC_CORE_AUTO ? (umma_fits ? SC_CORE_UMMA : SC_CORE_CSA) : (int)p->core;
    if (variant == SC_CORE_UMMA_PAIR) variant = SC_CORE_UMMA;       // same family: one operand layout, two kernels
    if (variant == SC_CORE_UMMA && !umma_fits) variant = SC_CORE_CSA;
    return variant;
}

static bool params_ok(const sc_params *p)
{
    if (!p) return false;
    if (p->mode != SC_BIPOLAR_XNOR && p->mode != SC_UNIPOLAR_AND) return false;
    if (p->scale_a < SC_SCALE_NONE || p->scale_a > SC_SCALE_PER_TENSOR) return false;
    if (p->scale_w < SC_SCALE_NONE || p->scale_w > SC_SCALE_PER_TENSOR) return false;
    if (p->group < 1) return false;
    if (p->stream_id >= (1u << 31)) return false;
    if (p->core > SC_CORE_UMMA_PAIR) return false;
    if ((p->quant != SC_QUANT_DIRECT257 && p->quant != SC_QUANT_INT8_THEN_257) || p->reserved != 0) return false;
    return true;
}

// The tensor-core family has two kernels: one SM per tile, and pairs of SMs.  AUTO lets the plan choose from the lengths
// (device data), an explicit request fixes it; batched calls and calls with too many row tiles stay on single SMs.
struct PairLaunch {
    int mode;               // 0 never (the two-SM kernel is not enqueued), 1 the plan decides, 2 always
    int clusters;           // CTA pairs the two-SM kernel runs with
    int32_t col_tiles;      // its column tiles
};
static bool choose_pair(sc_ctx_impl *c, const sc_params *params, bool umma, int64_t m_pad, int64_t N, int64_t B, int64_t max_units,
                        PairLaunch *out)
{
    out->mode = 0;
    out->clusters = 0;
    out->col_tiles = (int32_t)((N + pair_core_tile_cols() - 1) / pair_core_tile_cols());
    if (!umma || B != 1 || m_pad / kTileM > pair_core_max_row_tiles() || params->core == SC_CORE_UMMA) return true;
    out->mode = params->core == SC_CORE_UMMA_PAIR ? 2 : 1;
    if (pair_core_clusters(params->mode, c->sm_count, &out->clusters) != cudaSuccess) return false;
    if (out->clusters < 1) out->mode = 0;
    if (out->mode == 1) {
        // The plan selects the two-SM core only if its tiling costs at most 50 % more MMA time than the one-SM core's (its
        // measured advantage on long pieces; shorter pieces tighten the condition).  Where the shape and Lmax alone already
        // rule that out (an odd row tile, a ragged last column tile, short streams: ragged lengths only add to it), the two-SM
        // kernel is not enqueued at all.
        const int64_t row_tiles = m_pad / kTileM, pairs = (row_tiles + 1) / 2;
        const int64_t t_pair = pairs * out->col_tiles * pair_core_tile_cols() * 2;
        const int64_t tile_n = umma_tile_cols(N);
        const int64_t t_single = row_tiles * ((N + tile_n - 1) / tile_n) * tile_n;
        // (max_units: stage units of the longest possible piece, from Lmax; shorter pieces only tighten the condition)
        if (t_pair * (max_units + kPairDrainUnits) * 100 > t_single * (max_units + kPieceChargeUnits) * kPairAdvantagePct) out->mode = 0;
    }
    return true;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// sigma of one operand into `sigma` (one entry per stream row)
// X is `batch` consecutive [rows x cols] tensors; the weight operand may be stored transposed ([cols x rows]).
static cudaError_t compute_scales(sc_ctx_impl *ctx, const float *X, int64_t rows, int64_t cols, int tensor_id,
                                  int scale, float *sigma, cudaStream_t st, int64_t batch = 1, int w_transposed = 0)
{
    int32_t *status = ctx->scratch + kSlotStatus;
    const int64_t stream_rows = (tensor_id == 0 ? rows : cols) * batch;
    int32_t *slot = ctx->scratch + (tensor_id == 0 ? kSlotTensorMaxA : kSlotTensorMaxW);
    if (scale == SC_SCALE_PER_ROW) {
        if (tensor_id == 0) return launch_row_absmax(X, rows * batch, cols, nullptr, sigma, status, st);
        if (w_transposed) return launch_row_absmax(X, cols * batch, rows, nullptr, sigma, status, st);
        return launch_col_absmax(X, rows, cols, sigma, status, st, batch);
    }
    // NONE still scans the tensor once so that non-finite inputs are reported
    cudaError_t e = launch_tensor_absmax(X, rows * cols * batch, slot, status, st);
    if (e != cudaSuccess) return e;
    return launch_fill_sigma(sigma, stream_rows, scale == SC_SCALE_PER_TENSOR ? slot : nullptr, st);
}

}  // namespace sc

using namespace sc;

extern "C" {

const char *sc_status_string(sc_status s)
{
    switch (s) {
        case SC_OK: return "ok";
        case SC_ERR_ARG: return "bad argument";
        case SC_ERR_SHAPE: return "bad shape";
        case SC_ERR_LENGTH: return "stream length out of range";
        case SC_ERR_NONFINITE: return "non-finite input";
        case SC_ERR_BUDGET: return "average budget below the minimum length";
        case SC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SC_ERR_CUDA: return "CUDA call failed";
        case SC_ERR_TIMEOUT: return "bounded device wait ran out";
    }
    return "unknown status";
}

sc_status sc_create(sc_ctx **ctx_out, int device)
{
    if (!ctx_out) return SC_ERR_ARG;
    *ctx_out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return SC_ERR_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return SC_ERR_CUDA;
    sc_ctx_impl *c = new (std::nothrow) sc_ctx_impl();
    if (!c) return SC_ERR_ARG;
    c->device = device;
    c->scratch = nullptr;
    c->profiling = false;
    c->profile_valid = false;
    if (cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaMalloc(&c->scratch, kScratchBytes) != cudaSuccess ||
        cudaMemset(c->scratch, 0, kScratchBytes) != cudaSuccess ||
        cudaEventCreate(&c->ev0) != cudaSuccess || cudaEventCreate(&c->ev1) != cudaSuccess) {
        if (c->scratch) cudaFree(c->scratch);
        delete c;
        return SC_ERR_CUDA;
    }
    for (int k = 0; k < SC_PROFILE_PHASES; ++k)
        if (cudaEventCreate(&c->phase_ev[k]) != cudaSuccess) { cudaFree(c->scratch); delete c; return SC_ERR_CUDA; }
    if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_plan, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_a_done, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_rows_done, cudaEventDisableTiming) != cudaSuccess) {
        cudaFree(c->scratch); delete c; return SC_ERR_CUDA;
    }
    c->overlap = true;
    *ctx_out = reinterpret_cast<sc_ctx *>(c);
    return SC_OK;
}

sc_status sc_destroy(sc_ctx *ctx)
{
    if (!ctx) return SC_ERR_ARG;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    cudaSetDevice(c->device);
    cudaEventDestroy(c->ev0);
    cudaEventDestroy(c->ev1);
    for (int k = 0; k < SC_PROFILE_PHASES; ++k) cudaEventDestroy(c->phase_ev[k]);
    cudaEventDestroy(c->ev_fork); cudaEventDestroy(c->ev_plan); cudaEventDestroy(c->ev_join);
    cudaEventDestroy(c->ev_a_done); cudaEventDestroy(c->ev_rows_done);
    cudaStreamDestroy(c->side);
    cudaFree(c->scratch);
    delete c;
    return SC_OK;
}

sc_status sc_device_status(sc_ctx *ctx, int32_t *code_host)
{
    if (!ctx || !code_host) return SC_ERR_ARG;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    if (cudaSetDevice(c->device) != cudaSuccess) return SC_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return SC_ERR_CUDA;
    int32_t code = 0;
    if (cudaMemcpy(&code, c->scratch + kSlotStatus, sizeof(code), cudaMemcpyDeviceToHost) != cudaSuccess)
        return SC_ERR_CUDA;
    if (cudaMemset(c->scratch + kSlotStatus, 0, sizeof(int32_t)) != cudaSuccess ||
        cudaMemset(c->scratch + kSlotTimeoutSite, 0, 3 * sizeof(int32_t)) != cudaSuccess)
        return SC_ERR_CUDA;
    *code_host = code;
    return SC_OK;
}

sc_status sc_row_stats(sc_ctx *ctx, const float *A, int64_t M, int64_t K, float *g, void *stream)
{
    if (!ctx || !A || !g) return SC_ERR_ARG;
    if (M <= 0 || K <= 0) return SC_ERR_SHAPE;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    cudaError_t e = launch_row_absmax(A, M, K, g, nullptr, c->scratch + kSlotStatus, (cudaStream_t)stream);
    return e == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

sc_status sc_assign_lengths(sc_ctx *ctx, const float *g, int64_t M, int32_t group, double avg_budget, int32_t Lmin,
                            int32_t Lmax, int32_t *L_out, double *realized_avg, void *stream)
{
    if (!ctx || !g || !L_out || group < 1 || !(avg_budget >= 0.0) || !isfinite(avg_budget)) return SC_ERR_ARG;
    if (M <= 0 || M >= (1LL << 31)) return SC_ERR_SHAPE;
    if (Lmin < 0 || Lmax < Lmin || Lmax > SC_L_CAP) return SC_ERR_LENGTH;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    cudaStream_t st = (cudaStream_t)stream;
    if (launch_assign_lengths(g, M, group, avg_budget, Lmin, Lmax, L_out, c->scratch, st) != cudaSuccess)
        return SC_ERR_CUDA;
    if (realized_avg) {
        long long total = 0;
        if (cudaMemcpyAsync(&total, c->scratch + kSlotRealizedTotal, sizeof(total), cudaMemcpyDeviceToHost, st) !=
                cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
            return SC_ERR_CUDA;
        *realized_avg = (double)total / (double)M;
    }
    return SC_OK;
}

sc_status sc_ladder_lengths(sc_ctx *ctx, const float *g, int64_t M, int32_t group, const int32_t *ladder,
                            const float *tau, int32_t levels, int32_t *L_out, void *stream)
{
    if (!ctx || !g || !L_out || !ladder || group < 1 || levels < 1 || levels > 64 || (levels > 1 && !tau))
        return SC_ERR_ARG;
    if (M <= 0 || M >= (1LL << 31)) return SC_ERR_SHAPE;
    for (int k = 0; k < levels; ++k)
        if (ladder[k] < 0 || ladder[k] > SC_L_CAP) return SC_ERR_LENGTH;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    return launch_ladder_lengths(g, M, group, ladder, tau, levels, L_out, c->scratch, (cudaStream_t)stream) ==
                   cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

size_t sc_stream_bytes(int64_t stream_rows, int64_t depth, int32_t Lmax, int32_t mode)
{
    if (stream_rows <= 0 || depth <= 0 || Lmax <= 0) return 0;
    const int64_t kw = (depth + 31) / 32;
    return sizeof(uint32_t) * (size_t)Lmax * (size_t)kw * (size_t)planes_per_step(mode) *
           (size_t)round_up(stream_rows, kTileM);
}

sc_status sc_encode(sc_ctx *ctx, const float *X, int64_t rows, int64_t cols, int32_t tensor_id,
                    const int32_t *L_or_null, int32_t Lmax, const sc_params *params, void *streams_out,
                    float *scales_out, void *stream)
{
    if (!ctx || !X || !streams_out || !scales_out || !params_ok(params) || (tensor_id != 0 && tensor_id != 1))
        return SC_ERR_ARG;
    if (!aligned16(streams_out)) return SC_ERR_ARG;
    if (rows <= 0 || cols <= 0 || rows >= (1LL << 24) || cols >= (1LL << 24)) return SC_ERR_SHAPE;
    if (Lmax < 1 || Lmax > SC_L_CAP) return SC_ERR_LENGTH;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    cudaStream_t st = (cudaStream_t)stream;
    const int scale = tensor_id == 0 ? params->scale_a : params->scale_w;
    if (compute_scales(c, X, rows, cols, tensor_id, scale, scales_out, st) != cudaSuccess) return SC_ERR_CUDA;
    EncodeArgs a;
    a.X = X; a.rows = rows; a.cols = cols; a.tensor_id = tensor_id; a.mode = params->mode;
    a.stream_rows = tensor_id == 0 ? rows : cols;
    a.depth = tensor_id == 0 ? cols : rows;
    a.kw = (a.depth + 31) / 32;
    a.r_pad = round_up(a.stream_rows, kTileM);
    a.perm = nullptr; a.l_sorted = L_or_null; a.lmax_actual = nullptr; a.Lmax = Lmax;
    a.sigma = scales_out; a.seed = params->seed; a.stream_id = params->stream_id;
    a.streams = static_cast<uint32_t *>(streams_out); a.status = c->scratch + kSlotStatus;
    a.reverse_bytes = 0;
    a.quant = params->quant;
    return launch_encode(a, st) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

sc_status sc_debug_unpack(sc_ctx *ctx, const void *streams, int64_t stream_rows, int64_t depth, int32_t Lmax,
                          int32_t mode, uint8_t *bits_out, uint8_t *neg_out, void *stream)
{
    if (!ctx || !streams || !bits_out) return SC_ERR_ARG;
    if (stream_rows <= 0 || depth <= 0 || Lmax < 1) return SC_ERR_SHAPE;
    return launch_unpack(static_cast<const uint32_t *>(streams), stream_rows, depth, Lmax, mode, bits_out, neg_out,
                         (cudaStream_t)stream) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

size_t sc_workspace_bytes(int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params)
{
    if (!params_ok(params) || M <= 0 || K <= 0 || N <= 0 || Lmax < 1 || Lmax > SC_L_CAP) return 0;
    return layout_workspace(M, K, N, Lmax, params->mode, true).total;
}

// Padding of the output columns of one product: a single product is padded for every core (prepared weights may be
// used by either family); stacked products only for the core that will run, which keeps narrow products small.
static int64_t batched_col_pad(const sc_params *p, int64_t K, int32_t Lmax, int64_t B, int64_t N)
{
    if (B <= 1) return kColPad;
    if (pick_variant(p, K, Lmax) != SC_CORE_UMMA) return kTileN;
    // the tensor-core core's own tiles: its column tile follows N (umma_tile_cols), and a product takes exactly its tiles
    const int64_t tile_n = umma_tile_cols(N);
    return (N + tile_n - 1) / tile_n * tile_n;
}

// Shared body of sc_matmul (W given, everything derived per call) and sc_matmul_prepared (pw given).
// and of sc_matmul_batched (B products stacked along the rows of A and the columns of W; M, N per product).
static sc_status matmul_impl(sc_ctx *ctx, const float *A, const float *W, const sc_weights_impl *pw, int64_t M,
                             int64_t K, int64_t N, const int32_t *L, int32_t Lmax, const sc_params *params,
                             int32_t *P, float *C, void *ws, size_t ws_bytes, void *stream, int64_t B = 1,
                             int w_transposed = 0)
{
    if (!ctx || !A || (!W && !pw) || !C || !params_ok(params)) return SC_ERR_ARG;
    if (B < 1 || B > 65535 || (pw && (B != 1 || w_transposed))) return SC_ERR_ARG;
    if (M <= 0 || K <= 0 || N <= 0 || K > (1LL << 20)) return SC_ERR_SHAPE;
    if (B * round_up(M, kTileM) >= (1LL << 24) || B * round_up(N, kColPad) >= (1LL << 24)) return SC_ERR_SHAPE;
    if (Lmax < 1 || Lmax > SC_L_CAP || (int64_t)K * Lmax >= (1LL << 30)) return SC_ERR_LENGTH;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return SC_ERR_WORKSPACE;
    const int64_t col_pad = batched_col_pad(params, K, Lmax, B, N);
    const Workspace w = layout_workspace(M, K, N, Lmax, params->mode, P == nullptr, pw == nullptr, B, col_pad);
    if (ws_bytes < w.total) return SC_ERR_WORKSPACE;
    if (params->core == SC_CORE_SIMPLE && (B == 1 ? M : w.m_pad) > 65535) return SC_ERR_SHAPE;
    const int64_t m_pad_b = round_up(M, kTileM), n_pad_b = round_up(N, col_pad);   // per product
    const int64_t Mt = B * M;                                                      // stacked rows

    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    // the core follows the layout the weights were prepared for
    int variant = pick_variant(params, K, Lmax);
    if (pw) {
        if (pw->umma) variant = SC_CORE_UMMA;                      // fits: Lmax <= the prepared Lmax
        else if (variant == SC_CORE_UMMA) variant = SC_CORE_CSA;
    }
    const bool umma = variant == SC_CORE_UMMA;

    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *base = static_cast<uint8_t *>(ws);
    float *sigma_a = reinterpret_cast<float *>(base + w.sigma_a);
    float *sigma_w_ws = reinterpret_cast<float *>(base + w.sigma_w);
    const float *sigma_w = pw ? pw->sigma_w : sigma_w_ws;
    int32_t *l_rows = reinterpret_cast<int32_t *>(base + w.l_rows);
    int32_t *perm = reinterpret_cast<int32_t *>(base + w.perm);
    int32_t *l_sorted = reinterpret_cast<int32_t *>(base + w.l_sorted);
    PlanHeader *plan = reinterpret_cast<PlanHeader *>(base + w.plan);
    int32_t *acc = P ? P : reinterpret_cast<int32_t *>(base + w.acc);
    uint32_t *a_streams = reinterpret_cast<uint32_t *>(base + w.a_streams);
    uint32_t *w_streams_ws = reinterpret_cast<uint32_t *>(base + w.w_streams);
    const uint32_t *w_streams = pw ? pw->w_streams : w_streams_ws;
    int32_t *pop_w_ws = reinterpret_cast<int32_t *>(base + w.pop_w);
    const int32_t *pop_w = pw ? pw->pop_w : pop_w_ws;
    const int ppq_alloc = planes_per_step(params->mode);                 // planes per position the buffers are sized for
    const int ppq = planes_per_step_for(params->mode, umma);             // ... and as written for the core that runs
    const int pos_block = pos_block_for(params->mode, umma);
    uint32_t *w_sign_ws = reinterpret_cast<uint32_t *>(base + w.w_sign);
    const uint32_t *w_sign = pw ? pw->w_sign : w_sign_ws;
    uint32_t *a_sign = reinterpret_cast<uint32_t *>(base + w.a_sign);
    const bool signs = umma && params->mode == SC_UNIPOLAR_AND;
    PairLaunch pair;
    const int64_t l_round = params->mode == SC_UNIPOLAR_AND ? round_up(Lmax, kPosBlockSigned) : Lmax;
    if (!choose_pair(c, params, umma, w.m_pad, N, B, (l_round * w.kw + kStagePlanes - 1) / kStagePlanes, &pair)) return SC_ERR_CUDA;
    const int pair_mode = pair.mode, pair_clusters = pair.clusters;
    const int32_t pair_col_tiles = pair.col_tiles;

    auto mark = [&](int k) { if (c->profiling) cudaEventRecord(c->phase_ev[k], st); };
    c->profile_valid = false;
    // The W-side work (scales, encode, popcount tables) does not depend on the A side except for the longest length of
    // the call, which the plan writes: it runs on the context's side stream, forked from and joined back into the caller's
    // stream by events (valid under stream capture as well), and the plan then goes first so that the side stream does
    // not wait for it.  With phase timing on, everything stays on the caller's stream in the order of the phases.
    const bool fork = !pw && c->overlap && !c->profiling;
    cudaStream_t sw = fork ? c->side : st;          // the stream of the W-side work
    const int32_t tile_n = umma_tile_cols(N);                        // column tile of the one-SM tensor-core core
    const int64_t n_col_tiles = umma ? (N + tile_n - 1) / tile_n : (N + kTileN - 1) / kTileN;
    // a1: scales (the per-row scale of A is also the row metric of Sec. 4.4)
    auto scales = [&]() -> bool {
        if (!fork && compute_scales(c, A, M, K, 0, params->scale_a, sigma_a, st, B) != cudaSuccess) return false;
        if (fork && (cudaEventRecord(c->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(c->side, c->ev_fork, 0) != cudaSuccess))
            return false;
        if (!pw && compute_scales(c, W, K, N, 1, params->scale_w, sigma_w_ws, sw, B, w_transposed) != cudaSuccess) return false;
        return true;
    };
    // a3: row ordering by length and the work list
    auto plan_rows = [&]() -> bool {
        if (launch_plan(L, M, params->group, Lmax, w.kw, ppq, m_pad_b, n_col_tiles, umma ? 0 : c->sm_count * 16,
                        umma ? c->sm_count : 0, l_rows, perm, l_sorted, plan, c->scratch, st, B, pos_block, pair_col_tiles,
                        pair_mode ? pair_clusters : 0, pair_mode == 2, tile_n) != cudaSuccess)
            return false;
        // the W encode stops at the longest length of the call
        if (fork && (cudaEventRecord(c->ev_plan, st) != cudaSuccess || cudaStreamWaitEvent(c->side, c->ev_plan, 0) != cudaSuccess))
            return false;
        return cudaMemsetAsync(acc, 0, sizeof(int32_t) * (size_t)Mt * (size_t)N, st) == cudaSuccess;
    };
    mark(0);
    if (fork) {
        if (!scales() || !plan_rows()) return SC_ERR_CUDA;
        if (compute_scales(c, A, M, K, 0, params->scale_a, sigma_a, st, B) != cudaSuccess) return SC_ERR_CUDA;
    } else {
        if (!scales()) return SC_ERR_CUDA;
        mark(1);
        if (!plan_rows()) return SC_ERR_CUDA;
    }

    mark(2);
    // a4: encode both operands (A in sorted row order)
    EncodeArgs ea;
    ea.X = A; ea.rows = Mt; ea.cols = K; ea.tensor_id = 0; ea.mode = params->mode;
    ea.stream_rows = Mt; ea.depth = K; ea.kw = w.kw; ea.r_pad = w.m_pad;
    ea.perm = perm; ea.l_sorted = l_sorted; ea.lmax_actual = c->scratch + kSlotLmaxActual; ea.Lmax = Lmax;
    ea.sigma = sigma_a; ea.seed = params->seed; ea.stream_id = params->stream_id;
    ea.streams = a_streams; ea.status = c->scratch + kSlotStatus; ea.reverse_bytes = 0;
    ea.quant = params->quant;
    ea.pos_block = pos_block;
    ea.signs = signs ? a_sign : nullptr;
    if (launch_encode(ea, st) != cudaSuccess) return SC_ERR_CUDA;
    mark(3);
    const bool and_form = umma && params->mode == SC_BIPOLAR_XNOR;    // AND counts + popcount corrections
    if (!pw) {
        EncodeArgs ew = ea;
        ew.X = W; ew.rows = w_transposed ? N : K; ew.cols = w_transposed ? K : N; ew.tensor_id = 1;
        ew.stream_rows = B * N; ew.depth = K; ew.r_pad = w.n_pad;
        ew.w_transposed = w_transposed;
        if (B > 1) { ew.batch_pad = n_pad_b; ew.batch_real = N; }
        ew.perm = nullptr; ew.l_sorted = nullptr; ew.sigma = sigma_w_ws; ew.streams = w_streams_ws;
        ew.reverse_bytes = umma ? 1 : 0;
        ew.signs = signs ? w_sign_ws : nullptr;
        if (launch_encode(ew, sw) != cudaSuccess) return SC_ERR_CUDA;
        if (and_form && launch_col_corrections(w_streams_ws, w.n_pad, (int32_t)w.kw, Lmax,
                                               c->scratch + kSlotLmaxActual, pop_w_ws, sw) != cudaSuccess)
            return SC_ERR_CUDA;
        if (fork && (cudaEventRecord(c->ev_join, c->side) != cudaSuccess || cudaStreamWaitEvent(st, c->ev_join, 0) != cudaSuccess))
            return SC_ERR_CUDA;
    }

    // a5-a7: gate + popcount accumulation
    CoreArgs ca;
    ca.a_streams = a_streams; ca.w_streams = w_streams;
    ca.m_pad = w.m_pad; ca.n_pad = w.n_pad;
    ca.a_planes = w.a_planes / ppq_alloc * ppq;                          // planes the operands really have
    ca.w_planes = w.w_planes / ppq_alloc * ppq;
    ca.w_sign = signs ? w_sign : nullptr; ca.a_sign = signs ? a_sign : nullptr; ca.pos_block = pos_block;
    ca.tile_n = tile_n;
    ca.M = Mt; ca.N = N; ca.mode = params->mode;
    ca.tiles_m = (int32_t)(m_pad_b / kTileM); ca.w_batch_cols = n_pad_b;
    ca.variant = variant;
    ca.perm = perm; ca.l_sorted = l_sorted; ca.plan = plan; ca.kw = (int32_t)w.kw; ca.ppq = ppq;
    ca.acc = acc; ca.scratch = c->scratch; ca.sm_count = c->sm_count; ca.Lmax = Lmax;
    ca.pop_a = reinterpret_cast<int32_t *>(base + w.pop_a);
    ca.pop_w = pop_w;
    // The row popcounts of A feed the decode only: they run on the side stream beside the core (their small CTAs fit on
    // the SMs next to the core's one CTA each), forked after the encode of A and joined before the decode.
    const bool fork_rows = and_form && c->overlap && !c->profiling;
    if (fork_rows) {
        if (cudaEventRecord(c->ev_a_done, st) != cudaSuccess || cudaStreamWaitEvent(c->side, c->ev_a_done, 0) != cudaSuccess ||
            launch_row_corrections(ca, c->side) != cudaSuccess || cudaEventRecord(c->ev_rows_done, c->side) != cudaSuccess)
            return SC_ERR_CUDA;
    } else if (and_form && launch_row_corrections(ca, st) != cudaSuccess) {
        return SC_ERR_CUDA;                                                              // counted with the W encode phase
    }
    mark(4);
    if (umma) {
        // both kernels are enqueued; the one the plan did not select returns at once
        if (launch_core_umma(ca, st) != cudaSuccess) return SC_ERR_CUDA;
        if (pair_mode && launch_core_umma_pair(ca, pair_clusters, pair_mode == 2, st) != cudaSuccess) return SC_ERR_CUDA;
    } else if (launch_core(ca, st) != cudaSuccess) {
        return SC_ERR_CUDA;
    }

    mark(5);
    if (fork_rows && cudaStreamWaitEvent(st, c->ev_rows_done, 0) != cudaSuccess) return SC_ERR_CUDA;
    // a8: decode
    if (and_form) {
        if (launch_decode_and(acc, Mt, N, K, w.n_pad, l_rows, ca.pop_a, ca.pop_w, sigma_a, sigma_w, P, C, st, M,
                              n_pad_b) != cudaSuccess)
            return SC_ERR_CUDA;
    } else if (launch_decode(params->mode, acc, Mt, N, K, l_rows, sigma_a, sigma_w, P, C, st, M) != cudaSuccess) {
        return SC_ERR_CUDA;
    }
    mark(6);
    c->profile_valid = c->profiling;
    return SC_OK;
}

sc_status sc_matmul(sc_ctx *ctx, const float *A, const float *W, int64_t M, int64_t K, int64_t N, const int32_t *L,
                    int32_t Lmax, const sc_params *params, int32_t *P, float *C, void *ws, size_t ws_bytes,
                    void *stream)
{
    if (!W) return SC_ERR_ARG;
    return matmul_impl(ctx, A, W, nullptr, M, K, N, L, Lmax, params, P, C, ws, ws_bytes, stream);
}

size_t sc_workspace_bytes_batched(int64_t B, int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params)
{
    if (!params_ok(params) || B < 1 || B > 65535 || M <= 0 || K <= 0 || N <= 0 || Lmax < 1 || Lmax > SC_L_CAP) return 0;
    return layout_workspace(M, K, N, Lmax, params->mode, true, true, B, batched_col_pad(params, K, Lmax, B, N)).total;
}

sc_status sc_matmul_batched(sc_ctx *ctx, const float *A, const float *W, int64_t B, int64_t M, int64_t K, int64_t N,
                            int32_t w_transposed, const int32_t *L, int32_t Lmax, const sc_params *params, int32_t *P,
                            float *C, void *ws, size_t ws_bytes, void *stream)
{
    if (!W || (w_transposed != 0 && w_transposed != 1)) return SC_ERR_ARG;
    return matmul_impl(ctx, A, W, nullptr, M, K, N, L, Lmax, params, P, C, ws, ws_bytes, stream, B, w_transposed);
}

// ---- the paper's own generator: Sobol-8 streams with conditional bitstream generation --------------------
static bool cbsg_args_ok(const sc_params *p, int64_t M, int64_t K, int64_t N)
{
    if (!params_ok(p) || p->mode != SC_BIPOLAR_XNOR) return false;
    if (p->core != SC_CORE_AUTO && p->core != SC_CORE_UMMA && p->core != SC_CORE_UMMA_PAIR) return false;
    return M > 0 && K > 0 && N > 0;
}

size_t sc_workspace_bytes_cbsg(int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params)
{
    if (!cbsg_args_ok(params, M, K, N) || Lmax < 1 || Lmax > 256 || K * 2 * Lmax > (1LL << 24)) return 0;
    return align_up(layout_workspace(M, K, N, 2 * Lmax, SC_BIPOLAR_XNOR, true).total, 256) + align_up(kCbsgTableBytes, 256);
}

sc_status sc_matmul_cbsg(sc_ctx *ctx, const float *A, const float *W, int64_t M, int64_t K, int64_t N, const int32_t *L,
                         int32_t Lmax, const sc_params *params, int32_t *P, float *C, void *ws, size_t ws_bytes,
                         void *stream)
{
    if (!ctx || !A || !W || !C || !cbsg_args_ok(params, M, K, N)) return SC_ERR_ARG;
    if (M >= (1LL << 24) || N >= (1LL << 24)) return SC_ERR_SHAPE;
    if (Lmax < 1 || Lmax > 256) return SC_ERR_LENGTH;                   // one period of the 8-bit sequences
    const int32_t core_lmax = 2 * Lmax;                                 // code positions of the longest row
    if (K * core_lmax > (1LL << 24)) return SC_ERR_SHAPE;               // int32 headroom of the tensor-core accumulators
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return SC_ERR_WORKSPACE;
    const Workspace w = layout_workspace(M, K, N, core_lmax, SC_BIPOLAR_XNOR, P == nullptr);
    const size_t tables_at = align_up(w.total, 256);                    // the code tables follow the usual regions
    if (ws_bytes < tables_at + align_up(kCbsgTableBytes, 256)) return SC_ERR_WORKSPACE;

    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *base = static_cast<uint8_t *>(ws);
    float *sigma_a = reinterpret_cast<float *>(base + w.sigma_a);
    float *sigma_w = reinterpret_cast<float *>(base + w.sigma_w);
    int32_t *l_rows = reinterpret_cast<int32_t *>(base + w.l_rows);
    int32_t *perm = reinterpret_cast<int32_t *>(base + w.perm);
    int32_t *l_sorted = reinterpret_cast<int32_t *>(base + w.l_sorted);
    PlanHeader *plan = reinterpret_cast<PlanHeader *>(base + w.plan);
    int32_t *acc = P ? P : reinterpret_cast<int32_t *>(base + w.acc);
    uint32_t *a_streams = reinterpret_cast<uint32_t *>(base + w.a_streams);
    uint32_t *w_streams = reinterpret_cast<uint32_t *>(base + w.w_streams);
    // the row popcounts of the Philox path are not needed here: their space holds the core lengths (<= M entries)
    int32_t *l_core = reinterpret_cast<int32_t *>(base + w.pop_a);
    uint32_t *tables = reinterpret_cast<uint32_t *>(base + tables_at);
    int32_t *status = c->scratch + kSlotStatus;
    const int64_t n_groups = (M + params->group - 1) / params->group;

    auto mark = [&](int k) { if (c->profiling) cudaEventRecord(c->phase_ev[k], st); };
    c->profile_valid = false;
    mark(0);
    if (compute_scales(c, A, M, K, 0, params->scale_a, sigma_a, st) != cudaSuccess) return SC_ERR_CUDA;
    if (compute_scales(c, W, K, N, 1, params->scale_w, sigma_w, st) != cudaSuccess) return SC_ERR_CUDA;
    mark(1);
    if (launch_cbsg_setup(params->seed, params->stream_id, tables, L, n_groups, Lmax, l_core, status, st) != cudaSuccess)
        return SC_ERR_CUDA;
    const int32_t tile_n = umma_tile_cols(N);
    const int64_t n_col_tiles = (N + tile_n - 1) / tile_n;
    PairLaunch pair;
    if (!choose_pair(c, params, true, w.m_pad, N, 1, ((int64_t)core_lmax * w.kw + kStagePlanes - 1) / kStagePlanes, &pair)) return SC_ERR_CUDA;
    if (launch_plan(l_core, M, params->group, core_lmax, w.kw, 1, w.m_pad, n_col_tiles, 0, c->sm_count, l_rows,
                    perm, l_sorted, plan, c->scratch, st, 1, 1, pair.col_tiles, pair.mode ? pair.clusters : 0,
                    pair.mode == 2, tile_n) != cudaSuccess)
        return SC_ERR_CUDA;
    if (cudaMemsetAsync(acc, 0, sizeof(int32_t) * (size_t)M * (size_t)N, st) != cudaSuccess) return SC_ERR_CUDA;
    mark(2);
    if (launch_cbsg_encode(A, M, K, 0, w.m_pad, perm, l_sorted, c->scratch + kSlotLmaxActual, L, params->group, Lmax,
                           sigma_a, tables, a_streams, 0, status, st, params->quant) != cudaSuccess)
        return SC_ERR_CUDA;
    mark(3);
    if (launch_cbsg_encode(W, K, N, 1, w.n_pad, nullptr, nullptr, c->scratch + kSlotLmaxActual, nullptr, 1, Lmax,
                           sigma_w, tables, w_streams, 1, status, st, params->quant) != cudaSuccess)
        return SC_ERR_CUDA;
    mark(4);
    CoreArgs ca;
    ca.a_streams = a_streams; ca.w_streams = w_streams;
    ca.m_pad = w.m_pad; ca.n_pad = w.n_pad; ca.a_planes = w.a_planes; ca.w_planes = w.w_planes;
    ca.M = M; ca.N = N; ca.mode = SC_BIPOLAR_XNOR; ca.variant = SC_CORE_UMMA;
    ca.tiles_m = (int32_t)(w.m_pad / kTileM); ca.w_batch_cols = w.n_pad;
    ca.perm = perm; ca.l_sorted = l_sorted; ca.plan = plan; ca.kw = (int32_t)w.kw; ca.ppq = 1;
    ca.acc = acc; ca.scratch = c->scratch; ca.sm_count = c->sm_count; ca.Lmax = core_lmax;
    ca.pop_a = nullptr; ca.pop_w = nullptr;
    ca.tile_n = tile_n;
    if (launch_core_umma(ca, st) != cudaSuccess) return SC_ERR_CUDA;
    if (pair.mode && launch_core_umma_pair(ca, pair.clusters, pair.mode == 2, st) != cudaSuccess) return SC_ERR_CUDA;
    mark(5);
    if (launch_cbsg_decode(acc, M, N, K, L, params->group, Lmax, sigma_a, sigma_w, P, C, st) != cudaSuccess)
        return SC_ERR_CUDA;
    mark(6);
    c->profile_valid = c->profiling;
    return SC_OK;
}

sc_status sc_cbsg_scc(sc_ctx *ctx, const int32_t *Ta, const int32_t *Tw, int64_t n, int32_t L, uint64_t seed,
                      uint32_t stream_id, int32_t *counts, double *scc, void *ws, size_t ws_bytes, void *stream)
{
    if (!ctx || !Ta || !Tw || !scc || n <= 0 || stream_id >= (1u << 31)) return SC_ERR_ARG;
    if (L < 0 || L > 256) return SC_ERR_LENGTH;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 || ws_bytes < align_up(kCbsgTableBytes, 256) + 256)
        return SC_ERR_WORKSPACE;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    cudaStream_t st = (cudaStream_t)stream;
    uint32_t *tables = static_cast<uint32_t *>(ws);
    int32_t *dummy = reinterpret_cast<int32_t *>(static_cast<uint8_t *>(ws) + align_up(kCbsgTableBytes, 256));
    if (launch_cbsg_setup(seed, stream_id, tables, nullptr, 1, 1, dummy, c->scratch + kSlotStatus, st) != cudaSuccess)
        return SC_ERR_CUDA;
    return launch_cbsg_scc(tables, Ta, Tw, n, L, counts, scc, c->scratch + kSlotStatus, st) == cudaSuccess ? SC_OK
                                                                                                         : SC_ERR_CUDA;
}

size_t sc_weights_bytes(int64_t K, int64_t N, int32_t Lmax, const sc_params *params)
{
    if (!params_ok(params) || K <= 0 || N <= 0 || Lmax < 1 || Lmax > SC_L_CAP) return 0;
    return layout_weights(K, N, Lmax, params->mode).total;
}

sc_status sc_weights_prepare(sc_ctx *ctx, const float *W, int64_t K, int64_t N, int32_t Lmax, const sc_params *params,
                             void *wbuf, size_t wbuf_bytes, void *stream, sc_weights **out)
{
    if (out) *out = nullptr;
    if (!ctx || !W || !out || !params_ok(params)) return SC_ERR_ARG;
    if (K <= 0 || N <= 0 || N >= (1LL << 24) || K > (1LL << 20)) return SC_ERR_SHAPE;
    if (Lmax < 1 || Lmax > SC_L_CAP || (int64_t)K * Lmax >= (1LL << 30)) return SC_ERR_LENGTH;
    if (!wbuf || (reinterpret_cast<uintptr_t>(wbuf) & 255u) != 0) return SC_ERR_WORKSPACE;
    const WeightsLayout wl = layout_weights(K, N, Lmax, params->mode);
    if (wbuf_bytes < wl.total) return SC_ERR_WORKSPACE;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t *base = static_cast<uint8_t *>(wbuf);
    float *sigma_w = reinterpret_cast<float *>(base + wl.sigma_w);
    int32_t *pop_w = reinterpret_cast<int32_t *>(base + wl.pop_w);
    uint32_t *w_streams = reinterpret_cast<uint32_t *>(base + wl.w_streams);
    const bool umma = pick_variant(params, K, Lmax) == SC_CORE_UMMA;
    const bool and_form = umma && params->mode == SC_BIPOLAR_XNOR;

    if (compute_scales(c, W, K, N, 1, params->scale_w, sigma_w, st) != cudaSuccess) return SC_ERR_CUDA;
    EncodeArgs ew;
    ew.X = W; ew.rows = K; ew.cols = N; ew.tensor_id = 1; ew.mode = params->mode;
    ew.stream_rows = N; ew.depth = K; ew.kw = wl.kw; ew.r_pad = wl.n_pad;
    ew.perm = nullptr; ew.l_sorted = nullptr; ew.lmax_actual = nullptr; ew.Lmax = Lmax;
    ew.sigma = sigma_w; ew.seed = params->seed; ew.stream_id = params->stream_id;
    ew.streams = w_streams; ew.status = c->scratch + kSlotStatus; ew.reverse_bytes = umma ? 1 : 0;
    ew.quant = params->quant;
    ew.pos_block = pos_block_for(params->mode, umma);
    uint32_t *w_sign = reinterpret_cast<uint32_t *>(base + wl.w_sign);
    const bool signs = umma && params->mode == SC_UNIPOLAR_AND;
    ew.signs = signs ? w_sign : nullptr;
    if (launch_encode(ew, st) != cudaSuccess) return SC_ERR_CUDA;
    if (and_form && launch_col_corrections(w_streams, wl.n_pad, (int32_t)wl.kw, Lmax, nullptr, pop_w, st) != cudaSuccess)
        return SC_ERR_CUDA;

    sc_weights_impl *h = new (std::nothrow) sc_weights_impl();
    if (!h) return SC_ERR_ARG;
    h->magic = kWeightsMagic;
    h->device = c->device;
    h->K = K; h->N = N; h->Lmax = Lmax;
    h->mode = params->mode; h->scale_w = params->scale_w; h->quant = params->quant;
    h->seed = params->seed; h->stream_id = params->stream_id;
    h->umma = umma;
    h->sigma_w = sigma_w;
    h->pop_w = and_form ? pop_w : nullptr;
    h->w_streams = w_streams;
    h->w_sign = signs ? w_sign : nullptr;
    *out = reinterpret_cast<sc_weights *>(h);
    return SC_OK;
}

sc_status sc_weights_release(sc_weights *weights)
{
    sc_weights_impl *h = reinterpret_cast<sc_weights_impl *>(weights);
    if (!h || h->magic != kWeightsMagic) return SC_ERR_ARG;
    h->magic = 0;
    delete h;
    return SC_OK;
}

size_t sc_workspace_bytes_prepared(int64_t M, int64_t K, int64_t N, int32_t Lmax, const sc_params *params)
{
    if (!params_ok(params) || M <= 0 || K <= 0 || N <= 0 || Lmax < 1 || Lmax > SC_L_CAP) return 0;
    return layout_workspace(M, K, N, Lmax, params->mode, true, false).total;
}

sc_status sc_matmul_prepared(sc_ctx *ctx, const float *A, const sc_weights *weights, int64_t M, const int32_t *L,
                             int32_t Lmax, const sc_params *params, int32_t *P, float *C, void *ws, size_t ws_bytes,
                             void *stream)
{
    const sc_weights_impl *h = reinterpret_cast<const sc_weights_impl *>(weights);
    if (!ctx || !h || h->magic != kWeightsMagic || !params_ok(params)) return SC_ERR_ARG;
    if (h->device != reinterpret_cast<sc_ctx_impl *>(ctx)->device) return SC_ERR_ARG;
    if (params->mode != h->mode || params->scale_w != h->scale_w || params->quant != h->quant || params->seed != h->seed ||
        params->stream_id != h->stream_id)
        return SC_ERR_ARG;
    if (Lmax > h->Lmax) return SC_ERR_LENGTH;
    // an explicit request for a core the buffer was not laid out for cannot be served
    if (params->core != SC_CORE_AUTO && (params->core == SC_CORE_UMMA || params->core == SC_CORE_UMMA_PAIR) != h->umma) return SC_ERR_ARG;
    return matmul_impl(ctx, A, nullptr, h, M, h->K, h->N, L, Lmax, params, P, C, ws, ws_bytes, stream);
}

sc_status sc_surrogate_noise(sc_ctx *ctx, const float *Y, int64_t M, int64_t N, const int32_t *L, int32_t group,
                             double coeff, uint64_t seed, uint32_t stream_id, float *out, void *stream)
{
    if (!ctx || !Y || !out || group < 1 || !(coeff >= 0.0) || !isfinite(coeff) || stream_id >= (1u << 31)) return SC_ERR_ARG;
    if (M <= 0 || N <= 0 || M >= (1LL << 31) || N >= (1LL << 31)) return SC_ERR_SHAPE;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    return launch_surrogate(Y, M, N, L, group, coeff, seed, stream_id, out, c->scratch + kSlotStatus,
                            (cudaStream_t)stream) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

sc_status sc_profile_enable(sc_ctx *ctx, int32_t on)
{
    if (!ctx) return SC_ERR_ARG;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    c->profiling = on != 0;
    c->profile_valid = false;
    return SC_OK;
}

sc_status sc_profile_read(sc_ctx *ctx, float *ms_out)
{
    if (!ctx || !ms_out) return SC_ERR_ARG;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    for (int k = 0; k < SC_PROFILE_PHASES; ++k) ms_out[k] = 0.0f;
    if (!c->profile_valid) return SC_ERR_ARG;
    if (cudaEventSynchronize(c->phase_ev[6]) != cudaSuccess) return SC_ERR_CUDA;
    for (int k = 0; k < 6; ++k)
        if (cudaEventElapsedTime(&ms_out[k], c->phase_ev[k], c->phase_ev[k + 1]) != cudaSuccess) return SC_ERR_CUDA;
    if (cudaEventElapsedTime(&ms_out[6], c->phase_ev[0], c->phase_ev[6]) != cudaSuccess) return SC_ERR_CUDA;
    return SC_OK;
}

sc_status sc_launch_count(sc_ctx *ctx, int64_t *count_host)
{
    if (!ctx || !count_host) return SC_ERR_ARG;
    *count_host = (int64_t)launches_so_far();
    return SC_OK;
}

sc_status sc_last_core_selected(sc_ctx *ctx, int32_t *pair_host)
{
    if (!ctx || !pair_host) return SC_ERR_ARG;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    if (cudaDeviceSynchronize() != cudaSuccess) return SC_ERR_CUDA;
    if (cudaMemcpy(pair_host, c->scratch + kSlotPairSelected, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) return SC_ERR_CUDA;
    return SC_OK;
}

int32_t sc_selftest_comparator(void)
{
    int32_t mismatches = 0;
    for (int32_t T = 0; T <= 256; ++T) {
        // 256 draws packed 32 per word: draw value r sits in word r / 32, bit r % 32
        for (int wblk = 0; wblk < 8; ++wblk) {
            uint32_t planes[8];
            for (int k = 0; k < 8; ++k) {
                planes[k] = 0u;
                for (int b = 0; b < 32; ++b) planes[k] |= (uint32_t)(((wblk * 32 + b) >> k) & 1) << b;
            }
            const uint32_t got = draws_below(planes, T);
            for (int b = 0; b < 32; ++b)
                if (((got >> b) & 1u) != (uint32_t)((wblk * 32 + b) < T ? 1 : 0)) ++mismatches;
        }
    }
    return mismatches;
}

// value of an e2m1 nibble (sign, two exponent bits, one mantissa bit)
static double e2m1_value(uint32_t nib)
{
    static const double mag[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};
    return (nib & 8u) ? -mag[nib & 7u] : mag[nib & 7u];
}
// sum over the 32 nibble positions of the products of two expanded operands (4 words each)
static double expanded_dot(const uint32_t a[4], const uint32_t w[4])
{
    double s = 0.0;
    for (int m = 0; m < 4; ++m)
        for (int j = 0; j < 8; ++j) s += e2m1_value((a[m] >> (4 * j)) & 15u) * e2m1_value((w[m] >> (4 * j)) & 15u);
    return s;
}

int32_t sc_selftest_expansion(void)
{
    int32_t mismatches = 0;
    uint32_t rng = 0x9E3779B9u;
    auto next = [&]() { rng ^= rng << 13; rng ^= rng >> 17; rng ^= rng << 5; return rng; };
    // 32 x 32 single-element pairs, then dense random words
    for (int trial = 0; trial < 32 * 32 + 4096; ++trial) {
        uint32_t za, zw, sa, sw;          // stream bits and sign bits of the 32 depth elements (bit e = element e)
        if (trial < 32 * 32) { za = 1u << (trial / 32); zw = 1u << (trial % 32); sa = (trial & 1) ? za : 0u; sw = (trial & 2) ? zw : 0u; }
        else { za = next(); zw = next(); sa = next(); sw = next(); }
        // bipolar: the activation plane word is za itself; the weight plane word holds element w_bit_element(b) at bit b
        uint32_t w_plane = 0u;
        for (int b = 0; b < 32; ++b) w_plane |= ((zw >> w_bit_element(b)) & 1u) << b;
        uint32_t ea[4], ew[4];
        u_expand_bits<false>(za, ea);
        u_expand_bits<true>(w_plane, ew);
        if (expanded_dot(ea, ew) != (double)__builtin_popcount(za & zw)) ++mismatches;
        // unipolar: magnitude planes (the weight's in reversed order) with the nibble sign words of the elements' signs;
        // signs count only where both stream bits are set
        uint32_t w_sign = 0u;
        for (int b = 0; b < 32; ++b) w_sign |= ((sw >> w_bit_element(b)) & 1u) << b;
        uint32_t sn_a[4], sn_w[4];
        sign_nibble_words(sa, false, sn_a);
        sign_nibble_words(w_sign, true, sn_w);
        u_expand_signed<false>(za, sn_a, ea);
        u_expand_signed<true>(w_plane, sn_w, ew);
        int32_t expect = 0;
        for (int e = 0; e < 32; ++e)
            if ((za >> e) & (zw >> e) & 1u) expect += (((sa >> e) ^ (sw >> e)) & 1u) ? -1 : 1;
        if (expanded_dot(ea, ew) != (double)expect) ++mismatches;
        if ((za & sa) == 0u) {             // the unsigned rule for activations without a negative stream bit
            u_expand_bits<false>(za, ea);
            if (expanded_dot(ea, ew) != (double)expect) ++mismatches;
        }
        // position blocks: every (position, depth word) pair of a stream of 21 positions x 5 depth words gets its own plane
        if (trial == 0) {
            bool seen[24 * 5] = {false};
            for (int l = 0; l < 21; ++l)
                for (int w = 0; w < 5; ++w) {
                    const int64_t pi = plane_index(l, w, 5, kPosBlockSigned);
                    if (pi < 0 || pi >= 24 * 5 || seen[pi]) ++mismatches; else seen[pi] = true;
                    if (plane_index(l, w, 5, 1) != (int64_t)l * 5 + w) ++mismatches;
                    if (plane_index_pow2(l, w, 5, 3) != pi || plane_index_pow2(l, w, 5, 0) != (int64_t)l * 5 + w) ++mismatches;
                }
        }
    }
    return mismatches;
}

sc_status sc_selftest_bounded_wait(sc_ctx *ctx, int64_t limit_cycles, int32_t *site_host, int64_t *cycles_host)
{
    if (!ctx || !site_host || !cycles_host || limit_cycles < 1 || limit_cycles > 2000000000LL) return SC_ERR_ARG;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    if (cudaSetDevice(c->device) != cudaSuccess) return SC_ERR_CUDA;
    long long cyc[2] = {0, 0};
    if (run_bounded_wait_selftest(c, (long long)limit_cycles, site_host, cyc) != cudaSuccess) return SC_ERR_CUDA;
    cycles_host[0] = cyc[0];
    cycles_host[1] = cyc[1];
    return SC_OK;
}

sc_status sc_microbench(sc_ctx *ctx, int32_t kind, int32_t iters, float *ms_out, double *words_out)
{
    if (!ctx || !ms_out || !words_out || kind < 0 || kind > 9 || iters < 1 || iters > (1 << 22)) return SC_ERR_ARG;
    sc_ctx_impl *c = reinterpret_cast<sc_ctx_impl *>(ctx);
    if (cudaSetDevice(c->device) != cudaSuccess) return SC_ERR_CUDA;
    if (kind >= 8) return run_mxf4_rate(c, kind == 8 ? 192 : 256, iters, ms_out, words_out) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
    return run_microbench(c, kind, iters, ms_out, words_out) == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

}  // extern "C"
