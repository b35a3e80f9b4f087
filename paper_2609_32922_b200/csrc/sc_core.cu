// Bit-serial GEMM core: the gate and the popcount accumulation of Eq. (1) over packed stream planes,
// with one stream length per row (Sec. 4.2: every row ends at its own length l_i).
//
//   bipolar : X_ij = sum_{planes p < Q_i} popc( A[p][i] xor W[p][j] )          (XNOR count = K L_i - X_ij)
//   unipolar: S_ij = sum_{steps}  popc(a & w) - 2 popc( (a_neg & w) xor (w_neg & a) )
//
// Persistent CTAs pull work items (row tile, column tile, plane chunk) from a ticket counter.  A CTA
// owns a 128 x 128 output tile for a chunk of planes; operand tiles (128 words x 16 planes) arrive by
// 2-D TMA into a 4-stage shared-memory ring guarded by mbarriers; each of the 256 threads keeps an
// 8 x 8 register tile of int32 accumulators and evaluates one LOP3 + POPC + IADD per 32 stream
// bit-ops (or the carry-save form: 3 planes -> 2 POPC).  Rows whose stream has ended are masked
// through the third LOP3 input, so rows of different length share a tile without divergence.
// Partial sums of the chunks of a tile meet in global memory through integer atomics (exact in any order).
#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

constexpr int kCoreThreads = 256;
constexpr int kStageWords = kStagePlanes * kTileM;                       // words of one operand per stage
constexpr uint32_t kStageBytes = 2u * kStageWords * sizeof(uint32_t);    // A + W
constexpr long long kWaitCycles = 1500000000LL;                          // bound of every mbarrier wait (~1 s)

struct CoreDev {
    const int32_t *perm, *l_sorted;
    const PlanHeader *plan;
    int32_t *acc;
    int32_t *scratch;
    int64_t N;
    int32_t planes_per_len;
    int32_t tiles_m;                  // row tiles per product (batched calls stack products along rows / columns)
    int64_t w_batch_cols;             // padded W stream rows per product
};

// ---- mbarrier / TMA primitives -------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitCycles and returns false; never spins forever.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > kWaitCycles) return false;
    return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int32_t x, int32_t y, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}

// ---- per-stage arithmetic ------------------------------------------------------------------------
// Thread (tx, ty) owns rows {4 ty .. 4 ty + 3, 64 + 4 ty ..} and columns {4 tx .. 4 tx + 3, 64 + 4 tx ..}
// of the tile: every shared-memory read is a conflict-free 16-byte vector.
__device__ __forceinline__ void load8(const uint32_t *plane, int base4, uint32_t v[8])
{
    const uint4 lo = *reinterpret_cast<const uint4 *>(plane + base4);
    const uint4 hi = *reinterpret_cast<const uint4 *>(plane + 64 + base4);
    v[0] = lo.x; v[1] = lo.y; v[2] = lo.z; v[3] = lo.w;
    v[4] = hi.x; v[5] = hi.y; v[6] = hi.z; v[7] = hi.w;
}

template <bool kCsa>
__device__ __forceinline__ void stage_bipolar_full(const uint32_t *As, const uint32_t *Ws, int ty4, int tx4,
                                                   int32_t acc[8][8])
{
    if (!kCsa) {
#pragma unroll
        for (int kk = 0; kk < kStagePlanes; kk += 2) {
            uint32_t a0[8], w0[8], a1[8], w1[8];
            load8(As + kk * kTileM, ty4, a0);
            load8(Ws + kk * kTileN, tx4, w0);
            load8(As + (kk + 1) * kTileM, ty4, a1);
            load8(Ws + (kk + 1) * kTileN, tx4, w1);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] += __popc(a0[i] ^ w0[j]) + __popc(a1[i] ^ w1[j]);
        }
    } else {
        // carry-save: three planes -> sum and carry words -> 2 POPC for 96 bit-ops
#pragma unroll
        for (int kk = 0; kk + 2 < kStagePlanes; kk += 3) {
            uint32_t a0[8], w0[8], a1[8], w1[8], a2[8], w2[8];
            load8(As + kk * kTileM, ty4, a0);
            load8(Ws + kk * kTileN, tx4, w0);
            load8(As + (kk + 1) * kTileM, ty4, a1);
            load8(Ws + (kk + 1) * kTileN, tx4, w1);
            load8(As + (kk + 2) * kTileM, ty4, a2);
            load8(Ws + (kk + 2) * kTileN, tx4, w2);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t x0 = a0[i] ^ w0[j], x1 = a1[i] ^ w1[j], x2 = a2[i] ^ w2[j];
                    const uint32_t s = x0 ^ x1 ^ x2;
                    const uint32_t c = (x0 & x1) | (x2 & (x0 | x1));
                    acc[i][j] += __popc(s) + 2 * __popc(c);
                }
        }
#pragma unroll
        for (int kk = kStagePlanes / 3 * 3; kk < kStagePlanes; ++kk) {
            uint32_t a0[8], w0[8];
            load8(As + kk * kTileM, ty4, a0);
            load8(Ws + kk * kTileN, tx4, w0);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] += __popc(a0[i] ^ w0[j]);
        }
    }
}

// Ragged / partial stage: plane p of the stage counts for row i only while first_plane + p < row_planes[i].
__device__ __forceinline__ void stage_bipolar_masked(const uint32_t *As, const uint32_t *Ws, int ty4, int tx4,
                                                     int32_t acc[8][8], int n_planes, int32_t first_plane,
                                                     const int32_t row_planes[8])
{
#pragma unroll 2
    for (int kk = 0; kk < n_planes; ++kk) {
        uint32_t a[8], w[8], m[8];
        load8(As + kk * kTileM, ty4, a);
        load8(Ws + kk * kTileN, tx4, w);
#pragma unroll
        for (int i = 0; i < 8; ++i) m[i] = (first_plane + kk < row_planes[i]) ? 0xFFFFFFFFu : 0u;
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] += __popc((a[i] ^ w[j]) & m[i]);
    }
}

// Unipolar: planes come in pairs (magnitude stream, magnitude AND sign).
__device__ __forceinline__ void stage_unipolar(const uint32_t *As, const uint32_t *Ws, int ty4, int tx4,
                                               int32_t acc[8][8], int n_planes, int32_t first_plane,
                                               const int32_t row_planes[8], bool masked)
{
#pragma unroll 2
    for (int kk = 0; kk < n_planes; kk += 2) {
        uint32_t a[8], an[8], w[8], wn[8];
        load8(As + kk * kTileM, ty4, a);
        load8(As + (kk + 1) * kTileM, ty4, an);
        load8(Ws + kk * kTileN, tx4, w);
        load8(Ws + (kk + 1) * kTileN, tx4, wn);
        if (masked) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (first_plane + kk >= row_planes[i]) { a[i] = 0u; an[i] = 0u; }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t both = a[i] & w[j];                      // AND gate
                const uint32_t negs = (an[i] & w[j]) ^ (wn[j] & a[i]);   // set bits whose product is negative
                acc[i][j] += __popc(both) - 2 * __popc(negs);
            }
    }
}

// ---- the persistent kernel -----------------------------------------------------------------------
template <int kMode, bool kCsa>
__global__ void __launch_bounds__(kCoreThreads, (kCsa || kMode == SC_UNIPOLAR_AND) ? 1 : 2)
core_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, CoreDev p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint32_t *ring = reinterpret_cast<uint32_t *>(smem_raw);                    // kStages x (A | W)
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem_raw + (size_t)kStages * kStageBytes);
    int32_t *s_row_planes = reinterpret_cast<int32_t *>(bars + kStages);       // [128]
    int32_t *s_perm = s_row_planes + kTileM;                                    // [128]
    int32_t *s_ticket = s_perm + kTileM;

    const int tid = threadIdx.x;
    const int tx4 = (tid & 15) * 4, ty4 = (tid >> 4) * 4;
    const uint32_t ring_addr = smem_u32(ring), bars_addr = smem_u32(bars);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(bars_addr + 8u * s, 1u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const PlanHeader plan = *p.plan;
    const int32_t *prefix = reinterpret_cast<const int32_t *>(p.plan + 1);
    const int32_t *tile_planes = prefix + plan.n_row_tiles + 1;
    uint32_t it = 0;                       // stages consumed so far by this CTA (ring position and parity)

    auto issue = [&](uint32_t index, int32_t row0, int32_t col0, int32_t plane) {
        const uint32_t s = index % kStages;
        const uint32_t bar = bars_addr + 8u * s;
        const uint32_t dst = ring_addr + s * kStageBytes;
        mbar_expect_tx(bar, kStageBytes);
        tma_load_2d(dst, &map_a, row0, plane, bar);
        tma_load_2d(dst + kStageWords * 4u, &map_w, col0, plane, bar);
    };

    while (true) {
        if (tid == 0) *s_ticket = atomicAdd(p.scratch + kSlotTicket, 1);
        __syncthreads();
        const int32_t item = *s_ticket;
        if (item >= plan.total_items) break;

        // item -> (row tile, plane chunk, column tile)
        int32_t lo = 0, hi = plan.n_row_tiles;             // prefix[lo] <= item < prefix[hi]
        while (hi - lo > 1) {
            const int32_t mid = (lo + hi) >> 1;
            if (__ldg(prefix + mid) <= item) lo = mid; else hi = mid;
        }
        const int32_t rt = lo;
        const int32_t local = item - __ldg(prefix + rt);
        const int32_t chunk_idx = local / plan.n_col_tiles, ct = local - chunk_idx * plan.n_col_tiles;
        const int32_t tile_end = __ldg(tile_planes + rt);
        const int32_t q0 = chunk_idx * plan.chunk_planes;
        const int32_t q1 = min(q0 + plan.chunk_planes, tile_end);
        const int32_t n_steps = (q1 - q0 + kStagePlanes - 1) / kStagePlanes;
        const int32_t w_col0 = (int32_t)((rt / p.tiles_m) * p.w_batch_cols) + ct * kTileN;   // the product's own columns

        if (tid < kTileM) {
            const int64_t r = (int64_t)rt * kTileM + tid;
            s_row_planes[tid] = __ldg(p.l_sorted + r) * p.planes_per_len;
            s_perm[tid] = __ldg(p.perm + r);
        }
        __syncthreads();

        int32_t row_planes[8];
        int32_t min_planes = 0x7FFFFFFF;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            row_planes[i] = s_row_planes[(i < 4 ? ty4 + i : 64 + ty4 + i - 4)];
            min_planes = min(min_planes, row_planes[i]);
        }

        int32_t acc[8][8];
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[i][j] = 0;

        if (tid == 0)
            for (int s = 0; s < kStages - 1 && s < n_steps; ++s)
                issue(it + s, rt * kTileM, w_col0, q0 + s * kStagePlanes);

        bool failed = false;
        int32_t step = 0;
        for (; step < n_steps; ++step) {
            if (tid == 0 && step + kStages - 1 < n_steps)
                issue(it + step + kStages - 1, rt * kTileM, w_col0, q0 + (step + kStages - 1) * kStagePlanes);
            const uint32_t index = it + step, s = index % kStages;
            const bool ok = mbar_wait(bars_addr + 8u * s, (index / kStages) & 1u);
            const uint32_t *As = ring + (size_t)s * (kStageBytes / 4), *Ws = As + kStageWords;
            const int32_t first = q0 + step * kStagePlanes;
            const int n_planes = min(kStagePlanes, q1 - first);
            if (kMode == SC_BIPOLAR_XNOR) {
                if (n_planes == kStagePlanes && first + kStagePlanes <= min_planes)
                    stage_bipolar_full<kCsa>(As, Ws, ty4, tx4, acc);
                else
                    stage_bipolar_masked(As, Ws, ty4, tx4, acc, n_planes, first, row_planes);
            } else {
                stage_unipolar(As, Ws, ty4, tx4, acc, n_planes, first, row_planes,
                               first + kStagePlanes > min_planes);
            }
            if (__syncthreads_or(!ok)) { failed = true; break; }   // also frees the stage for the next TMA
        }
        if (failed) {
            // a wait ran out: record it, give the copies still in flight a bounded time to land, leave
            if (tid == 0) {
                report(p.scratch + kSlotStatus, SC_ERR_TIMEOUT);
                for (int32_t pending = step + 1; pending < n_steps && pending < step + kStages; ++pending) {
                    const uint32_t index = it + pending;
                    (void)mbar_wait(bars_addr + 8u * (index % kStages), (index / kStages) & 1u);
                }
            }
            __syncthreads();
            return;
        }
        it += (uint32_t)n_steps;

        // partial sums of this chunk -> global accumulators (original row order)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int rl = (i < 4 ? ty4 + i : 64 + ty4 + i - 4);
            const int32_t src = s_perm[rl];
            if (src < 0 || row_planes[i] <= q0) continue;
            int32_t *out = p.acc + (int64_t)src * p.N;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t col = (int64_t)ct * kTileN + (j < 4 ? tx4 + j : 64 + tx4 + j - 4);
                if (col < p.N) atomicAdd(out + col, acc[i][j]);
            }
        }
        // the next iteration's first __syncthreads orders these reads of s_perm / s_row_planes
        // before they are overwritten
    }
}

// ---- reference variant without shared memory or TMA: one thread per output ---------------------------
template <int kMode>
__global__ void __launch_bounds__(256)
core_simple_kernel(const uint32_t *__restrict__ A, const uint32_t *__restrict__ W, int64_t m_pad, int64_t n_pad,
                   int64_t M_sorted, CoreDev p)
{
    const int64_t col = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t r = blockIdx.y;
    if (r >= M_sorted || col >= p.N) return;
    const int32_t src = p.perm[r];
    if (src < 0) return;
    const int32_t planes = p.l_sorted[r] * p.planes_per_len;
    const int64_t wc = (r / ((int64_t)p.tiles_m * kTileM)) * p.w_batch_cols + col;      // the product's own columns
    int32_t acc = 0;
    if (kMode == SC_BIPOLAR_XNOR) {
        for (int32_t q = 0; q < planes; ++q) acc += __popc(A[(int64_t)q * m_pad + r] ^ W[(int64_t)q * n_pad + wc]);
    } else {
        for (int32_t q = 0; q < planes; q += 2) {
            const uint32_t a = A[(int64_t)q * m_pad + r], an = A[(int64_t)(q + 1) * m_pad + r];
            const uint32_t w = W[(int64_t)q * n_pad + wc], wn = W[(int64_t)(q + 1) * n_pad + wc];
            acc += __popc(a & w) - 2 * __popc((an & w) ^ (wn & a));
        }
    }
    p.acc[(int64_t)src * p.N + col] = acc;
}

// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// planes x row-words matrix of uint32, box = box_words words x kStagePlanes planes
bool make_plane_map(CUtensorMap *map, const uint32_t *base, int64_t row_words, int64_t planes, int box_words,
                    int box_planes)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)row_words, (cuuint64_t)planes};
    cuuint64_t strides[1] = {(cuuint64_t)row_words * sizeof(uint32_t)};
    cuuint32_t box[2] = {(cuuint32_t)box_words, (cuuint32_t)box_planes};
    cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<uint32_t *>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of the int32 accumulators [rows][cols] for bulk tensor reductions of 32 x 32 boxes staged in shared memory in
// the 128-byte swizzle (16-byte chunk c of box row r at chunk c ^ (r & 7): conflict-free 16-byte stores by one lane per row).
// Needs a 16-byte aligned base and cols % 4 == 0 (the row stride in bytes is a multiple of 16).
bool make_acc_map(CUtensorMap *map, int32_t *acc, int64_t rows, int64_t cols)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || (cols & 3) != 0 || (reinterpret_cast<uintptr_t>(acc) & 15u) != 0) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * sizeof(int32_t)};
    cuuint32_t box[2] = {32u, 32u};
    cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_INT32, 2, acc, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr size_t kCoreSmem = (size_t)kStages * kStageBytes + kStages * 8 + (2 * kTileM + 4) * sizeof(int32_t);

template <int kMode, bool kCsa>
static cudaError_t launch_core_variant(const CUtensorMap &ma, const CUtensorMap &mw, const CoreDev &dev, int sm_count,
                                       cudaStream_t st)
{
    auto kernel = core_kernel<kMode, kCsa>;
    static bool configured = false;
    static int per_sm = 1;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCoreSmem);
        if (e != cudaSuccess) return e;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kCoreThreads, kCoreSmem);
        if (e != cudaSuccess) return e;
        if (per_sm < 1) per_sm = 1;
        configured = true;
    }
    kernel<<<sm_count * per_sm, kCoreThreads, kCoreSmem, st>>>(ma, mw, dev);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_core(const CoreArgs &a, cudaStream_t st)
{
    CoreDev dev;
    dev.perm = a.perm;
    dev.l_sorted = a.l_sorted;
    dev.plan = a.plan;
    dev.acc = a.acc;
    dev.scratch = a.scratch;
    dev.N = a.N;
    dev.planes_per_len = a.kw * a.ppq;
    dev.tiles_m = a.tiles_m;
    dev.w_batch_cols = a.w_batch_cols;

    if (a.variant == SC_CORE_SIMPLE) {
        // one grid row per sorted position (a single product keeps its real rows first; stacked products interleave
        // padding, which the kernel skips)
        const int64_t sorted_rows = a.w_batch_cols < a.n_pad ? a.m_pad : a.M;
        dim3 grid((unsigned)((a.N + 255) / 256), (unsigned)sorted_rows);
        if (a.mode == SC_BIPOLAR_XNOR)
            core_simple_kernel<SC_BIPOLAR_XNOR><<<grid, 256, 0, st>>>(a.a_streams, a.w_streams, a.m_pad, a.n_pad, sorted_rows, dev);
        else
            core_simple_kernel<SC_UNIPOLAR_AND><<<grid, 256, 0, st>>>(a.a_streams, a.w_streams, a.m_pad, a.n_pad, sorted_rows, dev);
        count_launches(1);
        return cudaGetLastError();
    }

    CUtensorMap ma, mw;
    if (!make_plane_map(&ma, a.a_streams, a.m_pad, a.a_planes, kTileM, kStagePlanes) ||
        !make_plane_map(&mw, a.w_streams, a.n_pad, a.w_planes, kTileN, kStagePlanes))
        return cudaErrorInvalidValue;
    if (a.mode == SC_UNIPOLAR_AND) return launch_core_variant<SC_UNIPOLAR_AND, false>(ma, mw, dev, a.sm_count, st);
    if (a.variant == SC_CORE_CSA) return launch_core_variant<SC_BIPOLAR_XNOR, true>(ma, mw, dev, a.sm_count, st);
    return launch_core_variant<SC_BIPOLAR_XNOR, false>(ma, mw, dev, a.sm_count, st);
}

}  // namespace sc
