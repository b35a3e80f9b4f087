// Row ordering and work list for ragged stream lengths (Sec. 4.2: every row ends at its own length l_i).
// Rows are counting-sorted by length, longest first, so that a 128-row tile holds rows of similar
// length; each row tile is then cut into work items of `chunk_planes` stream planes per column tile.
// One CTA per product sorts its rows; one CTA builds the work list over all row tiles.
#include "sc_device.cuh"
#include "sc_internal.h"

namespace sc {

constexpr int kPlanThreads = 1024;

// Two-SM core (sc_core_umma2.cu): it has one accumulator, so a piece boundary drains its pipeline (about kPairDrainUnits stage
// units, against the kPieceChargeUnits of the one-SM core), it works on pairs of row tiles and on 256-column tiles (an odd row
// tile or a ragged last column tile is padding), and on long pieces it needs a third less time per multiply-accumulate.  It is
// selected when its estimated time is the shorter one:
//     t_pair (u + kPairDrainUnits) <= 1.50 t_single (u + kPieceChargeUnits),   u = min(mean units per piece, shortest tile pair),
// t = stage units x column tiles x tile columns / SMs per tile (MMA time up to a common factor).  Measured against the forced
// choices on the ViT-L/14 sweep and the ragged configurations (profiles/core_umma_pair_kernel_*.md).
// (kPairDrainUnits, kPairAdvantagePct, kPieceChargeUnits: sc_internal.h; the host applies the same rule to the longest
// possible piece to decide whether the two-SM kernel is enqueued at all.)

struct PairChoice {
    int32_t col_tiles;      // column tiles of the two-SM core (0: that core is not available for the call)
    int32_t clusters;       // CTA pairs it runs with
    int32_t force;          // select it whatever the lengths are
    int32_t single_cols;    // columns per tile of the one-SM core (its n_col_tiles tiles are compared with)
};

__device__ void finish_plan(int32_t n_row_tiles, int32_t n_col_tiles, int32_t target_items, int32_t wave_ctas,
                            int32_t planes_per_len, PlanHeader *__restrict__ plan, int32_t *scratch,
                            unsigned long long *s_cost /* 64 */, int32_t *s_scan /* 34 */, PairChoice pair)
{
    __shared__ int32_t s_pair_min;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t *prefix = reinterpret_cast<int32_t *>(plan + 1);
    int32_t *tile_planes = prefix + n_row_tiles + 1;
    int32_t *s_max = s_scan + 32, *s_chunk = s_scan + 33;
    // the longest tile (tile 0 of the product with the longest row) and, for the ALU cores, the total work
    if (tid < 64) s_cost[tid] = 0ull;
    if (tid == 0) { *s_max = 0; s_pair_min = 0x7FFFFFFF; }
    __syncthreads();
    if (pair.clusters > 0) {
        // stage units of the row-tile pairs (the first, longer tile of a pair decides) per column tile of that core
        unsigned long long units = 0, with_work = 0, single_units = 0;
        int32_t shortest = 0x7FFFFFFF;
        for (int32_t T = tid; 2 * T < n_row_tiles; T += kPlanThreads) {
            const int32_t u = (tile_planes[2 * T] + kStagePlanes - 1) / kStagePlanes;
            if (u > 0) { units += (unsigned long long)u; ++with_work; shortest = min(shortest, u); }
            single_units += (unsigned long long)u;
            if (2 * T + 1 < n_row_tiles) single_units += (unsigned long long)((tile_planes[2 * T + 1] + kStagePlanes - 1) / kStagePlanes);
        }
        if (with_work) {
            atomicAdd(&s_cost[1], units); atomicAdd(&s_cost[2], with_work); atomicAdd(&s_cost[3], single_units);
            atomicMin(&s_pair_min, shortest);
        }
    }
    int32_t mine = 0;
    unsigned long long work = 0;
    for (int32_t rt = tid; rt < n_row_tiles; rt += kPlanThreads) {
        mine = max(mine, tile_planes[rt]);
        work += (unsigned long long)tile_planes[rt] * n_col_tiles;
    }
    if (mine) atomicMax(s_max, mine);
    if (wave_ctas <= 0 && work) atomicAdd(&s_cost[0], work);
    __syncthreads();
    const int32_t longest = *s_max;

    // ALU cores: dynamic tickets over items of `chunk` planes, about target_items of them.  Tensor-core core
    // (wave_ctas > 0): the unit is one TMA stage of kStagePlanes planes; every CTA later takes an equal, contiguous run
    // of the stage units of all tiles (cutting tiles wherever its run begins and ends), so the prefix sums below count
    // stages.
    if (tid == 0) {
        long long chunk;
        if (wave_ctas > 0) {
            chunk = kStagePlanes;
        } else {
            // chunk so that about `target_items` items exist, never below 8 stages per item
            chunk = (long long)((s_cost[0] + target_items - 1) / target_items);
            const long long min_chunk = 8 * kStagePlanes;
            if (chunk < min_chunk) chunk = min_chunk;
            chunk = (chunk + kStagePlanes - 1) / kStagePlanes * kStagePlanes;
        }
        if (chunk > 0x3FFFFFF0LL) chunk = 0x3FFFFFF0LL;
        *s_chunk = (int32_t)chunk;
    }
    __syncthreads();
    const int32_t chunk = *s_chunk;
    const int32_t charge = wave_ctas > 0 ? kPieceChargeUnits : 0;

    // exclusive prefix sums of the items per tile: every thread owns a run of consecutive tiles
    const int32_t per = (n_row_tiles + kPlanThreads - 1) / kPlanThreads;
    const int32_t t0 = min(tid * per, n_row_tiles), t1 = min(t0 + per, n_row_tiles);
    int32_t local = 0;
    // items of one row tile: per column tile its chunks, plus (tensor-core core) the charge for the piece boundary
    auto tile_items = [&](int32_t planes) { return planes > 0 ? ((planes + chunk - 1) / chunk + charge) * n_col_tiles : 0; };
    for (int32_t rt = t0; rt < t1; ++rt) local += tile_items(tile_planes[rt]);
    int32_t incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int32_t w = s_scan[lane];
        int32_t wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t up = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += up;
        }
        s_scan[lane] = wi - w;                        // exclusive prefix of the warp totals
    }
    __syncthreads();
    int32_t run = s_scan[warp] + incl - local;
    for (int32_t rt = t0; rt < t1; ++rt) {
        prefix[rt] = run;
        run += tile_items(tile_planes[rt]);
    }
    if (tid == kPlanThreads - 1) {
        prefix[n_row_tiles] = run;
        plan->total_items = run;
        plan->chunk_planes = chunk;
        plan->n_row_tiles = n_row_tiles;
        plan->n_col_tiles = n_col_tiles;
        plan->lmax_actual = longest / planes_per_len;
        int32_t use_pair = 0;
        if (pair.clusters > 0 && s_cost[2] > 0) {
            const long long pieces = (long long)s_cost[2] * pair.col_tiles + pair.clusters;
            const long long mean = (long long)s_cost[1] * pair.col_tiles / pieces;
            // MMA time of the two tilings, up to a common factor: units x column tiles x tile columns / SMs per tile
            const long long t_pair = (long long)s_cost[1] * pair.col_tiles * 256 * 2;
            const long long t_single = (long long)s_cost[3] * n_col_tiles * pair.single_cols;
            const long long u = min(mean, (long long)s_pair_min);
            use_pair = (pair.force || t_pair * (u + kPairDrainUnits) * 100 <= t_single * (u + kPieceChargeUnits) * kPairAdvantagePct) ? 1 : 0;
        }
        plan->pad[0] = use_pair;                      // which tensor-core core runs: 1 = the two-SM core
        plan->pad[1] = charge;                        // virtual units in front of every (row tile, column tile) in the prefix sums
        scratch[kSlotTicket] = 0;
        scratch[kSlotPairSelected] = use_pair;
        scratch[kSlotAnyNegA] = 0;                    // the encode of A sets it again if it meets a negative element
        scratch[kSlotLmaxActual] = longest / planes_per_len;
    }
}

// One CTA per product: counting sort of its M rows by length (longest first) into its own m_pad sorted
// positions; source rows are numbered over all products (b * M + i).  A single product finishes the plan
// in the same launch; several need plan_finish_kernel afterwards.
__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t *__restrict__ L, int64_t M, int32_t group, int32_t Lmax, int32_t planes_per_len, int32_t pos_block,
            int64_t m_pad, int32_t n_col_tiles, int32_t target_items, int32_t wave_ctas,
            int32_t *__restrict__ l_rows,
            int32_t *__restrict__ perm, int32_t *__restrict__ l_sorted, PlanHeader *__restrict__ plan,
            int32_t *scratch, PairChoice pair)
{
    __shared__ int32_t bins[SC_L_CAP + 1];       // bins[v]: rows with length v, then running offsets
    __shared__ int32_t warp_sums[32];
    __shared__ unsigned long long s_cost[64];
    __shared__ int32_t s_scan[34];
    const int tid = threadIdx.x;
    int32_t *status = scratch + kSlotStatus;
    const int64_t row0 = (int64_t)blockIdx.x * M;        // first source row of this product
    perm += (int64_t)blockIdx.x * m_pad;
    l_sorted += (int64_t)blockIdx.x * m_pad;

    for (int v = tid; v <= SC_L_CAP; v += kPlanThreads) bins[v] = 0;
    __syncthreads();

    bool bad = false;
    for (int64_t i = tid; i < M; i += kPlanThreads) {
        int32_t v = L ? __ldg(L + (row0 + i) / group) : Lmax;
        if (v < 0 || v > Lmax) { bad = true; v = v < 0 ? 0 : Lmax; }
        l_rows[row0 + i] = v;
        atomicAdd(&bins[v], 1);
    }
    if (bad) report(status, SC_ERR_LENGTH);
    __syncthreads();

    // exclusive scan in DESCENDING length order: thread t owns length SC_L_CAP - t; length 0 goes last.
    {
        const int v = SC_L_CAP - tid;                 // 1024 .. 1
        const int32_t mine = bins[v];
        int32_t incl = mine;
        const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int32_t w = warp_sums[lane], wi = w;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int32_t up = __shfl_up_sync(0xFFFFFFFFu, wi, o);
                if (lane >= o) wi += up;
            }
            warp_sums[lane] = wi - w;                 // exclusive prefix of the warp totals
        }
        __syncthreads();
        const int32_t excl = warp_sums[warp] + incl - mine;
        __syncthreads();
        bins[v] = excl;                               // first sorted position of length v
        if (tid == kPlanThreads - 1) bins[0] = excl + mine;   // rows of length 0 follow every other row
    }
    __syncthreads();

    for (int64_t i = tid; i < M; i += kPlanThreads) {
        const int32_t v = l_rows[row0 + i];
        const int32_t pos = atomicAdd(&bins[v], 1);
        perm[pos] = (int32_t)(row0 + i);
        l_sorted[pos] = v;
    }
    for (int64_t p = M + tid; p < m_pad; p += kPlanThreads) {   // padding rows: no source row, length 0
        perm[p] = -1;
        l_sorted[p] = 0;
    }
    __syncthreads();
    __threadfence_block();

    const int32_t tiles_m = (int32_t)(m_pad / kTileM);
    const int32_t n_row_tiles = tiles_m * (int32_t)gridDim.x;
    int32_t *prefix = reinterpret_cast<int32_t *>(plan + 1);
    int32_t *tile_planes = prefix + n_row_tiles + 1 + (int64_t)blockIdx.x * tiles_m;
    for (int32_t rt = tid; rt < tiles_m; rt += kPlanThreads)
        // the longest row of the tile, in whole blocks of stream positions
        tile_planes[rt] = (l_sorted[(int64_t)rt * kTileM] + pos_block - 1) / pos_block * pos_block * planes_per_len;
    __syncthreads();
    if (gridDim.x == 1) finish_plan(n_row_tiles, n_col_tiles, target_items, wave_ctas, planes_per_len, plan, scratch, s_cost, s_scan, pair);
}

__global__ void __launch_bounds__(kPlanThreads)
plan_finish_kernel(int32_t n_row_tiles, int32_t n_col_tiles, int32_t target_items, int32_t wave_ctas,
                   int32_t planes_per_len, PlanHeader *__restrict__ plan, int32_t *scratch)
{
    __shared__ unsigned long long s_cost[64];
    __shared__ int32_t s_scan[34];
    finish_plan(n_row_tiles, n_col_tiles, target_items, wave_ctas, planes_per_len, plan, scratch, s_cost, s_scan, PairChoice{0, 0, 0, kTileNUmma});
}

cudaError_t launch_plan(const int32_t *L, int64_t M, int32_t group, int32_t Lmax, int64_t kw, int ppq, int64_t m_pad,
                        int64_t n_col_tiles, int32_t target_items, int32_t wave_ctas, int32_t *l_rows,
                        int32_t *perm, int32_t *l_sorted, PlanHeader *plan, int32_t *scratch, cudaStream_t st,
                        int64_t batch, int32_t pos_block, int32_t pair_col_tiles, int32_t pair_clusters, int32_t pair_force,
                        int32_t single_tile_cols)
{
    const PairChoice pair{pair_col_tiles, batch == 1 ? pair_clusters : 0, pair_force, single_tile_cols};
    if (batch < 1 || batch > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    plan_kernel<<<(unsigned)batch, kPlanThreads, 0, st>>>(L, M, group, Lmax, (int32_t)(kw * ppq), pos_block, m_pad, (int32_t)n_col_tiles,
                                                        target_items, wave_ctas, l_rows, perm, l_sorted, plan, scratch, pair);
    count_launches(1);
    if (batch > 1) {
        plan_finish_kernel<<<1, kPlanThreads, 0, st>>>((int32_t)(batch * (m_pad / kTileM)), (int32_t)n_col_tiles, target_items,
                                                      wave_ctas, (int32_t)(kw * ppq), plan, scratch);
        count_launches(1);
    }
    return cudaGetLastError();
}

}  // namespace sc
