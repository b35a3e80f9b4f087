// Tensor-core GEMM core: the popcount accumulation of Eq. (1) as a dense contraction on the 5th-gen tensor
// cores (tcgen05.mma, accumulators in tensor memory).
//
// The sum over (inner dimension d, stream position l) of a_{id,l} AND w_{dj,l} is a matrix product of 0/1
// matrices over K*L columns.  Bit planes cannot be fed to the tensor cores directly, so each CTA expands
// them on chip, 1 stream bit -> one 4-bit float (e2m1), for tcgen05.mma kind::mxf4 (block-scaled, all scales 2^0,
// K = 64 per instruction: twice the rate of the 8-bit kinds and half the shared-memory bytes per bit); the fp32
// accumulators hold exact integers as long as K L <= 2^24.
// The activation operand (128 rows) is expanded straight into tensor memory (tcgen05.st) and read by
// the MMA from there; the weight operand (192 columns) is expanded into the shared-memory layout the MMA reads
// (K-major, no swizzle: 8-row x 16-byte core matrices).  Only the weight operand therefore crosses shared memory.
// Rows whose stream has ended are zeroed during the expansion, so ragged lengths cost nothing extra.
//   bipolar : a set bit becomes a power of two chosen so that every product is exactly 1; the MMA yields the AND
//             count, and the decode pass turns it into the XNOR count,
//             XNOR = K L_i - pop(A_i, l < L_i) - pop(W_j, l < L_i) + 2 AND;
//   unipolar: the same powers of two with a sign bit: both operands come as magnitude planes plus, per (depth word,
//             row / column), the signs of its 32 elements as four nibble words (the activations' are skipped when the
//             call has no negative stream bit); positions are stored in blocks of 8 so that an operand stage is 8
//             positions of one depth word and one set of sign words serves the stage; the MMA yields the signed count.
//
// Warp roles (one CTA of 28 warps per SM, persistent; each CTA owns an equal contiguous run of the stage units of all
// tiles, see u_piece):
//   warp 0        TMA producer: 192-column x 48-plane bit tiles of W (three plan units per box: the W expander
//                 warps synchronise with the producer once per box) into a 2-stage ring
//   warp 1, 27    MMA issuers (warp 1 also allocates tensor memory): one lane of each issues tcgen05.mma
//                 (M=128, N=192, four K-steps per operand stage); issuer i owns the operand stages s with s % 2 == i
//   warps 2-5     epilogue: tcgen05.ld the 128 x 192 accumulators, stage each lane's 128-byte row piece in shared
//                 memory, bulk reduce-add into global memory
//   warps 6-17    A expanders, three groups of four (one row per thread, the warp's own quarter of the
//                 tensor-memory lanes); group g fills every third operand stage; the plane words come straight
//                 from global memory (128 consecutive bytes per warp and plane), one own stage ahead
//   warps 18-26   W expanders, three groups of three (two columns per thread), from the TMA ring
// Tensor memory: one or two accumulators (192 columns each), the A ring (32 columns per stage) and 32 columns of scale
// factors.
// Every wait is bounded; a wait that runs out sets SC_ERR_TIMEOUT and records where, all roles drain, tensor
// memory is freed.
#include <type_traits>

#include "sc_device.cuh"
#include "sc_internal.h"
#include "sc_umma.cuh"

namespace sc {

constexpr int kUN = kTileNUmma;                // 192 output columns per tile
constexpr int kRawUnits = 3;                   // plan units (kStagePlanes planes each) per TMA box / raw stage
constexpr int kRawPlanes = kRawUnits * kStagePlanes;
constexpr int kRawStages = 2;
constexpr int kOpSteps = 4;                    // MMA K-steps (32 bytes of K each) per operand stage
constexpr int kOpStages = 4;
constexpr int kEpiFirstWarp = 2, kEpiWarps = 4;
// Expander warps work in groups; group g of a kind fills every groups-th operand stage.  An MMA issuer owns
// fixed stages (a waiter that skipped a use of a stage could not tell the barrier's phases apart by parity;
// the expanders, which may skip uses, wait on barriers that alternate between even and odd uses instead).
constexpr int kAGroups = 3;                    // activation expanders: groups of ...
constexpr int kAFirstWarp = 6, kAWarps = 4;    // ... 4 warps (one per tensor-memory lane quarter)
constexpr int kWGroups = 3;                    // weight expanders: groups of ...
constexpr int kWCols = 2;                      // (columns per W expander thread)
constexpr int kWWarps = kTileNUmma / (32 * kWCols);   // ... 3 warps (64 columns each)
constexpr int kFillWarps = kAWarps + kWWarps;  // arrivals per operand stage
constexpr int kWFirstWarp = kAFirstWarp + kAGroups * kAWarps;
constexpr int kAllExpWarps = kAGroups * kAWarps + kWGroups * kWWarps;
constexpr int kIssuers = 2;                    // MMA issuer threads; issuer i owns the stages s with s % kIssuers == i
constexpr int kIssuerBWarp = kAFirstWarp + kAllExpWarps;   // issuers 1.. live in the last warps
constexpr int kUThreads = 32 * (kIssuerBWarp + kIssuers - 1);
static_assert(kOpStages % kIssuers == 0, "an issuer must own fixed operand stages");
static_assert(kUThreads <= 1024, "one CTA");

constexpr uint32_t kRawStageBytes = kRawPlanes * kUN * 4;         // W planes of one box (36 KB); A planes are read from global memory
constexpr uint32_t kLboB = kUN * 16;           // bytes between consecutive 16-byte K chunks of the W operand
constexpr uint32_t kOpStageBytes = kOpSteps * 2 * kLboB;          // 24 KB
constexpr int kEpiStride = 36;                 // words per staged row (144 B: 16-byte aligned, conflict-free vector stores)
constexpr uint32_t kEpiBytes = kEpiWarps * 2 * 32 * kEpiStride * 4;   // two staging buffers per epilogue warp
constexpr uint32_t kAccCols = kUN;             // columns of one accumulator
constexpr uint32_t kTmemCols = 512;

enum UBar : int {
    kRawFull = 0, kRawEmpty = kRawFull + kRawStages, kOpFull = kRawEmpty + kRawStages,
    kOpEmpty = kOpFull + kOpStages, kAccFull = kOpEmpty + 2 * kOpStages, kAccEmpty = kAccFull + 2,
    kAccStarted = kAccEmpty + 2, kNumBars = kAccStarted + 2
};
constexpr size_t kUmmaSmem = (size_t)kRawStages * kRawStageBytes + (size_t)kOpStages * kOpStageBytes + kEpiBytes +
                             kNumBars * 8 + 16;
// Tensor memory, 4-bit form (kind::mxf4, block scaled): the last 32 columns hold the scale factors (all 2^0), which
// leaves two accumulators an A ring of three stages only, one stage less than the W ring.  For long tiles that A ring is
// what bounds the pipeline, so a kernel whose pieces are long keeps one accumulator and a four-stage A ring instead: the
// MMAs of the next piece then wait for the epilogue of the last one (a pipeline drain per piece).  Measured on uniform
// lengths: -10 % at 64 stage units per piece, +5 % at 256, +10 % at 1024.  The choice follows the plan (device data),
// every role takes the same one.
// (The A ring is never deeper than the W ring: the A expanders arrive on the barrier of the W stage, and further ahead
// their arrival would fall into the stage's previous use.)  The 8-bit form has no scale factors: two accumulators and
// four A stages fit.
constexpr uint32_t kSfCols = 32;
constexpr uint32_t kSfCol = kTmemCols - kSfCols;
constexpr int32_t kSingleAccUnits = 176;   // mean stage units per piece from which one accumulator is faster
static_assert(2 * kAccCols + 3 * kOpSteps * 8 + kSfCols <= kTmemCols && kAccCols + 4 * kOpSteps * 8 + kSfCols <= kTmemCols &&
              2 * kAccCols + 4 * kOpSteps * 8 <= kTmemCols && kOpStages >= 4, "tensor memory budget");

static_assert(kAFirstWarp % 4 == 2 && kAWarps == 4 && kTileNUmma % (32 * kWCols) == 0, "lane-quarter / column mapping");

struct UmmaDev {
    const uint32_t *a_streams;        // A planes [plane][m_pad]
    int64_t m_pad;
    const int32_t *perm, *l_sorted;
    const PlanHeader *plan;
    int32_t *acc;
    int32_t *scratch;
    int64_t N;
    int32_t planes_per_len;           // W planes (= K-step halves) per stream position: the depth words
    int32_t pos_block;                // stream positions are stored in blocks of this many (1: position-major)
    int32_t tiles_m;                  // row tiles per product (batched calls stack products along rows / columns)
    int64_t w_batch_cols;             // padded W stream rows per product
    const uint32_t *w_sign;           // unipolar: [depth word][n_pad][4] nibble sign words of W ...
    const uint32_t *a_sign;           // ... and [depth word][m_pad][4] of A
    int64_t n_pad;                    // padded W stream rows in all
    int32_t tile_n;                   // output columns per tile: a multiple of 32, at most kUN (the shared-memory layout, the
                                      // TMA box and the accumulator are kUN wide; columns from tile_n on are not expanded,
                                      // not multiplied and not read back)
};

// (The bit -> 4-bit float expansions u_expand_bits / u_expand_signed_a / u_expand_signed_w live in sc_device.cuh,
// shared with the host self-test.)

struct UItem {
    int32_t rt, ct, q0, q1, n_raw;
    int32_t adv;            // how far the walk moves on (the piece's units plus any hand-over charge walked over)
};

// Work decomposition: the plan lists, per row tile, the running total of stage units (one unit = one TMA stage of
// kStagePlanes planes of one (row tile, column tile)).  CTA c owns the contiguous run [c T / G, (c + 1) T / G) of the
// T units, cutting tiles where its run begins and ends: all CTAs get the same amount of work whatever the tile
// count is, and the pieces of a cut tile meet in the global accumulators.  Every role of a CTA walks the same pieces.
// A piece boundary (accumulator hand-over, pipeline refill) costs about as much as a few units, so the plan charges every
// (row tile, column tile) `charge` virtual units in front of its real ones (PlanHeader.pad[1]): CTAs whose runs cross
// many short tiles receive fewer real units, and all CTAs finish together when lengths are ragged.
__device__ __forceinline__ int32_t u_run_begin(const PlanHeader &plan, int32_t cta)
{
    return (int32_t)((long long)plan.total_items * cta / (long long)gridDim.x);
}

// The next piece with work at or after position `pos` of the run ending at `end` (n_raw == 0: none is left).
__device__ __forceinline__ UItem u_piece(const PlanHeader &plan, const int32_t *prefix, const int32_t *tile_planes,
                                         int32_t pos, int32_t end)
{
    const int32_t charge = plan.pad[1];
    UItem it;
    it.n_raw = 0;
    it.adv = 0;
    while (pos < end) {
        int32_t lo = 0, hi = plan.n_row_tiles;           // largest row tile with prefix <= pos (skips empty tiles)
        while (hi - lo > 1) {
            const int32_t mid = (lo + hi) >> 1;
            if (__ldg(prefix + mid) <= pos) lo = mid; else hi = mid;
        }
        const int32_t planes = __ldg(tile_planes + lo);
        const int32_t stages = (planes + kStagePlanes - 1) / kStagePlanes;
        const int32_t charged = stages + charge;         // positions of one column tile: the charge, then the real units
        const int32_t local = pos - __ldg(prefix + lo);
        const int32_t ct = local / charged;
        const int32_t x0 = local - ct * charged;
        const int32_t x1 = min(charged, x0 + (end - pos));
        const int32_t s0 = max(x0 - charge, 0), s1 = max(x1 - charge, 0);
        it.adv += x1 - x0;
        pos += x1 - x0;
        if (s1 > s0) {
            it.rt = lo;
            it.ct = ct;
            it.q0 = s0 * kStagePlanes;
            it.q1 = min(s1 * kStagePlanes, planes);
            it.n_raw = s1 - s0;
            return it;
        }
    }
    return it;
}

// kNarrow: the tile is narrower than kUN columns (UmmaDev.tile_n, narrow products); otherwise the width is the constant
// kUN and every test against it folds away (the kernel is sensitive to each instruction on its expander paths).
template <int kMode, bool kNarrow>
__global__ void __launch_bounds__(kUThreads, 1)
core_umma_kernel(const __grid_constant__ CUtensorMap map_w, UmmaDev p)
{
    const int32_t tile_n = kNarrow ? p.tile_n : kUN;
    // An MMA K-step of 64 elements is two (depth word, position) pairs = two planes of either operand.
    constexpr int kPpq = 2;
    constexpr int kStepsPerRaw = kStagePlanes / kPpq;              // MMA steps in one raw stage
    constexpr int kOpsPerRaw = kStepsPerRaw / kOpSteps;            // operand stages in one raw stage
    constexpr int kStagePp = kOpSteps * kPpq;                      // (depth word, position) pairs of one operand stage
    static_assert(kStagePp == kPosBlockSigned, "a signed operand stage is one block of positions of one depth word");

    if (p.plan->pad[0] != 0) return;                   // the plan gave this call to the two-SM core (same in every CTA)
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *raw = smem;
    uint8_t *ops = smem + (size_t)kRawStages * kRawStageBytes;
    uint32_t *epi = reinterpret_cast<uint32_t *>(ops + (size_t)kOpStages * kOpStageBytes);
    uint64_t *bars = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(epi) + kEpiBytes);
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(bars + kNumBars);
    volatile int32_t *s_abort = reinterpret_cast<volatile int32_t *>(s_tmem + 1);
    int32_t *s_single = reinterpret_cast<int32_t *>(s_tmem + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t bars_addr = u_smem(bars), raw_addr = u_smem(raw), ops_addr = u_smem(ops);
    auto bar = [&](int which) { return bars_addr + 8u * (uint32_t)which; };

    if (tid == 0) {
        for (int s = 0; s < kRawStages; ++s) { u_mbar_init(bar(kRawFull + s), 1); u_mbar_init(bar(kRawEmpty + s), kWGroups * kWWarps); }
        for (int s = 0; s < kOpStages; ++s) u_mbar_init(bar(kOpFull + s), kFillWarps);
        for (int s = 0; s < 2 * kOpStages; ++s) u_mbar_init(bar(kOpEmpty + s), 1);
        for (int s = 0; s < 2; ++s) {
            u_mbar_init(bar(kAccFull + s), kIssuers);   // one arrival from each MMA issuer
            u_mbar_init(bar(kAccEmpty + s), kEpiWarps);
            u_mbar_init(bar(kAccStarted + s), 1);
        }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(u_smem(s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const PlanHeader plan = *p.plan;
    const int32_t *prefix = reinterpret_cast<const int32_t *>(p.plan + 1);
    const int32_t *tile_planes = prefix + plan.n_row_tiles + 1;
    if (warp == 2) {
        // stage units per piece: the mean (pieces = tiles with work + one cut per CTA) and the shortest tile (CTAs get
        // equal runs of units, so the CTA that owns the shortest tiles has the most pieces)
        int32_t n = 0, shortest = 0x7FFFFFFF;
        for (int32_t rt = lane; rt < plan.n_row_tiles; rt += 32) {
            const int32_t planes = __ldg(tile_planes + rt);
            if (planes > 0) { ++n; shortest = min(shortest, (planes + kStagePlanes - 1) / kStagePlanes); }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            n += __shfl_xor_sync(0xFFFFFFFFu, n, o);
            shortest = min(shortest, __shfl_xor_sync(0xFFFFFFFFu, shortest, o));
        }
        const int32_t mean = (plan.total_items - plan.pad[1] * n * plan.n_col_tiles) / (n * plan.n_col_tiles + (int32_t)gridDim.x);
        if (lane == 0) *s_single = min(mean, shortest) >= kSingleAccUnits ? 1 : 0;
    }
    u_fence_before();
    __syncthreads();
    u_fence_after();
    const uint32_t tmem_base = *s_tmem;
    const bool single = *s_single != 0;                            // one accumulator, four A stages
    const uint32_t a_ring_col = (single ? 1u : 2u) * kAccCols;     // first column of the A ring
    const bool a_three = !single;                                  // depth of the A ring: three stages, else four
    auto a_slot = [&](uint32_t op) { return a_three ? op % 3u : op & 3u; };
    {
        // scale factors: every byte 0x7F = 2^0 (ue8m0), whatever the scale layout picks
        if (warp >= kAFirstWarp && warp < kAFirstWarp + kAWarps) {
            uint32_t ones[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) ones[k] = 0x7F7F7F7Fu;
#pragma unroll
            for (uint32_t c = 0; c < kSfCols; c += 8)
                u_tmem_st8(tmem_base + kSfCol + c + ((((uint32_t)warp & 3u) * 32u) << 16), ones);
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        u_fence_before();
        __syncthreads();
        u_fence_after();
    }

    // The first role that gives up records where (wait site, warp, CTA, its counters) for the host to read.
    auto give_up = [&](int site, uint32_t cnt_a, uint32_t cnt_b) {
        if (*s_abort == 0 && atomicCAS(p.scratch + kSlotTimeoutSite, 0, site | (warp << 8) | ((int)blockIdx.x << 16)) == 0) {
            p.scratch[kSlotTimeoutSite + 1] = (int32_t)cnt_a;
            p.scratch[kSlotTimeoutSite + 2] = (int32_t)cnt_b;
        }
        *s_abort = 1;
        report(p.scratch + kSlotStatus, SC_ERR_TIMEOUT);
    };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t raw_cnt = 0;
            bool ok = true;
            for (int32_t pos = u_run_begin(plan, blockIdx.x), end = u_run_begin(plan, blockIdx.x + 1); pos < end && ok && !*s_abort;) {
                const UItem it = u_piece(plan, prefix, tile_planes, pos, end);
                pos += it.adv;
                if (it.n_raw == 0) break;
                // one box holds kRawUnits units; the last box of a piece may reach past it (those planes are not used)
                for (int32_t k = 0; k < (it.n_raw + kRawUnits - 1) / kRawUnits; ++k, ++raw_cnt) {
                    const uint32_t s = raw_cnt % kRawStages;
                    ok = u_mbar_wait(bar(kRawEmpty + s), ((raw_cnt / kRawStages) & 1u) ^ 1u, s_abort);
                    if (!ok) break;
                    u_mbar_expect_tx(bar(kRawFull + s), kRawStageBytes);
                    const uint32_t dst = raw_addr + s * kRawStageBytes;
                    u_tma_load_2d(dst, &map_w, (int32_t)((it.rt / p.tiles_m) * p.w_batch_cols) + it.ct * tile_n,
                                  it.q0 + k * kRawPlanes, bar(kRawFull + s));
                }
            }
            if (!ok) give_up(1, raw_cnt, 0);
        }
    } else if (warp == 1 || warp >= kIssuerBWarp) {
        // ---------------- MMA issuers ----------------
        // A thread that has issued tcgen05.mma stalls in its next barrier operation or fence until those MMAs
        // have drained, and while it stalls it issues nothing: with one issuer the tensor pipe idles a few
        // hundred cycles per operand stage.  Several issuers (lane 0 of different warps) therefore take turns:
        // issuer i owns the operand stages s with s % kIssuers == i, so while one drains, tests the barrier of
        // its next stage and commits, another one's MMAs run.  Owning fixed stages also means that an issuer
        // has itself consumed a stage's previous use before it waits for the next one (parity waits cannot
        // tell phases two apart).  The pipe executes MMAs in issue order; the only order that matters
        // between the issuers is that the MMA that overwrites the accumulator (first stage of an item) is
        // issued before any other MMA of the item: the others wait for a barrier that its issuer arrives on
        // right after that MMA.  Each issuer commits the stages it issued and arrives once per item on the
        // accumulator barrier (a commit after its last stage, a plain arrival if it had none).
        if (lane == 0) {
            const uint32_t me = warp == 1 ? 0u : (uint32_t)(warp - kIssuerBWarp + 1);
            uint32_t op_cnt = 0, acc_cnt = 0;
            bool ok = true;
            int site = 0;
            const uint64_t desc0 = u_smem_desc(ops_addr, kLboB);
            constexpr uint32_t kStepDesc = (2u * kLboB) >> 4, kStageDesc = kOpStageBytes >> 4;
            const uint32_t idesc = u_idesc_fp4(kTileM, (uint32_t)tile_n);
            for (int32_t pos = u_run_begin(plan, blockIdx.x), end = u_run_begin(plan, blockIdx.x + 1); pos < end && ok && !*s_abort;) {
                const UItem it = u_piece(plan, prefix, tile_planes, pos, end);
                pos += it.adv;
                if (it.n_raw == 0) break;
                const uint32_t b = single ? 0u : acc_cnt & 1u, acc_phase = (single ? acc_cnt : acc_cnt >> 1) & 1u;
                const uint32_t first = op_cnt % kIssuers;        // owner of the item's first stage: it overwrites
                site = 2;
                ok = u_mbar_wait(bar(kAccEmpty + b), acc_phase ^ 1u, s_abort);
                if (ok && me != first) { site = 3; ok = u_mbar_wait(bar(kAccStarted + b), acc_phase, s_abort); }
                if (!ok) break;
                site = 4;
                const uint32_t d_tmem = tmem_base + b * kAccCols;
                const int32_t n_ops = it.n_raw * kOpsPerRaw;
                const int32_t j0 = (int32_t)((me + kIssuers - first) % kIssuers);      // the issuer's first stage of the item
                for (int32_t j = j0; j < n_ops; j += kIssuers) {
                    const uint32_t op = op_cnt + (uint32_t)j;
                    const uint32_t t = op % kOpStages, use = op / kOpStages;
                    ok = u_mbar_wait(bar(kOpFull + t), use & 1u, s_abort);
                    if (!ok) break;
                    u_fence_after();
                    const uint64_t bdesc = desc0 + (uint64_t)(t * kStageDesc);
                    const uint32_t a_base = tmem_base + a_ring_col + a_slot(op) * (kOpSteps * 8u);
#pragma unroll
                    for (int st = 0; st < kOpSteps; ++st) {
                        u_mma_fp4_ts(d_tmem, a_base + st * 8u, bdesc + (uint64_t)(st * kStepDesc), idesc,
                                     (uint32_t)((j | st) != 0), tmem_base + kSfCol, tmem_base + kSfCol + 16u);
                        if (j == 0 && st == 0) u_mbar_arrive(bar(kAccStarted + b));     // the overwrite is in the pipe
                    }
                    // frees the operand stage when these MMAs have read it (even and odd uses of a stage have
                    // barriers of their own)
                    u_commit(bar(kOpEmpty + t + kOpStages * (use & 1u)));
                }
                if (!ok) break;
                if (j0 < n_ops) u_commit(bar(kAccFull + b));     // this issuer's share of the accumulator is complete
                else u_mbar_arrive(bar(kAccFull + b));           // (it had no stage in this item)
                op_cnt += (uint32_t)n_ops;
                ++acc_cnt;
            }
            if (!ok) give_up(site, op_cnt, acc_cnt);
        }
    } else if (warp < kAFirstWarp) {
        // ---------------- epilogue ----------------
        const uint32_t quarter = (uint32_t)warp & 3u;      // a warp may only touch TMEM lanes 32 (warp % 4) ..
        // A lane reads 32 consecutive columns of its own row: one 128-byte piece of an output row.  It stages the piece in
        // shared memory and hands it to a bulk reduce-add into the global accumulators (the SM's own atomic path retires
        // about one lane per cycle, several times slower).  Pieces that cannot be 16-byte aligned, or that hang over the
        // last column, go through a transposed loop of coalesced reductions instead.
        uint32_t *tile0 = epi + (warp - kEpiFirstWarp) * (2 * 32 * kEpiStride);
        const bool bulk_ok = (p.N & 3) == 0 && (reinterpret_cast<uintptr_t>(p.acc) & 15u) == 0;
        uint32_t acc_cnt = 0, chunk_cnt = 0;
        for (int32_t pos = u_run_begin(plan, blockIdx.x), end = u_run_begin(plan, blockIdx.x + 1); pos < end && !*s_abort;) {
            const UItem it = u_piece(plan, prefix, tile_planes, pos, end);
            pos += it.adv;
                if (it.n_raw == 0) break;
            const int64_t r = (int64_t)it.rt * kTileM + quarter * 32 + lane;
            int32_t src = __ldg(p.perm + r);
            // nothing of this row in the chunk: its stream ends at or before the first position block of the chunk
            if (__ldg(p.l_sorted + r) <= it.q0 / (p.pos_block * p.planes_per_len) * p.pos_block) src = -1;
            const uint32_t b = single ? 0u : acc_cnt & 1u, acc_phase = (single ? acc_cnt : acc_cnt >> 1) & 1u;
            if (!u_mbar_wait_warp(bar(kAccFull + b), acc_phase, s_abort, lane)) { if (lane == 0) give_up(5, acc_cnt, 0); break; }
            u_fence_after();
#pragma unroll 1
            for (int c = 0; c * 32 < tile_n; ++c, ++chunk_cnt) {
                uint32_t v[32];
                u_tmem_ld32(tmem_base + b * kAccCols + (uint32_t)c * 32u + ((quarter * 32u) << 16), v);
                // the accumulators hold exact fp32 integers
#pragma unroll
                for (int k = 0; k < 32; ++k) v[k] = (uint32_t)__float2int_rn(__uint_as_float(v[k]));
                uint32_t *buf = tile0 + (chunk_cnt & 1u) * (32 * kEpiStride);
                // the bulk operation that read this buffer two chunks ago has finished reading
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                const int64_t col0 = (int64_t)it.ct * tile_n + c * 32;
                // columns of this chunk that exist: inside the tile and inside the matrix
                const int32_t width = (int32_t)min((int64_t)min(32, tile_n - c * 32), p.N - col0);
                if (bulk_ok && width > 0 && (width & 3) == 0) {
                    uint4 *dst = reinterpret_cast<uint4 *>(buf + lane * kEpiStride);
#pragma unroll
                    for (int j = 0; j < 8; ++j) dst[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    if (src >= 0)
                        asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.s32 [%0], [%1], %2;"
                                     ::"l"(p.acc + (int64_t)src * p.N + col0), "r"(u_smem(dst)), "r"((uint32_t)width * 4u) : "memory");
                } else if (width > 0) {
                    __syncwarp();
#pragma unroll
                    for (int k = 0; k < 32; ++k) buf[lane * kEpiStride + k] = v[k];
                    __syncwarp();
                    const int64_t col = col0 + lane;
#pragma unroll 4
                    for (int rr = 0; rr < 32; ++rr) {
                        const int32_t s_rr = __shfl_sync(0xFFFFFFFFu, src, rr);
                        const uint32_t val = buf[rr * kEpiStride + lane];
                        if (s_rr >= 0 && lane < width && val != 0u) atomicAdd(p.acc + (int64_t)s_rr * p.N + col, (int32_t)val);
                    }
                    __syncwarp();
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            u_fence_before();
            __syncwarp();
            if (lane == 0) u_mbar_arrive(bar(kAccEmpty + b));
            ++acc_cnt;
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");      // all reductions of this warp have been performed
    } else if (warp < kWFirstWarp) {
        // ---------------- A expanders: one row per thread, bit planes from global memory into tensor memory ----
        // Group g fills the operand stages n with n % kAGroups == g.  The plane words of a stage come straight from
        // global memory (a warp reads 128 consecutive bytes of a plane); to hide that latency the words of the group's
        // next stage are requested before the current one is expanded, so the walk over pieces and stages runs as two
        // iterators, one stage of the group apart.
        const uint32_t quarter = (uint32_t)warp & 3u;
        const int group = (warp - kAFirstWarp) / kAWarps;
        const int row = (int)(quarter * 32 + lane);
        // Unipolar activations without a negative stream bit in the call (post-ReLU / GELU outputs, attention
        // probabilities) skip the sign words; the two cases are compiled separately so that the unsigned one carries no
        // registers for them.
        const bool a_signed_call = kMode == SC_UNIPOLAR_AND && __ldg(p.scratch + kSlotAnyNegA) != 0;
        auto run_expander = [&](auto signed_tag) {
        constexpr bool a_signed = decltype(signed_tag)::value;
        constexpr int kStagePl = kStagePp;            // A plane words of one operand stage held in registers
        constexpr int kSignWords = a_signed ? 4 : 1;
        struct AIter {
            int32_t pos, end, j, n_ops, my_len, rt, q0, q1, n_raw, adv;
            uint32_t op;
            bool valid;
        };
        auto load_piece = [&](AIter &x) {
            x.valid = x.pos < x.end;
            if (!x.valid) return;
            const UItem it = u_piece(plan, prefix, tile_planes, x.pos, x.end);
            x.adv = it.adv;
            if (it.n_raw == 0) { x.valid = false; return; }
            x.rt = it.rt; x.q0 = it.q0; x.q1 = it.q1; x.n_raw = it.n_raw;
            x.n_ops = it.n_raw * kOpsPerRaw;
            x.j = 0;
            x.my_len = __ldg(p.l_sorted + (int64_t)it.rt * kTileM + row);
        };
        auto advance = [&](AIter &x, int n) {
            for (int a = 0; a < n && x.valid; ++a) {
                ++x.op;
                if (++x.j == x.n_ops) { x.pos += x.adv; load_piece(x); }
            }
        };
        auto fetch = [&](const AIter &x, uint32_t (&dst)[kStagePl], uint32_t (&sgn)[kSignWords]) {
            const int32_t pp0 = x.q0 + x.j * kStagePp;              // first (depth word, position) pair of the stage
            // A row contributes the pairs below the end of this piece whose position lies below its own length; in a
            // stage these are the leading ones: position-major, the pairs below l_i * (depth words); in blocks of 8
            // positions, the stage is positions lb .. lb + 7 of one depth word.
            int32_t n_act;
            if (kMode == SC_BIPOLAR_XNOR) n_act = min(x.my_len * p.planes_per_len, x.q1) - pp0;
            else n_act = min(x.my_len - pp0 / (kPosBlockSigned * p.planes_per_len) * kPosBlockSigned, x.q1 - pp0);
            const uint32_t *src = p.a_streams + (int64_t)pp0 * p.m_pad + (int64_t)x.rt * kTileM + row;
#pragma unroll
            for (int q = 0; q < kStagePl; ++q) dst[q] = q < n_act ? __ldcs(src + (int64_t)q * p.m_pad) : 0u;
            if (a_signed) {
                const int32_t wd = pp0 % (kPosBlockSigned * p.planes_per_len) / kPosBlockSigned;
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p.a_sign) + (int64_t)wd * p.m_pad + (int64_t)x.rt * kTileM + row);
                sgn[0] = v.x; sgn[1 % kSignWords] = v.y; sgn[2 % kSignWords] = v.z; sgn[3 % kSignWords] = v.w;
            }
        };
        AIter cur;
        cur.pos = u_run_begin(plan, blockIdx.x); cur.end = u_run_begin(plan, blockIdx.x + 1); cur.op = 0u;
        load_piece(cur);
        advance(cur, group);
        AIter nxt = cur;
        advance(nxt, kAGroups);
        uint32_t now[kStagePl], ahead[kStagePl], now_s[kSignWords], ahead_s[kSignWords];
        if (cur.valid) fetch(cur, now, now_s);
        bool ok = true;
        while (cur.valid && ok && !*s_abort) {
            if (nxt.valid) fetch(nxt, ahead, ahead_s);
            const uint32_t op_cnt = cur.op, t = op_cnt % kOpStages;
            // The slot of the A ring (depth D) was last read by the MMAs of operand stage op_cnt - D; its barrier is the
            // "stage free" barrier of that operand stage (even and odd uses of a W stage signal different barriers).
            // The A expanders also arrive on the "stage full" barrier of W stage t, whose previous use was operand stage
            // op_cnt - kOpStages.  The two issuers run independently, so with a three-stage A ring the slot can be free
            // (stage op_cnt - 3 consumed) while that previous use has not even been issued yet; an arrival then would be
            // counted in the wrong phase.  Its consumption is therefore awaited first (normally long complete).
            if (a_three && op_cnt >= (uint32_t)kOpStages) {
                const uint32_t puse = op_cnt / kOpStages - 1u;
                ok = u_mbar_wait_warp(bar(kOpEmpty + t + kOpStages * (puse & 1u)), (puse >> 1) & 1u, s_abort, lane);
                if (!ok) break;
            }
            const uint32_t depth = a_three ? 3u : (uint32_t)kOpStages;
            if (op_cnt >= depth) {
                const uint32_t prev = op_cnt - depth, pt = prev % kOpStages, puse = prev / kOpStages;
                ok = u_mbar_wait_warp(bar(kOpEmpty + pt + kOpStages * (puse & 1u)), (puse >> 1) & 1u, s_abort, lane);
                if (!ok) break;
            }
            const uint32_t a_col = tmem_base + a_ring_col + a_slot(op_cnt) * (kOpSteps * 8u) + ((quarter * 32u) << 16);
#pragma unroll
            for (int st = 0; st < kOpSteps; ++st) {
                uint32_t out[8];
                if (!a_signed) {
                    u_expand_bits<false>(now[2 * st], out);
                    u_expand_bits<false>(now[2 * st + 1], out + 4);
                } else {
                    u_expand_signed<false>(now[2 * st], now_s, out);
                    u_expand_signed<false>(now[2 * st + 1], now_s, out + 4);
                }
                u_tmem_st8(a_col + st * 8u, out);
            }
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            u_fence_before();
            __syncwarp();
            if (lane == 0) u_mbar_arrive(bar(kOpFull + t));
#pragma unroll
            for (int q = 0; q < kStagePl; ++q) now[q] = ahead[q];
#pragma unroll
            for (int q = 0; q < kSignWords; ++q) now_s[q] = ahead_s[q];
            cur = nxt;
            advance(nxt, kAGroups);
        }
        if (!ok && lane == 0) give_up(7, cur.op, 0);
        };
        if constexpr (kMode == SC_UNIPOLAR_AND) {
            if (a_signed_call) run_expander(std::true_type{});
            else run_expander(std::false_type{});
        } else {
            run_expander(std::false_type{});
        }
    } else {
        // ---------------- W expanders: two columns per thread, bit planes from the TMA ring into shared memory ----
        const int group = (warp - kWFirstWarp) / kWWarps;
        const int row = ((warp - kWFirstWarp) % kWWarps) * 32 + lane;            // first W column of the thread
        uint32_t raw_cnt = 0, op_cnt = 0;
        int site = 0;
        bool ok = true;
        for (int32_t pos = u_run_begin(plan, blockIdx.x), end = u_run_begin(plan, blockIdx.x + 1); pos < end && ok && !*s_abort;) {
            const UItem it = u_piece(plan, prefix, tile_planes, pos, end);
            pos += it.adv;
                if (it.n_raw == 0) break;
            for (int32_t k = 0; k < (it.n_raw + kRawUnits - 1) / kRawUnits && ok; ++k, ++raw_cnt) {
                const uint32_t s = raw_cnt % kRawStages;
                const int ops_here = min(kRawUnits, it.n_raw - k * kRawUnits) * kOpsPerRaw;    // units present in this box
                // Unipolar: the sign words of this group's stages of the box (a box holds kRawUnits * kOpsPerRaw stages, the
                // group fills every kWGroups-th) are requested from global memory before the box is awaited, so that their
                // latency hides behind that wait.  A stage is eight positions of one depth word: one sign word per column.
                constexpr int kOwnMax = (kRawUnits * kOpsPerRaw + kWGroups - 1) / kWGroups;
                uint4 sg_box[kOwnMax][kWCols];
                if (kMode == SC_UNIPOLAR_AND) {
                    const int first_own = (group + kWGroups - (int)(op_cnt % kWGroups)) % kWGroups;
                    const uint4 *sign_col = reinterpret_cast<const uint4 *>(p.w_sign) + (int64_t)(it.rt / p.tiles_m) * p.w_batch_cols +
                                            (int64_t)it.ct * tile_n + row;
#pragma unroll
                    for (int o = 0; o < kOwnMax; ++o) {
                        const int i = first_own + o * kWGroups;
                        const int32_t pp0 = it.q0 + k * kRawPlanes + i * kStagePp;
                        const int32_t wd = pp0 % (kPosBlockSigned * p.planes_per_len) / kPosBlockSigned;
#pragma unroll
                        for (int c = 0; c < kWCols; ++c)
                            sg_box[o][c] = (i < ops_here && row + c * (kUN / kWCols) < tile_n)
                                               ? __ldg(sign_col + (int64_t)wd * p.n_pad + c * (kUN / kWCols)) : make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                int own = 0;
                site = 6;
                ok = u_mbar_wait_warp(bar(kRawFull + s), (raw_cnt / kRawStages) & 1u, s_abort, lane);
                if (!ok) break;
                site = 8;
                const uint32_t *raw_w = reinterpret_cast<const uint32_t *>(raw + (size_t)s * kRawStageBytes);
                for (int i = 0; i < ops_here; ++i, ++op_cnt) {
                    if ((int)(op_cnt % kWGroups) != group) continue;        // another group's stage
                    const uint32_t t = op_cnt % kOpStages;
                    // the bit words of this operand stage are read before the stage's buffer is awaited, so the
                    // shared-memory latency hides behind the wait
                    constexpr int kStagePl = kStagePp;            // raw planes of one operand stage
                    uint32_t pl[kWCols][kStagePl];
                    uint4 sg[kWCols];
#pragma unroll
                    for (int c = 0; c < kWCols; ++c) {
                        const int idx = row + c * (kUN / kWCols);
                        if (idx >= tile_n) continue;               // beyond the tile: nothing to expand
#pragma unroll
                        for (int q = 0; q < kStagePl; ++q) pl[c][q] = raw_w[(i * kStagePl + q) * kUN + idx];
                        if (kMode == SC_UNIPOLAR_AND) sg[c] = own == 0 ? sg_box[0][c] : sg_box[kOwnMax - 1][c];
                    }
                    ++own;
                    // Use u of a stage waits for the MMAs of use u - 1.  Even and odd uses signal different barriers: a warp
                    // that fills only every third use of a stage would otherwise see the parity it waits for while the
                    // barrier is still two uses behind.
                    if (op_cnt >= (uint32_t)kOpStages) {
                        const uint32_t puse = op_cnt / kOpStages - 1u;
                        ok = u_mbar_wait_warp(bar(kOpEmpty + t + kOpStages * (puse & 1u)), (puse >> 1) & 1u, s_abort, lane);
                    }
                    if (!ok) break;
#pragma unroll
                    for (int c = 0; c < kWCols; ++c) {
                        if (row + c * (kUN / kWCols) >= tile_n) continue;
                        uint8_t *op_b = ops + (size_t)t * kOpStageBytes + (row + c * (kUN / kWCols)) * 16;
                        uint32_t sn[4] = {0u, 0u, 0u, 0u};
                        if (kMode == SC_UNIPOLAR_AND) { sn[0] = sg[c].x; sn[1] = sg[c].y; sn[2] = sg[c].z; sn[3] = sg[c].w; }
#pragma unroll
                        for (int st = 0; st < kOpSteps; ++st) {
                            uint32_t out[8];
                            if (kMode == SC_BIPOLAR_XNOR) {
                                u_expand_bits<true>(pl[c][2 * st], out);
                                u_expand_bits<true>(pl[c][2 * st + 1], out + 4);
                            } else {
                                u_expand_signed<true>(pl[c][2 * st], sn, out);
                                u_expand_signed<true>(pl[c][2 * st + 1], sn, out + 4);
                            }
                            uint8_t *dst = op_b + 2u * st * kLboB;
                            *reinterpret_cast<uint4 *>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
                            *reinterpret_cast<uint4 *>(dst + kLboB) = make_uint4(out[4], out[5], out[6], out[7]);
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA
                    __syncwarp();
                    if (lane == 0) u_mbar_arrive(bar(kOpFull + t));
                }
                if (!ok) break;
                __syncwarp();
                if (lane == 0) u_mbar_arrive(bar(kRawEmpty + s));
            }
        }
        if (!ok && lane == 0) give_up(site, raw_cnt, op_cnt);
    }

    u_fence_before();
    __syncthreads();
    if (warp == 1) {
        u_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---- the bounded wait running out, on purpose ------------------------------------------------------------
// One CTA, two warps, no tensor-core or TMA work: warp 0 waits with the core's own bounded wait on a barrier that
// nobody ever arrives on, with a short limit; when the limit passes it records the wait site beside the status word
// and raises the abort flag, exactly as a role of the core does.  Warp 1 waits on a second such barrier with the
// default (long) limit and must leave through the abort flag.  The kernel then returns normally.
constexpr int kSelftestWaitSite = 99;
__global__ void __launch_bounds__(64)
bounded_wait_selftest_kernel(long long limit_cycles, int32_t *scratch, long long *cycles_out)
{
    __shared__ uint64_t bars[2];
    __shared__ int32_t s_abort_word;
    volatile int32_t *s_abort = &s_abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        u_mbar_init(u_smem(&bars[0]), 1);
        u_mbar_init(u_smem(&bars[1]), 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const long long t0 = clock64();
    bool ok;
    if (warp == 0) {
        ok = u_mbar_wait_warp_limit(u_smem(&bars[0]), 0u, s_abort, lane, limit_cycles);
        if (!ok && lane == 0) {
            if (atomicCAS(scratch + kSlotTimeoutSite, 0, kSelftestWaitSite | (warp << 8) | ((int)blockIdx.x << 16)) == 0) {
                scratch[kSlotTimeoutSite + 1] = 1;
                scratch[kSlotTimeoutSite + 2] = 2;
            }
            *s_abort = 1;
            report(scratch + kSlotStatus, SC_ERR_TIMEOUT);
        }
    } else {
        ok = u_mbar_wait_warp(u_smem(&bars[1]), 0u, s_abort, lane);      // leaves when warp 0 gives up
    }
    if (lane == 0) cycles_out[warp] = ok ? -1 : clock64() - t0;
}

cudaError_t run_bounded_wait_selftest(sc_ctx_impl *ctx, long long limit_cycles, int32_t site_out[3], long long cycles_out[2])
{
    long long *cyc = reinterpret_cast<long long *>(ctx->scratch + 1024);
    cudaError_t e = cudaMemset(cyc, 0, 2 * sizeof(long long));
    if (e != cudaSuccess) return e;
    bounded_wait_selftest_kernel<<<1, 64>>>(limit_cycles, ctx->scratch, cyc);
    count_launches(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return e;
    e = cudaMemcpy(cycles_out, cyc, 2 * sizeof(long long), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return e;
    return cudaMemcpy(site_out, ctx->scratch + kSlotTimeoutSite, 3 * sizeof(int32_t), cudaMemcpyDeviceToHost);
}

// ---- popcount corrections of the bipolar mode ---------------------------------------------------------
// pop_a[source row] += ones in planes [p0, p0 + 64) of the row, below the row's own end.
__global__ void __launch_bounds__(256)
row_popcount_kernel(const uint32_t *__restrict__ A, int64_t m_pad, const int32_t *__restrict__ perm,
                    const int32_t *__restrict__ l_sorted, int32_t planes_per_len, int32_t *__restrict__ pop_a)
{
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= m_pad) return;
    const int32_t src = perm[r];
    if (src < 0) return;
    const int32_t end = l_sorted[r] * planes_per_len;
    const int32_t p0 = blockIdx.y * 64, p1 = min(p0 + 64, end);
    int32_t s = 0;
    for (int32_t q = p0; q < p1; ++q) s += __popc(__ldg(A + (int64_t)q * m_pad + r));
    if (s) atomicAdd(pop_a + src, s);
}

// cnt[(l + 1) * n_pad + j] = ones of column j at stream position l (all depth words); row 0 is zero.
// Positions at or beyond *lmax_actual (when given) are skipped.  One thread per (position, column).
__global__ void __launch_bounds__(256)
col_popcount_kernel(const uint32_t *__restrict__ W, int64_t n_pad, int32_t kw, const int32_t *__restrict__ lmax_actual,
                    int32_t *__restrict__ cnt)
{
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t l = blockIdx.y;
    if (j >= n_pad) return;
    if (l == 0) cnt[j] = 0;
    if (lmax_actual && l >= *lmax_actual) return;
    int32_t s = 0;
    const uint32_t *src = W + (int64_t)l * kw * n_pad + j;
#pragma unroll 8
    for (int32_t w = 0; w < kw; ++w) s += __popc(__ldg(src + (int64_t)w * n_pad));
    cnt[(int64_t)(l + 1) * n_pad + j] = s;
}

// in place: cnt[l][j] <- sum_{l' <= l} cnt[l'][j]  (so row l holds the ones of the positions below l).
// A block owns 32 columns; its 32 x 32 threads split the positions into 32 runs: running sums inside a run, the runs'
// totals scanned through shared memory, the offset of a run added in a second pass.
__global__ void __launch_bounds__(1024)
col_prefix_kernel(int32_t *__restrict__ cnt, int64_t n_pad, const int32_t *__restrict__ lmax_actual, int32_t Lmax)
{
    __shared__ int32_t tot[32][33];
    const int cx = threadIdx.x, ly = threadIdx.y;
    const int64_t j = (int64_t)blockIdx.x * 32 + cx;
    const int32_t L = lmax_actual ? min(__ldg(lmax_actual), Lmax) : Lmax;
    const int32_t run = (L + 31) / 32;
    const int32_t l0 = ly * run, l1 = min(l0 + run, L);
    int32_t sum = 0;
    if (j < n_pad)
        for (int32_t l = l0; l < l1; ++l) {
            sum += cnt[(int64_t)(l + 1) * n_pad + j];
            cnt[(int64_t)(l + 1) * n_pad + j] = sum;
        }
    tot[ly][cx] = sum;
    __syncthreads();
    int32_t offset = 0;
    for (int k = 0; k < ly; ++k) offset += tot[k][cx];
    if (j < n_pad && offset)
        for (int32_t l = l0; l < l1; ++l) cnt[(int64_t)(l + 1) * n_pad + j] += offset;
}

// Ones of every row of A below its own end (bipolar tensor-core form).
cudaError_t launch_row_corrections(const CoreArgs &a, cudaStream_t st)
{
    cudaError_t e = cudaMemsetAsync(a.pop_a, 0, sizeof(int32_t) * (size_t)a.M, st);
    if (e != cudaSuccess) return e;
    const int32_t ppl = a.kw * a.ppq;
    dim3 ga((unsigned)((a.m_pad + 255) / 256), (unsigned)((a.a_planes + 63) / 64));
    row_popcount_kernel<<<ga, 256, 0, st>>>(a.a_streams, a.m_pad, a.perm, a.l_sorted, ppl, a.pop_a);
    count_launches(1);
    return cudaGetLastError();
}

// Prefix ones of every W column for each length 0 .. Lmax (or up to *lmax_actual when given).
cudaError_t launch_col_corrections(const uint32_t *w_streams, int64_t n_pad, int32_t kw, int32_t Lmax,
                                   const int32_t *lmax_actual, int32_t *pop_w, cudaStream_t st)
{
    dim3 gw((unsigned)((n_pad + 255) / 256), (unsigned)Lmax);
    col_popcount_kernel<<<gw, 256, 0, st>>>(w_streams, n_pad, kw, lmax_actual, pop_w);
    col_prefix_kernel<<<(unsigned)((n_pad + 31) / 32), dim3(32, 32), 0, st>>>(pop_w, n_pad, lmax_actual, Lmax);
    count_launches(2);
    return cudaGetLastError();
}

// ---- host side ---------------------------------------------------------------------------------------
bool make_plane_map(CUtensorMap *map, const uint32_t *base, int64_t row_words, int64_t planes, int box_words,
                    int box_planes);

template <int kMode, bool kNarrow>
static cudaError_t launch_umma_mode(const CUtensorMap &mw, const UmmaDev &dev, int sm_count,
                                    cudaStream_t st)
{
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(core_umma_kernel<kMode, kNarrow>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)kUmmaSmem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    core_umma_kernel<kMode, kNarrow><<<sm_count, kUThreads, kUmmaSmem, st>>>(mw, dev);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_core_umma(const CoreArgs &a, cudaStream_t st)
{
    CUtensorMap mw;
    if (!make_plane_map(&mw, a.w_streams, a.n_pad, a.w_planes, kUN, kRawPlanes)) return cudaErrorInvalidValue;
    UmmaDev dev;
    dev.a_streams = a.a_streams; dev.m_pad = a.m_pad;
    dev.perm = a.perm; dev.l_sorted = a.l_sorted; dev.plan = a.plan; dev.acc = a.acc; dev.scratch = a.scratch;
    dev.N = a.N; dev.planes_per_len = a.kw; dev.pos_block = a.pos_block;
    dev.w_sign = a.w_sign; dev.a_sign = a.a_sign; dev.n_pad = a.n_pad;
    dev.tile_n = a.tile_n;
    if (a.tile_n < 32 || a.tile_n > kUN || a.tile_n % 32 != 0) return cudaErrorInvalidValue;
    if (a.mode == SC_UNIPOLAR_AND && (a.pos_block != kPosBlockSigned || !a.w_sign || !a.a_sign)) return cudaErrorInvalidValue;
    if (a.mode != SC_UNIPOLAR_AND && a.pos_block != 1) return cudaErrorInvalidValue;
    dev.tiles_m = a.tiles_m; dev.w_batch_cols = a.w_batch_cols;
    const bool narrow = a.tile_n != kUN;
    if (a.mode == SC_UNIPOLAR_AND)
        return narrow ? launch_umma_mode<SC_UNIPOLAR_AND, true>(mw, dev, a.sm_count, st)
                      : launch_umma_mode<SC_UNIPOLAR_AND, false>(mw, dev, a.sm_count, st);
    return narrow ? launch_umma_mode<SC_BIPOLAR_XNOR, true>(mw, dev, a.sm_count, st)
                  : launch_umma_mode<SC_BIPOLAR_XNOR, false>(mw, dev, a.sm_count, st);
}

}  // namespace sc
