// Two-SM tensor-core GEMM core: the popcount accumulation of Eq. (1) on tcgen05.mma.cta_group::2.
//
// Same contraction and operand encodings as the one-SM core (bits expanded on chip to 4-bit floats, kind::mxf4, exact fp32
// sums; see sc_core_umma.cu), but a tile is 256 rows x 256 columns owned by a PAIR of CTAs on neighbouring SMs (a cluster
// of two): CTA r of the pair holds row tile 2 T + r of the sorted rows (128 rows: its own activation ring and its own
// 128 x 256 accumulator in its tensor memory) and expands columns [128 r, 128 r + 128) of the weight tile into its own
// shared memory; one MMA instruction issued by the first CTA (the leader) multiplies both halves.  Per multiply-accumulate
// a CTA therefore expands 40 % fewer operand bits than with a 128 x 192 tile, writes and reads half the weight bytes
// through shared memory, and the operand rings are six stages deep in both memories (the hand-over chain MMA done ->
// refill -> MMA takes longer than two or three stages of MMAs, which is what bounds the one-SM core).
// The price: one accumulator only (256 of the 512 tensor-memory columns), so the MMAs of a piece wait for the epilogue
// of the previous one.  The plan therefore selects this core for calls whose pieces are long; short pieces run on the
// one-SM core (both kernels are launched, the one not selected returns at once: the choice is device data).
//
// Synchronisation across the pair: "stage full" and "accumulator free" barriers live in the leader and receive remote
// arrivals from the other CTA's warps (plain arrivals: see p_arrive_cta; the waits acquire at cluster scope); "stage free" and
// "accumulator full" are signalled in BOTH CTAs by one multicast tcgen05.commit of the issuing thread.  Each CTA loads its
// own half of the weight tile with its own TMA loads (no multicast loads anywhere).  Every wait is bounded; a wait that runs
// out sets SC_ERR_TIMEOUT, raises the abort flag of both CTAs, all roles drain, both CTAs meet at the cluster barrier and
// free their tensor memory.
// Epilogue: a piece that is a whole tile overwrites the zeroed outputs with plain stores; a piece of a cut tile adds its
// share with bulk reductions (several times dearer for the warp: with one accumulator the MMAs wait for it).
#include <type_traits>

#include "sc_device.cuh"
#include "sc_internal.h"
#include "sc_umma.cuh"

namespace sc {

namespace {

constexpr int kPN = 256;                       // output columns of a pair's tile
constexpr int kPH = kPN / 2;                   // ... of which each CTA expands this many
constexpr int kPRawUnits = 3;                  // plan units (kStagePlanes planes each) per TMA box
constexpr int kPRawPlanes = kPRawUnits * kStagePlanes;
constexpr int kPRawStages = 2;
constexpr int kPOpSteps = 4;                   // MMA K-steps per operand stage
constexpr int kPOpStages = 6;                  // depth of both operand rings
constexpr int kPStagePp = kPOpSteps * 2;       // planes of one operand stage
constexpr int kPOpsPerRaw = kStagePlanes / kPStagePp;
constexpr int kPEpiFirstWarp = 2, kPEpiWarps = 4;
constexpr int kPAFirstWarp = 6, kPAWarps = 4;    // activation expanders: kAG groups (a template parameter: 3, or 2 for short calls) of 4 warps
constexpr int kPWGroups = 3, kPWCols = 2, kPWWarps = kPH / (32 * kPWCols);
__host__ __device__ constexpr int p_w_first_warp(int ag) { return kPAFirstWarp + ag * kPAWarps; }
constexpr int kPIssuers = 2;
__host__ __device__ constexpr int p_issuer_b_warp(int ag) { return p_w_first_warp(ag) + kPWGroups * kPWWarps; }
__host__ __device__ constexpr int p_threads(int ag) { return 32 * (p_issuer_b_warp(ag) + kPIssuers - 1); }
static_assert(kPOpStages % kPIssuers == 0 && kPOpStages % 3 == 0 && kPOpStages % 2 == 0 && kPOpStages % kPWGroups == 0,
              "issuers and expander groups own fixed ring slots");
static_assert(kPAFirstWarp % 4 == 2 && kPAWarps == 4 && kPStagePp == kPosBlockSigned && p_threads(3) <= 1024, "role layout");

constexpr uint32_t kPRawStageBytes = kPRawPlanes * kPH * 4;     // 24 KB
constexpr uint32_t kPLbo = kPH * 16;                            // bytes between the two 16-byte K chunks of a K-step
constexpr uint32_t kPOpStageBytes = kPOpSteps * 2 * kPLbo;      // 16 KB
constexpr int kPEpiStride = 36;
constexpr uint32_t kPEpiBytes = kPEpiWarps * 2 * 32 * kPEpiStride * 4;
constexpr uint32_t kPTmemCols = 512;
constexpr uint32_t kPARingCol = kPN;                            // accumulator: columns 0 .. 255
constexpr uint32_t kPSfCol = 448, kPSfCols = 64;                // scale factors (every byte 2^0): A's at 448, B's at 480
static_assert(kPARingCol + kPOpStages * kPOpSteps * 8 <= kPSfCol && kPSfCol + kPSfCols == kPTmemCols, "tensor memory budget");
constexpr int kPShortCallStages = 1024;                         // below this many stages per CTA pair (twice as many for bipolar calls): two activation expander groups
constexpr int kPMaxPairs = 1024;                                // row-tile pairs whose unit prefix fits the shared-memory table

// "stage full" is four barriers per ring slot -- the activation and the weight expanders of either CTA arrive on a
// barrier of their own, the issuer awaits all four -- because arrivals on one barrier are served one after another.
enum PBar : int {
    kPRawFull = 0, kPRawEmpty = kPRawFull + kPRawStages, kPOpFull = kPRawEmpty + kPRawStages,
    kPOpEmpty = kPOpFull + 4 * kPOpStages, kPAccFull = kPOpEmpty + 2 * kPOpStages, kPAccEmpty = kPAccFull + 1,
    kPAccStarted = kPAccEmpty + 1, kPNumBars = kPAccStarted + 1
};
constexpr size_t kPairSmem = (size_t)kPRawStages * kPRawStageBytes + (size_t)kPOpStages * kPOpStageBytes + kPEpiBytes +
                             (kPMaxPairs + 1) * 4 + 12 + kPNumBars * 8 + 16;

struct PairDev {
    const uint32_t *a_streams;        // A planes [plane][m_pad]
    int64_t m_pad;
    const int32_t *perm, *l_sorted;
    const PlanHeader *plan;
    int32_t *acc;
    int32_t *scratch;
    int64_t N;
    int32_t planes_per_len, pos_block;
    int32_t n_col_tiles;              // column tiles of kPN columns
    int32_t force;                    // run whatever the plan selected
    const uint32_t *w_sign, *a_sign;  // unipolar: nibble sign words
    int64_t n_pad;
    int32_t acc_map_ok;               // the tensor map of the accumulators is valid (aligned, N % 4 == 0)
};

__device__ __forceinline__ uint32_t p_cluster_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void p_cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `cta` of the pair: the plain form, a release at CTA scope.
// What the arrival hands over never needs more.  Operand A and the accumulators live in tensor memory, ordered by
// tcgen05.wait and tcgen05.fence::before_thread_sync.  Operand W is written by ordinary stores to the ARRIVING CTA's own
// shared memory and published to the async proxy by fence.proxy.async before the arrival; the two-SM MMA reads each CTA's
// half of W from that CTA's own shared memory, so the leader's issuing thread passes on only the barrier's phase.  A release
// at cluster scope adds a fence that costs each expander warp a quarter of its time: measured, 13 - 20 % of the kernel's
// time, all of it on the W side, which is the critical path.
__device__ __forceinline__ void p_arrive_cta(uint32_t bar, uint32_t cta)
{
    asm volatile("{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\t"
                 "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}" ::"r"(bar), "r"(cta) : "memory");
}
__device__ __forceinline__ void p_store_cta(uint32_t addr, uint32_t cta, uint32_t value)
{
    asm volatile("{\n\t.reg .b32 ra;\n\tmapa.shared::cluster.u32 ra, %0, %1;\n\tst.shared::cluster.u32 [ra], %2;\n\t}"
                 ::"r"(addr), "r"(cta), "r"(value) : "memory");
}
__device__ __forceinline__ bool p_mbar_try_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded, abortable wait on a barrier that also receives arrivals from the other CTA
__device__ __forceinline__ bool p_mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int32_t *abort_flag)
{
    long long t0 = 0;
    for (uint32_t spins = 1;; ++spins) {
        if (p_mbar_try_cluster(bar, parity)) return true;
        if ((spins & 63u) == 0u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kUWaitCycles) return false;
        }
    }
}
// The same wait by a whole warp on the four consecutive barriers from `bar0` at once: lane k polls barrier k % 4, so the four
// polls are one instruction and their latencies overlap.  (Polled one after the other by one thread they cost about 350 clocks
// each even when complete, which made the issuing threads the bottleneck of the kernel.)  Uniform result.
__device__ __forceinline__ bool p_mbar_wait4_warp(uint32_t bar0, uint32_t parity, volatile int32_t *abort_flag, int lane)
{
    const uint32_t mine = bar0 + 8u * (uint32_t)(lane & 3);
    long long t0 = 0;
    for (uint32_t spins = 1;; ++spins) {
        const bool done = p_mbar_try_cluster(mine, parity);
        if (__all_sync(0xFFFFFFFFu, done)) return true;
        if ((spins & 63u) == 0u) {
            bool stop = *abort_flag != 0;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kUWaitCycles) stop = true;
            if (__any_sync(0xFFFFFFFFu, stop)) return false;
        }
    }
}
// D[tmem of both CTAs] (+)= A[tmem of both CTAs] x B[shared memory of both CTAs], 256 x 256 x 64
__device__ __forceinline__ void p_mma_fp4_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate,
                                             uint32_t sfa_tmem, uint32_t sfb_tmem)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.scale_vec::2X [%0], [%1], %2, %3, [%5], [%6], p;\n\t}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem) : "memory");
}
// the barrier at this offset in BOTH CTAs receives one arrival when the MMAs issued so far by this thread are complete
__device__ __forceinline__ void p_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}

struct PItem {
    int32_t pair, ct, q0, q1, n_raw;
    bool whole;             // the piece is the whole (tile pair, column tile): nothing else adds to these outputs
};

// stage units of a pair per column tile: the longer (first) row tile of the pair decides
__device__ __forceinline__ int32_t p_units(int32_t planes) { return (planes + kStagePlanes - 1) / kStagePlanes; }

__device__ __forceinline__ PItem p_piece(const int32_t *s_prefix, int32_t n_pairs, const int32_t *tile_planes, int32_t n_col_tiles,
                                         int32_t pos, int32_t end)
{
    int32_t lo = 0, hi = n_pairs;                          // largest pair with prefix <= pos (skips empty pairs)
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (s_prefix[mid] <= pos) lo = mid; else hi = mid;
    }
    PItem it;
    it.pair = lo;
    const int32_t planes = __ldg(tile_planes + 2 * lo);
    const int32_t stages = p_units(planes);
    const int32_t local = pos - s_prefix[lo];
    it.ct = local / stages;
    const int32_t s0 = local - it.ct * stages;
    const int32_t s1 = min(stages, s0 + (end - pos));
    it.q0 = s0 * kStagePlanes;
    it.q1 = min(s1 * kStagePlanes, planes);
    it.n_raw = s1 - s0;
    it.whole = s0 == 0 && s1 == stages;
    (void)n_col_tiles;
    return it;
}

// kAG: groups of activation expander warps.  Three keep up with long pieces; with two the CTA is 22 warps instead of 26, which
// is 1 - 3 % faster on calls of a few hundred stages per CTA pair (measured: config 2 0.204 -> 0.198 ms) and 1.5 - 3 % slower on
// long ones; the host picks by the stages a pair can get at most.
template <int kMode, int kAG>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(p_threads(kAG), 1)
core_umma_pair_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_acc, PairDev p)
{
    constexpr int kPAGroups = kAG, kPWFirstWarp = p_w_first_warp(kAG), kPIssuerBWarp = p_issuer_b_warp(kAG), kPThreads = p_threads(kAG);
    const PlanHeader plan = *p.plan;
    if (!p.force && plan.pad[0] == 0) return;              // the plan chose the one-SM core (same decision in every CTA)
    const int32_t n_pairs = (plan.n_row_tiles + 1) / 2;
    if (n_pairs > kPMaxPairs) return;                      // (the host does not launch such calls)

    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t *raw = smem;
    uint8_t *ops = smem + (size_t)kPRawStages * kPRawStageBytes;
    uint32_t *epi = reinterpret_cast<uint32_t *>(ops + (size_t)kPOpStages * kPOpStageBytes);
    int32_t *s_prefix = reinterpret_cast<int32_t *>(reinterpret_cast<uint8_t *>(epi) + kPEpiBytes);
    uint64_t *bars = reinterpret_cast<uint64_t *>(s_prefix + kPMaxPairs + 1 + 3);
    uint32_t *s_tmem = reinterpret_cast<uint32_t *>(bars + kPNumBars);
    volatile int32_t *s_abort = reinterpret_cast<volatile int32_t *>(s_tmem + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = p_cluster_rank();
    const int32_t cluster = (int32_t)(blockIdx.x >> 1), n_clusters = (int32_t)(gridDim.x >> 1);
    const uint32_t bars_addr = u_smem(bars), raw_addr = u_smem(raw), ops_addr = u_smem(ops);
    auto bar = [&](int which) { return bars_addr + 8u * (uint32_t)which; };
    const int32_t *tile_planes = reinterpret_cast<const int32_t *>(p.plan + 1) + plan.n_row_tiles + 1;

    if (tid == 0) {
        for (int s = 0; s < kPRawStages; ++s) { u_mbar_init(bar(kPRawFull + s), 1); u_mbar_init(bar(kPRawEmpty + s), kPWGroups * kPWWarps); }
        for (int s = 0; s < kPOpStages; ++s)
            for (int k = 0; k < 4; ++k) u_mbar_init(bar(kPOpFull + 4 * s + k), k < 2 ? kPAWarps : kPWWarps);
        for (int s = 0; s < 2 * kPOpStages; ++s) u_mbar_init(bar(kPOpEmpty + s), 1);
        u_mbar_init(bar(kPAccFull), kPIssuers);
        u_mbar_init(bar(kPAccEmpty), 2 * kPEpiWarps);
        u_mbar_init(bar(kPAccStarted), 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // running totals of the stage units of the pairs: s_prefix[T] = units of pairs 0 .. T - 1
    for (int32_t T = tid; T < n_pairs; T += kPThreads) s_prefix[T + 1] = p_units(__ldg(tile_planes + 2 * T)) * p.n_col_tiles;
    if (tid == 0) s_prefix[0] = 0;
    __syncthreads();
    if (warp == 2) {
        // inclusive scan by one warp: every lane owns a run of consecutive entries
        const int32_t per = (n_pairs + 31) / 32;
        const int32_t t0 = min(lane * per, n_pairs), t1 = min(t0 + per, n_pairs);
        int32_t local = 0;
        for (int32_t T = t0; T < t1; ++T) local += s_prefix[T + 1];
        int32_t incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += up;
        }
        int32_t run = incl - local;
        for (int32_t T = t0; T < t1; ++T) { run += s_prefix[T + 1]; s_prefix[T + 1] = run; }
    }
    p_cluster_sync();                                      // barriers of both CTAs initialised (also a CTA-wide barrier)
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(u_smem(s_tmem)), "r"(kPTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    u_fence_before();
    __syncthreads();
    u_fence_after();
    const uint32_t tmem_base = *s_tmem;
    if (warp >= kPAFirstWarp && warp < kPAFirstWarp + kPAWarps) {
        // scale factors: every byte 0x7F = 2^0 (ue8m0), whatever the scale layout picks
        uint32_t ones[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) ones[k] = 0x7F7F7F7Fu;
#pragma unroll
        for (uint32_t c = 0; c < kPSfCols; c += 8) u_tmem_st8(tmem_base + kPSfCol + c + ((((uint32_t)warp & 3u) * 32u) << 16), ones);
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    u_fence_before();
    p_cluster_sync();                                      // scale factors of both CTAs in place before the first MMA
    u_fence_after();

    const int32_t total = s_prefix[n_pairs];
    const int32_t run0 = (int32_t)((long long)total * cluster / n_clusters);
    const int32_t run1 = (int32_t)((long long)total * (cluster + 1) / n_clusters);
    const int32_t ppl = p.planes_per_len;

    // The first role that gives up records where; both CTAs of the pair are told to drain.
    auto give_up = [&](int site, uint32_t cnt_a, uint32_t cnt_b) {
        if (*s_abort == 0 && atomicCAS(p.scratch + kSlotTimeoutSite, 0, (site + 32) | (warp << 8) | ((int)blockIdx.x << 16)) == 0) {
            p.scratch[kSlotTimeoutSite + 1] = (int32_t)cnt_a;
            p.scratch[kSlotTimeoutSite + 2] = (int32_t)cnt_b;
        }
        *s_abort = 1;
        p_store_cta(u_smem(const_cast<int32_t *>(s_abort)), rank ^ 1u, 1u);
        report(p.scratch + kSlotStatus, SC_ERR_TIMEOUT);
    };

    if (warp == 0) {
        // ---------------- TMA producer: this CTA's half of the weight tile ----------------
        if (lane == 0) {
            uint32_t raw_cnt = 0;
            bool ok = true;
            for (int32_t pos = run0; pos < run1 && ok && !*s_abort;) {
                const PItem it = p_piece(s_prefix, n_pairs, tile_planes, p.n_col_tiles, pos, run1);
                pos += it.n_raw;
                for (int32_t k = 0; k < (it.n_raw + kPRawUnits - 1) / kPRawUnits; ++k, ++raw_cnt) {
                    const uint32_t s = raw_cnt % kPRawStages;
                    ok = u_mbar_wait(bar(kPRawEmpty + s), ((raw_cnt / kPRawStages) & 1u) ^ 1u, s_abort);
                    if (!ok) break;
                    u_mbar_expect_tx(bar(kPRawFull + s), kPRawStageBytes);
                    u_tma_load_2d(raw_addr + s * kPRawStageBytes, &map_w, it.ct * kPN + (int32_t)rank * kPH,
                                  it.q0 + k * kPRawPlanes, bar(kPRawFull + s));
                }
            }
            if (!ok) give_up(1, raw_cnt, 0);
        }
    } else if (warp == 1 || warp >= kPIssuerBWarp) {
        // ---------------- MMA issuers (leader CTA): issuer i owns the stages n with n % kPIssuers == i ----------------
        // The whole warp walks the pieces and polls (one barrier per lane); lane 0 issues.  The path of an issuer per stage is
        // kept short: it, not the tensor pipe, bounds the kernel as soon as it takes longer than kPIssuers stages of MMAs.
        if (rank == 0) {
            const uint32_t me = warp == 1 ? 0u : (uint32_t)(warp - kPIssuerBWarp + 1);
            uint32_t op_cnt = 0, acc_cnt = 0;                     // stages / pieces before the current piece
            bool ok = true;
            int site = 0;
            const uint64_t desc0 = u_smem_desc(ops_addr, kPLbo);
            constexpr uint32_t kStepDesc = (2u * kPLbo) >> 4, kStageDesc = kPOpStageBytes >> 4;
            constexpr uint32_t idesc = u_idesc_fp4(256u, (uint32_t)kPN);
            for (int32_t pos = run0; pos < run1 && ok && !*s_abort;) {
                const PItem it = p_piece(s_prefix, n_pairs, tile_planes, p.n_col_tiles, pos, run1);
                pos += it.n_raw;
                const uint32_t acc_phase = acc_cnt & 1u;
                const uint32_t first = op_cnt % kPIssuers;        // owner of the piece's first stage: it overwrites
                site = 2;
                {
                    int good = 1;
                    if (lane == 0) good = p_mbar_wait_cluster(bar(kPAccEmpty), acc_phase ^ 1u, s_abort) ? 1 : 0;
                    ok = __shfl_sync(0xFFFFFFFFu, good, 0) != 0;
                }
                if (ok && me != first) { site = 3; ok = u_mbar_wait_warp(bar(kPAccStarted), acc_phase, s_abort, lane); }
                if (!ok) break;
                site = 4;
                const int32_t n_ops = it.n_raw * kPOpsPerRaw;
                const int32_t j0 = (int32_t)((me + kPIssuers - first) % kPIssuers);
                for (int32_t j = j0; j < n_ops; j += kPIssuers) {
                    const uint32_t op = op_cnt + (uint32_t)j;
                    const uint32_t t = op % kPOpStages, use = op / kPOpStages;
                    ok = p_mbar_wait4_warp(bar(kPOpFull + 4 * t), use & 1u, s_abort, lane);
                    if (!ok) break;
                    u_fence_after();
                    if (lane == 0) {
                        const uint64_t bdesc = desc0 + (uint64_t)(t * kStageDesc);
                        const uint32_t a_base = tmem_base + kPARingCol + t * (kPOpSteps * 8u);
#pragma unroll
                        for (int st = 0; st < kPOpSteps; ++st) {
                            p_mma_fp4_ts(tmem_base, a_base + st * 8u, bdesc + (uint64_t)(st * kStepDesc), idesc,
                                         (uint32_t)((j | st) != 0), tmem_base + kPSfCol, tmem_base + kPSfCol + 32u);
                            if (j == 0 && st == 0) u_mbar_arrive(bar(kPAccStarted));       // the overwrite is in the pipe
                        }
                        // frees the ring slot in both CTAs when these MMAs have read it (even and odd uses of a slot signal
                        // barriers of their own)
                        p_commit_pair(bar(kPOpEmpty + t + kPOpStages * (use & 1u)));
                    }
                }
                if (!ok) break;
                if (lane == 0) {
                    if (j0 < n_ops) p_commit_pair(bar(kPAccFull));    // this issuer's share of the accumulators is complete
                    else { p_arrive_cta(bar(kPAccFull), 0u); p_arrive_cta(bar(kPAccFull), 1u); }      // (no stage of its own in this piece)
                }
                op_cnt += (uint32_t)n_ops;
                ++acc_cnt;
            }
            if (!ok && lane == 0) give_up(site, op_cnt, acc_cnt);
        }
    } else if (warp < kPAFirstWarp) {
        // ---------------- epilogue: this CTA's 128 rows of the 256 x 256 accumulator ----------------
        const uint32_t quarter = (uint32_t)warp & 3u;
        uint32_t *tile0 = epi + (warp - kPEpiFirstWarp) * (2 * 32 * kPEpiStride);
        const bool bulk_ok = (p.N & 3) == 0 && (reinterpret_cast<uintptr_t>(p.acc) & 15u) == 0;
        uint32_t acc_cnt = 0, chunk_cnt = 0;
        for (int32_t pos = run0; pos < run1 && !*s_abort;) {
            const PItem it = p_piece(s_prefix, n_pairs, tile_planes, p.n_col_tiles, pos, run1);
            pos += it.n_raw;
            const int32_t rt = 2 * it.pair + (int32_t)rank;
            int32_t src = -1;
            if (rt < plan.n_row_tiles) {
                const int64_t r = (int64_t)rt * kTileM + quarter * 32 + lane;
                src = __ldg(p.perm + r);
                // nothing of this row in the chunk: its stream ends at or before the first position block of the chunk
                if (__ldg(p.l_sorted + r) <= it.q0 / (p.pos_block * ppl) * p.pos_block) src = -1;
            }
            // A cut piece whose 32 rows of this warp are consecutive rows of the output (uniform or grouped lengths: the stable
            // sort keeps them together) adds each 32 x 32 chunk with ONE bulk tensor reduction instead of 32 row pieces.
            int32_t run_row = -1;
            if (p.acc_map_ok && !it.whole) {
                const unsigned valid = __ballot_sync(0xFFFFFFFFu, src >= 0);
                if (valid != 0u) {
                    const int first = __ffs((int)valid) - 1;
                    const int32_t ref = __shfl_sync(0xFFFFFFFFu, src, first) - first;
                    if (ref >= 0 && __all_sync(0xFFFFFFFFu, src < 0 || src == ref + lane)) run_row = ref;
                }
            }
            if (!u_mbar_wait_warp(bar(kPAccFull), acc_cnt & 1u, s_abort, lane)) { if (lane == 0) give_up(5, acc_cnt, 0); break; }
            u_fence_after();
            if (__any_sync(0xFFFFFFFFu, src >= 0)) {
#pragma unroll 1
                for (int c = 0; c < kPN / 32; ++c, ++chunk_cnt) {
                    uint32_t v[32];
                    u_tmem_ld32(tmem_base + (uint32_t)c * 32u + ((quarter * 32u) << 16), v);
#pragma unroll
                    for (int k = 0; k < 32; ++k) v[k] = (uint32_t)__float2int_rn(__uint_as_float(v[k]));   // exact fp32 integers
                    uint32_t *buf = tile0 + (chunk_cnt & 1u) * (32 * kPEpiStride);
                    asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");     // the buffer's previous reduction has read it
                    __syncwarp();                          // ... whichever lane issued it (lane 0 issues the tensor reductions)
                    const int64_t col0 = (int64_t)it.ct * kPN + c * 32;
                    if (it.whole) {
                        // No other piece adds to this tile: the zeroed outputs are simply overwritten, straight from the
                        // registers (eight 16-byte stores per row piece; a dozen instructions per chunk).  With one accumulator
                        // the MMAs wait for the epilogue, and the bulk reduction below costs the warp about 2000 clocks per chunk.
                        if (src >= 0) {
                            int32_t *row = p.acc + (int64_t)src * p.N + col0;
                            if (bulk_ok && col0 + 32 <= p.N) {
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    reinterpret_cast<uint4 *>(row)[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                            } else {
#pragma unroll
                                for (int k = 0; k < 32; ++k)
                                    if (col0 + k < p.N) row[k] = (int32_t)v[k];
                            }
                        }
                    } else if (run_row >= 0 && col0 < p.N) {
                        // (rows of the warp without a stream in this piece hold zeros or do not exist: a lane without a row
                        // adds nothing; rows and columns beyond the matrix are clipped by the tensor map)
                        uint8_t *dense = reinterpret_cast<uint8_t *>(tile0) + (chunk_cnt & 1u) * 5120u;
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<uint4 *>(dense + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                src >= 0 ? make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]) : make_uint4(0u, 0u, 0u, 0u);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0)
                            asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                                         ::"l"(reinterpret_cast<uint64_t>(&map_acc)), "r"((int32_t)col0), "r"(run_row), "r"(u_smem(dense))
                                         : "memory");
                    } else if (bulk_ok && col0 + 32 <= p.N) {
                        uint4 *dst = reinterpret_cast<uint4 *>(buf + lane * kPEpiStride);
#pragma unroll
                        for (int j = 0; j < 8; ++j) dst[j] = make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        if (src >= 0)
                            asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.s32 [%0], [%1], 128;"
                                         ::"l"(p.acc + (int64_t)src * p.N + col0), "r"(u_smem(dst)) : "memory");
                    } else if (col0 < p.N) {
                        __syncwarp();
#pragma unroll
                        for (int k = 0; k < 32; ++k) buf[lane * kPEpiStride + k] = v[k];
                        __syncwarp();
                        const int64_t col = col0 + lane;
#pragma unroll 4
                        for (int rr = 0; rr < 32; ++rr) {
                            const int32_t s_rr = __shfl_sync(0xFFFFFFFFu, src, rr);
                            const uint32_t val = buf[rr * kPEpiStride + lane];
                            if (s_rr >= 0 && col < p.N && val != 0u) atomicAdd(p.acc + (int64_t)s_rr * p.N + col, (int32_t)val);
                        }
                        __syncwarp();
                    }
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            u_fence_before();
            __syncwarp();
            if (lane == 0) p_arrive_cta(bar(kPAccEmpty), 0u);
            ++acc_cnt;
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    } else if (warp < kPWFirstWarp) {
        // ---------------- A expanders: one row per thread, bit planes from global memory into this CTA's tensor memory ----
        const uint32_t quarter = (uint32_t)warp & 3u;
        const int group = (warp - kPAFirstWarp) / kPAWarps;
        const int row = (int)(quarter * 32 + lane);
        const bool a_signed_call = kMode == SC_UNIPOLAR_AND && __ldg(p.scratch + kSlotAnyNegA) != 0;
        auto run_expander = [&](auto signed_tag) {
            constexpr bool a_signed = decltype(signed_tag)::value;
            constexpr int kSignWords = a_signed ? 4 : 1;
            // The walk over this group's stages: `it` names the next stage to request from global memory.  The expander is on
            // the critical path of the core, so the walk is kept cheap: a running plane pointer, the number of planes the
            // row still takes part in as a running count, whole-group steps.
            struct AIter {
                int32_t pos, j, n_ops, n_raw, lim;         // lim: planes of the piece this row takes part in (position-major)
                int32_t my_len, q0, q1, rt;                // (blocked positions: needed to find the stage's position block)
                uint32_t op;
                bool valid;
                const uint32_t *src;                       // this row's word of plane q0 + 8 j
            };
            const int64_t stage_stride = (int64_t)kPStagePp * p.m_pad;
            auto load_piece = [&](AIter &x) {
                x.valid = x.pos < run1;
                if (!x.valid) return;
                const PItem pc = p_piece(s_prefix, n_pairs, tile_planes, p.n_col_tiles, x.pos, run1);
                x.rt = 2 * pc.pair + (int32_t)rank; x.q0 = pc.q0; x.q1 = pc.q1; x.n_raw = pc.n_raw;
                x.n_ops = pc.n_raw * kPOpsPerRaw;
                x.j = 0;
                // the second row tile of the last pair may not exist: no row, nothing to read
                x.my_len = x.rt < plan.n_row_tiles ? __ldg(p.l_sorted + (int64_t)x.rt * kTileM + row) : 0;
                x.lim = min(x.my_len * ppl, pc.q1) - pc.q0;
                x.src = p.a_streams + (int64_t)pc.q0 * p.m_pad + (int64_t)x.rt * kTileM + row;
            };
            auto advance = [&](AIter &x) {                 // to the group's next stage
                x.op += kPAGroups;
                x.j += kPAGroups;
                x.src += kPAGroups * stage_stride;
                if (x.j >= x.n_ops) {
                    int32_t over = x.j - x.n_ops;
                    x.pos += x.n_raw;
                    load_piece(x);
                    while (x.valid && over >= x.n_ops) { over -= x.n_ops; x.pos += x.n_raw; load_piece(x); }
                    if (x.valid) { x.j = over; x.src += over * stage_stride; }
                }
            };
            auto fetch = [&](const AIter &x, uint32_t (&dst)[kPStagePp], uint32_t (&sgn)[kSignWords]) {
                int32_t n_act;                                 // leading planes of the stage the row takes part in
                if (kMode == SC_BIPOLAR_XNOR) {
                    n_act = x.lim - x.j * kPStagePp;
                } else {
                    const int32_t pp0 = x.q0 + x.j * kPStagePp;    // blocks of 8 positions: the stage is positions lb .. lb + 7
                    n_act = min(x.my_len - pp0 / (kPosBlockSigned * ppl) * kPosBlockSigned, x.q1 - pp0);
                }
#pragma unroll
                for (int q = 0; q < kPStagePp; ++q) dst[q] = q < n_act ? __ldg(x.src + (int64_t)q * p.m_pad) : 0u;
                if (a_signed) {
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (n_act > 0) {
                        const int32_t wd = (x.q0 + x.j * kPStagePp) % (kPosBlockSigned * ppl) / kPosBlockSigned;
                        v = __ldg(reinterpret_cast<const uint4 *>(p.a_sign) + (int64_t)wd * p.m_pad + (int64_t)x.rt * kTileM + row);
                    }
                    sgn[0] = v.x; sgn[1 % kSignWords] = v.y; sgn[2 % kSignWords] = v.z; sgn[3 % kSignWords] = v.w;
                }
            };
            bool ok = true;
            // expands one stage (operand stage op_cnt) from the words in `w` into the ring slot and hands it over
            auto process = [&](const uint32_t (&w)[kPStagePp], const uint32_t (&ws)[kSignWords], uint32_t op_cnt) {
                const uint32_t t = op_cnt % kPOpStages;
                if (op_cnt >= (uint32_t)kPOpStages) {          // the slot's previous use has been read by its MMAs
                    const uint32_t puse = op_cnt / kPOpStages - 1u;
                    ok = u_mbar_wait_warp(bar(kPOpEmpty + t + kPOpStages * (puse & 1u)), (puse >> 1) & 1u, s_abort, lane);
                    if (!ok) return;
                }
                const uint32_t a_col = tmem_base + kPARingCol + t * (kPOpSteps * 8u) + ((quarter * 32u) << 16);
#pragma unroll
                for (int st = 0; st < kPOpSteps; ++st) {
                    uint32_t out[8];
                    if (!a_signed) {
                        u_expand_bits<false>(w[2 * st], out);
                        u_expand_bits<false>(w[2 * st + 1], out + 4);
                    } else {
                        u_expand_signed<false>(w[2 * st], ws, out);
                        u_expand_signed<false>(w[2 * st + 1], ws, out + 4);
                    }
                    u_tmem_st8(a_col + st * 8u, out);
                }
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                u_fence_before();
                __syncwarp();
                if (lane == 0) p_arrive_cta(bar(kPOpFull + 4 * t + rank), 0u);
            };
            AIter it;
            it.pos = run0; it.op = 0u;
            load_piece(it);
            if (it.valid && group > 0) {                       // the group's first stage
                it.op = (uint32_t)(group - kPAGroups); it.j = group - kPAGroups; it.src += (int64_t)(group - kPAGroups) * stage_stride;
                advance(it);
            }
            // Two register sets take turns.  The words of a stage are requested right after the group's previous hand-over and
            // used two hand-overs later: they have a whole period of the group to land, and no load of the thread is in flight
            // when it arrives on the barrier.
            uint32_t w0[kPStagePp], w1[kPStagePp], s0[kSignWords], s1[kSignWords];
            uint32_t op0 = it.op, op1 = 0u;
            bool v0 = it.valid, v1 = false;
            if (v0) { fetch(it, w0, s0); advance(it); }
            v1 = it.valid; op1 = it.op;
            if (v1) { fetch(it, w1, s1); advance(it); }
            while (v0 && ok && !*s_abort) {
                process(w0, s0, op0);
                if (!ok || *s_abort) break;
                v0 = it.valid; op0 = it.op;
                if (v0) { fetch(it, w0, s0); advance(it); }
                if (!v1) break;
                process(w1, s1, op1);
                if (!ok || *s_abort) break;
                v1 = it.valid; op1 = it.op;
                if (v1) { fetch(it, w1, s1); advance(it); }
            }
            if (!ok && lane == 0) give_up(7, op0, op1);
        };
        if constexpr (kMode == SC_UNIPOLAR_AND) {
            if (a_signed_call) run_expander(std::true_type{});
            else run_expander(std::false_type{});
        } else {
            run_expander(std::false_type{});
        }
    } else {
        // ---------------- W expanders: two columns per thread, bit planes from the TMA ring into shared memory ----
        const int group = (warp - kPWFirstWarp) / kPWWarps;
        const int row = ((warp - kPWFirstWarp) % kPWWarps) * 32 + lane;           // first column of the thread (of this CTA's 128)
        uint32_t raw_cnt = 0, op_cnt = 0;
        int site = 0;
        bool ok = true;
        for (int32_t pos = run0; pos < run1 && ok && !*s_abort;) {
            const PItem it = p_piece(s_prefix, n_pairs, tile_planes, p.n_col_tiles, pos, run1);
            pos += it.n_raw;
            for (int32_t k = 0; k < (it.n_raw + kPRawUnits - 1) / kPRawUnits && ok; ++k, ++raw_cnt) {
                const uint32_t s = raw_cnt % kPRawStages;
                const int ops_here = min(kPRawUnits, it.n_raw - k * kPRawUnits) * kPOpsPerRaw;
                // unipolar: the sign words of this group's stages of the box, requested before the box is awaited
                constexpr int kOwnMax = (kPRawUnits * kPOpsPerRaw + kPWGroups - 1) / kPWGroups;
                uint4 sg_box[kOwnMax][kPWCols];
                if (kMode == SC_UNIPOLAR_AND) {
                    const int first_own = (group + kPWGroups - (int)(op_cnt % kPWGroups)) % kPWGroups;
                    const int64_t col = (int64_t)it.ct * kPN + (int64_t)rank * kPH + row;
#pragma unroll
                    for (int o = 0; o < kOwnMax; ++o) {
                        const int i = first_own + o * kPWGroups;
                        const int32_t pp0 = it.q0 + k * kPRawPlanes + i * kPStagePp;
                        const int32_t wd = pp0 % (kPosBlockSigned * ppl) / kPosBlockSigned;
#pragma unroll
                        for (int c = 0; c < kPWCols; ++c) {
                            const int64_t cc = col + c * (kPH / kPWCols);
                            sg_box[o][c] = (i < ops_here && cc < p.n_pad)
                                               ? __ldg(reinterpret_cast<const uint4 *>(p.w_sign) + (int64_t)wd * p.n_pad + cc)
                                               : make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                }
                int own = 0;
                site = 6;
                ok = u_mbar_wait_warp(bar(kPRawFull + s), (raw_cnt / kPRawStages) & 1u, s_abort, lane);
                if (!ok) break;
                site = 8;
                const uint32_t *raw_w = reinterpret_cast<const uint32_t *>(raw + (size_t)s * kPRawStageBytes);
                for (int i = 0; i < ops_here; ++i, ++op_cnt) {
                    if ((int)(op_cnt % kPWGroups) != group) continue;
                    const uint32_t t = op_cnt % kPOpStages;
                    uint32_t pl[kPWCols][kPStagePp];
                    uint4 sg[kPWCols];
#pragma unroll
                    for (int c = 0; c < kPWCols; ++c) {
                        const int idx = row + c * (kPH / kPWCols);
#pragma unroll
                        for (int q = 0; q < kPStagePp; ++q) pl[c][q] = raw_w[(i * kPStagePp + q) * kPH + idx];
                        if (kMode == SC_UNIPOLAR_AND) sg[c] = own == 0 ? sg_box[0][c] : sg_box[kOwnMax - 1][c];
                    }
                    ++own;
                    if (op_cnt >= (uint32_t)kPOpStages) {
                        const uint32_t puse = op_cnt / kPOpStages - 1u;
                        ok = u_mbar_wait_warp(bar(kPOpEmpty + t + kPOpStages * (puse & 1u)), (puse >> 1) & 1u, s_abort, lane);
                    }
                    if (!ok) break;
#pragma unroll
                    for (int c = 0; c < kPWCols; ++c) {
                        uint8_t *op_b = ops + (size_t)t * kPOpStageBytes + (row + c * (kPH / kPWCols)) * 16;
                        uint32_t sn[4] = {0u, 0u, 0u, 0u};
                        if (kMode == SC_UNIPOLAR_AND) { sn[0] = sg[c].x; sn[1] = sg[c].y; sn[2] = sg[c].z; sn[3] = sg[c].w; }
#pragma unroll
                        for (int st = 0; st < kPOpSteps; ++st) {
                            uint32_t out[8];
                            if (kMode == SC_BIPOLAR_XNOR) {
                                u_expand_bits<true>(pl[c][2 * st], out);
                                u_expand_bits<true>(pl[c][2 * st + 1], out + 4);
                            } else {
                                u_expand_signed<true>(pl[c][2 * st], sn, out);
                                u_expand_signed<true>(pl[c][2 * st + 1], sn, out + 4);
                            }
                            uint8_t *dst = op_b + 2u * st * kPLbo;
                            *reinterpret_cast<uint4 *>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
                            *reinterpret_cast<uint4 *>(dst + kPLbo) = make_uint4(out[4], out[5], out[6], out[7]);
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA
                    __syncwarp();
                    if (lane == 0) p_arrive_cta(bar(kPOpFull + 4 * t + 2 + rank), 0u);
                }
                if (!ok) break;
                __syncwarp();
                if (lane == 0) u_mbar_arrive(bar(kPRawEmpty + s));
            }
        }
        if (!ok && lane == 0) give_up(site, raw_cnt, op_cnt);
    }

    u_fence_before();
    __syncthreads();
    p_cluster_sync();                                      // neither CTA frees tensor memory or exits while the other still works
    if (warp == 1) {
        u_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kPTmemCols) : "memory");
    }
}

}  // namespace

bool make_plane_map(CUtensorMap *map, const uint32_t *base, int64_t row_words, int64_t planes, int box_words,
                    int box_planes);
bool make_acc_map(CUtensorMap *map, int32_t *acc, int64_t rows, int64_t cols);

// Clusters of two CTAs of the pair kernel that can be resident at once (one CTA per SM): the grid is sized to that.
template <int kMode, int kAG>
static cudaError_t pair_clusters_variant(int sm_count, int *clusters)
{
    static int cached = -1;
    if (cached < 0) {
        cudaError_t e = cudaFuncSetAttribute(core_umma_pair_kernel<kMode, kAG>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairSmem);
        if (e != cudaSuccess) return e;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(sm_count / 2 * 2));
        cfg.blockDim = dim3(p_threads(kAG));
        cfg.dynamicSmemBytes = kPairSmem;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, core_umma_pair_kernel<kMode, kAG>, &cfg);
        if (e != cudaSuccess) return e;
        cached = n < sm_count / 2 ? n : sm_count / 2;
    }
    *clusters = cached;
    return cudaSuccess;
}

// (the smaller of the two variants' counts: the plan is built before the variant is picked)
template <int kMode>
static cudaError_t pair_clusters_mode(int sm_count, int *clusters)
{
    int c3 = 0, c2 = 0;
    cudaError_t e = pair_clusters_variant<kMode, 3>(sm_count, &c3);
    if (e != cudaSuccess) return e;
    e = pair_clusters_variant<kMode, 2>(sm_count, &c2);
    if (e != cudaSuccess) return e;
    *clusters = c3 < c2 ? c3 : c2;
    return cudaSuccess;
}

cudaError_t pair_core_clusters(int mode, int sm_count, int *clusters)
{
    return mode == SC_UNIPOLAR_AND ? pair_clusters_mode<SC_UNIPOLAR_AND>(sm_count, clusters)
                                   : pair_clusters_mode<SC_BIPOLAR_XNOR>(sm_count, clusters);
}

int pair_core_tile_cols() { return kPN; }
int pair_core_max_row_tiles() { return 2 * kPMaxPairs; }

cudaError_t launch_core_umma_pair(const CoreArgs &a, int clusters, bool force, cudaStream_t st)
{
    if (clusters < 1) return cudaErrorInvalidValue;
    CUtensorMap mw;
    if (!make_plane_map(&mw, a.w_streams, a.n_pad, a.w_planes, kPH, kPRawPlanes)) return cudaErrorInvalidValue;
    PairDev dev;
    dev.a_streams = a.a_streams; dev.m_pad = a.m_pad;
    dev.perm = a.perm; dev.l_sorted = a.l_sorted; dev.plan = a.plan; dev.acc = a.acc; dev.scratch = a.scratch;
    dev.N = a.N; dev.planes_per_len = a.kw; dev.pos_block = a.pos_block;
    dev.n_col_tiles = (int32_t)((a.N + kPN - 1) / kPN);
    dev.force = force ? 1 : 0;
    dev.w_sign = a.w_sign; dev.a_sign = a.a_sign; dev.n_pad = a.n_pad;
    CUtensorMap macc = mw;                                 // (a valid map in any case; used only if acc_map_ok)
    dev.acc_map_ok = make_acc_map(&macc, a.acc, a.M, a.N) ? 1 : 0;
    if (a.mode == SC_UNIPOLAR_AND && (a.pos_block != kPosBlockSigned || !a.w_sign || !a.a_sign)) return cudaErrorInvalidValue;
    if (a.mode != SC_UNIPOLAR_AND && a.pos_block != 1) return cudaErrorInvalidValue;
    // Stages a CTA pair gets at most (every row at Lmax): short calls run the variant with two activation expander groups.
    const int64_t pairs = (a.m_pad / kTileM + 1) / 2;
    const int64_t units = ((int64_t)a.Lmax * a.kw + kStagePlanes - 1) / kStagePlanes;
    const bool short_call = pairs * dev.n_col_tiles * units * kPOpsPerRaw / clusters <
                            (a.mode == SC_UNIPOLAR_AND ? kPShortCallStages : 2 * kPShortCallStages);
    if (a.mode == SC_UNIPOLAR_AND) {
        if (short_call) core_umma_pair_kernel<SC_UNIPOLAR_AND, 2><<<2 * clusters, p_threads(2), kPairSmem, st>>>(mw, macc, dev);
        else core_umma_pair_kernel<SC_UNIPOLAR_AND, 3><<<2 * clusters, p_threads(3), kPairSmem, st>>>(mw, macc, dev);
    } else {
        if (short_call) core_umma_pair_kernel<SC_BIPOLAR_XNOR, 2><<<2 * clusters, p_threads(2), kPairSmem, st>>>(mw, macc, dev);
        else core_umma_pair_kernel<SC_BIPOLAR_XNOR, 3><<<2 * clusters, p_threads(3), kPairSmem, st>>>(mw, macc, dev);
    }
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace sc
