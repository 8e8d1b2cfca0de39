// Greedy tokens straight from the AR view's last hidden states: the LM-head product
// logits[r][v] = hidden[r][:] . lm_head[v][:] on the 5th-generation tensor cores with the
// per-row argmax of Eq. 8 taken in the accumulator read-out, so the [rows][vocab] logits
// never reach memory.  bf16 operands, fp32 accumulation, the comparison on the fp32 sums.
//
// Tiling.  An item is (tile of BM hidden rows, tile of bn <= 256 vocabulary entries, bn chosen
// by the host so that the items fill whole waves of the grid); its product
// runs over the hidden dimension in stages of 64 columns (one 128-byte swizzle panel).  A
// persistent grid of one CTA per SM takes items round-robin with the row tile varying
// fastest, so the CTAs that share a vocabulary tile read it at the same time and it crosses
// HBM once.  Rows past the end of `hidden`, vocabulary entries past V and a ragged last stage
// are zero-filled by the TMA unit; the read-out skips the padded vocabulary entries and never
// writes padded rows.
//
// Two one-SM shapes (and an optional two-SM one, further down), all using the 512 TMEM columns
// as two 128 x 256 fp32 accumulators:
//   MT = 1 (at most 128 rows: the LM head is streamed once and HBM binds).  BM = 128, four
//          stages of 16 + 32 KB; the accumulators alternate between items, so the product of
//          the next item runs under the read-out of this one.
//   MT = 2 (more rows: the tensor pipe binds).  BM = 256, three stages of 32 + 32 KB; the two
//          accumulators hold the two row halves of one item, which takes a third off the
//          bytes the SM pulls from L2 per MMA.  Within a stage the MMAs of the first half are issued
//          first, so its read-out overlaps the last MMAs of the second half, and the read-out
//          of the second half the first MMAs of the next item.
//
// One CTA: warp 0 producer (one lane issues the TMA loads of every stage), warp 1 TMEM
// allocation and MMA issue (128x256x16 MMAs, four per accumulator and stage), then four
// read-out warps per accumulator: thread = one row (TMEM lane); 256 fp32 sums are scanned in
// increasing vocabulary order with a strict '>' (the lowest id wins ties, a NaN never wins)
// and one (value, id) pair per (row, vocabulary tile) is stored.  The pairs are folded per
// row, and the accept rule applied, by the finalize kernel of the logits-based consensus.
//
// Every mbarrier wait is bounded: on expiry the CTA records ORTHRUS_DEV_WAIT_TIMEOUT in the
// status word, drains the copies it armed, frees its TMEM and returns.
#include <cstdlib>
#include <mutex>
#include <unordered_map>
#include "common.cuh"
#include "tc_ptx.cuh"

namespace orthrus {
namespace {

constexpr int BN = 256, BK = 64;
constexpr int W_BYTES = BN * BK * 2, XSUB_BYTES = 128 * BK * 2;
template <int MT> struct Shape {
    static constexpr int BM = 128 * MT;
    static constexpr int NSTAGE = MT == 1 ? 4 : 3;
    static constexpr int NTHREADS = 64 + 128 * MT;
    static constexpr int X_BYTES = MT * XSUB_BYTES;
    static constexpr int STAGE_BYTES = X_BYTES + W_BYTES;
    static constexpr int OFF_BAR = NSTAGE * STAGE_BYTES;
    static constexpr int OFF_MISC = OFF_BAR + 16 * 8;
    static constexpr int SMEM_BYTES = OFF_MISC + 64;
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
    static_assert(2 * SMEM_BYTES > 228 * 1024, "one CTA per SM: it takes all 512 TMEM columns");
    enum { BAR_FULL = 0, BAR_EMPTY = NSTAGE, BAR_TFULL = 2 * NSTAGE, BAR_TEMPTY = BAR_TFULL + 2,
           BAR_DONE = BAR_TEMPTY + 2, NUM_BARS };
    static_assert(NUM_BARS <= 16, "barrier area");
};
constexpr uint32_t TM_COLS = 2 * BN;

__device__ inline uint64_t policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ inline uint64_t policy_evict_normal() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

struct HeadMaps { CUtensorMap x, w; };

// Read-out of one accumulator row: this thread's TMEM lane, columns [0, n_valid) from column
// address `taddr`, scanned in increasing order with a strict '>' (the lowest id wins ties, a
// NaN never wins).  Nothing compares greater than -inf: then idx stays 0x7fffffff.
__device__ inline void scan_accumulator(uint32_t taddr, int n_valid, int v0, float &best, int &bidx)
{
    best = -INFINITY;
    bidx = 0x7fffffff;
#pragma unroll 1
    for (int c = 0; c < n_valid; c += 64) {
        uint32_t r[64];
        tmem_ld32(taddr + c, r);
        tmem_ld32(taddr + c + 32, r + 32);
        tmem_ld_wait();
        if (c + 64 <= n_valid) {
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const float x = __uint_as_float(r[j]);
                if (x > best) { best = x; bidx = v0 + c + j; }
            }
        } else {
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                const float x = __uint_as_float(r[j]);
                if (c + j < n_valid && x > best) { best = x; bidx = v0 + c + j; }
            }
        }
    }
}

template <int MT>
__global__ void __launch_bounds__(Shape<MT>::NTHREADS, 1)
lm_head_argmax_kernel(const __grid_constant__ HeadMaps tm, const int R, const int V, const int n_k,
                      const int n_m, const int n_n, const int bn, ArgPart *parts, int32_t *status)
{
    using S = Shape<MT>;
    constexpr int NSTAGE = S::NSTAGE, STAGE_BYTES = S::STAGE_BYTES, X_BYTES = S::X_BYTES, BM = S::BM;
    constexpr int BAR_FULL = S::BAR_FULL, BAR_EMPTY = S::BAR_EMPTY, BAR_TFULL = S::BAR_TFULL,
                  BAR_TEMPTY = S::BAR_TEMPTY, BAR_DONE = S::BAR_DONE;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + S::OFF_MISC + 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + S::OFF_MISC);
    auto bar = [&](int i) { return sbase + S::OFF_BAR + i * 8; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_items = n_m * n_n;

    if (tid == 0) *abort_flag = (sbase & 1023u) == 0 ? 0 : 1;   // swizzled tiles need 1 KB alignment
    if (warp == 0 && lane == 0) {
        for (int i = 0; i < 2 * NSTAGE; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(BAR_TFULL), 1); mbar_init(bar(BAR_TFULL + 1), 1);
        mbar_init(bar(BAR_TEMPTY), 4); mbar_init(bar(BAR_TEMPTY + 1), 4);
        mbar_init(bar(BAR_DONE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        prefetch_map(&tm.x); prefetch_map(&tm.w);
    } else if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    griddep_launch();                         // the finalize kernel may be placed now; it waits for this grid

    // accumulator and its use count for row half `a` of this CTA's item number `li`
    auto acc_of = [](int li, int a) { return MT == 1 ? (li & 1) : a; };
    auto use_of = [](int li) { return MT == 1 ? (li >> 1) : li; };

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0 && !*abort_flag) {
            const uint64_t pol_x = policy_evict_last();
            // the LM head is read once when there is a single row tile
            const uint64_t pol_w = n_m == 1 ? policy_evict_first() : policy_evict_normal();
            int g = 0;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const int m = it % n_m, n = it / n_m;
                for (int ks = 0; ks < n_k && ok; ++ks, ++g) {
                    const int stage = g % NSTAGE, use = g / NSTAGE;
                    if (use > 0) ok = mbar_wait(bar(BAR_EMPTY + stage), (use - 1) & 1, abort_flag);
                    if (!ok) break;
                    const uint32_t dst = sbase + stage * STAGE_BYTES;
                    mbar_expect_tx(bar(BAR_FULL + stage), (uint32_t)(X_BYTES + bn * BK * 2));
                    tma_load_2d(dst, &tm.x, ks * BK, m * BM, bar(BAR_FULL + stage), pol_x);
                    tma_load_2d(dst + X_BYTES, &tm.w, ks * BK, n * bn, bar(BAR_FULL + stage), pol_w);
                }
            }
            if (*abort_flag) {
                // give the copies that were armed a bounded time to land before smem is released
                for (int j = max(0, g - NSTAGE); j < g; ++j) {
                    int dummy = 0;
                    mbar_wait(bar(BAR_FULL + j % NSTAGE), (j / NSTAGE) & 1, &dummy);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issue
        const uint32_t IDESC = make_idesc((uint32_t)bn, 0);     // both operands K-major
        int g = 0, li = 0;
        bool ok = !*abort_flag;
        ok = __all_sync(0xffffffffu, ok);
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++li) {
            const int use = use_of(li);
            for (int ks = 0; ks < n_k && ok; ++ks, ++g) {
                const int stage = g % NSTAGE, suse = g / NSTAGE;
                ok = mbar_wait_warp(bar(BAR_FULL + stage), suse & 1, abort_flag);
                if (!ok) break;
                const uint32_t x_addr = sbase + stage * STAGE_BYTES, w_addr = x_addr + X_BYTES;
#pragma unroll
                for (int a = 0; a < MT; ++a) {
                    const int acc = acc_of(li, a);
                    // the accumulator must have been read out before the item's first MMA clears it
                    if (ks == 0 && use > 0) {
                        ok = mbar_wait_warp(bar(BAR_TEMPTY + acc), (use - 1) & 1, abort_flag);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    if (lane == 0) {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk)
                            umma_ss(tmem + acc * BN, make_desc(x_addr + a * XSUB_BYTES + kk * 32, 16, 1024),
                                    make_desc(w_addr + kk * 32, 16, 1024), IDESC, (ks > 0) || (kk > 0));
                        if (a == MT - 1) umma_commit(bar(BAR_EMPTY + stage));
                        if (ks == n_k - 1) umma_commit(bar(BAR_TFULL + acc));
                    }
                    __syncwarp();
                }
            }
        }
        // every MMA issued so far must have retired before TMEM is freed
        if (lane == 0) umma_commit(bar(BAR_DONE));
        __syncwarp();
        { int dummy = 0; mbar_wait_warp(bar(BAR_DONE), 0, &dummy); }
        tc_fence_before();
    } else {
        // ------------------------------------------------------------------ read-out
        const int quarter = warp & 3;                           // the TMEM lanes this warp may read
        const int a = (warp - 2) >> 2;                          // row half (MT = 2)
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        int li = 0;
        bool ok = !*abort_flag;
        ok = __all_sync(0xffffffffu, ok);
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++li) {
            const int m = it % n_m, n = it / n_m;
            const int acc = acc_of(li, a), use = use_of(li);
            ok = mbar_wait_warp(bar(BAR_TFULL + acc), use & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const int v0 = n * bn;
            const int n_valid = min(bn, V - v0);                // columns past it hold nothing of this item
            float best;
            int bidx;
            scan_accumulator(lane_base + acc * BN, n_valid, v0, best, bidx);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_TEMPTY + acc));
            const int row = m * BM + a * 128 + quarter * 32 + lane;
            if (row < R) parts[(long long)row * n_n + n] = ArgPart{best, bidx};
        }
        tc_fence_before();
    }

    __syncthreads();
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
    if (tid == 0 && *abort_flag && status) atomicOr(status, ORTHRUS_DEV_WAIT_TIMEOUT);
}

// ---------------------------------------------------------------------------- two-SM shape
//
// Opt-in (ORTHRUS_LM_HEAD_PAIR=1) for more than 128 rows: the two CTAs of a cluster share
// every item of 256 rows x bn vocabulary entries through one MMA of M = 256
// (tcgen05.mma.cta_group::2, issued by the leader, CTA rank 0).  Each CTA stages its own 128
// hidden rows and its own half of the LM-head tile (bn / 2 rows), so an SM loads and reads
// from shared memory two thirds of what the one-SM 256-row shape needs per flop, and keeps its
// two accumulators for alternate items, so the read-out is hidden.  Stages are 128 hidden
// columns wide (two swizzle panels per operand, 64 KB per CTA, three stages): with 64-column
// stages the per-stage barrier round and commits were measured to cost a quarter of the time.
// Each CTA reads its 128 result rows out of its own TMEM.
//
// Barriers (same offsets in both CTAs): both producers' loads complete on the leader's FULL
// barrier; the leader's MMA warp commits to the EMPTY and TFULL barriers of both CTAs (one
// commit each); the read-out warps of both CTAs arrive on the leader's TEMPTY barrier.  No
// load or commit is a cluster broadcast.
//
// Measured on the serving shape (1024 x 128256 x 4096): 769 us against 750 us for the one-SM
// 256-row shape on the same box (735 against 732 us with a single broadcast commit per stage
// in a scratch build): both run at the power cap, so the one-SM shape stays the default.
namespace pair {
constexpr int NSTAGE = 3;
constexpr int NTHREADS = 192;
constexpr int KPANELS = 2;                             // 64-column panels per stage
constexpr int WPANEL_BYTES = W_BYTES / 2;              // up to 128 LM-head rows x 64 columns
constexpr int X_BYTES = KPANELS * XSUB_BYTES;          // 128 rows of hidden x 128 columns
constexpr int STAGE_BYTES = X_BYTES + KPANELS * WPANEL_BYTES;
constexpr int OFF_BAR = NSTAGE * STAGE_BYTES;
constexpr int OFF_MISC = OFF_BAR + 24 * 8;
constexpr int SMEM_BYTES = OFF_MISC + 64;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
static_assert(2 * SMEM_BYTES > 228 * 1024, "one CTA per SM: it takes all 512 TMEM columns");
enum { BAR_FULL = 0, BAR_EMPTY = NSTAGE, BAR_TFULL = 2 * NSTAGE, BAR_TEMPTY = BAR_TFULL + 2,
       BAR_DONE = BAR_TEMPTY + 2, NUM_BARS };
static_assert(NUM_BARS <= 24, "barrier area");
}  // namespace pair

// D[tmem of both CTAs] (+)= A . B with M = 256 over the CTA pair
__device__ inline void umma_ss_pair(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
// arrival on a barrier of either CTA (cluster-window address) once the pair's MMAs so far retire
__device__ inline void umma_commit_pair(uint32_t bar_cluster) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar_cluster) : "memory");
}
// tile load into this CTA's shared memory whose bytes are counted on a barrier of either CTA
__device__ inline void tma_load_2d_pair(uint32_t dst, const CUtensorMap *tm, int c0, int c1, uint32_t bar_cluster,
                                        uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
                 " [%0], [%1, {%2, %3}], [%4], %5;"
                 ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar_cluster), "l"(policy) : "memory");
}
// the same arrival on the barrier at this offset in both CTAs of the pair: one commit per CTA,
// the peer's barrier addressed through the cluster window
__device__ inline void umma_commit_both(uint32_t bar) {
    umma_commit_pair(bar);
    umma_commit_pair(map_to_rank(bar, 1));
}
__device__ inline void mbar_arrive_cluster(uint32_t bar_cluster) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
// instruction descriptor as make_idesc, for M = 256 over the pair
__host__ __device__ constexpr uint32_t make_idesc_pair(uint32_t n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((256u >> 4) << 24);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(pair::NTHREADS, 1)
lm_head_argmax_pair_kernel(const __grid_constant__ HeadMaps tm, const int R, const int V, const int n_k,
                           const int n_m, const int n_n, const int bn, ArgPart *parts, int32_t *status)
{
    using namespace pair;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);
    auto bar = [&](int i) { return sbase + OFF_BAR + i * 8; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = (int)cluster_rank();                       // 0: leader
    const int n_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;
    const int n_items = n_m * n_n;
    const int half = bn >> 1;                                   // LM-head rows per CTA and item

    if (tid == 0) *abort_flag = (sbase & 1023u) == 0 ? 0 : 1;   // swizzled tiles need 1 KB alignment
    if (warp == 0 && lane == 0) {
        for (int i = 0; i < 2 * NSTAGE; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(BAR_TFULL), 1); mbar_init(bar(BAR_TFULL + 1), 1);
        mbar_init(bar(BAR_TEMPTY), 8); mbar_init(bar(BAR_TEMPTY + 1), 8);   // 4 warps of each CTA
        mbar_init(bar(BAR_DONE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        prefetch_map(&tm.x); prefetch_map(&tm.w);
    } else if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                       // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    griddep_launch();                         // the finalize kernel may be placed now; it waits for this grid

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (both CTAs)
        if (lane == 0 && !*abort_flag) {
            const uint64_t pol_x = policy_evict_last();
            const uint64_t pol_w = n_m == 1 ? policy_evict_first() : policy_evict_normal();
            const uint32_t stage_tx = 2u * KPANELS * (uint32_t)(XSUB_BYTES + half * BK * 2);   // both CTAs' bytes
            int g = 0;
            bool ok = true;
            for (int it = cluster_id; it < n_items && ok; it += n_clusters) {
                const int m = it % n_m, n = it / n_m;
                for (int ks = 0; ks < n_k && ok; ++ks, ++g) {
                    const int stage = g % NSTAGE, use = g / NSTAGE;
                    if (use > 0) ok = mbar_wait(bar(BAR_EMPTY + stage), (use - 1) & 1, abort_flag);
                    if (!ok) break;
                    const uint32_t dst = sbase + stage * STAGE_BYTES;
                    const uint32_t full = map_to_rank(bar(BAR_FULL + stage), 0);
                    if (rank == 0) mbar_expect_tx(bar(BAR_FULL + stage), stage_tx);
#pragma unroll
                    for (int pnl = 0; pnl < KPANELS; ++pnl) {
                        const int col = (ks * KPANELS + pnl) * BK;   // past H: zero-filled
                        tma_load_2d_pair(dst + pnl * XSUB_BYTES, &tm.x, col, m * 256 + rank * 128, full, pol_x);
                        tma_load_2d_pair(dst + X_BYTES + pnl * WPANEL_BYTES, &tm.w, col, n * bn + rank * half,
                                         full, pol_w);
                    }
                }
            }
            if (*abort_flag && rank == 0) {
                // give the copies that were armed a bounded time to land before smem is released
                for (int j = max(0, g - NSTAGE); j < g; ++j) {
                    int dummy = 0;
                    mbar_wait(bar(BAR_FULL + j % NSTAGE), (j / NSTAGE) & 1, &dummy);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issue (leader)
        if (rank == 0) {
            const uint32_t IDESC = make_idesc_pair((uint32_t)bn);
            int g = 0, li = 0;
            bool ok = !*abort_flag;
            ok = __all_sync(0xffffffffu, ok);
            for (int it = cluster_id; it < n_items && ok; it += n_clusters, ++li) {
                const int buf = li & 1, buse = li >> 1;
                if (buse > 0) ok = mbar_wait_warp(bar(BAR_TEMPTY + buf), (buse - 1) & 1, abort_flag);
                if (!ok) break;
                for (int ks = 0; ks < n_k && ok; ++ks, ++g) {
                    const int stage = g % NSTAGE, use = g / NSTAGE;
                    ok = mbar_wait_warp(bar(BAR_FULL + stage), use & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    if (lane == 0) {
                        const uint32_t x_addr = sbase + stage * STAGE_BYTES, w_addr = x_addr + X_BYTES;
#pragma unroll
                        for (int kk = 0; kk < KPANELS * BK / 16; ++kk)
                            umma_ss_pair(tmem + buf * BN,
                                         make_desc(x_addr + (kk >> 2) * XSUB_BYTES + (kk & 3) * 32, 16, 1024),
                                         make_desc(w_addr + (kk >> 2) * WPANEL_BYTES + (kk & 3) * 32, 16, 1024),
                                         IDESC, (ks > 0) || (kk > 0));
                        umma_commit_both(bar(BAR_EMPTY + stage));
                        if (ks == n_k - 1) umma_commit_both(bar(BAR_TFULL + buf));
                    }
                    __syncwarp();
                }
            }
            // every MMA issued so far must have retired before TMEM is freed
            if (lane == 0) umma_commit_pair(bar(BAR_DONE));
            __syncwarp();
            { int dummy = 0; mbar_wait_warp(bar(BAR_DONE), 0, &dummy); }
        }
        tc_fence_before();
    } else {
        // ------------------------------------------------------------------ read-out (both CTAs)
        const int quarter = warp & 3;                           // the TMEM lanes this warp may read
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16);
        int li = 0;
        bool ok = !*abort_flag;
        ok = __all_sync(0xffffffffu, ok);
        for (int it = cluster_id; it < n_items && ok; it += n_clusters, ++li) {
            const int m = it % n_m, n = it / n_m;
            const int buf = li & 1, buse = li >> 1;
            ok = mbar_wait_warp(bar(BAR_TFULL + buf), buse & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const int v0 = n * bn;
            const int n_valid = min(bn, V - v0);
            float best;
            int bidx;
            scan_accumulator(lane_base + buf * BN, n_valid, v0, best, bidx);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_rank(bar(BAR_TEMPTY + buf), 0));
            const int row = m * 256 + rank * 128 + quarter * 32 + lane;
            if (row < R) parts[(long long)row * n_n + n] = ArgPart{best, bidx};
        }
        tc_fence_before();
    }

    // neither CTA may leave, or free its TMEM, while the other can still signal its barriers or
    // the leader's MMAs can still write its TMEM
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
    if (tid == 0 && *abort_flag && status) atomicOr(status, ORTHRUS_DEV_WAIT_TIMEOUT);
}

struct Map2Key {
    const void *ptr; unsigned long long inner, outer; unsigned box_outer;
    bool operator==(const Map2Key &o) const {
        return ptr == o.ptr && inner == o.inner && outer == o.outer && box_outer == o.box_outer;
    }
};
struct Map2KeyHash {
    size_t operator()(const Map2Key &k) const {
        size_t x = std::hash<const void *>()(k.ptr);
        for (unsigned long long v : {k.inner, k.outer, (unsigned long long)k.box_outer})
            x = (x ^ v) * 0x9E3779B97F4A7C15ull;
        return x;
    }
};

// A map over a row-major bf16 matrix [outer][inner]: boxes of 64 columns x box_outer rows,
// 128-byte swizzle, zero fill outside the matrix.  Cached by (pointer, shape).
bool get_map_2d(const void *ptr, unsigned long long inner, unsigned long long outer, unsigned box_outer,
                CUtensorMap *out)
{
    static std::mutex mu;
    static std::unordered_map<Map2Key, CUtensorMap, Map2KeyHash> cache;
    std::lock_guard<std::mutex> lock(mu);
    const Map2Key key{ptr, inner, outer, box_outer};
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
    const cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
    const cuuint32_t box[2] = {(cuuint32_t)BK, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap tm;
    const CUresult r = fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides,
                          box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache.size() > 1024) cache.clear();
    cache.emplace(key, tm);
    *out = tm;
    return true;
}

template <int MT>
cudaError_t launch_shape(const HeadMaps &tm, int R, int V, int H, int bn, ArgPart *parts, int32_t *status,
                         cudaStream_t st)
{
    using S = Shape<MT>;
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static bool configured[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (dev < 0 || dev >= kMaxDevices || !configured[dev]) {
            e = cudaFuncSetAttribute(lm_head_argmax_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     S::SMEM_BYTES);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < kMaxDevices) configured[dev] = true;
        }
    }
    const int n_m = (R + S::BM - 1) / S::BM, n_n = (V + bn - 1) / bn, n_k = (H + BK - 1) / BK;
    const long long n_items = (long long)n_m * n_n;
    const int grid = (int)(n_items < num_sms() ? n_items : num_sms());
    lm_head_argmax_kernel<MT><<<grid, S::NTHREADS, S::SMEM_BYTES, st>>>(tm, R, V, n_k, n_m, n_n, bn, parts,
                                                                       status);
    count_launch();
    return cudaGetLastError();
}

// Clusters of two CTAs of the pair kernel the current device can keep resident (0: not asked
// for with ORTHRUS_LM_HEAD_PAIR=1, none, or the query failed); looked up once per device.
int pair_clusters()
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int cached[kMaxDevices];
    static bool known[kMaxDevices] = {};
    static const bool enabled = [] { const char *e = getenv("ORTHRUS_LM_HEAD_PAIR"); return e && atoi(e) == 1; }();
    if (!enabled) return 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    std::lock_guard<std::mutex> lock(mu);
    if (known[dev]) return cached[dev];
    int n = 0;
    if (cudaFuncSetAttribute(lm_head_argmax_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             pair::SMEM_BYTES) == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * num_sms(), 1, 1);
        cfg.blockDim = dim3(pair::NTHREADS);
        cfg.dynamicSmemBytes = pair::SMEM_BYTES;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (cudaOccupancyMaxActiveClusters(&n, lm_head_argmax_pair_kernel, &cfg) != cudaSuccess) n = 0;
    }
    (void)cudaGetLastError();
    if (n > num_sms() / 2) n = num_sms() / 2;
    cached[dev] = n; known[dev] = true;
    return n;
}

cudaError_t launch_pair(const HeadMaps &tm, int R, int V, int H, int bn, int clusters, ArgPart *parts,
                        int32_t *status, cudaStream_t st)
{
    const int n_m = (R + 255) / 256, n_n = (V + bn - 1) / bn;
    const int n_k = (H + pair::KPANELS * BK - 1) / (pair::KPANELS * BK);
    const long long n_items = (long long)n_m * n_n;
    const int n_cl = (int)(n_items < clusters ? n_items : clusters);
    lm_head_argmax_pair_kernel<<<2 * n_cl, pair::NTHREADS, pair::SMEM_BYTES, st>>>(tm, R, V, n_k, n_m, n_n, bn,
                                                                                  parts, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

// Width of the vocabulary tiles (the N of the MMAs, from 128 to 256): the one whose item count
// fills the waves of the persistent grid best.  The busiest CTA (or CTA pair) works through
// waves x (width + a per-item overhead worth about 16 columns); ties go to the wider tile,
// which re-reads the hidden rows less often.  `pairs` > 0: the two-SM shape on that many
// clusters, widths in multiples of 32 (each CTA holds half a tile).
static int tile_width(int R, int V, int pairs)
{
    const int n_m = R > 128 ? (R + 255) / 256 : 1;
    const int workers = pairs > 0 ? pairs : num_sms(), step = pairs > 0 ? 32 : 16;
    int best_bn = BN;
    long long best_cost = -1;
    for (int bn = BN; bn >= 128; bn -= step) {
        const long long items = (long long)n_m * ((V + bn - 1) / bn);
        const long long waves = (items + workers - 1) / workers;
        const long long cost = waves * (bn + 16);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_bn = bn; }
    }
    return best_bn;
}

// the shape a problem runs in on the current device: clusters of the two-SM shape (0: one-SM
// shapes) and the tile width
static void plan(int R, int V, int *pairs, int *bn)
{
    *pairs = R > 128 ? pair_clusters() : 0;
    *bn = tile_width(R, V, *pairs);
}

int lm_head_vocab_tiles(int R, int V)
{
    int pairs, bn;
    plan(R, V, &pairs, &bn);
    return (V + bn - 1) / bn;
}

int lm_head_max_vocab_tiles(int V) { return (V + 127) / 128; }

bool lm_head_supported() { return encode_fn() != nullptr; }

// parts: [rows][lm_head_vocab_tiles(R, V)] (value, id) pairs.  Returns cudaErrorNotSupported when
// the tensor maps cannot be built.
cudaError_t launch_lm_head_argmax(const void *hidden, const void *lm_head, int R, int V, int H,
                                  ArgPart *parts, int32_t *status, cudaStream_t st)
{
    int pairs, bn;
    plan(R, V, &pairs, &bn);
    const int mt = R > 128 ? 2 : 1;
    HeadMaps tm;
    if (!get_map_2d(hidden, (unsigned long long)H, (unsigned long long)R, pairs > 0 ? 128 : 128 * mt, &tm.x) ||
        !get_map_2d(lm_head, (unsigned long long)H, (unsigned long long)V, pairs > 0 ? bn / 2 : bn, &tm.w))
        return cudaErrorNotSupported;
    if (pairs > 0) return launch_pair(tm, R, V, H, bn, pairs, parts, status, st);
    return mt == 2 ? launch_shape<2>(tm, R, V, H, bn, parts, status, st)
                   : launch_shape<1>(tm, R, V, H, bn, parts, status, st);
}

}  // namespace orthrus
