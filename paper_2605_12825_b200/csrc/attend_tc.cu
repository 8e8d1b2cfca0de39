// Split-KV flash-decode block attention on the 5th-generation tensor cores
// (tcgen05.mma with TMEM accumulators), bf16, head_dim 128, both views.
//
// Work decomposition.  A unit is one (sequence, KV head); its query tile is the GQA
// group times the block width, M = G*K logical rows (row r = i*G + g), padded to the
// 128 rows of the MMA.  The S CTAs of a thread-block cluster share one unit: the unit's
// 64-position prefix tiles plus the tile of block keys are shared out evenly.  Clusters are handed out longest sequence first, so that a ragged
// batch packs well onto the SMs.
//
// One CTA (192 threads, 112 KB of shared memory, 256 TMEM columns: two fit on an SM).
//   warps 0-3  softmax.  Thread r owns TMEM lane r = query row r: it reads the 64 scores
//              of a tile, keeps the running max / sum of the online softmax, and writes
//              the bf16 probabilities back into TMEM over the scores, where the P.V
//              product reads them as its A operand.
//   warp 4     producer: one lane issues every TMA load (Q tile, K and V tiles of the
//              cache, the block K/V tile) into a ring of five 16 KB slots, in the order
//              the MMAs consume them.
//   warp 5     TMEM allocation and MMA issue: S = Q.K^T into one of two score buffers
//              (so that QK(t+1) runs under softmax(t)), then O += P.V.
// Units of at most 64 rows run a variant of this CTA (see the kernel's comment): probabilities
// through shared memory, the two products issued by two warps.
// The output accumulator O stays in TMEM for the whole CTA.  The running max is only
// raised when a tile exceeds it by more than 2^8; then, and only then, the owner threads
// rescale their O rows in TMEM.  Probabilities are bounded by 2^8, which fp32 sums and
// bf16 operands carry without loss, and the result is the exact softmax because the
// same shift is used for the numerator and the denominator.
//
// Merge of the S partial results of a unit, inside the kernel (there is no second launch),
// through the workspace, which stays in L2: every softmax thread stores its partial row (max, sum, unnormalised O) straight from the
// registers its TMEM read-out filled, in a chunk-major layout ([16-byte column chunk][row])
// so that a warp's 32 rows land in 512 contiguous bytes; one cluster barrier publishes the
// rows; then the work is shared out as (32-row group, column chunk) tasks, one warp each,
// round-robin over the cluster's CTAs and their warps: lane = row, all S partials of the
// task are requested at once (again 512 contiguous bytes per request), weighted, summed,
// normalised and written.  A CTA leaves as soon as its tasks are done.  (Reading the peers'
// shared memory instead was measured slower at every cluster size: remote loads are round
// trips with few requests in flight.)
//
// Programmatic dependent launch.  The kernel waits for the preceding kernel of the
// stream (griddepcontrol.wait) before it reads anything that kernel may have written,
// and then lets its own successor start.  With ORTHRUS_LAYER_CACHE_QUIESCENT the prefix
// K/V tiles are requested before that wait, so the next call's loads are in flight
// while this call is still computing.
//
// Every mbarrier wait is bounded: on expiry the CTA records ORTHRUS_DEV_WAIT_TIMEOUT in
// the status word, drains the copies it armed, still takes part in the cluster barriers,
// frees its TMEM and returns.
#include <cuda.h>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <unordered_map>
#include "common.cuh"
#include "tc_ptx.cuh"

namespace orthrus {
namespace {

constexpr int HD = 128;                  // head_dim
constexpr int MROWS = 128;               // MMA M
constexpr int TN = 64;                   // key positions per tile
constexpr int QSUB_BYTES = MROWS * 128;  // a [128 rows][64 cols] bf16 sub-tile of Q
constexpr int SUB_BYTES = TN * 128;      // a [64 rows][64 cols] bf16 sub-tile of K or V
constexpr int SLOT_BYTES = 2 * SUB_BYTES;
constexpr int MAX_BARS = 40;

// Two shapes of CTA.  NT = 1: one 128-row query tile, 192 threads, 112 KB of shared memory and
// 256 TMEM columns, so that two CTAs share an SM.  NT = 2 (units wider than 128 rows): two
// 128-row query tiles of the same unit share ONE ring of K/V tiles, so every cache byte is
// loaded once for both; 320 threads (two softmax warpgroups), 224 KB of shared memory, all
// 512 TMEM columns: one CTA per SM, with a ring twice as deep.
template <int NT> struct Shape {
    static constexpr int NSLOT = NT == 1 ? 5 : 10;             // ring slots, one K or V tile each
    // warps: 4 softmax warps per query tile, the producer, one MMA-issuing warp per query tile
    // (a thread is held for about a hundred cycles per tcgen05.mma it issues, whatever the
    //  shape: the two tiles' MMAs of a key tile are issued side by side, not one after the other)
    static constexpr int NTHREADS = 32 * (4 * NT + 1 + NT);
    static constexpr int PRODUCER_WARP = 4 * NT, MMA_WARP = 4 * NT + 1;    // MMA warps: MMA_WARP + ti
    // shared memory map (offsets from a 1024-byte aligned base)
    static constexpr int OFF_Q = 0;                            // NT x [128][128] bf16, 2 sub-tiles each
    static constexpr int OFF_RING = OFF_Q + NT * 2 * QSUB_BYTES;
    static constexpr int OFF_BAR = OFF_RING + NSLOT * SLOT_BYTES;
    static constexpr int OFF_MISC = OFF_BAR + MAX_BARS * 8;    // tmem base, abort flag, unit
    static constexpr int SMEM_BYTES = OFF_MISC + 64;
    // mbarriers: per ring slot, per query tile and score buffer
    static constexpr int BAR_FULL = 0, BAR_EMPTY = NSLOT, BAR_QFULL = 2 * NSLOT;
    static constexpr int BAR_SFULL = BAR_QFULL + 1;            // + ti * 2 + buffer
    static constexpr int BAR_PFULL = BAR_SFULL + 2 * NT;       // + ti * 2 + buffer
    static constexpr int BAR_PVDONE = BAR_PFULL + 2 * NT;      // + ti
    static constexpr int BAR_ALLDONE = BAR_PVDONE + NT;        // + ti
    // small-row form of the narrow shape: "scores of buffer b read" and "P buffer b consumed"
    static constexpr int BAR_SREAD = BAR_ALLDONE + NT;         // + buffer
    static constexpr int BAR_PFREE = BAR_SREAD + 2;            // + buffer
    static constexpr int NUM_BARS = BAR_PFREE + 2;
    static_assert(NUM_BARS <= MAX_BARS, "barrier area");
    // TMEM columns: the NT output accumulators, then two score buffers per query tile
    static constexpr uint32_t TM_COLS = 256 * NT;
    static constexpr uint32_t tm_o(int ti) { return (uint32_t)ti * HD; }
    static constexpr uint32_t tm_s(int ti, int sb) { return (uint32_t)(NT * HD + ti * 2 * TN + sb * TN); }
};
static_assert(2 * (Shape<1>::SMEM_BYTES + 1024) <= 228 * 1024, "two CTAs per SM");
static_assert(Shape<2>::SMEM_BYTES <= 227 * 1024, "one CTA per SM");
constexpr float RESCALE_THRESHOLD = 8.f;                  // log2 units
struct TcMaps { CUtensorMap k, v, q, kb, vb; };

// Merge through the workspace.  A task is (32-row group, 16-byte column chunk) of a unit; lane =
// row of the group.  Tasks go round-robin to the cluster's CTAs and their warps.  A warp takes
// LOADS / SP tasks per round (SP = cluster size rounded up to a power of two), so that LOADS
// 16-byte loads per lane are in flight whatever the cluster size (sixteen in the narrow shape,
// eight in the wide one, which has fewer registers per thread); every load of a warp covers
// 512 contiguous bytes.  grp_o: the cluster's S partial tiles, each [32 chunks][128 rows] of
// float4; grp_ml: (max, sum) per [CTA][row].  store(R, chunk, acc, 1 / sum).
template <int SP, int LOADS, class Store>
__device__ inline void l2_merge_tasks(int S, int rank, int warp, int lane, int n_warps, int n_tasks, int rows_here,
                                      const float4 *grp_o, const float2 *grp_ml, Store store)
{
    constexpr int TB = LOADS / SP > 0 ? LOADS / SP : 1;
    // task index of (round, slot u) for this warp: consecutive tasks of a round sit S * n_warps apart
    for (int t0 = rank + warp * S; t0 < n_tasks; t0 += S * n_warps * TB) {
        float2 ml[TB][SP];
        float4 o[TB][SP];
#pragma unroll
        for (int u = 0; u < TB; ++u) {
            const int task = t0 + u * S * n_warps;
            const int R = (task / (HD / 4)) * 32 + lane, c = task % (HD / 4);
            const bool live = task < n_tasks && R < rows_here;
#pragma unroll
            for (int j = 0; j < SP; ++j)
                if (j < S && live) {
                    ml[u][j] = __ldcg(grp_ml + j * MROWS + R);
                    o[u][j] = __ldcg(grp_o + (long long)j * (MROWS * HD / 4) + c * MROWS + R);
                }
        }
#pragma unroll
        for (int u = 0; u < TB; ++u) {
            const int task = t0 + u * S * n_warps;
            const int R = (task / (HD / 4)) * 32 + lane, c = task % (HD / 4);
            if (task < n_tasks && R < rows_here) {
                float mmax = -INFINITY;
#pragma unroll
                for (int j = 0; j < SP; ++j)
                    if (j < S && ml[u][j].y > 0.f) mmax = fmaxf(mmax, ml[u][j].x);
                float L = 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < SP; ++j)
                    if (j < S && ml[u][j].y > 0.f) {      // a partial without keys was never written
                        const float w = ex2(ml[u][j].x - mmax);
                        L = fmaf(w, ml[u][j].y, L);
                        acc.x = fmaf(w, o[u][j].x, acc.x); acc.y = fmaf(w, o[u][j].y, acc.y);
                        acc.z = fmaf(w, o[u][j].z, acc.z); acc.w = fmaf(w, o[u][j].w, acc.w);
                    }
                store(R, c, acc, 1.f / L);
            }
        }
    }
}

// One query tile's merge, kept out of line so that its registers (sixteen 16-byte loads in flight
// per lane) do not add to those of the streaming loop.  out_tile: the output row of the tile's
// first block position and first head of the group; row R = i * G + g lies (i * Hq + g) rows on.
template <int LOADS>
__device__ __forceinline__ void merge_tile_body(int S, int rank, int warp, int lane, int n_warps, int rows_here,
                                                const float4 *grp_o, const float2 *grp_ml, __nv_bfloat16 *out_tile,
                                                int G, int Hq)
{
    const int n_tasks = ((rows_here + 31) >> 5) * (HD / 4);
    auto run = [&](auto sp) {
        l2_merge_tasks<decltype(sp)::value, LOADS>(S, rank, warp, lane, n_warps, n_tasks, rows_here, grp_o, grp_ml,
                                            [&](int R, int c, const float4 &acc, float inv) {
            __nv_bfloat16 *row = out_tile + ((long long)(R / G) * Hq + R % G) * HD;
            reinterpret_cast<uint2 *>(row)[c] =
                make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
        });
    };
    if (S <= 2) run(std::integral_constant<int, 2>());
    else if (S <= 4) run(std::integral_constant<int, 4>());
    else if (S <= 8) run(std::integral_constant<int, 8>());
    else run(std::integral_constant<int, 16>());
}
template <int LOADS>
__device__ __noinline__ void merge_tile(int S, int rank, int warp, int lane, int n_warps, int rows_here,
                                        const float4 *grp_o, const float2 *grp_ml, __nv_bfloat16 *out_tile,
                                        int G, int Hq)
{
    merge_tile_body<LOADS>(S, rank, warp, lane, n_warps, rows_here, grp_o, grp_ml, out_tile, G, Hq);
}

// Thread r of a softmax warpgroup owns query row r of its tile (TMEM lane r) and all 64 columns of
// a key tile.  blockIdx.z counts groups of NT query tiles; warpgroup ti works on tile z * NT + ti.
//
// PACK (multi-block mask, Eq. 6): the p.nb blocks of a sequence, p.kb_width positions each, lie
// back to back on the position axis (p.K = nb * kb_width), so a 128-row query tile holds the rows
// of several blocks and the prefix is streamed once for all of them.  Row i belongs to block
// j = i / kb_width, sees the prefix below its own anchor cache_len[b * nb + j] and the keys of its
// own block only; the CTA streams up to the largest anchor among the blocks of its query tile,
// then the 64-key tiles of the block axis that hold those blocks' keys.
//
// SM (at most 64 query rows, narrow shape, not packed): the chain score tile -> softmax -> P.V ->
// next score tile is what a short chunk waits for, and an issuing thread is held about 110 cycles
// per tcgen05.mma.  Here the probabilities go to shared memory (the unused upper halves of the
// query tile's two sub-tiles) instead of back into the score buffer, so a score buffer is free
// again as soon as its softmax threads have read it, and the two products are issued by two
// warps.  256 threads: warps 0-3 softmax (200 registers after setmaxnreg), 4 producer, 5 Q.K^T,
// 6 P.V, 7 idle (56 registers).
template <int NT, bool PACK, bool SM>
__global__ void __launch_bounds__(SM ? 256 : Shape<NT>::NTHREADS, NT == 1 ? 2 : 1)
attend_tc_kernel(const AttnParams p, const __grid_constant__ TcMaps tm, const int S, const int kb_rows,
                 const int quiescent)
{
    using C = Shape<NT>;
    constexpr int W = TN;                     // score columns per softmax thread
    static_assert(!SM || (NT == 1 && !PACK), "the small-row form is a variant of the plain narrow shape");
    constexpr int NSLOT = C::NSLOT, NTHREADS = SM ? 256 : C::NTHREADS;
    constexpr int OFF_Q = C::OFF_Q, OFF_RING = C::OFF_RING, OFF_BAR = C::OFF_BAR, OFF_MISC = C::OFF_MISC;
    constexpr int BAR_FULL = C::BAR_FULL, BAR_EMPTY = C::BAR_EMPTY, BAR_QFULL = C::BAR_QFULL;
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);
    volatile int *seq_slot = reinterpret_cast<volatile int *>(smem + OFF_MISC + 16);
    auto bar = [&](int i) { return sbase + OFF_BAR + i * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = S > 1 ? (int)cluster_rank() : 0;
    const int order = blockIdx.y;
    // query tile ti of this CTA: kb_rows block positions x G heads (at most 128 rows); the last
    // group of a unit may hold fewer than NT tiles
    // (packed form: anchors usually grow along a sequence, so the last query tiles, which stream the
    //  longest prefixes, are handed out first)
    const int zt = PACK ? (int)(gridDim.z - 1 - blockIdx.z) : (int)blockIdx.z;
    auto tile_i0 = [&](int ti) { return (zt * NT + ti) * kb_rows; };
    auto tile_rows = [&](int ti) { return max(0, min(p.K - tile_i0(ti), kb_rows)) * p.G; };
    const bool aligned = (sbase & 1023u) == 0;                // swizzled tiles need 1 KB alignment

    // ------------------------------------------------------------------ prologue
    if (tid == 0) { *abort_flag = aligned ? 0 : 1; *seq_slot = 0; }
    if (warp == C::PRODUCER_WARP && lane == 0) {
        int n_tiles_q = 0;                                    // query tiles with rows = MMA warps at work
        for (int ti = 0; ti < NT; ++ti) n_tiles_q += tile_rows(ti) > 0;
        for (int i = 0; i < NSLOT; ++i) {
            mbar_init(bar(BAR_FULL + i), 1);
            mbar_init(bar(BAR_EMPTY + i), max(1, n_tiles_q));  // every MMA warp releases a slot
        }
        mbar_init(bar(BAR_QFULL), 1);
        for (int ti = 0; ti < NT; ++ti) {
            const int n_act = max(1, (tile_rows(ti) + 31) >> 5);      // softmax warps with rows
            for (int sb = 0; sb < 2; ++sb) {
                mbar_init(bar(C::BAR_SFULL + ti * 2 + sb), 1);
                mbar_init(bar(C::BAR_PFULL + ti * 2 + sb), n_act);
            }
            mbar_init(bar(C::BAR_PVDONE + ti), 1);
            mbar_init(bar(C::BAR_ALLDONE + ti), 1);
            if constexpr (SM)
                for (int sb = 0; sb < 2; ++sb) {
                    mbar_init(bar(C::BAR_SREAD + sb), n_act);
                    mbar_init(bar(C::BAR_PFREE + sb), 1);
                }
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        prefetch_map(&tm.k); prefetch_map(&tm.v); prefetch_map(&tm.q);
        prefetch_map(&tm.kb); prefetch_map(&tm.vb);
    } else if (warp == C::MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(C::TM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // Nothing written by earlier work of the stream has been read so far.
    if (!quiescent) griddep_wait();

    // ------------------------------------------------------------------ which unit
    // clusters are ordered longest prefix first (ties by sequence index)
    int b = order / p.Hkv;
    const int h = order % p.Hkv;
    const int len_hi = (int)p.len_cap;
    static_assert(!PACK || NT == 1, "the packed form runs one query tile per CTA");
    if (!PACK && p.B > 1 && p.B <= 128) {
        const int want = b;
        for (int i = tid; i < p.B; i += NTHREADS) {
            const int Pi = min(max(__ldg(p.cache_len + i), 0), len_hi);
            int before = 0;
            for (int j = 0; j < p.B; ++j) {
                const int Pj = min(max(__ldg(p.cache_len + j), 0), len_hi);
                before += (Pj > Pi) || (Pj == Pi && j < i);
            }
            if (before == want) *seq_slot = i;
        }
        __syncthreads();
        b = *seq_slot;
    }
    int P;
    int bt_lo = 0, n_blk = 1;               // first tile of block keys on the block axis, how many
    if constexpr (PACK) {
        // blocks j_lo..j_hi have rows in this query tile: stream up to their largest anchor
        const int i0 = tile_i0(0), i1 = min(p.K, i0 + kb_rows) - 1;
        const int j_lo = i0 / p.kb_width, j_hi = i1 / p.kb_width;
        bt_lo = j_lo * p.kb_width / TN;
        n_blk = ((j_hi + 1) * p.kb_width - 1) / TN - bt_lo + 1;
        P = 0;
        bool bad = false;
        for (int j = j_lo; j <= j_hi; ++j) {
            const int a = __ldg(p.cache_len + (long long)b * p.nb + j);
            bad |= a < 0 || a > len_hi;
            P = max(P, min(max(a, 0), len_hi));
        }
        if (bad && tid == 0 && rank == 0 && p.status) atomicOr(p.status, ORTHRUS_DEV_BAD_CACHE_LEN);
    } else {
        P = p.cache_len[b];
        if (P < 0 || P > len_hi) {
            if (tid == 0 && rank == 0 && p.status) atomicOr(p.status, ORTHRUS_DEV_BAD_CACHE_LEN);
            P = P < 0 ? 0 : len_hi;
        }
    }
    // the unit's tiles: n_pre prefix tiles followed by the tile(s) of block keys, shared out evenly
    const uint32_t n_pre = (uint32_t)(P + TN - 1) / TN;
    const uint32_t t0 = (uint32_t)rank * (n_pre + n_blk) / (uint32_t)S;
    const uint32_t t1 = (uint32_t)(rank + 1) * (n_pre + n_blk) / (uint32_t)S;
    const int n_tiles = (int)(t1 - t0);
    // prefix tiles of this CTA; the tiles behind them are block tiles (one, in the last CTA of the
    // cluster, unless the form is packed)
    const int n_mine = max(0, min(n_tiles, (int)n_pre - (int)t0));
    const bool active = n_tiles > 0 && aligned;
    const int row_base = (int)(((long long)(PACK ? b : b / p.nb) * p.Hkv + h) * p.capacity);   // row of position 0

    // The ring holds K and V tiles in the order the MMAs consume them: K0, K1, V0, K2, V1, ...,
    // K(n-1), V(n-2), V(n-1) (the product P.V of a tile is issued after the scores of the next
    // one), so that slots are freed in the order they were filled and a V tile does not sit
    // in the ring while its softmax is still to come.  Item j lives in slot j % NSLOT.
    auto item_of_k = [&](int t) { return t == 0 ? 0 : 2 * t - 1; };
    auto item_of_v = [&](int t) { return min(2 * t + 2, 2 * n_tiles - 1); };
    const uint64_t stream_policy = policy_evict_first();
    auto issue_item = [&](int j) {
        const int slot = j % NSLOT;
        const bool is_v = j == 2 * n_tiles - 1 || (j > 0 && (j & 1) == 0);
        const int t = is_v ? (j == 2 * n_tiles - 1 ? n_tiles - 1 : j / 2 - 1) : (j + 1) / 2;
        const uint32_t dst = sbase + OFF_RING + slot * SLOT_BYTES;
        const uint32_t fb = bar(BAR_FULL + slot);
        mbar_expect_tx(fb, SLOT_BYTES);
        if (t < n_mine) {
            const CUtensorMap *m = is_v ? &tm.v : &tm.k;
            const int row = row_base + ((int)t0 + t) * TN;
            tma_load_2d(dst, m, 0, row, fb, stream_policy);
            tma_load_2d(dst + SUB_BYTES, m, 64, row, fb, stream_policy);
        } else if (PACK) {        // tile bt of the block axis: rows >= nb * kb_width arrive as zeros
            const CUtensorMap *m = is_v ? &tm.vb : &tm.kb;
            const int bt = bt_lo + (int)t0 + t - (int)n_pre;
            tma_load_4d(dst, m, 0, h, bt * TN, b, fb);
            tma_load_4d(dst + SUB_BYTES, m, 64, h, bt * TN, b, fb);
        } else if (p.blk_in_cache) {
            // block tile = the 64 cache rows from P on: rows >= K hold whatever follows the block
            // (masked out of the scores; cleared in the V tile before its product)
            const CUtensorMap *m = is_v ? &tm.v : &tm.k;
            tma_load_2d(dst, m, 0, row_base + P, fb, stream_policy);
            tma_load_2d(dst + SUB_BYTES, m, 64, row_base + P, fb, stream_policy);
        } else {                  // block tile: rows >= K are out of bounds and arrive as zeros
            const CUtensorMap *m = is_v ? &tm.vb : &tm.kb;
            tma_load_4d(dst, m, 0, h, 0, b, fb);
            tma_load_4d(dst + SUB_BYTES, m, 64, h, 0, b, fb);
        }
    };
    int produced = 0;                                         // ring items armed so far
    if (quiescent) {
        // the cache rows below cache_len are not being written by the preceding kernel:
        // request the first prefix tiles before waiting for it
        if (active && warp == C::PRODUCER_WARP && lane == 0)
            while (produced < (n_mine < n_tiles ? item_of_k(n_mine) : 2 * n_tiles) && produced < NSLOT) {
                issue_item(produced); ++produced;     // (stops before the block tile's first item)
            }
        griddep_wait();
    }
    griddep_launch();

    if constexpr (SM) {
        // the softmax warps take the registers the other four warps do not need
        if (warp < 4) asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
        else asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    }
    if (warp < 4 * NT) {
        const int ti = warp >> 2, wq = warp & 3;              // query tile, quarter of its TMEM lanes
        const int r = tid - ti * MROWS;
        const int rows_here = tile_rows(ti);
        const bool valid = r < rows_here;
        const bool warp_active = wq * 32 < rows_here;
        const int i_row = tile_i0(ti) + r / p.G;
        const uint32_t lane_base = tmem + ((uint32_t)(wq * 32) << 16);
        const uint32_t TM_O = C::tm_o(ti);
        float m_run = -INFINITY, l_run = 0.f;
        bool have_o = false;
        int a_row = 0, k0_row = 0;          // packed form: this row's anchor, first key of its block
        if constexpr (PACK) {
            if (valid) {
                const int j_row = i_row / p.kb_width;
                a_row = min(max(__ldg(p.cache_len + (long long)b * p.nb + j_row), 0), len_hi);
                k0_row = j_row * p.kb_width;
            }
        }
        if (active && warp_active) {
            // -------------------------------------------------------------- softmax
            const float sc = p.scale_log2;
            const float2 sc2 = make_float2(sc, sc);
            bool ok = true;
            for (int t = 0; t < n_tiles; ++t) {
                const int sb = t & 1;
                ok = mbar_wait_warp(bar(C::BAR_SFULL + ti * 2 + sb), (t >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t TM_S = C::tm_s(ti, sb);
                uint32_t s[W];
#pragma unroll
                for (int c = 0; c < W / 32; ++c) tmem_ld32(lane_base + TM_S + c * 32, s + c * 32);
                tmem_ld_wait();
                if constexpr (SM) {                            // the buffer may take the scores of tile t + 2
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(C::BAR_SREAD + sb));
                }
                // visible columns of this row in this tile: [lo, lim)
                int lim, lo = 0;
                if constexpr (PACK) {
                    if (t < n_mine) {
                        lim = min(TN, a_row - ((int)t0 + t) * TN);
                    } else {
                        const int c0 = k0_row - (bt_lo + (int)t0 + t - (int)n_pre) * TN;
                        lo = max(c0, 0);
                        lim = min(TN, c0 + p.kb_width);
                    }
                    if (lim <= lo) { lim = 0; lo = 0; }
                } else {
                    if (t < n_mine) lim = min(TN, P - ((int)t0 + t) * TN);
                    else lim = p.causal ? min(p.K, i_row + 1) : p.K;
                }
                lim = valid ? lim : 0;
                float mx;
                if (lim == W && lo == 0) {
                    float m4[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        m4[q] = max3(__uint_as_float(s[q]), __uint_as_float(s[q + 4]), __uint_as_float(s[q + 8]));
#pragma unroll
                    for (int j = 12; j + 8 <= W; j += 8)
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            m4[q] = max3(m4[q], __uint_as_float(s[j + q]), __uint_as_float(s[j + q + 4]));
#pragma unroll
                    for (int q = 0; q < 4; ++q) m4[q] = fmaxf(m4[q], __uint_as_float(s[W - 4 + q]));
                    mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                } else {
                    // a ragged or block tile: only the 16-column groups that hold visible keys
                    mx = -INFINITY;
#pragma unroll
                    for (int c = 0; c < W; c += 16) {
                        if (c < lim && c + 16 > lo) {
#pragma unroll
                            for (int j = c; j < c + 16; ++j) if (j < lim && j >= lo) mx = fmaxf(mx, __uint_as_float(s[j]));
                        }
                    }
                }
                const float m_new = fmaxf(m_run, mx * sc);
                const bool need = m_new > m_run + RESCALE_THRESHOLD;   // also the first finite maximum
                if (__any_sync(0xffffffffu, need)) {
                    const float alpha = need ? ex2(m_run - m_new) : 1.f;
                    if (need) { m_run = m_new; l_run *= alpha; }
                    if (t > 0) {
                        // O holds the products of tiles 0..t-1 and nothing is adding to it now
                        ok = mbar_wait_warp(bar(C::BAR_PVDONE + ti), (t - 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll 1
                        for (int c4 = 0; c4 < HD / 32; ++c4) {
                            uint32_t o[32];
                            tmem_ld32(lane_base + TM_O + c4 * 32, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                            tmem_st32(lane_base + TM_O + c4 * 32, o);
                        }
                    }
                }
                const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
                const float2 nm2 = make_float2(neg_m, neg_m);
                uint32_t pk[W / 2];                            // this thread's probabilities, packed bf16
                float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
                if (lim == W && lo == 0) {
#pragma unroll
                    for (int j = 0; j < W; j += 4) {
                        float2 a = __ffma2_rn(make_float2(__uint_as_float(s[j]), __uint_as_float(s[j + 1])), sc2, nm2);
                        float2 c = __ffma2_rn(make_float2(__uint_as_float(s[j + 2]), __uint_as_float(s[j + 3])), sc2, nm2);
                        a.x = ex2(a.x); a.y = ex2(a.y); c.x = ex2(c.x); c.y = ex2(c.y);
                        acc0 = __fadd2_rn(acc0, a);
                        acc1 = __fadd2_rn(acc1, c);
                        pk[j >> 1] = pack_bf16(a.x, a.y);
                        pk[(j >> 1) + 1] = pack_bf16(c.x, c.y);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < W; c += 16) {
                        if (c < lim && c + 16 > lo) {
#pragma unroll
                            for (int j = c; j < c + 16; j += 2) {
                                float p0 = ex2(fmaf(__uint_as_float(s[j]), sc, neg_m));
                                float p1 = ex2(fmaf(__uint_as_float(s[j + 1]), sc, neg_m));
                                if (j >= lim || j < lo) p0 = 0.f;
                                if (j + 1 >= lim || j + 1 < lo) p1 = 0.f;
                                acc0.x += p0; acc0.y += p1;
                                pk[j >> 1] = pack_bf16(p0, p1);
                            }
                        } else {
#pragma unroll
                            for (int j = c; j < c + 16; j += 2) pk[j >> 1] = 0u;
                        }
                    }
                }
                l_run += (acc0.x + acc0.y) + (acc1.x + acc1.y);
                if constexpr (SM) {
                    // P row r into shared memory buffer sb ([64 rows][64 keys] bf16, 128-byte swizzle),
                    // once the product of tile t - 2 has read that buffer
                    if (t >= 2) {
                        ok = mbar_wait_warp(bar(C::BAR_PFREE + sb), ((t >> 1) - 1) & 1, abort_flag);
                        if (!ok) break;
                    }
                    unsigned char *prow = smem + OFF_Q + (sb ? 3 : 1) * (QSUB_BYTES / 2) + r * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        *reinterpret_cast<uint4 *>(prow + ((c ^ (r & 7)) << 4)) =
                            make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                    fence_proxy_async();
                } else {
                    // P over the scores, 2 bf16 per 32-bit column
                    tmem_st32(lane_base + TM_S, pk);
                    tmem_st_wait();
                    tc_fence_before();
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(C::BAR_PFULL + ti * 2 + sb));
            }
            // BAR_PVDONE cannot be used here: a parity wait cannot tell phase k from phase k-2, and
            // by now the barrier may be one or two phases ahead of what this thread last observed
            if (ok) ok = mbar_wait_warp(bar(C::BAR_ALLDONE + ti), 0, abort_flag);
            if (ok) tc_fence_after();
            have_o = ok;
        }

        if (S == 1) {
            // ---------------------------------------------------------- direct output
            // the whole unit was here: normalise and write the final rows
            if (have_o) {
                const float inv = 1.f / l_run;
                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.out) +
                    (((long long)b * p.K + i_row) * p.Hq + h * p.G + (r % p.G)) * HD;
#pragma unroll 1
                for (int c4 = 0; c4 < HD / 32; ++c4) {
                    uint32_t o[32];
                    tmem_ld32(lane_base + TM_O + c4 * 32, o);
                    tmem_ld_wait();
                    if (valid) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint4 w;
                            w.x = pack_bf16(__uint_as_float(o[c * 8 + 0]) * inv, __uint_as_float(o[c * 8 + 1]) * inv);
                            w.y = pack_bf16(__uint_as_float(o[c * 8 + 2]) * inv, __uint_as_float(o[c * 8 + 3]) * inv);
                            w.z = pack_bf16(__uint_as_float(o[c * 8 + 4]) * inv, __uint_as_float(o[c * 8 + 5]) * inv);
                            w.w = pack_bf16(__uint_as_float(o[c * 8 + 6]) * inv, __uint_as_float(o[c * 8 + 7]) * inv);
                            reinterpret_cast<uint4 *>(dst)[c4 * 4 + c] = w;
                        }
                    }
                }
            }
        } else {
            // ---------------------------------------------------------- partial rows to the workspace
            // straight from the registers of the TMEM read-out: element (chunk c, row r) of this
            // CTA's [32 chunks][128 rows] array of 16-byte chunks, so a warp stores 512 contiguous bytes
            const long long cta_lin = (((long long)blockIdx.z * NT + ti) * gridDim.y + order) * S + rank;
            float4 *my_o = reinterpret_cast<float4 *>(p.part_o + cta_lin * (MROWS * HD));
            float2 *my_ml = reinterpret_cast<float2 *>(p.part_ml + cta_lin * (MROWS * 2));
            if (have_o) {
                // the narrow shape reads the whole row out at once (one wait instead of four), the
                // wide one, with fewer registers per thread, in two halves; 16-byte stores follow
                constexpr int PIECE = (NT == 1 && !SM) ? HD : HD / 2;
#pragma unroll 1
                for (int c0 = 0; c0 < HD; c0 += PIECE) {
                    uint32_t o[PIECE];
#pragma unroll
                    for (int c4 = 0; c4 < PIECE / 32; ++c4) tmem_ld32(lane_base + TM_O + c0 + c4 * 32, o + c4 * 32);
                    tmem_ld_wait();
                    if (valid) {
#pragma unroll
                        for (int c = 0; c < PIECE / 4; ++c)
                            __stcg(my_o + (c0 / 4 + c) * MROWS + r,
                                   make_float4(__uint_as_float(o[c * 4]), __uint_as_float(o[c * 4 + 1]),
                                               __uint_as_float(o[c * 4 + 2]), __uint_as_float(o[c * 4 + 3])));
                    }
                }
            }
            // (a CTA without tiles has empty rows: sum 0, and its O rows are never read)
            if (valid) __stcg(my_ml + r, make_float2(have_o ? m_run : -INFINITY, have_o ? l_run : 0.f));
        }
        tc_fence_before();
        if constexpr (SM) {
            // These warps hold the registers the merge wants, so they finish the unit here: the
            // CTA-wide barrier the other warps take below (after it the TMEM is freed), then the
            // cluster barrier and this CTA's share of the merge.
            asm volatile("bar.sync 0;" ::: "memory");
            if (S == 1) return;
            cluster_sync_all();
            const int rows_here0 = tile_rows(0);
            __nv_bfloat16 *out_tile = static_cast<__nv_bfloat16 *>(p.out) +
                                      (((long long)b * p.K + tile_i0(0)) * p.Hq + h * p.G) * HD;
            const long long grp_lin = ((long long)blockIdx.z * gridDim.y + order) * S;
            merge_tile_body<16>(S, rank, warp, lane, 4, rows_here0,
                                reinterpret_cast<const float4 *>(p.part_o + grp_lin * (MROWS * HD)),
                                reinterpret_cast<const float2 *>(p.part_ml + grp_lin * (MROWS * 2)), out_tile, p.G, p.Hq);
            return;
        }
    } else if (warp == C::PRODUCER_WARP) {
        // ------------------------------------------------------------------ producer
        if (active && lane == 0) {
            // the query rows of every tile: box = 64 columns x G heads x kb_rows positions
            int n_q = 0;
            for (int ti = 0; ti < NT; ++ti) n_q += tile_rows(ti) > 0;
            mbar_expect_tx(bar(BAR_QFULL), (uint32_t)(n_q * 2 * 128 * p.G * kb_rows));
            for (int ti = 0; ti < NT; ++ti)
                if (tile_rows(ti) > 0) {
                    const uint32_t q_dst = sbase + OFF_Q + ti * 2 * QSUB_BYTES;
                    tma_load_4d(q_dst, &tm.q, 0, h * p.G, tile_i0(ti), b, bar(BAR_QFULL));
                    tma_load_4d(q_dst + QSUB_BYTES, &tm.q, 64, h * p.G, tile_i0(ti), b, bar(BAR_QFULL));
                }
            bool ok = true;
            const int n_items = 2 * n_tiles;
            while (produced < n_items && ok) {
                const int slot = produced % NSLOT, use = produced / NSLOT;
                if (use > 0) ok = mbar_wait(bar(BAR_EMPTY + slot), (use - 1) & 1, abort_flag);
                if (ok) { issue_item(produced); ++produced; }
            }
            if (*abort_flag) {
                // give the copies that were armed a bounded time to land before smem is released
                for (int j = max(0, produced - NSLOT); j < produced; ++j) {   // latest use of each slot
                    int dummy = 0;
                    mbar_wait(bar(BAR_FULL + j % NSLOT), (j / NSLOT) & 1, &dummy);
                }
                int dummy = 0;
                mbar_wait(bar(BAR_QFULL), 0, &dummy);
            }
        }
    } else if (active && (SM ? warp <= C::MMA_WARP + 1 : tile_rows(warp - C::MMA_WARP) > 0)) {
        // ------------------------------------------------------------------ MMA issue, query tile ti
        const int ti = SM ? 0 : warp - C::MMA_WARP;
        constexpr uint32_t IDESC_QK = make_idesc(TN, 0);      // A = Q, B = K tile, both K-major
        constexpr uint32_t IDESC_PV = make_idesc(HD, 1);      // A = P (TMEM), B = V tile (MN-major)
        const uint32_t q_addr = sbase + OFF_Q + ti * 2 * QSUB_BYTES;
        auto issue_qk = [&](int t) -> bool {
            const int j = item_of_k(t), slot = j % NSLOT;
            if (!mbar_wait_warp(bar(BAR_FULL + slot), (j / NSLOT) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t k_addr = sbase + OFF_RING + slot * SLOT_BYTES;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {        // 16 head-dim columns per MMA
                    umma_ss(tmem + C::tm_s(ti, t & 1),
                            make_desc(q_addr + (kk >> 2) * QSUB_BYTES + (kk & 3) * 32, 16, 1024),
                            make_desc(k_addr + (kk >> 2) * SUB_BYTES + (kk & 3) * 32, 16, 1024),
                            IDESC_QK, kk > 0);
                }
                umma_commit(bar(BAR_EMPTY + slot));
                umma_commit(bar(C::BAR_SFULL + ti * 2 + (t & 1)));
            }
            __syncwarp();
            return true;
        };
        auto issue_pv = [&](int t) -> bool {
            const int j = item_of_v(t), slot = j % NSLOT;
            if (!mbar_wait_warp(bar(BAR_FULL + slot), (j / NSLOT) & 1, abort_flag)) return false;
            // Only the 16-key groups that hold keys are multiplied (an instruction costs its issuing
            // thread the same whatever its size): the block's own tile is K keys wide, a ragged
            // prefix tile ends at the prefix.  In the last group, V rows past the keys may hold
            // anything where they come from the cache, and 0 * NaN would poison the product, so
            // they are cleared before the MMA reads them (by every MMA warp: the same zeros, and
            // no warp has to wait for another); rows of the block's own tensor past K arrive as zeros.
            const bool from_cache = t < n_mine || p.blk_in_cache;
            const int nv = t < n_mine ? min(TN, P - ((int)t0 + t) * TN) : (PACK ? TN : p.K);
            const int n_kk = (nv + 15) >> 4;
            if (from_cache && nv < n_kk * 16) {
                unsigned char *vt = smem + OFF_RING + slot * SLOT_BYTES;
                for (int e = lane; e < (n_kk * 16 - nv) * 16; e += 32) {
                    const int rr = nv + (e >> 4), c = e & 15;
                    *reinterpret_cast<uint4 *>(vt + sw_off(rr, c, SUB_BYTES)) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async();
                __syncwarp();
            }
            if (!mbar_wait_warp(bar(C::BAR_PFULL + ti * 2 + (t & 1)), (t >> 1) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t v_addr = sbase + OFF_RING + slot * SLOT_BYTES;
#pragma unroll
                for (int kk = 0; kk < TN / 16; ++kk) {        // 16 key positions per MMA
                    if (kk >= n_kk) break;
                    if constexpr (SM)
                        umma_ss(tmem + C::tm_o(ti),
                                make_desc(sbase + OFF_Q + ((t & 1) ? 3 : 1) * (QSUB_BYTES / 2) + kk * 32, 16, 1024),
                                make_desc(v_addr + kk * 2048, SUB_BYTES, 1024), IDESC_PV, (t > 0) || (kk > 0));
                    else
                        umma_ts(tmem + C::tm_o(ti), tmem + C::tm_s(ti, t & 1) + kk * 8,
                                make_desc(v_addr + kk * 2048, SUB_BYTES, 1024), IDESC_PV, (t > 0) || (kk > 0));
                }
                umma_commit(bar(BAR_EMPTY + slot));
                umma_commit(bar(C::BAR_PVDONE + ti));
                if constexpr (SM) umma_commit(bar(C::BAR_PFREE + (t & 1)));
                if (t == n_tiles - 1) umma_commit(bar(C::BAR_ALLDONE + ti));
            }
            __syncwarp();
            return true;
        };
        bool ok = true;
        if constexpr (SM) {
            if (warp == C::MMA_WARP) {
                // scores of tile t go into buffer t & 1 once the softmax threads of tile t - 2 have
                // read theirs out of it (one completion of that barrier per use of the buffer, so
                // the waiter is never more than one phase behind)
                ok = mbar_wait_warp(bar(BAR_QFULL), 0, abort_flag);
                if (ok) tc_fence_after();
                for (int t = 0; t < n_tiles && ok; ++t) {
                    if (t >= 2) {
                        ok = mbar_wait_warp(bar(C::BAR_SREAD + (t & 1)), ((t >> 1) - 1) & 1, abort_flag);
                        if (ok) tc_fence_after();
                    }
                    if (ok) ok = issue_qk(t);
                }
            } else {
                for (int t = 0; t < n_tiles && ok; ++t) ok = issue_pv(t);
            }
        } else {
            ok = mbar_wait_warp(bar(BAR_QFULL), 0, abort_flag);
            if (ok) { tc_fence_after(); ok = issue_qk(0); }
            for (int t = 0; t < n_tiles && ok; ++t) {
                if (t + 1 < n_tiles) ok = issue_qk(t + 1);
                if (ok) ok = issue_pv(t);
            }
        }
        // every MMA of this warp must have retired before TMEM is freed
        if (ok) mbar_wait_warp(bar(C::BAR_ALLDONE + ti), 0, abort_flag);
        tc_fence_before();
    }

    // ---------------------------------------------------------------------- merge
    __syncthreads();
    tc_fence_after();
    if (warp == C::MMA_WARP)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TM_COLS) : "memory");
    if (tid == (SM ? 128 : 0) && *abort_flag && p.status) atomicOr(p.status, ORTHRUS_DEV_WAIT_TIMEOUT);
    if (S == 1) return;
    constexpr int NWARPS = NTHREADS / 32;
    // The cluster is what guarantees that the CTAs waiting for one another are resident
    // together.  Release / acquire at cluster scope: every CTA's partial rows are in place.
    cluster_sync_all();
    if constexpr (!SM) {                  // (in the small-row form the softmax warps merge; they never come here)
        for (int ti = 0; ti < NT; ++ti) {
            const int rows_here = tile_rows(ti);
            if (rows_here == 0) break;
            __nv_bfloat16 *out_tile = static_cast<__nv_bfloat16 *>(p.out) +
                                      (((long long)b * p.K + tile_i0(ti)) * p.Hq + h * p.G) * HD;
            const long long grp_lin = (((long long)blockIdx.z * NT + ti) * gridDim.y + order) * S;
            merge_tile<NT == 1 ? 16 : 8>(S, rank, warp, lane, NWARPS, rows_here,
                       reinterpret_cast<const float4 *>(p.part_o + grp_lin * (MROWS * HD)),
                       reinterpret_cast<const float2 *>(p.part_ml + grp_lin * (MROWS * 2)), out_tile, p.G, p.Hq);
        }
    }
}

#include "attend_tc_stream.cuh"

// ---------------------------------------------------------------------------- host side

}  // namespace

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

namespace {

// Tensor maps over bf16 tensors whose innermost dimension is the 128-wide head: up to four
// dimensions, boxes of 64 columns with the 128-byte swizzle.  Cached by (pointer, shape).
struct MapKey {
    const void *ptr; unsigned long long d1, d2, d3; unsigned b1, b2;
    bool operator==(const MapKey &o) const {
        return ptr == o.ptr && d1 == o.d1 && d2 == o.d2 && d3 == o.d3 && b1 == o.b1 && b2 == o.b2;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey &k) const {
        size_t x = std::hash<const void *>()(k.ptr);
        for (unsigned long long v : {k.d1, k.d2, k.d3, (unsigned long long)k.b1, (unsigned long long)k.b2})
            x = (x ^ v) * 0x9E3779B97F4A7C15ull;
        return x;
    }
};

// dims: (128, d1, d2, d3) row-major with d3 outermost; box (64, b1, b2, 1).  rank = 2 when
// d2 == 0 (then the box is (64, b1)).
bool get_map(const void *ptr, unsigned long long d1, unsigned long long d2, unsigned long long d3,
             unsigned b1, unsigned b2, CUtensorMap *out)
{
    static std::mutex mu;
    static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
    std::lock_guard<std::mutex> lock(mu);
    const MapKey key{ptr, d1, d2, d3, b1, b2};
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const int rank = d2 == 0 ? 2 : 4;
    const cuuint64_t dims[4] = {(cuuint64_t)HD, (cuuint64_t)d1, (cuuint64_t)d2, (cuuint64_t)d3};
    const cuuint64_t strides[3] = {(cuuint64_t)HD * 2, (cuuint64_t)HD * 2 * d1, (cuuint64_t)HD * 2 * d1 * d2};
    const cuuint32_t box[4] = {64, b1, b2, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap tm;
    const CUresult r = fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void *>(ptr), dims,
                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache.size() > 4096) cache.clear();
    cache.emplace(key, tm);
    *out = tm;
    return true;
}

}  // namespace

// block positions per query tile of 128 rows
static int tc_kb_rows(int G, int K) { return K < MROWS / G ? K : MROWS / G; }

int tc_row_tiles(int G, int K)
{
    if (G < 1 || G > MROWS) return 0;
    const int kb = tc_kb_rows(G, K);
    return (K + kb - 1) / kb;
}

// Query tiles per CTA.  Units wider than one 128-row tile run one CTA per query tile by default:
// the CTAs of a unit walk the cache in step, so the second read of every K/V tile is an L2 hit
// (measured DRAM read 545 MB for 539 MB of cache at 256 rows) and two CTAs per SM overlap better
// than one wide CTA.  ORTHRUS_TC_ROW_TILES_PER_CTA=2 selects the shape whose two query tiles share
// one K/V ring (measured 8 % slower at 256 rows; kept for measurements).
int tc_tiles_per_cta(int G, int K)
{
    static const int forced = [] { const char *e = getenv("ORTHRUS_TC_ROW_TILES_PER_CTA"); return e ? atoi(e) : 0; }();
    return (forced == 2 && tc_row_tiles(G, K) >= 2) ? 2 : 1;
}

// CTAs along the query-tile axis of the grid
int tc_cta_groups(int G, int K)
{
    const int nt = tc_tiles_per_cta(G, K);
    return (tc_row_tiles(G, K) + nt - 1) / nt;
}

bool tc_driver_ok() { return encode_fn() != nullptr; }

// CTAs of the shape with nt query tiles one SM of the current device keeps resident: what its
// shared memory holds (each CTA also costs the 1 KB the system reserves per block), at most what
// the 512 TMEM columns allow.  2 and 1 on a B200.  Asked once per device; those values are assumed
// where there is no device.
int tc_ctas_per_sm(int nt)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int smem_cached[kMaxDevices] = {};
    const int smem_bytes = nt == 2 ? Shape<2>::SMEM_BYTES : Shape<1>::SMEM_BYTES;
    const int by_tmem = nt == 2 ? 1 : 2;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { (void)cudaGetLastError(); return by_tmem; }
    std::lock_guard<std::mutex> lock(mu);
    if (!smem_cached[dev]) {
        int smem_per_sm = 0;
        if (cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            return by_tmem;
        }
        smem_cached[dev] = smem_per_sm;
    }
    const int n = smem_cached[dev] / (smem_bytes + 1024);
    return n < 1 ? 1 : (n > by_tmem ? by_tmem : n);
}

namespace {

template <int NT, bool PACK = false, bool SM = false>
cudaError_t configure_kernel()
{   // function attributes belong to a device: set them once on each device that launches
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static bool configured[kMaxDevices] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
        e = cudaFuncSetAttribute(attend_tc_kernel<NT, PACK, SM>, cudaFuncAttributeMaxDynamicSharedMemorySize, Shape<NT>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(attend_tc_kernel<NT, PACK, SM>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    return cudaSuccess;
}

template <int NT>
int max_cluster_of_shape()
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 16;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev]) return cached[dev];
    int best = 16;
    if (configure_kernel<NT>() == cudaSuccess) {
        for (int s = 16; s >= 2; s >>= 1) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(s, 1, 1);
            cfg.blockDim = dim3(Shape<NT>::NTHREADS);
            cfg.dynamicSmemBytes = Shape<NT>::SMEM_BYTES;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = s; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, attend_tc_kernel<NT, false, false>, &cfg) == cudaSuccess && n > 0) { best = s; break; }
            best = s >> 1;
        }
        if (best < 1) best = 1;
    } else {
        (void)cudaGetLastError();
    }
    cached[dev] = best;
    return best;
}

}  // namespace

// Largest cluster size (a power of two up to 16) the current device can co-schedule for the shape
// with nt query tiles; 16 on a full B200.  Without a device (or if the query fails) 16 is assumed
// and a launch that cannot be scheduled reports its error.
int tc_max_cluster(int nt) { return nt == 2 ? max_cluster_of_shape<2>() : max_cluster_of_shape<1>(); }
int tc_tile_positions() { return TN; }

template <int NT, bool PACK = false, bool SM = false>
static cudaError_t launch_tc(const AttnParams &p, const TcMaps &tm, int kb, int flags, cudaStream_t st)
{
    const int S = p.n_splits;
    cudaError_t e = configure_kernel<NT, PACK, SM>();
    if (e != cudaSuccess) return e;
    const int row_tiles = (p.K + kb - 1) / kb;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, p.B * p.Hkv, (row_tiles + NT - 1) / NT);
    cfg.blockDim = dim3(SM ? 256 : Shape<NT>::NTHREADS);
    cfg.dynamicSmemBytes = Shape<NT>::SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (S > 1) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = S;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    if (!(flags & ORTHRUS_LAYER_NO_EARLY_LAUNCH)) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    e = cudaLaunchKernelEx(&cfg, attend_tc_kernel<NT, PACK, SM>, p, tm, S, kb, (flags & ORTHRUS_LAYER_CACHE_QUIESCENT) ? 1 : 0);
    count_launch();
    return e;
}

// The persistent kernel serves one query tile per unit and ranks at most 128 batch entries.
bool tc_stream_shape(int B, int G, int K) { return B <= STREAM_MAX_B && G >= 1 && G * K <= MROWS && K <= TN; }

// Workspace of the persistent kernel behind the header: two partial tiles and their (max, sum)
// rows per CTA, then one arrival counter per unit (zero between calls).
size_t tc_stream_workspace_bytes(int B, int Hkv, int n_ctas)
{
    return (size_t)n_ctas * 2 * (MROWS * HD * sizeof(float) + MROWS * 2 * sizeof(float)) +
           (((size_t)B * Hkv * sizeof(int32_t) + 255) / 256) * 256;
}

cudaError_t launch_attend_tc_stream(const AttnParams &p, int n_ctas, void *ws_body, int flags, cudaStream_t st)
{
    TcMaps tm;
    const unsigned long long rows = (unsigned long long)(p.B / p.nb) * p.Hkv * p.capacity;
    if (!get_map(p.k_cache, rows, 0, 0, TN, 0, &tm.k) || !get_map(p.v_cache, rows, 0, 0, TN, 0, &tm.v) ||
        !get_map(p.q, p.Hq, p.K, p.B, p.G, p.K, &tm.q))
        return cudaErrorInvalidValue;
    if (p.blk_in_cache) {
        tm.kb = tm.k; tm.vb = tm.v;
    } else if (!get_map(p.k_blk, p.Hkv, p.K, p.B, 1, TN, &tm.kb) || !get_map(p.v_blk, p.Hkv, p.K, p.B, 1, TN, &tm.vb)) {
        return cudaErrorInvalidValue;
    }
    {   // function attributes belong to a device: set them once on each device that launches
        constexpr int kMaxDevices = 64;
        static std::mutex mu;
        static bool configured[kMaxDevices] = {};
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mu);
        if (!configured[dev]) {
            e = cudaFuncSetAttribute(attend_tc_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, STREAM_SMEM_BYTES);
            if (e != cudaSuccess) return e;
            configured[dev] = true;
        }
    }
    StreamArgs sa;
    unsigned char *base = static_cast<unsigned char *>(ws_body);
    sa.part_o = reinterpret_cast<float4 *>(base);
    sa.part_ml = reinterpret_cast<float2 *>(base + (size_t)n_ctas * 2 * MROWS * HD * sizeof(float));
    sa.counters = reinterpret_cast<int32_t *>(base + (size_t)n_ctas * 2 * (MROWS * HD + MROWS * 2) * sizeof(float));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ctas, 1, 1);
    cfg.blockDim = dim3(Shape<1>::NTHREADS);
    cfg.dynamicSmemBytes = STREAM_SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    int n_attr = 0;
    if (!(flags & ORTHRUS_LAYER_NO_EARLY_LAUNCH)) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attend_tc_stream_kernel, p, tm, sa);
    count_launch();
    return e;
}

cudaError_t launch_attend_tc(const AttnParams &p, int flags, cudaStream_t st)
{
    const int kb = tc_kb_rows(p.G, p.K);
    TcMaps tm;
    const unsigned long long rows = (unsigned long long)(p.B / p.nb) * p.Hkv * p.capacity;
    if (!get_map(p.k_cache, rows, 0, 0, TN, 0, &tm.k) || !get_map(p.v_cache, rows, 0, 0, TN, 0, &tm.v) ||
        !get_map(p.q, p.Hq, p.K, p.B, p.G, kb, &tm.q))
        return cudaErrorInvalidValue;
    if (p.blk_in_cache) {
        tm.kb = tm.k; tm.vb = tm.v;           // unused: the block tile comes through the cache maps
    } else if (!get_map(p.k_blk, p.Hkv, p.K, p.B, 1, TN, &tm.kb) || !get_map(p.v_blk, p.Hkv, p.K, p.B, 1, TN, &tm.vb)) {
        return cudaErrorInvalidValue;
    }
    if (tc_tiles_per_cta(p.G, p.K) == 2) return launch_tc<2>(p, tm, kb, flags, st);
    // at most 64 query rows: the form with the probabilities in shared memory and two issuing warps
    // (ORTHRUS_TC_SMALL_ROWS=0 keeps the common form: a measurement knob)
    static const bool small_rows = [] { const char *e = getenv("ORTHRUS_TC_SMALL_ROWS"); return !(e && e[0] == '0'); }();
    if (small_rows && p.G * p.K <= MROWS / 2) return launch_tc<1, false, true>(p, tm, kb, flags, st);
    return launch_tc<1>(p, tm, kb, flags, st);
}

// Packed multi-block form: p.B sequences, p.nb blocks of p.kb_width positions each on one position
// axis of p.K = nb * kb_width, anchors in p.cache_len[B][nb].
cudaError_t launch_attend_tc_packed(const AttnParams &p, int flags, cudaStream_t st)
{
    const int kb = tc_kb_rows(p.G, p.K);
    TcMaps tm;
    const unsigned long long rows = (unsigned long long)p.B * p.Hkv * p.capacity;
    if (!get_map(p.k_cache, rows, 0, 0, TN, 0, &tm.k) || !get_map(p.v_cache, rows, 0, 0, TN, 0, &tm.v) ||
        !get_map(p.q, p.Hq, p.K, p.B, p.G, kb, &tm.q) ||
        !get_map(p.k_blk, p.Hkv, p.K, p.B, 1, TN, &tm.kb) || !get_map(p.v_blk, p.Hkv, p.K, p.B, 1, TN, &tm.vb))
        return cudaErrorInvalidValue;
    return launch_tc<1, true>(p, tm, kb, flags, st);
}

}  // namespace orthrus
