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
// The output accumulator O stays in TMEM for the whole CTA.  The running max is only
// raised when a tile exceeds it by more than 2^8; then, and only then, the owner threads
// rescale their O rows in TMEM.  Probabilities are bounded by 2^8, which fp32 sums and
// bf16 operands carry without loss, and the result is the exact softmax because the
// same shift is used for the numerator and the denominator.
//
// Narrow units (M <= 64) can optionally load their query rows twice and run two independent
// softmax streams over the two column halves of every tile, so that all 128 softmax
// threads work; the two streams are folded together in shared memory before the merge.
//
// Merge.  Every softmax thread puts its partial row (max, sum, unnormalised O straight out
// of TMEM) into its CTA's idle ring.  Row r of the tile is merged and written by cluster
// rank r % S.  Small exchanges (cluster size x rows < 1024) are read straight out of the
// peers' shared memory, between two cluster barriers.  Larger ones go through the
// workspace (L2): each CTA copies its rows out with 512-byte coalesced stores, one cluster
// barrier publishes them, the owners read them back and a CTA leaves as soon as its own
// rows are written; for those sizes the SM-to-SM path was measured to be slower.  There is
// no second kernel.
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
#include <mutex>
#include <unordered_map>
#include "common.cuh"
#include "tc_ptx.cuh"

namespace orthrus {
namespace {

constexpr int HD = 128;                  // head_dim
constexpr int MROWS = 128;               // MMA M
constexpr int TN = 64;                   // key positions per tile
constexpr int NTHREADS = 192;
constexpr int NSLOT = 5;                 // ring slots, one K or V tile each
constexpr int QSUB_BYTES = MROWS * 128;  // a [128 rows][64 cols] bf16 sub-tile of Q
constexpr int SUB_BYTES = TN * 128;      // a [64 rows][64 cols] bf16 sub-tile of K or V
constexpr int SLOT_BYTES = 2 * SUB_BYTES;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                                   // [128][128] bf16, 2 sub-tiles
constexpr int OFF_RING = OFF_Q + 2 * QSUB_BYTES;           // NSLOT x 16 KB
constexpr int OFF_OPART = OFF_RING;                        // float [128][128], after the last MMA
constexpr int OFF_ML = OFF_OPART + MROWS * HD * 4;         // float [128][2], inside the ring
constexpr int OFF_BAR = OFF_RING + NSLOT * SLOT_BYTES;     // mbarriers
constexpr int OFF_MISC = OFF_BAR + 24 * 8;                 // tmem base, abort flag, unit
constexpr int SMEM_BYTES = OFF_MISC + 64;
static_assert(OFF_ML + MROWS * 8 <= OFF_BAR, "partial rows must fit in the idle ring");
static_assert(2 * (SMEM_BYTES + 1024) <= 228 * 1024, "two CTAs per SM");

enum { BAR_FULL = 0, BAR_EMPTY = NSLOT, BAR_QFULL = 2 * NSLOT, BAR_SFULL, BAR_PFULL = BAR_SFULL + 2,
       BAR_PVDONE = BAR_PFULL + 2, BAR_ALLDONE, NUM_BARS };
static_assert(NUM_BARS <= 24, "barrier area");

constexpr uint32_t TM_O = 0, TM_S = 128, TM_COLS = 256;   // TMEM column map
constexpr float RESCALE_THRESHOLD = 8.f;                  // log2 units
// a cluster whose partial rows add up to this many (cluster size x rows per CTA) or more
// exchanges them through the L2 workspace instead of distributed shared memory
constexpr int kL2ExchangeRows = 1024;

struct TcMaps { CUtensorMap k, v, q, kb, vb; };

// Split merge.  Row R of a tile is merged and written by cluster rank R % S: a warp per row,
// lane j holds the weight of the partial result of rank j, every lane four output columns.
// load_ml(j, R) returns (max, sum) of rank j's partial row R, load_o(j, R) this lane's four
// columns of it.  The loads of a batch are all issued before the first is used.
template <class LoadML, class LoadO, class Store>
__device__ inline void merge_rows(int S, int rank, int my_rows, int warp, int lane, int n_warps,
                                  LoadML load_ml, LoadO load_o, Store store)
{
    if (my_rows <= n_warps) {
        // at most one row per warp: all of the row's partial results are requested at once
        if (warp < my_rows) {
            const int R = rank + warp * S;
            float mj = -INFINITY, lj = 0.f;
            if (lane < S) { const float2 t2 = load_ml(lane, R); mj = t2.x; lj = t2.y; }
            float4 v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u)
                if (u < S) v[u] = load_o(u, R);
            float mmax = mj;
#pragma unroll
            for (int off = 16; off; off >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, off));
            const float wj = (lj > 0.f) ? ex2(mj - mmax) : 0.f;
            float L = wj * lj;
#pragma unroll
            for (int off = 16; off; off >>= 1) L += __shfl_xor_sync(0xffffffffu, L, off);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const float w = (u < S) ? __shfl_sync(0xffffffffu, wj, u) : 0.f;
                // a partial without keys has weight 0 and its row was never written
                if (w != 0.f) {
                    acc.x = fmaf(w, v[u].x, acc.x); acc.y = fmaf(w, v[u].y, acc.y);
                    acc.z = fmaf(w, v[u].z, acc.z); acc.w = fmaf(w, v[u].w, acc.w);
                }
            }
            store(R, acc, 1.f / L);
        }
        return;
    }
    for (int s0 = warp; s0 < my_rows; s0 += 4 * n_warps) {
        float mj[4], lj[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int R = rank + min(s0 + q * n_warps, my_rows - 1) * S;
            mj[q] = -INFINITY; lj[q] = 0.f;
            if (lane < S && s0 + q * n_warps < my_rows) { const float2 t2 = load_ml(lane, R); mj[q] = t2.x; lj[q] = t2.y; }
        }
        float4 acc[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        float wj[4] = {0.f, 0.f, 0.f, 0.f}, L[4] = {1.f, 1.f, 1.f, 1.f};
        for (int j0 = 0; j0 < S; j0 += 4) {
            float4 v[4][4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int R = rank + min(s0 + q * n_warps, my_rows - 1) * S;
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (j0 + u < S && s0 + q * n_warps < my_rows) v[q][u] = load_o(j0 + u, R);
            }
            if (j0 == 0) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    float mmax = mj[q];
#pragma unroll
                    for (int off = 16; off; off >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, off));
                    wj[q] = (lj[q] > 0.f) ? ex2(mj[q] - mmax) : 0.f;
                    L[q] = wj[q] * lj[q];
#pragma unroll
                    for (int off = 16; off; off >>= 1) L[q] += __shfl_xor_sync(0xffffffffu, L[q], off);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float w = (j0 + u < S) ? __shfl_sync(0xffffffffu, wj[q], min(j0 + u, 31)) : 0.f;
                    // a partial without keys has weight 0 and its row was never written
                    if (w != 0.f) {
                        acc[q].x = fmaf(w, v[q][u].x, acc[q].x); acc[q].y = fmaf(w, v[q][u].y, acc[q].y);
                        acc[q].z = fmaf(w, v[q][u].z, acc[q].z); acc[q].w = fmaf(w, v[q][u].w, acc[q].w);
                    }
                }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (s0 + q * n_warps < my_rows) store(rank + (s0 + q * n_warps) * S, acc[q], 1.f / L[q]);
    }
}

// NSUB = 1: thread r of the softmax warps owns query row r and all 64 columns of a tile.
// NSUB = 2 (units of at most 64 rows): the query rows are loaded twice, rows 64..127 being a
// copy of rows 0..63; thread r works on logical row r % 64 and on columns [32*(r/64), +32)
// of every tile only, so all 128 threads have work.  The two halves are independent
// online-softmax streams (own max, own sum, own O row in TMEM) that are folded together
// at the end exactly like the partial results of different CTAs.
template <int NSUB>
__global__ void __launch_bounds__(NTHREADS, 2)
attend_tc_kernel(const AttnParams p, const __grid_constant__ TcMaps tm, const int S, const int kb_rows,
                 const int quiescent)
{
    constexpr int W = TN / NSUB;              // score columns per softmax thread
    constexpr int MPAD = MROWS / NSUB;        // logical rows per sub-stream
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);
    volatile int *seq_slot = reinterpret_cast<volatile int *>(smem + OFF_MISC + 16);
    auto bar = [&](int i) { return sbase + OFF_BAR + i * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = S > 1 ? (int)cluster_rank() : 0;
    const int order = blockIdx.y, rt = blockIdx.z;
    // this row tile: kb_rows block positions x G heads (at most MPAD rows)
    const int i0 = rt * kb_rows;
    const int rows_here = min(p.K - i0, kb_rows) * p.G;
    const int n_act = NSUB * ((rows_here + 31) >> 5);         // softmax warps with rows
    const bool aligned = (sbase & 1023u) == 0;                // swizzled tiles need 1 KB alignment

    // ------------------------------------------------------------------ prologue
    if (tid == 0) { *abort_flag = aligned ? 0 : 1; *seq_slot = 0; }
    if (warp == 4 && lane == 0) {
        for (int i = 0; i < 2 * NSLOT; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(BAR_QFULL), 1);
        mbar_init(bar(BAR_SFULL), 1); mbar_init(bar(BAR_SFULL + 1), 1);
        mbar_init(bar(BAR_PFULL), n_act); mbar_init(bar(BAR_PFULL + 1), n_act);
        mbar_init(bar(BAR_PVDONE), 1);
        mbar_init(bar(BAR_ALLDONE), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        prefetch_map(&tm.k); prefetch_map(&tm.v); prefetch_map(&tm.q);
        prefetch_map(&tm.kb); prefetch_map(&tm.vb);
    } else if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(TM_COLS) : "memory");
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
    const int len_hi = (int)(p.capacity - p.K);
    if (p.B > 1 && p.B <= 128) {
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
    int P = p.cache_len[b];
    if (P < 0 || P > len_hi) {
        if (tid == 0 && rank == 0 && p.status) atomicOr(p.status, ORTHRUS_DEV_BAD_CACHE_LEN);
        P = P < 0 ? 0 : len_hi;
    }
    // the unit's tiles: n_pre prefix tiles followed by the tile of block keys, shared out evenly
    const uint32_t n_pre = (uint32_t)(P + TN - 1) / TN;
    const uint32_t t0 = (uint32_t)rank * (n_pre + 1) / (uint32_t)S;
    const uint32_t t1 = (uint32_t)(rank + 1) * (n_pre + 1) / (uint32_t)S;
    const int n_tiles = (int)(t1 - t0);
    const bool owner = rank == S - 1;                         // its last tile is the block tile
    const int n_mine = n_tiles - (owner ? 1 : 0);             // prefix tiles of this CTA
    const bool active = n_tiles > 0 && aligned;
    const int row_base = (int)(((long long)b * p.Hkv + h) * p.capacity);   // row of position 0

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
        if (active && warp == 4 && lane == 0)
            while (produced < (owner ? item_of_k(n_tiles - 1) : 2 * n_tiles) && produced < NSLOT) {
                issue_item(produced); ++produced;     // (stops before the block tile's first item)
            }
        griddep_wait();
    }
    griddep_launch();

    if (warp < 4) {
        const int r = tid;
        const int sub = r / MPAD, Rl = r % MPAD;              // sub-stream, logical row in the tile
        const bool valid = Rl < rows_here;
        const bool warp_active = ((warp * 32) % MPAD) < rows_here;
        const int i_row = i0 + Rl / p.G;
        const int col0 = sub * W;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        float m_run = -INFINITY, l_run = 0.f;
        bool have_o = false;
        if (active && warp_active) {
            // -------------------------------------------------------------- softmax
            const float sc = p.scale_log2;
            const float2 sc2 = make_float2(sc, sc);
            bool ok = true;
            for (int t = 0; t < n_tiles; ++t) {
                const int sb = t & 1;
                ok = mbar_wait_warp(bar(BAR_SFULL + sb), (t >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t s[W];
#pragma unroll
                for (int c = 0; c < W / 32; ++c) tmem_ld32(lane_base + TM_S + sb * TN + col0 + c * 32, s + c * 32);
                tmem_ld_wait();
                // visible columns of this row in this tile, then in this thread's column range
                int lim;
                if (t < n_mine) lim = min(TN, P - ((int)t0 + t) * TN);
                else lim = p.causal ? min(p.K, i_row + 1) : p.K;
                lim = valid ? min(W, max(0, lim - col0)) : 0;
                float mx;
                if (lim == W) {
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
                        if (c < lim) {
#pragma unroll
                            for (int j = c; j < c + 16; ++j) if (j < lim) mx = fmaxf(mx, __uint_as_float(s[j]));
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
                        ok = mbar_wait_warp(bar(BAR_PVDONE), (t - 1) & 1, abort_flag);
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
                if (lim == W) {
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
                        if (c < lim) {
#pragma unroll
                            for (int j = c; j < c + 16; j += 2) {
                                float p0 = ex2(fmaf(__uint_as_float(s[j]), sc, neg_m));
                                float p1 = ex2(fmaf(__uint_as_float(s[j + 1]), sc, neg_m));
                                if (j >= lim) p0 = 0.f;
                                if (j + 1 >= lim) p1 = 0.f;
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
                // P over the scores, 2 bf16 per column: the row's 32 packed columns are this
                // thread's range and zeros for the range of the other sub-stream
                if constexpr (NSUB == 1) {
                    tmem_st32(lane_base + TM_S + sb * TN, pk);
                } else {
                    uint32_t zero[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) zero[j] = 0u;
                    tmem_st16(lane_base + TM_S + sb * TN + sub * 16, pk);
                    tmem_st16(lane_base + TM_S + sb * TN + (1 - sub) * 16, zero);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_PFULL + sb));
            }
            // BAR_PVDONE cannot be used here: a parity wait cannot tell phase k from phase k-2, and
            // by now the barrier may be one or two phases ahead of what this thread last observed
            if (ok) ok = mbar_wait_warp(bar(BAR_ALLDONE), 0, abort_flag);
            if (ok) tc_fence_after();
            have_o = ok;
        }

        if (S == 1 && NSUB == 1) {
            // ---------------------------------------------------------- direct output
            // the whole unit was here: normalise and write the final rows
            if (have_o) {
                const float inv = 1.f / l_run;
                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.out) +
                    (((long long)b * p.K + i_row) * p.Hq + h * p.G + (Rl % p.G)) * HD;
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
            // ---------------------------------------------------------- publish partial rows
            // every softmax thread puts its partial row (max, sum, unnormalised O straight out
            // of TMEM) into this CTA's ring, which is idle once the last product has retired
            if (have_o) {
#pragma unroll 1
                for (int c2 = 0; c2 < HD / 64; ++c2) {
                    uint32_t o[64];
                    tmem_ld32(lane_base + TM_O + c2 * 64, o);
                    tmem_ld32(lane_base + TM_O + c2 * 64 + 32, o + 32);
                    tmem_ld_wait();
#pragma unroll
                    for (int c = 0; c < 16; ++c)
                        *reinterpret_cast<uint4 *>(smem + OFF_OPART + r * 512 + (((c2 * 16 + c) ^ (r & 31)) << 4)) =
                            make_uint4(o[c * 4], o[c * 4 + 1], o[c * 4 + 2], o[c * 4 + 3]);
                }
            }
            if (valid && (have_o || !active)) {   // (threads without a row may get here before the ring is idle)
                float *ml = reinterpret_cast<float *>(smem + OFF_ML);
                ml[r * 2] = have_o ? m_run : -INFINITY;       // a CTA without tiles has empty rows
                ml[r * 2 + 1] = have_o ? l_run : 0.f;
            }
            if constexpr (NSUB == 2) {
                // fold the two sub-streams of a row together, in place in the first one's row:
                // a warp per logical row, lane c holds output columns 4c..4c+3
                named_bar_sync(1, 128);
                float *ml = reinterpret_cast<float *>(smem + OFF_ML);
                for (int R0 = warp; R0 < rows_here; R0 += 16) {   // four rows at a time, for latency
                    float2 ma[4], mb[4];
                    float4 va[4], vb[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int R = min(R0 + 4 * q, rows_here - 1), R2 = R + MPAD;
                        ma[q] = *reinterpret_cast<const float2 *>(ml + R * 2);
                        mb[q] = *reinterpret_cast<const float2 *>(ml + R2 * 2);
                        va[q] = *reinterpret_cast<const float4 *>(smem + OFF_OPART + R * 512 + ((lane ^ (R & 31)) << 4));
                        vb[q] = *reinterpret_cast<const float4 *>(smem + OFF_OPART + R2 * 512 + ((lane ^ (R2 & 31)) << 4));
                    }
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int R = R0 + 4 * q;
                        if (R < rows_here) {
                            // a sub-stream without keys has sum 0 and its row was never written
                            const bool ha = ma[q].y > 0.f, hb = mb[q].y > 0.f;
                            const float mm = fmaxf(ha ? ma[q].x : -INFINITY, hb ? mb[q].x : -INFINITY);
                            const float wa = ha ? ex2(ma[q].x - mm) : 0.f, wb = hb ? ex2(mb[q].x - mm) : 0.f;
                            float4 o;
                            o.x = wa * (ha ? va[q].x : 0.f) + wb * (hb ? vb[q].x : 0.f);
                            o.y = wa * (ha ? va[q].y : 0.f) + wb * (hb ? vb[q].y : 0.f);
                            o.z = wa * (ha ? va[q].z : 0.f) + wb * (hb ? vb[q].z : 0.f);
                            o.w = wa * (ha ? va[q].w : 0.f) + wb * (hb ? vb[q].w : 0.f);
                            *reinterpret_cast<float4 *>(smem + OFF_OPART + R * 512 + ((lane ^ (R & 31)) << 4)) = o;
                            if (lane == 0)
                                *reinterpret_cast<float2 *>(ml + R * 2) =
                                    make_float2(mm, wa * ma[q].y + wb * mb[q].y);
                        }
                    }
                }
            }
        }
        tc_fence_before();
    } else if (warp == 4) {
        // ------------------------------------------------------------------ producer
        if (active && lane == 0) {
            // the query rows of this tile: box = 64 columns x G heads x kb_rows positions,
            // once per sub-stream
            mbar_expect_tx(bar(BAR_QFULL), (uint32_t)(NSUB * 2 * 128 * p.G * kb_rows));
#pragma unroll
            for (int u = 0; u < NSUB; ++u) {
                tma_load_4d(sbase + OFF_Q + u * MPAD * 128, &tm.q, 0, h * p.G, i0, b, bar(BAR_QFULL));
                tma_load_4d(sbase + OFF_Q + QSUB_BYTES + u * MPAD * 128, &tm.q, 64, h * p.G, i0, b, bar(BAR_QFULL));
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
    } else if (active) {
        // ------------------------------------------------------------------ MMA issue
        const uint32_t q_addr = sbase + OFF_Q;
        constexpr uint32_t IDESC_QK = make_idesc(TN, 0);      // A = Q, B = K tile, both K-major
        constexpr uint32_t IDESC_PV = make_idesc(HD, 1);      // A = P (TMEM), B = V tile (MN-major)
        auto issue_qk = [&](int t) -> bool {
            const int j = item_of_k(t), slot = j % NSLOT;
            if (!mbar_wait_warp(bar(BAR_FULL + slot), (j / NSLOT) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t k_addr = sbase + OFF_RING + slot * SLOT_BYTES;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {        // 16 head-dim columns per MMA
                    umma_ss(tmem + TM_S + (t & 1) * TN,
                            make_desc(q_addr + (kk >> 2) * QSUB_BYTES + (kk & 3) * 32, 16, 1024),
                            make_desc(k_addr + (kk >> 2) * SUB_BYTES + (kk & 3) * 32, 16, 1024),
                            IDESC_QK, kk > 0);
                }
                umma_commit(bar(BAR_EMPTY + slot));
                umma_commit(bar(BAR_SFULL + (t & 1)));
            }
            __syncwarp();
            return true;
        };
        auto issue_pv = [&](int t) -> bool {
            const int j = item_of_v(t), slot = j % NSLOT;
            if (!mbar_wait_warp(bar(BAR_FULL + slot), (j / NSLOT) & 1, abort_flag)) return false;
            // a ragged prefix tile: V rows past the prefix may hold anything, and 0 * NaN would
            // poison the product, so they are cleared before the MMA reads them
            const int nv = t < n_mine ? min(TN, P - ((int)t0 + t) * TN) : TN;
            if (nv < TN) {
                unsigned char *vt = smem + OFF_RING + slot * SLOT_BYTES;
                for (int e = lane; e < (TN - nv) * 16; e += 32) {
                    const int rr = nv + (e >> 4), c = e & 15;
                    *reinterpret_cast<uint4 *>(vt + sw_off(rr, c, SUB_BYTES)) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async();
                __syncwarp();
            }
            if (!mbar_wait_warp(bar(BAR_PFULL + (t & 1)), (t >> 1) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t v_addr = sbase + OFF_RING + slot * SLOT_BYTES;
#pragma unroll
                for (int kk = 0; kk < TN / 16; ++kk) {        // 16 key positions per MMA
                    umma_ts(tmem + TM_O, tmem + TM_S + (t & 1) * TN + kk * 8,
                            make_desc(v_addr + kk * 2048, SUB_BYTES, 1024), IDESC_PV, (t > 0) || (kk > 0));
                }
                umma_commit(bar(BAR_EMPTY + slot));
                umma_commit(bar(BAR_PVDONE));
                if (t == n_tiles - 1) umma_commit(bar(BAR_ALLDONE));
            }
            __syncwarp();
            return true;
        };
        bool ok = mbar_wait_warp(bar(BAR_QFULL), 0, abort_flag);
        if (ok) { tc_fence_after(); ok = issue_qk(0); }
        for (int t = 0; t < n_tiles && ok; ++t) {
            if (t + 1 < n_tiles) ok = issue_qk(t + 1);
            if (ok) ok = issue_pv(t);
        }
        // every MMA must have retired before TMEM is freed
        if (ok) mbar_wait_warp(bar(BAR_ALLDONE), 0, abort_flag);
        tc_fence_before();
    }

    // ---------------------------------------------------------------------- merge
    __syncthreads();
    tc_fence_after();
    if (warp == 5)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TM_COLS) : "memory");
    if (tid == 0 && *abort_flag && p.status) atomicOr(p.status, ORTHRUS_DEV_WAIT_TIMEOUT);
    if (S == 1 && NSUB == 1) return;
    constexpr int NWARPS = NTHREADS / 32;
    if (S == 1) {
        // the two sub-streams of a lone CTA were folded in shared memory: normalise and write
        const float *ml = reinterpret_cast<const float *>(smem + OFF_ML);
        for (int R = warp; R < rows_here; R += NWARPS) {
            const float4 v = *reinterpret_cast<const float4 *>(smem + OFF_OPART + R * 512 + ((lane ^ (R & 31)) << 4));
            const float inv = 1.f / ml[R * 2 + 1];
            const int i = i0 + R / p.G, g = R % p.G;
            uint2 *dst = reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(p.out) +
                         (((long long)b * p.K + i) * p.Hq + h * p.G + g) * HD);
            dst[lane] = make_uint2(pack_bf16(v.x * inv, v.y * inv), pack_bf16(v.z * inv, v.w * inv));
        }
        return;
    }

    // How the CTAs of a cluster exchange their partial rows.  Small exchanges: each CTA reads
    // the rows it merges straight out of its peers' shared memory.  Large ones (cluster size x
    // rows >= 1024, e.g. 16 CTAs x 64 rows or 8 x 128): through the workspace, which lives in
    // L2; an all-to-all of that size over the SM-to-SM path moved about 5 bytes per cycle per
    // SM and took longer than the whole stream of keys.  The cluster is what guarantees that
    // the CTAs waiting for one another are resident together.
    const int my_rows = rank < rows_here ? (rows_here - rank + S - 1) / S : 0;
    auto store = [&](int R, const float4 &acc, float inv) {
        const int i = i0 + R / p.G, g = R % p.G;
        uint2 *dst = reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(p.out) +
                     (((long long)b * p.K + i) * p.Hq + h * p.G + g) * HD);
        dst[lane] = make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
    };
    if (S * rows_here >= kL2ExchangeRows) {
        const long long cta_lin = ((long long)rt * gridDim.y + order) * S + rank;
        float *my_o = p.part_o + cta_lin * (MROWS * HD);
        float *my_ml = p.part_ml + cta_lin * (MROWS * 2);
        const float *ml = reinterpret_cast<const float *>(smem + OFF_ML);
        // copy this CTA's rows out: a warp per row, 512 contiguous bytes
        for (int R0 = warp; R0 < rows_here; R0 += 4 * NWARPS) {
            float4 v[4];
            float2 t2[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int R = min(R0 + q * NWARPS, rows_here - 1);
                v[q] = *reinterpret_cast<const float4 *>(smem + OFF_OPART + R * 512 + ((lane ^ (R & 31)) << 4));
                t2[q] = *reinterpret_cast<const float2 *>(ml + R * 2);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int R = R0 + q * NWARPS;
                if (R < rows_here) {
                    // (the row of a CTA without keys was never written: only its sum 0 matters)
                    reinterpret_cast<float4 *>(my_o + R * HD)[lane] = v[q];
                    if (lane == 0) *reinterpret_cast<float2 *>(my_ml + R * 2) = t2[q];
                }
            }
        }
        cluster_sync_all();               // release / acquire at cluster scope: the rows are in place
        const float *grp_o = p.part_o + (cta_lin - rank) * (MROWS * HD);
        const float *grp_ml = p.part_ml + (cta_lin - rank) * (MROWS * 2);
        merge_rows(S, rank, my_rows, warp, lane, NWARPS,
                   [&](int j, int R) { return __ldcg(reinterpret_cast<const float2 *>(grp_ml + (long long)j * (MROWS * 2) + R * 2)); },
                   [&](int j, int R) { return __ldcg(reinterpret_cast<const float4 *>(grp_o + (long long)j * (MROWS * HD) + R * HD) + lane); },
                   store);
        return;                           // nobody reads this CTA's shared memory
    }
    cluster_sync_all();                   // every CTA's partial rows are in place
    merge_rows(S, rank, my_rows, warp, lane, NWARPS,
               [&](int j, int R) { return ld_cluster_f2(map_to_rank(sbase + OFF_ML + R * 8, j)); },
               [&](int j, int R) { return ld_cluster_f4(map_to_rank(sbase + OFF_OPART + R * 512 + ((lane ^ (R & 31)) << 4), j)); },
               store);
    cluster_sync_all();                   // peers may still be reading this CTA's rows
}

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

// Sub-streams per query row: 2 when a unit has at most 64 rows, else 1.
// Sub-streams per query row.  Two sub-streams halve the softmax time of a tile for units of
// at most 64 rows, but their extra fold step costs more than that at the tile counts per
// CTA measured so far, so they are opt-in (ORTHRUS_TC_NSUB=2) and one is the default.
static int tc_nsub(int G, int K)
{
    static const int forced = [] { const char *e = getenv("ORTHRUS_TC_NSUB"); return e ? atoi(e) : 0; }();
    return (forced == 2 && G * K <= 64) ? 2 : 1;
}
// block positions per query tile of 128 / nsub rows
static int tc_kb_rows(int G, int K, int nsub) { return K < (MROWS / nsub) / G ? K : (MROWS / nsub) / G; }

int tc_row_tiles(int G, int K)
{
    if (G < 1 || G > MROWS) return 0;
    const int kb = tc_kb_rows(G, K, tc_nsub(G, K));
    return (K + kb - 1) / kb;
}

bool tc_driver_ok() { return encode_fn() != nullptr; }

// CTAs of this kernel one SM of the current device keeps resident: what its shared memory holds
// (each CTA also costs the 1 KB the system reserves per block), at most the two that share
// the 512 TMEM columns.  2 on a B200.  Asked once per device; 2 assumed where there is none.
int tc_ctas_per_sm()
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { (void)cudaGetLastError(); return 2; }
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev]) return cached[dev];
    int smem_per_sm = 0;
    if (cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return 2;
    }
    int n = smem_per_sm / (SMEM_BYTES + 1024);
    n = n < 1 ? 1 : (n > 512 / (int)TM_COLS ? 512 / (int)TM_COLS : n);
    cached[dev] = n;
    return n;
}

// Largest cluster size (a power of two up to 16) the current device can co-schedule for this
// kernel; 16 on a full B200.  Without a device (or if the query fails) 16 is assumed and a
// launch that cannot be scheduled reports its error.
int tc_max_cluster()
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 16;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev]) return cached[dev];
    int best = 16;
    if (cudaFuncSetAttribute(attend_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(attend_tc_kernel<1>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
        for (int s = 16; s >= 2; s >>= 1) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(s, 1, 1);
            cfg.blockDim = dim3(NTHREADS);
            cfg.dynamicSmemBytes = SMEM_BYTES;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = s; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, attend_tc_kernel<1>, &cfg) == cudaSuccess && n > 0) { best = s; break; }
            best = s >> 1;
        }
        if (best < 1) best = 1;
    } else {
        (void)cudaGetLastError();
    }
    cached[dev] = best;
    return best;
}
int tc_tile_positions() { return TN; }
bool tc_exchange_in_workspace(int S, int M) { return S * (M < MROWS ? M : MROWS) >= kL2ExchangeRows; }

template <int NSUB>
static cudaError_t launch_tc(const AttnParams &p, const TcMaps &tm, int kb, int flags, cudaStream_t st)
{
    const int S = p.n_splits;
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
            e = cudaFuncSetAttribute(attend_tc_kernel<NSUB>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(attend_tc_kernel<NSUB>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            if (e != cudaSuccess) return e;
            configured[dev] = true;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, p.B * p.Hkv, (p.K + kb - 1) / kb);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
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
    cudaError_t e = cudaLaunchKernelEx(&cfg, attend_tc_kernel<NSUB>, p, tm, S, kb,
                                       (flags & ORTHRUS_LAYER_CACHE_QUIESCENT) ? 1 : 0);
    count_launch();
    return e;
}

cudaError_t launch_attend_tc(const AttnParams &p, int flags, cudaStream_t st)
{
    const int nsub = tc_nsub(p.G, p.K);
    const int kb = tc_kb_rows(p.G, p.K, nsub);
    TcMaps tm;
    const unsigned long long rows = (unsigned long long)p.B * p.Hkv * p.capacity;
    if (!get_map(p.k_cache, rows, 0, 0, TN, 0, &tm.k) || !get_map(p.v_cache, rows, 0, 0, TN, 0, &tm.v) ||
        !get_map(p.q, p.Hq, p.K, p.B, p.G, kb, &tm.q) ||
        !get_map(p.k_blk, p.Hkv, p.K, p.B, 1, TN, &tm.kb) || !get_map(p.v_blk, p.Hkv, p.K, p.B, 1, TN, &tm.vb))
        return cudaErrorInvalidValue;
    return nsub == 2 ? launch_tc<2>(p, tm, kb, flags, st) : launch_tc<1>(p, tm, kb, flags, st);
}

}  // namespace orthrus
