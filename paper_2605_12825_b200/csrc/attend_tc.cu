// Split-KV flash-decode block attention on the 5th-generation tensor cores
// (tcgen05.mma with TMEM accumulators), bf16, head_dim 128, both views.
//
// One CTA streams one split of one (sequence, KV head) unit.  The query tile is the GQA
// group times the block width: M = G*K logical rows.  The MMA is always 128 rows high;
// when M <= 64 (<= 32) the logical rows are replicated 2x (4x) and every replica
// ("sub-stream") owns a disjoint column range of each key tile, so all 128 softmax
// threads have work; sub-streams are independent online-softmax streams and are merged
// at the end exactly like splits.
//
// Warp roles:
//   warps 0-3  softmax: thread r owns TMEM lane r: row max, exp2, row sum; bf16
//              probabilities go to shared memory as the A operand of P.V
//   warps 4-7  accumulate: thread r keeps output row r (128 fp32) in registers and folds
//              in each tile's P.V product with the rescale factor of the online softmax
//   warp 8     producer: barrier set-up and TMA loads of K and V tiles (64-column boxes,
//              128-byte swizzle) into a ring of stages
//   warp 9     TMEM allocation and MMA issue (one elected lane)
// S = Q.K^T is double-buffered in TMEM so QK(t+1) overlaps softmax(t); each P.V product
// lands in one of two TMEM buffers and is drained by the accumulate warps.
//
// The splits of one unit form a thread-block cluster (<= 16 CTAs).  At the end every CTA
// publishes its partial rows (running max, running sum, unnormalised output) in its own
// shared memory; after a cluster barrier each CTA merges a slice of the rows straight out
// of its peers' shared memory (DSMEM) and writes the final bf16 output: no partials in
// global memory, no second kernel.  More than 16 splits fall back to global partials and
// the separate merge kernel.
//
// Every mbarrier wait is bounded: on expiry the CTA records ORTHRUS_DEV_WAIT_TIMEOUT in
// the status word, drains the copies it armed, still takes part in the cluster barriers,
// frees its TMEM and returns.
#include <cuda.h>
#include <mutex>
#include <unordered_map>
#include "common.cuh"

namespace orthrus {
#ifdef ORTHRUS_TC_TRACE
// development aid: per-CTA time stamps (ns) at fixed points, read back by a debug export
__device__ unsigned long long g_trace[4096 * 32];
#endif
namespace {

constexpr int HD = 128;                  // head_dim
constexpr int MROWS = 128;               // MMA M
constexpr int NTHREADS = 320;
constexpr int PSUB_BYTES = 128 * 128;    // a [128 rows][64 cols] bf16 sub-tile (Q, P)
constexpr int STAGE_BYTES_ALL = 64 * 1024;   // K ring and V ring, each

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_Q = 0;                               // [128][128] bf16
constexpr int OFF_P = OFF_Q + 2 * PSUB_BYTES;          // [128][TN] bf16
constexpr int OFF_K = OFF_P + 2 * PSUB_BYTES;          // K ring; reused for the partial rows
constexpr int OFF_V = OFF_K + STAGE_BYTES_ALL;         // V ring
constexpr int OFF_ALPHA = OFF_V + STAGE_BYTES_ALL;     // float [2][128]
constexpr int OFF_ML = OFF_ALPHA + 2 * 128 * 4;        // float [128][2]
constexpr int OFF_BAR = OFF_ML + 128 * 2 * 4;          // mbarriers
constexpr int NUM_BARS = 32;
constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;       // tmem base, abort flag
constexpr int SMEM_BYTES = OFF_MISC + 64;
constexpr int OFF_OPART = OFF_K;                       // float [128][128], chunk-swizzled

enum { BAR_KFULL = 0, BAR_VFULL = 4, BAR_KEMPTY = 8, BAR_VEMPTY = 12, BAR_SFULL = 16,
       BAR_OFULL = 18, BAR_OFREE = 20, BAR_AFULL = 22, BAR_PFULL = 24 };

__device__ inline uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

#ifdef ORTHRUS_TC_TRACE
__device__ inline unsigned long long gtimer() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
#define TRACE(slot) do { if ((slot) < 32) g_trace[((blockIdx.y * gridDim.x + blockIdx.x) & 4095) * 32 + (slot)] = gtimer(); } while (0)
#else
#define TRACE(slot) do { } while (0)
#endif

__device__ inline void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ inline void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ inline void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ inline bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                 " selp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) if the phase does not
// complete within about a second, or if another thread already gave up.
__device__ inline bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t it = 1; it < (1u << 24); ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 127) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > (1ll << 31)) break;
        }
    }
    *abort_flag = 1;
    return false;
}

__device__ inline void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ inline void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ inline uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ inline uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ inline float4 ld_cluster_f4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ inline float2 ld_cluster_f2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr));
    return v;
}

// shared-memory matrix descriptor, 128-byte swizzle
__device__ inline uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
// instruction descriptor: D fp32, A/B bf16, M = 128, N = n; b_mn = 1 when B is MN-major
__host__ __device__ constexpr uint32_t make_idesc(uint32_t n, uint32_t b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

__device__ inline void umma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
__device__ inline void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane (no wait: pair with tmem_ld_wait)
__device__ inline void tmem_ld32_nowait(uint32_t taddr, uint32_t *r) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
                   "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]),
                   "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
                   "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                   "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]),
                   "=r"(r[31])
                 : "r"(taddr));
}
__device__ inline void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ inline float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
// byte offset of 16-byte chunk `c` of row `r` in a tile stored as 128-byte-swizzled
// sub-tiles of 64 bf16 columns, `sub_bytes` apart
__device__ inline uint32_t sw_off(int r, int c, int sub_bytes) {
    return (uint32_t)((c >> 3) * sub_bytes + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

template <int TN, int NSUB>
__global__ void __launch_bounds__(NTHREADS, 1)
attend_tc_kernel(AttnParams p, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, int cluster_size)
{
    constexpr int NSTAGE = STAGE_BYTES_ALL / (TN * 256);      // 2 (TN=128) or 4 (TN=64)
    constexpr int KSUB_BYTES = TN * 128;                      // a [TN][64] bf16 sub-tile
    constexpr int TILE_BYTES = 2 * KSUB_BYTES;
    constexpr int W = TN / NSUB;                              // score columns per thread
    constexpr int MPAD = MROWS / NSUB;                        // logical rows per sub-stream
    constexpr uint32_t TM_S = 0, TM_O = 2 * TN;               // TMEM column bases
    static_assert(W % 32 == 0, "a thread reads whole 32-column TMEM chunks");

    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);
    float *alpha_buf = reinterpret_cast<float *>(smem + OFF_ALPHA);
    float *ml_buf = reinterpret_cast<float *>(smem + OFF_ML);
    auto bar = [&](int i) { return sbase + OFF_BAR + i * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit = blockIdx.x, split = blockIdx.y, rt = blockIdx.z;
    if (tid == 0) TRACE(0);
    const int b = unit / p.Hkv, h = unit % p.Hkv;
    const int P = clamp_cache_len(p, b);
    const int ls = last_split(P, p.chunk);
    const int pos0 = split * p.chunk;
    const int pos1 = min(P, pos0 + p.chunk);
    const int n_prefix = (split <= ls && pos1 > pos0) ? (pos1 - pos0 + TN - 1) / TN : 0;
    const int n_blk = (split == ls) ? 1 : 0;                 // the block tile comes first
    const int n_tiles = n_prefix + n_blk;
    const bool active = n_tiles > 0 && (sbase & 1023u) == 0;  // swizzled tiles need 1 KB alignment
    const int rows_here = min(p.M - rt * MROWS, MPAD);        // logical rows of this row tile

    if (tid == 0) *abort_flag = ((sbase & 1023u) != 0) ? 1 : 0;

    const int row_base = (int)((long long)unit * p.capacity);     // row of position 0 in the 2-D maps
    auto issue_prefix = [&](int t) {                              // t: tile index in this CTA
        const int st = t % NSTAGE;
        const int pos = pos0 + (t - n_blk) * TN;
        const uint32_t kdst = sbase + OFF_K + st * TILE_BYTES;
        const uint32_t vdst = sbase + OFF_V + st * TILE_BYTES;
        mbar_expect_tx(bar(BAR_KFULL + st), TILE_BYTES);
        tma_load_2d(kdst, &tm_k, 0, row_base + pos, bar(BAR_KFULL + st));
        tma_load_2d(kdst + KSUB_BYTES, &tm_k, 64, row_base + pos, bar(BAR_KFULL + st));
        mbar_expect_tx(bar(BAR_VFULL + st), TILE_BYTES);
        tma_load_2d(vdst, &tm_v, 0, row_base + pos, bar(BAR_VFULL + st));
        tma_load_2d(vdst + KSUB_BYTES, &tm_v, 64, row_base + pos, bar(BAR_VFULL + st));
    };
    int produced = n_blk;                    // tiles armed so far (the block tile is armed by the prologue)

    if (active) {
        if (warp == 8) {
            if (lane == 0) {
                for (int i = 0; i < 16; ++i) mbar_init(bar(i), 1);                // k/v full/empty
                mbar_init(bar(BAR_SFULL), 1); mbar_init(bar(BAR_SFULL + 1), 1);
                mbar_init(bar(BAR_OFULL), 1); mbar_init(bar(BAR_OFULL + 1), 1);
                mbar_init(bar(BAR_OFREE), 128); mbar_init(bar(BAR_OFREE + 1), 128);
                mbar_init(bar(BAR_AFULL), 128); mbar_init(bar(BAR_AFULL + 1), 128);
                mbar_init(bar(BAR_PFULL), 128);
                asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
                fence_proxy_async();
                // the first prefix tiles are requested before anything else happens
                while (produced < n_tiles && produced < NSTAGE) { issue_prefix(produced); ++produced; }
            }
        } else if (warp == 9) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                         ::"r"(smem_u32(tmem_slot)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            // warps 0-7: Q rows (replicated per sub-stream, zero-padded) and, in the owning
            // split, the block K/V rows (zero-padded to the tile) into the swizzled operand
            // layout; all global loads are issued before the first store
            const int t8 = tid;                                   // 0..255
            const uint4 zero = make_uint4(0, 0, 0, 0);
            const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(p.q);
            uint4 qv[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int e = t8 + k * 256, r = e >> 4, c = e & 15;
                const int Rl = r % MPAD, R = rt * MROWS + Rl;
                qv[k] = zero;
                if (Rl < rows_here) {
                    const int i = R / p.G, g = R % p.G;
                    qv[k] = __ldg(reinterpret_cast<const uint4 *>(
                                q + (((long long)b * p.K + i) * p.Hq + h * p.G + g) * HD) + c);
                }
            }
            uint4 kv[4], vv[4];
            if (n_blk) {
                const __nv_bfloat16 *kb = static_cast<const __nv_bfloat16 *>(p.k_blk);
                const __nv_bfloat16 *vb = static_cast<const __nv_bfloat16 *>(p.v_blk);
#pragma unroll
                for (int k = 0; k < 4; ++k) {                     // K <= 64 rows x 16 chunks
                    const int e = t8 + k * 256, r = e >> 4, c = e & 15;
                    kv[k] = zero; vv[k] = zero;
                    if (r < p.K) {
                        const long long off = (((long long)b * p.K + r) * p.Hkv + h) * HD;
                        kv[k] = __ldg(reinterpret_cast<const uint4 *>(kb + off) + c);
                        vv[k] = __ldg(reinterpret_cast<const uint4 *>(vb + off) + c);
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int e = t8 + k * 256, r = e >> 4, c = e & 15;
                *reinterpret_cast<uint4 *>(smem + OFF_Q + sw_off(r, c, PSUB_BYTES)) = qv[k];
            }
            if (NSUB > 1) {        // columns a sub-stream never writes must read as zero
                for (int e = t8; e < MROWS * (TN / 8); e += 256)
                    *reinterpret_cast<uint4 *>(smem + OFF_P + e * 16) = zero;
            }
            if (n_blk) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int e = t8 + k * 256, r = e >> 4, c = e & 15;
                    *reinterpret_cast<uint4 *>(smem + OFF_K + sw_off(r, c, KSUB_BYTES)) = kv[k];
                    *reinterpret_cast<uint4 *>(smem + OFF_V + sw_off(r, c, KSUB_BYTES)) = vv[k];
                }
                for (int e = t8 + 1024; e < TN * 16; e += 256) {  // V rows 64..TN-1 of the block tile
                    const int r = e >> 4, c = e & 15;
                    *reinterpret_cast<uint4 *>(smem + OFF_V + sw_off(r, c, KSUB_BYTES)) = zero;
                }
            }
            fence_proxy_async();
        }
    } else if (tid < MROWS) {
        ml_buf[tid * 2] = -INFINITY;          // an empty split publishes empty partial rows
        ml_buf[tid * 2 + 1] = 0.f;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = active ? *tmem_slot : 0u;
    if (tid == 0) TRACE(1);

    if (active && warp < 4) {
        // ------------------------------------------------------------------ softmax
        const int r = tid;
        const int sub = r / MPAD, Rl = r % MPAD;
        const int i_row = (rt * MROWS + Rl) / p.G;
        const int col0 = sub * W;
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16) + TM_S + col0;
        float m_run = -INFINITY, l_run = 0.f;
        for (int t = 0; t < n_tiles; ++t) {
            const int sb = t & 1;
            if (!mbar_wait(bar(BAR_SFULL + sb), (t >> 1) & 1, abort_flag)) break;
            tc_fence_after();
            if (tid == 0) TRACE(4 + 4 * t);
            uint32_t s[W];
#pragma unroll
            for (int c = 0; c < W / 32; ++c) tmem_ld32_nowait(lane_addr + sb * TN + c * 32, s + c * 32);
            tmem_ld_wait();
            const bool is_blk = t < n_blk;
            const int nv = is_blk ? p.K : min(TN, pos1 - (pos0 + (t - n_blk) * TN));
            // number of visible columns of this thread's range [col0, col0 + W)
            const int lim = min(W, max(0, ((is_blk && p.causal) ? min(nv, i_row + 1) : nv) - col0));
            float mx = -INFINITY;
            if (lim == W) {
#pragma unroll
                for (int j = 0; j < W; ++j) mx = fmaxf(mx, __uint_as_float(s[j]));
            } else {
#pragma unroll
                for (int j = 0; j < W; ++j) if (j < lim) mx = fmaxf(mx, __uint_as_float(s[j]));
            }
            const float m_new = fmaxf(m_run, mx * p.scale_log2);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;     // nothing visible so far
            const float alpha = ex2(m_run - m_use);
            m_run = m_new;
            if (tid == 0) TRACE(5 + 4 * t);
            // alpha slot (t&1) was last read by accumulate(t-2); P was last read by PV(t-1)
            if (t >= 2 && !mbar_wait(bar(BAR_OFREE + sb), ((t - 2) >> 1) & 1, abort_flag)) break;
            alpha_buf[sb * 128 + r] = alpha;
            mbar_arrive(bar(BAR_AFULL + sb));
            if (t >= 1 && !mbar_wait(bar(BAR_OFULL + ((t - 1) & 1)), ((t - 1) >> 1) & 1, abort_flag)) break;
            float lsum = 0.f;
#pragma unroll
            for (int c8 = 0; c8 < W / 8; ++c8) {
                uint32_t w[4];
#pragma unroll
                for (int j = 0; j < 8; j += 2) {
                    const int col = c8 * 8 + j;
                    float p0 = ex2(fmaf(__uint_as_float(s[col]), p.scale_log2, -m_use));
                    float p1 = ex2(fmaf(__uint_as_float(s[col + 1]), p.scale_log2, -m_use));
                    if (lim != W) {
                        if (col >= lim) p0 = 0.f;
                        if (col + 1 >= lim) p1 = 0.f;
                    }
                    lsum += p0 + p1;
                    w[j >> 1] = pack_bf16(p0, p1);
                }
                *reinterpret_cast<uint4 *>(smem + OFF_P + sw_off(r, col0 / 8 + c8, PSUB_BYTES)) =
                    make_uint4(w[0], w[1], w[2], w[3]);
            }
            l_run = l_run * alpha + lsum;
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(BAR_PFULL));
            if (tid == 0) TRACE(6 + 4 * t);
        }
        ml_buf[r * 2] = m_run;
        ml_buf[r * 2 + 1] = l_run;
    } else if (active && warp < 8) {
        // ------------------------------------------------------------------ accumulate
        const int r = tid - 128;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp - 4) * 32) << 16) + TM_O;
        float o[HD];
#pragma unroll
        for (int j = 0; j < HD; ++j) o[j] = 0.f;
        bool ok = true;
        for (int t = 0; t < n_tiles; ++t) {
            const int ob = t & 1;
            if (!mbar_wait(bar(BAR_AFULL + ob), (t >> 1) & 1, abort_flag)) { ok = false; break; }
            const float alpha = alpha_buf[ob * 128 + r];
            if (!mbar_wait(bar(BAR_OFULL + ob), (t >> 1) & 1, abort_flag)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t v[32];
                tmem_ld32_nowait(lane_addr + ob * 128 + c4 * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    o[c4 * 32 + j] = fmaf(o[c4 * 32 + j], alpha, __uint_as_float(v[j]));
            }
            tc_fence_before();
            mbar_arrive(bar(BAR_OFREE + ob));
            if (tid == 128) TRACE(7 + 4 * t);
        }
        // publish the partial row; the K ring is idle once the last P.V product has landed
        if (ok) {
#pragma unroll
            for (int c = 0; c < 32; ++c)
                *reinterpret_cast<float4 *>(smem + OFF_OPART + r * 512 + ((c ^ (r & 31)) << 4)) =
                    make_float4(o[c * 4], o[c * 4 + 1], o[c * 4 + 2], o[c * 4 + 3]);
        }
    } else if (active && warp == 8) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            if (n_blk) { mbar_arrive(bar(BAR_KFULL)); mbar_arrive(bar(BAR_VFULL)); }
            bool ok = true;
            for (int t = produced; t < n_tiles && ok; ++t) {
                const int st = t % NSTAGE, use = t / NSTAGE;
                // the stage was last used by tile t-NSTAGE: K is free after its QK, V after its PV
                ok = mbar_wait(bar(BAR_KEMPTY + st), (use - 1) & 1, abort_flag) &&
                     mbar_wait(bar(BAR_VEMPTY + st), (use - 1) & 1, abort_flag);
                if (ok) { issue_prefix(t); produced = t + 1; }
            }
            if (*abort_flag) {
                // give the copies that were armed a bounded time to land before smem is released
                for (int t = n_blk; t < produced; ++t) {
                    int dummy = 0;
                    mbar_wait(bar(BAR_KFULL + t % NSTAGE), (t / NSTAGE) & 1, &dummy);
                    dummy = 0;
                    mbar_wait(bar(BAR_VFULL + t % NSTAGE), (t / NSTAGE) & 1, &dummy);
                }
            }
        }
    } else if (active) {
        // ------------------------------------------------------------------ MMA issue
        const uint32_t q_addr = sbase + OFF_Q, p_addr = sbase + OFF_P;
        constexpr uint32_t IDESC_QK = make_idesc(TN, 0);      // A = Q, B = K tile, both K-major
        constexpr uint32_t IDESC_PV = make_idesc(HD, 1);      // A = P (K-major), B = V tile (MN-major)
        auto issue_qk = [&](int t) -> bool {
            const int st = t % NSTAGE;
            if (!mbar_wait(bar(BAR_KFULL + st), (t / NSTAGE) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                if (t < 4) TRACE(24 + t);
                const uint32_t k_addr = sbase + OFF_K + st * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < HD / 16; ++kk) {       // 16 head-dim columns per MMA
                    umma(tmem + TM_S + (t & 1) * TN,
                         make_desc(q_addr + (kk >> 2) * PSUB_BYTES + (kk & 3) * 32, 16, 1024),
                         make_desc(k_addr + (kk >> 2) * KSUB_BYTES + (kk & 3) * 32, 16, 1024),
                         IDESC_QK, kk > 0);
                }
                umma_commit(bar(BAR_KEMPTY + st));
                umma_commit(bar(BAR_SFULL + (t & 1)));
            }
            __syncwarp();
            return true;
        };
        auto issue_pv = [&](int u) -> bool {
            const int st = u % NSTAGE;
            if (!mbar_wait(bar(BAR_VFULL + st), (u / NSTAGE) & 1, abort_flag)) return false;
            // a ragged prefix tile: V rows past the chunk end may hold anything, and 0 * NaN
            // would poison the product, so they are cleared before the MMA reads them
            const bool is_blk = u < n_blk;
            const int nv = is_blk ? TN : min(TN, pos1 - (pos0 + (u - n_blk) * TN));
            if (nv < TN) {
                unsigned char *vt = smem + OFF_V + st * TILE_BYTES;
                for (int e = lane; e < (TN - nv) * 16; e += 32) {
                    const int rr = nv + (e >> 4), c = e & 15;
                    *reinterpret_cast<uint4 *>(vt + sw_off(rr, c, KSUB_BYTES)) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async();
                __syncwarp();
            }
            if (!mbar_wait(bar(BAR_PFULL), u & 1, abort_flag)) return false;
            if (u >= 2 && !mbar_wait(bar(BAR_OFREE + (u & 1)), ((u - 2) >> 1) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t v_addr = sbase + OFF_V + st * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < TN / 16; ++kk) {       // 16 key positions per MMA
                    umma(tmem + TM_O + (u & 1) * 128,
                         make_desc(p_addr + (kk >> 2) * PSUB_BYTES + (kk & 3) * 32, 16, 1024),
                         make_desc(v_addr + kk * 2048, KSUB_BYTES, 1024), IDESC_PV, kk > 0);
                }
                umma_commit(bar(BAR_VEMPTY + st));
                umma_commit(bar(BAR_OFULL + (u & 1)));
            }
            __syncwarp();
            return true;
        };
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            ok = issue_qk(t);
            if (ok && t > 0) ok = issue_pv(t - 1);
        }
        if (ok) ok = issue_pv(n_tiles - 1);
        if (ok)    // every MMA must have retired before the K ring is reused and TMEM is freed
            mbar_wait(bar(BAR_OFULL + ((n_tiles - 1) & 1)), ((n_tiles - 1) >> 1) & 1, abort_flag);
    }

    // ---------------------------------------------------------------------- merge
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid == 0) TRACE(2);
    if (active && warp == 9)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    if (tid == 0 && *abort_flag && p.status) atomicOr(p.status, ORTHRUS_DEV_WAIT_TIMEOUT);
    if (cluster_size > 1) cluster_sync_all();

    const int my_rank = cluster_size > 1 ? (int)cluster_rank() : 0;
    const int n_part = cluster_size * NSUB;                   // <= 32 partial rows per logical row
    const bool final_out = (cluster_size == p.n_splits);
    if (warp < 8) {
        const int pj_rank = lane / NSUB, pj_sub = lane % NSUB;
        for (int Rl = my_rank + cluster_size * warp; Rl < rows_here; Rl += cluster_size * 8) {
            float mj = -INFINITY, lj = 0.f;
            if (lane < n_part) {
                const uint32_t a = sbase + OFF_ML + (pj_sub * MPAD + Rl) * 8;
                const float2 v = ld_cluster_f2(cluster_size > 1 ? map_to_rank(a, pj_rank) : a);
                mj = v.x; lj = v.y;
            }
            float mmax = mj;
#pragma unroll
            for (int off = 16; off; off >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, off));
            const float wj = (lj > 0.f) ? ex2(mj - mmax) : 0.f;
            float L = wj * lj;
#pragma unroll
            for (int off = 16; off; off >>= 1) L += __shfl_xor_sync(0xffffffffu, L, off);
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
            for (int j = 0; j < n_part; ++j) {
                const float w = __shfl_sync(0xffffffffu, wj, j);
                if (w != 0.f) {
                    const int row = (j % NSUB) * MPAD + Rl;
                    const uint32_t a = sbase + OFF_OPART + row * 512 + ((lane ^ (row & 31)) << 4);
                    const float4 v = ld_cluster_f4(cluster_size > 1 ? map_to_rank(a, j / NSUB) : a);
                    acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y);
                    acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
                }
            }
            const int R = rt * MROWS + Rl;
            if (final_out) {
                const int i = R / p.G, g = R % p.G;
                const float inv = 1.f / L;
                uint2 *dst = reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(p.out) +
                             (((long long)b * p.K + i) * p.Hq + h * p.G + g) * HD);
                dst[lane] = make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
            } else {
                const long long row = ((long long)unit * p.n_splits + split) * p.M + R;
                reinterpret_cast<float4 *>(p.part_o + row * HD)[lane] = acc;
                if (lane == 0) { p.part_ml[row * 2] = mmax; p.part_ml[row * 2 + 1] = L; }
            }
        }
    }
    if (cluster_size > 1) cluster_sync_all();     // peers may still be reading this CTA's rows
    if (tid == 0) TRACE(3);
}

// ---------------------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

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

// 2-D view of a cache tensor: rows = B*Hkv*capacity positions, 128 bf16 columns;
// box = 64 columns x `box_rows` rows, 128-byte swizzle.  Maps are cached by key.
struct MapKey {
    const void *ptr; unsigned long long rows; int box_rows;
    bool operator==(const MapKey &o) const { return ptr == o.ptr && rows == o.rows && box_rows == o.box_rows; }
};
struct MapKeyHash {
    size_t operator()(const MapKey &k) const {
        return std::hash<const void *>()(k.ptr) ^ (std::hash<unsigned long long>()(k.rows) * 0x9E3779B97F4A7C15ull) ^
               (size_t)k.box_rows;
    }
};

bool get_map(const void *ptr, unsigned long long rows, int box_rows, CUtensorMap *out)
{
    static std::mutex mu;
    static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
    std::lock_guard<std::mutex> lock(mu);
    const MapKey key{ptr, rows, box_rows};
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)HD, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)HD * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap tm;
    const CUresult r = fn(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims,
                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (cache.size() > 4096) cache.clear();
    cache.emplace(key, tm);
    *out = tm;
    return true;
}

template <int TN, int NSUB>
cudaError_t launch_one(const AttnParams &p, int cluster, cudaStream_t st)
{
    const unsigned long long rows = (unsigned long long)p.B * p.Hkv * p.capacity;
    CUtensorMap tk, tv;
    if (!get_map(p.k_cache, rows, TN, &tk) || !get_map(p.v_cache, rows, TN, &tv)) return cudaErrorInvalidValue;
    auto kern = attend_tc_kernel<TN, NSUB>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.B * p.Hkv, p.n_splits, (p.M + MROWS - 1) / MROWS);
    cfg.blockDim = dim3(NTHREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    int n_attr = 0;
    if (cluster > 1) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 1;
        attr[n_attr].val.clusterDim.y = cluster;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, p, tk, tv, cluster);
    count_launch();
    return e;
}

}  // namespace

bool tc_path_supports(const AttnParams &p, int dtype)
{
    if (dtype != ORTHRUS_BF16 || p.d != HD || p.K > 64) return false;
    const unsigned long long rows = (unsigned long long)p.B * p.Hkv * p.capacity;
    return rows < 0x7fffffffull && encode_fn() != nullptr;
}

// Cluster size the kernel will use for a split count: all splits of a unit in one
// cluster when there are at most 16, otherwise none (global partials + merge kernel).
int tc_cluster_for_splits(int n_splits) { return n_splits <= 16 ? n_splits : 1; }

cudaError_t launch_attend_tc(const AttnParams &p, int tile, cudaStream_t st)
{
    const int cluster = tc_cluster_for_splits(p.n_splits);
    int nsub = p.M <= 32 ? 4 : (p.M <= 64 ? 2 : 1);
    while (nsub > 1 && (cluster * nsub > 32 || tile / nsub < 32)) nsub >>= 1;
    if (tile == 64) {
        return nsub >= 2 ? launch_one<64, 2>(p, cluster, st) : launch_one<64, 1>(p, cluster, st);
    }
    if (nsub == 4) return launch_one<128, 4>(p, cluster, st);
    if (nsub == 2) return launch_one<128, 2>(p, cluster, st);
    return launch_one<128, 1>(p, cluster, st);
}

}  // namespace orthrus

#ifdef ORTHRUS_TC_TRACE
extern "C" int orthrus_debug_read_trace(unsigned long long *host, int n_words)
{
    return (int)cudaMemcpyFromSymbol(host, orthrus::g_trace, sizeof(unsigned long long) * n_words);
}
#endif
