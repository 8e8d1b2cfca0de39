// Split-KV flash-decode block attention on the 5th-generation tensor cores
// (tcgen05.mma with TMEM accumulators), bf16, head_dim 128, both views.
//
// One CTA streams one split of one (sequence, KV head) unit.  The query tile is the
// GQA group times the block width (M = G*K <= 128 rows, zero-padded to the 128-row MMA).
// Warp roles:
//   warps 0-3  softmax: thread r owns score row r (TMEM lane r): row max, exp2, row
//              sum, bf16 probabilities written to shared memory as the A operand of PV
//   warps 4-7  accumulate: thread r keeps output row r (128 fp32) in registers and folds
//              in each tile's P.V product with the rescale factor of the online softmax
//   warp 8     producer: TMA loads of 128-position K and V tiles (two 64-column boxes
//              each, 128-byte swizzle) into a two-stage ring
//   warp 9     MMA issue (one elected lane) and TMEM allocation
// S = Q.K^T is double-buffered in TMEM so QK(t+1) overlaps softmax(t); each P.V product
// lands in its own TMEM buffer and is drained by the accumulate warps.
// Every wait on an mbarrier is bounded: on expiry the kernel records
// ORTHRUS_DEV_WAIT_TIMEOUT in the status word, drains what it armed, frees its TMEM and
// returns.
#include <cuda.h>
#include <mutex>
#include <unordered_map>
#include "common.cuh"

namespace orthrus {
namespace {

constexpr int HD = 128;            // head_dim
constexpr int TN = 128;            // key positions per tile
constexpr int MROWS = 128;         // MMA M
constexpr int SUB_BYTES = 128 * 128;          // one [128 rows][64 cols] bf16 sub-tile
constexpr int TILE_BYTES = 2 * SUB_BYTES;     // a [128][128] bf16 tile
constexpr int NSTAGE = 2;
constexpr int NTHREADS = 320;

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_Q = 0;
constexpr int OFF_P = OFF_Q + TILE_BYTES;
constexpr int OFF_K = OFF_P + TILE_BYTES;
constexpr int OFF_V = OFF_K + NSTAGE * TILE_BYTES;
constexpr int OFF_ALPHA = OFF_V + NSTAGE * TILE_BYTES;       // float [2][128]
constexpr int OFF_ML = OFF_ALPHA + 2 * 128 * 4;              // float [128][2]
constexpr int OFF_BAR = OFF_ML + 128 * 2 * 4;                // mbarriers
constexpr int NUM_BARS = 16;
constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;             // tmem base, abort flag
constexpr int SMEM_BYTES = OFF_MISC + 64;

enum { BAR_KFULL = 0, BAR_VFULL = 2, BAR_KEMPTY = 4, BAR_VEMPTY = 6, BAR_SFULL = 8,
       BAR_OFULL = 10, BAR_OFREE = 12, BAR_AFULL = 14 };   // each x2
constexpr int BAR_PFULL_OFF = OFF_MISC + 16;               // one more barrier, 8 bytes

__device__ inline uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

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
// instruction descriptor: D fp32, A/B bf16, M = 128, N = 128
constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t IDESC_QK = IDESC_BASE;                 // A, B both K-major
constexpr uint32_t IDESC_PV = IDESC_BASE | (1u << 16);    // B (V) is MN-major

__device__ inline void umma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
                 " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
}
__device__ inline void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                 ::"r"(bar) : "memory");
}
__device__ inline void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
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
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}
__device__ inline float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
// byte offset of 16-byte chunk `c` (0..15) of row `r` inside a [128][128] bf16 tile held
// as two 128-byte-swizzled [128][64] sub-tiles
__device__ inline uint32_t sw_off(int r, int c) {
    return (uint32_t)((c >> 3) * SUB_BYTES + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// 32 score columns of one row: probabilities 2^(s*scale - m), their sum, and the bf16
// values stored as four 16-byte chunks of the swizzled P operand tile
template <bool MASKED>
__device__ inline float softmax_chunk(unsigned char *smem, uint32_t s_addr, int r, int c4, int lim,
                                      float scale_log2, float m_new)
{
    float v[32];
    tmem_ld32(s_addr + c4 * 32, v);
    uint32_t w[16];
    float lsum = 0.f;
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
        float p0 = ex2(fmaf(v[j], scale_log2, -m_new));
        float p1 = ex2(fmaf(v[j + 1], scale_log2, -m_new));
        if (MASKED) {
            if (c4 * 32 + j >= lim) p0 = 0.f;
            if (c4 * 32 + j + 1 >= lim) p1 = 0.f;
        }
        lsum += p0 + p1;
        w[j >> 1] = pack_bf16(p0, p1);
    }
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4)
        *reinterpret_cast<uint4 *>(smem + OFF_P + sw_off(r, c4 * 4 + q4)) =
            make_uint4(w[q4 * 4], w[q4 * 4 + 1], w[q4 * 4 + 2], w[q4 * 4 + 3]);
    return lsum;
}

__global__ void __launch_bounds__(NTHREADS, 1)
attend_tc_kernel(AttnParams p, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);
    float *alpha_buf = reinterpret_cast<float *>(smem + OFF_ALPHA);
    float *ml_buf = reinterpret_cast<float *>(smem + OFF_ML);
    auto bar = [&](int i) { return sbase + OFF_BAR + i * 8; };
    const uint32_t bar_pfull = sbase + BAR_PFULL_OFF;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit = blockIdx.x, split = blockIdx.y, rt = blockIdx.z;
    const int b = unit / p.Hkv, h = unit % p.Hkv;
    const int P = clamp_cache_len(p, b);
    const int ls = last_split(P, p.chunk);
    if (split > ls) return;                                  // uniform: nothing armed yet
    const int pos0 = split * p.chunk;
    const int pos1 = min(P, pos0 + p.chunk);
    const int n_prefix = pos1 > pos0 ? (pos1 - pos0 + TN - 1) / TN : 0;
    const int n_blk = (split == ls) ? 1 : 0;                 // the block tile comes first
    const int n_tiles = n_prefix + n_blk;

    if ((sbase & 1023u) != 0) {                              // swizzled tiles need 1 KB alignment
        if (tid == 0 && p.status) atomicOr(p.status, ORTHRUS_DEV_WAIT_TIMEOUT);
        return;
    }

    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < 8; ++i) mbar_init(bar(i), 1);                 // k/v full/empty
        mbar_init(bar(BAR_SFULL), 1); mbar_init(bar(BAR_SFULL + 1), 1);
        mbar_init(bar(BAR_OFULL), 1); mbar_init(bar(BAR_OFULL + 1), 1);
        mbar_init(bar(BAR_OFREE), 128); mbar_init(bar(BAR_OFREE + 1), 128);
        mbar_init(bar(BAR_AFULL), 128); mbar_init(bar(BAR_AFULL + 1), 128);
        mbar_init(bar_pfull, 128);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                     ::"r"(smem_u32(tmem_slot)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // the producer arms the first prefix tiles before the cooperative prologue loads
    const int row_base = (int)((long long)unit * p.capacity);      // row of position 0 in the 2-D map
    auto issue_prefix = [&](int t) {                               // t: tile index in this CTA
        const int st = t & 1;
        const int pos = pos0 + (t - n_blk) * TN;
        const uint32_t kdst = sbase + OFF_K + st * TILE_BYTES;
        const uint32_t vdst = sbase + OFF_V + st * TILE_BYTES;
        mbar_expect_tx(bar(BAR_KFULL + st), TILE_BYTES);
        tma_load_2d(kdst, &tm_k, 0, row_base + pos, bar(BAR_KFULL + st));
        tma_load_2d(kdst + SUB_BYTES, &tm_k, 64, row_base + pos, bar(BAR_KFULL + st));
        mbar_expect_tx(bar(BAR_VFULL + st), TILE_BYTES);
        tma_load_2d(vdst, &tm_v, 0, row_base + pos, bar(BAR_VFULL + st));
        tma_load_2d(vdst + SUB_BYTES, &tm_v, 64, row_base + pos, bar(BAR_VFULL + st));
    };
    int produced = n_blk;                        // tiles armed so far (the block tile is armed below)
    if (warp == 8 && lane == 0) {
        while (produced < n_tiles && produced < NSTAGE) { issue_prefix(produced); ++produced; }
    }

    // prologue, all threads: Q rows (zero-padded) and, in the owning split, the block K/V
    // rows (V zero-padded to the full tile) into the swizzled operand layout
    {
        const uint4 zero = make_uint4(0, 0, 0, 0);
        const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(p.q);
        for (int e = tid; e < MROWS * 16; e += NTHREADS) {
            const int r = e >> 4, c = e & 15;
            const int R = rt * MROWS + r;
            uint4 v = zero;
            if (R < p.M) {
                const int i = R / p.G, g = R % p.G;
                v = __ldg(reinterpret_cast<const uint4 *>(
                        q + (((long long)b * p.K + i) * p.Hq + h * p.G + g) * HD) + c);
            }
            *reinterpret_cast<uint4 *>(smem + OFF_Q + sw_off(r, c)) = v;
        }
        if (n_blk) {
            const __nv_bfloat16 *kb = static_cast<const __nv_bfloat16 *>(p.k_blk);
            const __nv_bfloat16 *vb = static_cast<const __nv_bfloat16 *>(p.v_blk);
            for (int e = tid; e < TN * 16; e += NTHREADS) {
                const int r = e >> 4, c = e & 15;
                uint4 kv = zero, vv = zero;
                if (r < p.K) {
                    const long long off = (((long long)b * p.K + r) * p.Hkv + h) * HD;
                    kv = __ldg(reinterpret_cast<const uint4 *>(kb + off) + c);
                    vv = __ldg(reinterpret_cast<const uint4 *>(vb + off) + c);
                }
                *reinterpret_cast<uint4 *>(smem + OFF_K + sw_off(r, c)) = kv;
                *reinterpret_cast<uint4 *>(smem + OFF_V + sw_off(r, c)) = vv;
            }
        }
        fence_proxy_async();
    }
    __syncthreads();

    if (warp < 4) {
        // ------------------------------------------------------------------ softmax
        const int r = tid;
        const int R = rt * MROWS + r;
        const int i_row = R / p.G;
        const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
        float m_run = -INFINITY, l_run = 0.f;
        for (int t = 0; t < n_tiles; ++t) {
            const int sb = t & 1;
            if (!mbar_wait(bar(BAR_SFULL + sb), (t >> 1) & 1, abort_flag)) break;
            tc_fence_after();
            const bool is_blk = t < n_blk;
            const int nv = is_blk ? p.K : min(TN, pos1 - (pos0 + (t - n_blk) * TN));
            const int lim = (is_blk && p.causal) ? min(nv, i_row + 1) : nv;
            const uint32_t s_addr = lane_addr + sb * 128;
            float mx = -INFINITY;
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                float v[32];
                tmem_ld32(s_addr + c4 * 32, v);
                if (lim >= (c4 + 1) * 32) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) mx = fmaxf(mx, v[j]);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) if (c4 * 32 + j < lim) mx = fmaxf(mx, v[j]);
                }
            }
            const float m_new = fmaxf(m_run, mx * p.scale_log2);
            const float alpha = ex2(m_run - m_new);
            m_run = m_new;
            // alpha slot (t&1) was last read by accumulate(t-2); P was last read by PV(t-1)
            if (t >= 2 && !mbar_wait(bar(BAR_OFREE + sb), ((t - 2) >> 1) & 1, abort_flag)) break;
            alpha_buf[sb * 128 + r] = alpha;
            mbar_arrive(bar(BAR_AFULL + sb));
            if (t >= 1 && !mbar_wait(bar(BAR_OFULL + ((t - 1) & 1)), ((t - 1) >> 1) & 1, abort_flag)) break;
            float lsum = 0.f;
            if (lim >= TN) {
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4)
                    lsum += softmax_chunk<false>(smem, s_addr, r, c4, lim, p.scale_log2, m_new);
            } else {
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4)
                    lsum += softmax_chunk<true>(smem, s_addr, r, c4, lim, p.scale_log2, m_new);
            }
            l_run = l_run * alpha + lsum;
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar_pfull);
        }
        ml_buf[r * 2] = m_run;
        ml_buf[r * 2 + 1] = l_run;
    } else if (warp < 8) {
        // ------------------------------------------------------------------ accumulate
        const int r = tid - 128;
        const uint32_t lane_addr = tmem + ((uint32_t)((warp - 4) * 32) << 16) + 256;
        float o[HD];
#pragma unroll
        for (int j = 0; j < HD; ++j) o[j] = 0.f;
        for (int t = 0; t < n_tiles; ++t) {
            const int ob = t & 1;
            if (!mbar_wait(bar(BAR_AFULL + ob), (t >> 1) & 1, abort_flag)) break;
            const float alpha = alpha_buf[ob * 128 + r];
            if (!mbar_wait(bar(BAR_OFULL + ob), (t >> 1) & 1, abort_flag)) break;
            tc_fence_after();
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                float v[32];
                tmem_ld32(lane_addr + ob * 128 + c4 * 32, v);
#pragma unroll
                for (int j = 0; j < 32; ++j) o[c4 * 32 + j] = fmaf(o[c4 * 32 + j], alpha, v[j]);
            }
            tc_fence_before();
            mbar_arrive(bar(BAR_OFREE + ob));
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");       // m, l of the softmax warps are in ml_buf
        const int R = rt * MROWS + r;
        if (R < p.M && !*abort_flag) {
            const float l = ml_buf[r * 2 + 1];
            if (p.n_splits == 1) {
                const int i = R / p.G, g = R % p.G;
                uint4 *dst = reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(p.out) +
                             (((long long)b * p.K + i) * p.Hq + h * p.G + g) * HD);
                const float inv = 1.f / l;
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    dst[c] = make_uint4(pack_bf16(o[c * 8] * inv, o[c * 8 + 1] * inv),
                                        pack_bf16(o[c * 8 + 2] * inv, o[c * 8 + 3] * inv),
                                        pack_bf16(o[c * 8 + 4] * inv, o[c * 8 + 5] * inv),
                                        pack_bf16(o[c * 8 + 6] * inv, o[c * 8 + 7] * inv));
            } else {
                const long long row = ((long long)unit * p.n_splits + split) * p.M + R;
                float4 *dst = reinterpret_cast<float4 *>(p.part_o + row * HD);
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    dst[c] = make_float4(o[c * 4], o[c * 4 + 1], o[c * 4 + 2], o[c * 4 + 3]);
                p.part_ml[row * 2] = ml_buf[r * 2];
                p.part_ml[row * 2 + 1] = l;
            }
        }
    } else if (warp == 8) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            if (n_blk) { mbar_arrive(bar(BAR_KFULL)); mbar_arrive(bar(BAR_VFULL)); }
            bool ok = true;
            for (int t = produced; t < n_tiles && ok; ++t) {
                const int st = t & 1;
                // the stage was used by tile t-2: K freed after QK(t-2), V after PV(t-2)
                ok = mbar_wait(bar(BAR_KEMPTY + st), ((t - 2) >> 1) & 1, abort_flag) &&
                     mbar_wait(bar(BAR_VEMPTY + st), ((t - 2) >> 1) & 1, abort_flag);
                if (ok) { issue_prefix(t); produced = t + 1; }
            }
            if (*abort_flag) {
                // give the copies that were armed a bounded time to land before smem is released
                for (int t = n_blk; t < produced; ++t) {
                    int dummy = 0;
                    mbar_wait(bar(BAR_KFULL + (t & 1)), (t >> 1) & 1, &dummy);
                    dummy = 0;
                    mbar_wait(bar(BAR_VFULL + (t & 1)), (t >> 1) & 1, &dummy);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ MMA issue
        const uint32_t q_addr = sbase + OFF_Q, p_addr = sbase + OFF_P;
        auto issue_qk = [&](int t) -> bool {
            const int st = t & 1;
            if (!mbar_wait(bar(BAR_KFULL + st), (t >> 1) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t k_addr = sbase + OFF_K + st * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {             // 16 head-dim columns per MMA
                    const uint32_t off = (kk >> 2) * SUB_BYTES + (kk & 3) * 32;
                    umma(tmem + (t & 1) * 128, make_desc(q_addr + off, 16, 1024),
                         make_desc(k_addr + off, 16, 1024), IDESC_QK, kk > 0);
                }
                umma_commit(bar(BAR_KEMPTY + st));
                umma_commit(bar(BAR_SFULL + (t & 1)));
            }
            __syncwarp();
            return true;
        };
        auto issue_pv = [&](int u) -> bool {
            const int st = u & 1;
            if (!mbar_wait(bar(BAR_VFULL + st), (u >> 1) & 1, abort_flag)) return false;
            // a ragged prefix tile: V rows past the chunk end may hold anything, and 0 * NaN
            // would poison the product, so they are cleared before the MMA reads them
            const bool is_blk = u < n_blk;
            const int nv = is_blk ? TN : min(TN, pos1 - (pos0 + (u - n_blk) * TN));
            if (nv < TN) {
                unsigned char *vt = smem + OFF_V + st * TILE_BYTES;
                for (int e = lane; e < (TN - nv) * 16; e += 32) {
                    const int rr = nv + (e >> 4), c = e & 15;
                    *reinterpret_cast<uint4 *>(vt + sw_off(rr, c)) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async();
                __syncwarp();
            }
            if (!mbar_wait(bar_pfull, u & 1, abort_flag)) return false;
            if (u >= 2 && !mbar_wait(bar(BAR_OFREE + (u & 1)), ((u - 2) >> 1) & 1, abort_flag)) return false;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t v_addr = sbase + OFF_V + st * TILE_BYTES;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {             // 16 key positions per MMA
                    const uint64_t a = make_desc(p_addr + (kk >> 2) * SUB_BYTES + (kk & 3) * 32, 16, 1024);
                    const uint64_t bdesc = make_desc(v_addr + kk * 2048, SUB_BYTES, 1024);
                    umma(tmem + 256 + (u & 1) * 128, a, bdesc, IDESC_PV, kk > 0);
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
        if (ok && n_tiles > 0) ok = issue_pv(n_tiles - 1);
        if (ok) {
            // every MMA must have retired before TMEM is freed
            mbar_wait(bar(BAR_OFULL + ((n_tiles - 1) & 1)), ((n_tiles - 1) >> 1) & 1, abort_flag);
        }
    }
    if (warp < 4) asm volatile("bar.sync 1, 256;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 9) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
    if (tid == 0 && *abort_flag && p.status) atomicOr(p.status, ORTHRUS_DEV_WAIT_TIMEOUT);
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
// box = 64 columns x 128 rows, 128-byte swizzle.  Maps are cached by (pointer, rows).
struct MapKey {
    const void *ptr; unsigned long long rows;
    bool operator==(const MapKey &o) const { return ptr == o.ptr && rows == o.rows; }
};
struct MapKeyHash {
    size_t operator()(const MapKey &k) const {
        return std::hash<const void *>()(k.ptr) ^ (std::hash<unsigned long long>()(k.rows) * 0x9E3779B97F4A7C15ull);
    }
};

bool get_map(const void *ptr, unsigned long long rows, CUtensorMap *out)
{
    static std::mutex mu;
    static std::unordered_map<MapKey, CUtensorMap, MapKeyHash> cache;
    std::lock_guard<std::mutex> lock(mu);
    const MapKey key{ptr, rows};
    auto it = cache.find(key);
    if (it != cache.end()) { *out = it->second; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)HD, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)HD * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)TN};
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

}  // namespace

int tc_tile_positions() { return TN; }

bool tc_path_supports(const AttnParams &p, int dtype)
{
    if (dtype != ORTHRUS_BF16 || p.d != HD || p.K > 64) return false;
    const unsigned long long rows = (unsigned long long)p.B * p.Hkv * p.capacity;
    return rows < 0x7fffffffull && encode_fn() != nullptr;
}

cudaError_t launch_attend_tc(const AttnParams &p, cudaStream_t st)
{
    const unsigned long long rows = (unsigned long long)p.B * p.Hkv * p.capacity;
    CUtensorMap tk, tv;
    if (!get_map(p.k_cache, rows, &tk) || !get_map(p.v_cache, rows, &tv)) return cudaErrorInvalidValue;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(attend_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             SMEM_BYTES);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid(p.B * p.Hkv, p.n_splits, (p.M + MROWS - 1) / MROWS);
    attend_tc_kernel<<<grid, NTHREADS, SMEM_BYTES, st>>>(p, tk, tv);
    count_launch();
    return cudaGetLastError();
}

}  // namespace orthrus
