// Split-KV flash-decode block attention on warp-level tensor-core MMAs (bf16 inputs,
// fp32 accumulation), for both views.  The tile is the GQA group times the block
// width: M = G*K query rows of one (sequence, KV head) unit share every K/V row that
// is streamed.  One CTA = (unit, split, row tile of 16 rows per warp).  K/V tiles of 64
// positions travel global -> shared with 16-byte cp.async through a 3-stage ring, in
// an XOR-swizzled layout that ldmatrix reads without bank conflicts; the running
// max / sum of the online softmax live in registers and are reduced across the four
// lanes that share a row with shuffles.
#include "common.cuh"

namespace orthrus {
namespace {

constexpr int TN = 64;       // key positions per tile
constexpr int STAGES = 3;

__device__ inline uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ inline void cp_async16(uint32_t dst, const void *src, bool valid) {
    const int n = valid ? 16 : 0;      // src-size 0: the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(n));
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ inline void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ inline void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ inline void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ inline void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
                 "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ inline float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

template <int HD, int NWARPS>
__global__ void __launch_bounds__(NWARPS * 32) attend_mma_kernel(AttnParams p)
{
    constexpr int MT = NWARPS * 16;
    constexpr int ROW_BYTES = HD * 2;
    constexpr int ROW_CHUNKS = ROW_BYTES / 16;
    constexpr int TILE_BYTES = TN * ROW_BYTES;
    constexpr int NTHREADS = NWARPS * 32;
    extern __shared__ __align__(128) unsigned char smem_raw[];

    const int unit = blockIdx.x, split = blockIdx.y, rt = blockIdx.z;
    const int b = unit / p.Hkv, h = unit % p.Hkv;
    const int P = clamp_cache_len(p, b);
    const int ls = last_split(P, p.chunk);
    if (split > ls) return;
    const int pos0 = split * p.chunk;
    const int pos1 = min(P, pos0 + p.chunk);
    const int n_prefix_tiles = pos1 > pos0 ? (pos1 - pos0 + TN - 1) / TN : 0;
    const int n_blk_tiles = (split == ls) ? 1 : 0;         // K <= 64: one tile
    const int n_tiles = n_prefix_tiles + n_blk_tiles;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gq = lane >> 2, tq = lane & 3;               // row within 8, column pair
    const uint32_t smem_base = smem_u32(smem_raw);

    const long long cache_unit = (long long)(b / p.nb) * p.Hkv + h;      // whose cache this batch entry reads
    const __nv_bfloat16 *kc = static_cast<const __nv_bfloat16 *>(p.k_cache) + cache_unit * p.capacity * HD;
    const __nv_bfloat16 *vc = static_cast<const __nv_bfloat16 *>(p.v_cache) + cache_unit * p.capacity * HD;
    // the block's rows: K rows of the block tensors, or the cache rows behind the prefix
    const __nv_bfloat16 *kb = p.blk_in_cache ? kc + (long long)P * HD
        : static_cast<const __nv_bfloat16 *>(p.k_blk) + ((long long)b * p.K * p.Hkv + h) * HD;
    const __nv_bfloat16 *vb = p.blk_in_cache ? vc + (long long)P * HD
        : static_cast<const __nv_bfloat16 *>(p.v_blk) + ((long long)b * p.K * p.Hkv + h) * HD;

    // tile t: block tile first (if this split owns it), then the prefix tiles
    auto issue_tile = [&](int t, int stage) {
        const bool is_blk = t < n_blk_tiles;
        const int base = is_blk ? 0 : pos0 + (t - n_blk_tiles) * TN;
        const int nv = is_blk ? p.K : min(TN, pos1 - base);
        const long long row_stride = (is_blk && !p.blk_in_cache) ? (long long)p.Hkv * HD : HD;
        const __nv_bfloat16 *ks = is_blk ? kb : kc + (long long)base * HD;
        const __nv_bfloat16 *vs = is_blk ? vb : vc + (long long)base * HD;
        const uint32_t sk = smem_base + stage * 2 * TILE_BYTES;
        const uint32_t sv = sk + TILE_BYTES;
#pragma unroll
        for (int e = tid; e < TN * ROW_CHUNKS; e += NTHREADS) {
            const int r = e / ROW_CHUNKS, c = e % ROW_CHUNKS;
            const bool valid = r < nv;
            const long long off = valid ? r * row_stride + c * 8 : 0;
            const uint32_t so = r * ROW_BYTES + ((c ^ (r & 7)) << 4);
            cp_async16(sk + so, ks + off, valid);
            cp_async16(sv + so, vs + off, valid);
        }
    };

#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        if (s < n_tiles) issue_tile(s, s);
        cp_async_commit();
    }

    // query fragments straight from global memory (A operand, 16 rows x HD per warp)
    const int R0 = rt * MT + warp * 16 + gq;
    const int R1 = R0 + 8;
    const int i0 = R0 / p.G, i1 = R1 / p.G;
    uint32_t qf[HD / 16][4];
    {
        const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(p.q);
        const uint32_t *q0 = reinterpret_cast<const uint32_t *>(
            q + (((long long)b * p.K + i0) * p.Hq + h * p.G + R0 % p.G) * HD);
        const uint32_t *q1 = reinterpret_cast<const uint32_t *>(
            q + (((long long)b * p.K + i1) * p.Hq + h * p.G + R1 % p.G) * HD);
        const bool v0 = R0 < p.M, v1 = R1 < p.M;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
            qf[ks][0] = v0 ? __ldg(q0 + ks * 8 + tq) : 0u;
            qf[ks][1] = v1 ? __ldg(q1 + ks * 8 + tq) : 0u;
            qf[ks][2] = v0 ? __ldg(q0 + ks * 8 + 4 + tq) : 0u;
            qf[ks][3] = v1 ? __ldg(q1 + ks * 8 + 4 + tq) : 0u;
        }
    }

    float o[HD / 8][4];
#pragma unroll
    for (int j = 0; j < HD / 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    for (int t = 0; t < n_tiles; ++t) {
        cp_async_wait<STAGES - 2>();
        __syncthreads();
        {
            const int tn = t + STAGES - 1;
            if (tn < n_tiles) issue_tile(tn, tn % STAGES);
            cp_async_commit();
        }
        const int stage = t % STAGES;
        const uint32_t sk = smem_base + stage * 2 * TILE_BYTES;
        const uint32_t sv = sk + TILE_BYTES;

        // S = Q K^T  (16 x 64 per warp)
        float s[TN / 8][4];
#pragma unroll
        for (int j = 0; j < TN / 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < TN / 16; ++np) {
                const int r = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                const int c = ks * 2 + ((lane >> 3) & 1);
                uint32_t kf[4];
                ldmatrix_x4(kf, sk + r * ROW_BYTES + ((c ^ (r & 7)) << 4));
                mma_bf16(s[2 * np], qf[ks], kf[0], kf[1]);
                mma_bf16(s[2 * np + 1], qf[ks], kf[2], kf[3]);
            }
        }

        // masks: ragged tail of the prefix chunk; block rows past K; causal rule in the AR view
        const bool is_blk = t < n_blk_tiles;
        const int nv = is_blk ? p.K : min(TN, pos1 - (pos0 + (t - n_blk_tiles) * TN));
        if (nv < TN || (is_blk && p.causal)) {
            const int lim0 = (is_blk && p.causal) ? min(nv, i0 + 1) : nv;
            const int lim1 = (is_blk && p.causal) ? min(nv, i1 + 1) : nv;
#pragma unroll
            for (int j = 0; j < TN / 8; ++j) {
                const int col = j * 8 + tq * 2;
                if (col >= lim0) s[j][0] = -INFINITY;
                if (col + 1 >= lim0) s[j][1] = -INFINITY;
                if (col >= lim1) s[j][2] = -INFINITY;
                if (col + 1 >= lim1) s[j][3] = -INFINITY;
            }
        }

        // online softmax (scores kept in the log2 domain)
        float t0 = -INFINITY, t1 = -INFINITY;
#pragma unroll
        for (int j = 0; j < TN / 8; ++j) {
            t0 = fmaxf(t0, fmaxf(s[j][0], s[j][1]));
            t1 = fmaxf(t1, fmaxf(s[j][2], s[j][3]));
        }
        t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 1));
        t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 2));
        t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 1));
        t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 2));
        const float mn0 = fmaxf(m0, t0 * p.scale_log2);
        const float mn1 = fmaxf(m1, t1 * p.scale_log2);
        const float a0 = ex2(m0 - mn0), a1 = ex2(m1 - mn1);
        m0 = mn0; m1 = mn1;
        float ps0 = 0.f, ps1 = 0.f;
        uint32_t pf[TN / 16][4];
#pragma unroll
        for (int j = 0; j < TN / 8; ++j) {
            const float p0 = ex2(fmaf(s[j][0], p.scale_log2, -mn0));
            const float p1 = ex2(fmaf(s[j][1], p.scale_log2, -mn0));
            const float p2 = ex2(fmaf(s[j][2], p.scale_log2, -mn1));
            const float p3 = ex2(fmaf(s[j][3], p.scale_log2, -mn1));
            ps0 += p0 + p1;
            ps1 += p2 + p3;
            pf[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
            pf[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        l0 = l0 * a0 + ps0;
        l1 = l1 * a1 + ps1;
#pragma unroll
        for (int j = 0; j < HD / 8; ++j) {
            o[j][0] *= a0; o[j][1] *= a0; o[j][2] *= a1; o[j][3] *= a1;
        }

        // O += P V  (16 x HD per warp)
#pragma unroll
        for (int kk = 0; kk < TN / 16; ++kk) {
#pragma unroll
            for (int dp = 0; dp < HD / 16; ++dp) {
                const int r = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                const int c = dp * 2 + (lane >> 4);
                uint32_t vf[4];
                ldmatrix_x4_trans(vf, sv + r * ROW_BYTES + ((c ^ (r & 7)) << 4));
                mma_bf16(o[2 * dp], pf[kk], vf[0], vf[1]);
                mma_bf16(o[2 * dp + 1], pf[kk], vf[2], vf[3]);
            }
        }
    }
    cp_async_wait<0>();

    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    if (p.n_splits == 1) {
        __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(p.out);
        const float inv0 = 1.f / l0, inv1 = 1.f / l1;
        if (R0 < p.M) {
            uint32_t *dst = reinterpret_cast<uint32_t *>(
                out + (((long long)b * p.K + i0) * p.Hq + h * p.G + R0 % p.G) * HD);
#pragma unroll
            for (int j = 0; j < HD / 8; ++j) dst[j * 4 + tq] = pack_bf16(o[j][0] * inv0, o[j][1] * inv0);
        }
        if (R1 < p.M) {
            uint32_t *dst = reinterpret_cast<uint32_t *>(
                out + (((long long)b * p.K + i1) * p.Hq + h * p.G + R1 % p.G) * HD);
#pragma unroll
            for (int j = 0; j < HD / 8; ++j) dst[j * 4 + tq] = pack_bf16(o[j][2] * inv1, o[j][3] * inv1);
        }
    } else {
        const long long row_base = ((long long)unit * p.n_splits + split) * p.M;
        if (R0 < p.M) {
            float2 *dst = reinterpret_cast<float2 *>(p.part_o + (row_base + R0) * HD);
#pragma unroll
            for (int j = 0; j < HD / 8; ++j) dst[j * 4 + tq] = make_float2(o[j][0], o[j][1]);
            if (tq == 0) { p.part_ml[(row_base + R0) * 2] = m0; p.part_ml[(row_base + R0) * 2 + 1] = l0; }
        }
        if (R1 < p.M) {
            float2 *dst = reinterpret_cast<float2 *>(p.part_o + (row_base + R1) * HD);
#pragma unroll
            for (int j = 0; j < HD / 8; ++j) dst[j * 4 + tq] = make_float2(o[j][2], o[j][3]);
            if (tq == 0) { p.part_ml[(row_base + R1) * 2] = m1; p.part_ml[(row_base + R1) * 2 + 1] = l1; }
        }
    }
}

template <int HD, int NWARPS>
cudaError_t launch_one(const AttnParams &p, cudaStream_t st)
{
    constexpr int MT = NWARPS * 16;
    const int smem = STAGES * 2 * TN * HD * 2;
    auto kern = attend_mma_kernel<HD, NWARPS>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid(p.B * p.Hkv, p.n_splits, (p.M + MT - 1) / MT);
    kern<<<grid, NWARPS * 32, smem, st>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

int mma_tile_positions() { return TN; }

bool mma_path_supports(const AttnParams &p, int dtype)
{
    return dtype == ORTHRUS_BF16 && (p.d == 64 || p.d == 128) && p.K <= TN;
}

cudaError_t launch_attend_mma(const AttnParams &p, cudaStream_t st)
{
    const bool wide = p.M > 64;
    if (p.d == 128) return wide ? launch_one<128, 8>(p, st) : launch_one<128, 4>(p, st);
    return wide ? launch_one<64, 8>(p, st) : launch_one<64, 4>(p, st);
}

}  // namespace orthrus
