// General SIMT split-KV block attention (both views), fp32 arithmetic throughout.
// Serves the fp32 test mode and every shape the tensor-core paths do not take.
// One CTA = (unit, split, 32-row tile); a warp owns 8 query rows, keeps their
// output accumulators in registers and runs the online softmax with warp shuffles:
// lane j scores key j of a 32-position tile, the tile max and sum are butterfly
// reductions, and the probabilities are broadcast lane by lane for the PV update.
#include "common.cuh"

namespace orthrus {
namespace {

constexpr int TN = 32;   // key positions per tile
constexpr int MT = 32;   // query rows per CTA
constexpr int RW = 8;    // query rows per warp

__device__ inline float to_f(float x) { return x; }
__device__ inline float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ inline void from_f(float *p, float x) { *p = x; }
__device__ inline void from_f(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }

template <typename T, int DPL>
__global__ void __launch_bounds__(128) attend_simt_kernel(AttnParams p)
{
    constexpr int D = DPL * 32;
    extern __shared__ float smem[];
    float *sK = smem;                    // [TN][D+1]
    float *sV = sK + TN * (D + 1);       // [TN][D]
    float *sQ = sV + TN * D;             // [MT][D]

    const int unit = blockIdx.x, split = blockIdx.y, rt = blockIdx.z;
    const int b = unit / p.Hkv, h = unit % p.Hkv;
    const int P = clamp_cache_len(p, b);
    const int ls = last_split(P, p.chunk);
    if (split > ls) return;
    const int pos0 = split * p.chunk;
    const int pos1 = min(P, pos0 + p.chunk);
    const int n_prefix_tiles = pos1 > pos0 ? (pos1 - pos0 + TN - 1) / TN : 0;
    const int n_blk_tiles = (split == ls) ? (p.K + TN - 1) / TN : 0;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *q = static_cast<const T *>(p.q);
    const long long cache_unit = (long long)(b / p.nb) * p.Hkv + h;      // whose cache this batch entry reads
    const T *kc = static_cast<const T *>(p.k_cache) + (cache_unit * p.capacity) * D;
    const T *vc = static_cast<const T *>(p.v_cache) + (cache_unit * p.capacity) * D;
    const T *kb = static_cast<const T *>(p.k_blk);
    const T *vb = static_cast<const T *>(p.v_blk);

    // stage this CTA's query rows
    for (int e = tid; e < MT * D; e += blockDim.x) {
        const int r = e / D, c = e % D;
        const int R = rt * MT + r;
        float v = 0.f;
        if (R < p.M) {
            const int i = R / p.G, g = R % p.G;
            v = to_f(q[(((long long)b * p.K + i) * p.Hq + h * p.G + g) * D + c]);
        }
        sQ[r * D + c] = v;
    }

    float o[RW][DPL], m[RW], l[RW];
#pragma unroll
    for (int rr = 0; rr < RW; ++rr) {
        m[rr] = -INFINITY; l[rr] = 0.f;
#pragma unroll
        for (int k = 0; k < DPL; ++k) o[rr][k] = 0.f;
    }

    for (int t = 0; t < n_prefix_tiles + n_blk_tiles; ++t) {
        const bool is_blk = t >= n_prefix_tiles;
        const int base = is_blk ? (t - n_prefix_tiles) * TN : pos0 + t * TN;
        const int nv = is_blk ? min(TN, p.K - base) : min(TN, pos1 - base);
        __syncthreads();
        for (int e = tid; e < TN * D; e += blockDim.x) {
            const int j = e / D, c = e % D;
            float kx = 0.f, vx = 0.f;
            if (j < nv) {
                if (is_blk && p.blk_in_cache) {
                    const long long off = (long long)(P + base + j) * D + c;
                    kx = to_f(kc[off]); vx = to_f(vc[off]);
                } else if (is_blk) {
                    const long long off = (((long long)b * p.K + base + j) * p.Hkv + h) * D + c;
                    kx = to_f(kb[off]); vx = to_f(vb[off]);
                } else {
                    const long long off = (long long)(base + j) * D + c;
                    kx = to_f(kc[off]); vx = to_f(vc[off]);
                }
            }
            sK[j * (D + 1) + c] = kx;
            sV[j * D + c] = vx;
        }
        __syncthreads();
#pragma unroll
        for (int rr = 0; rr < RW; ++rr) {
            const int r = warp * RW + rr;
            const int R = rt * MT + r;
            if (R >= p.M) continue;                  // warp-uniform
            const int i = R / p.G;
            float s = 0.f;
            const float *qr = sQ + r * D;
            const float *kr = sK + lane * (D + 1);
#pragma unroll 8
            for (int c = 0; c < D; ++c) s = fmaf(qr[c], kr[c], s);
            s *= p.scale_log2;
            bool visible = lane < nv;
            if (is_blk && p.causal) visible = visible && (base + lane <= i);
            if (!visible) s = -INFINITY;
            float tmax = s;
#pragma unroll
            for (int off = 16; off; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
            const float m_new = fmaxf(m[rr], tmax);
            if (m_new == -INFINITY) continue;        // nothing visible yet (warp-uniform)
            const float alpha = exp2f(m[rr] - m_new);
            const float pj = exp2f(s - m_new);
            float psum = pj;
#pragma unroll
            for (int off = 16; off; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
            l[rr] = l[rr] * alpha + psum;
            m[rr] = m_new;
#pragma unroll
            for (int k = 0; k < DPL; ++k) o[rr][k] *= alpha;
            for (int j = 0; j < TN; ++j) {
                const float pb = __shfl_sync(0xffffffffu, pj, j);
                const float *vr = sV + j * D + lane;
#pragma unroll
                for (int k = 0; k < DPL; ++k) o[rr][k] = fmaf(pb, vr[32 * k], o[rr][k]);
            }
        }
    }

    // epilogue: final output when there is a single split, else the partial triple
#pragma unroll
    for (int rr = 0; rr < RW; ++rr) {
        const int R = rt * MT + warp * RW + rr;
        if (R >= p.M) continue;
        if (p.n_splits == 1) {
            const int i = R / p.G, g = R % p.G;
            T *dst = static_cast<T *>(p.out) + (((long long)b * p.K + i) * p.Hq + h * p.G + g) * D;
            const float inv = 1.f / l[rr];
#pragma unroll
            for (int k = 0; k < DPL; ++k) from_f(dst + lane + 32 * k, o[rr][k] * inv);
        } else {
            const long long row = ((long long)unit * p.n_splits + split) * p.M + R;
            float *dst = p.part_o + row * D;
#pragma unroll
            for (int k = 0; k < DPL; ++k) dst[lane + 32 * k] = o[rr][k];
            if (lane == 0) { p.part_ml[row * 2] = m[rr]; p.part_ml[row * 2 + 1] = l[rr]; }
        }
    }
}

template <typename T, int DPL>
cudaError_t launch_one(const AttnParams &p, cudaStream_t st)
{
    constexpr int D = DPL * 32;
    const size_t smem = sizeof(float) * (TN * (D + 1) + TN * D + MT * D);
    auto kern = attend_simt_kernel<T, DPL>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid(p.B * p.Hkv, p.n_splits, (p.M + MT - 1) / MT);
    kern<<<grid, 128, smem, st>>>(p);
    count_launch();
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_d(const AttnParams &p, cudaStream_t st)
{
    switch (p.d) {
    case 32: return launch_one<T, 1>(p, st);
    case 64: return launch_one<T, 2>(p, st);
    case 128: return launch_one<T, 4>(p, st);
    case 256: return launch_one<T, 8>(p, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_attend_simt(const AttnParams &p, int dtype, cudaStream_t st)
{
    return dtype == ORTHRUS_FP32 ? launch_d<float>(p, st) : launch_d<__nv_bfloat16>(p, st);
}

}  // namespace orthrus
