// Split-KV merge: for every query row, fold the per-split triples (running max m_s in
// the log2 domain, running sum l_s, unnormalised output O_s) into
//   m = max_s m_s,  l = sum_s 2^(m_s-m) l_s,  O = sum_s 2^(m_s-m) O_s / l.
// One warp per row; splits past the one holding the block keys were never written and
// are not read.
#include "common.cuh"

namespace orthrus {
namespace {

template <typename T>
__global__ void __launch_bounds__(256) combine_kernel(AttnParams p)
{
    const int unit = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = blockIdx.y * 8 + warp;
    if (R >= p.M) return;
    const int b = unit / p.Hkv, h = unit % p.Hkv;
    // the same clamp as the kernels that wrote the partial rows (they raised the status bit)
    int P = p.cache_len[b];
    const long long hi = max_served_len(p);
    P = P < 0 ? 0 : (P > hi ? (int)hi : P);
    const int ns = min(last_split(P, p.chunk) + 1, p.n_splits);
    const long long row0 = ((long long)unit * p.n_splits) * p.M + R;

    float mx = -INFINITY;
    for (int s = 0; s < ns; ++s) mx = fmaxf(mx, p.part_ml[(row0 + (long long)s * p.M) * 2]);
    float l = 0.f;
    for (int s = 0; s < ns; ++s) {
        const float *ml = p.part_ml + (row0 + (long long)s * p.M) * 2;
        l += exp2f(ml[0] - mx) * ml[1];
    }
    const float inv = 1.f / l;
    const int i = R / p.G, g = R % p.G;
    T *dst = static_cast<T *>(p.out) + (((long long)b * p.K + i) * p.Hq + h * p.G + g) * p.d;
    for (int c = lane; c < p.d; c += 32) {
        float acc = 0.f;
        for (int s = 0; s < ns; ++s) {
            const long long row = row0 + (long long)s * p.M;
            acc += exp2f(p.part_ml[row * 2] - mx) * p.part_o[row * p.d + c];
        }
        if constexpr (sizeof(T) == 4) dst[c] = acc * inv;
        else dst[c] = __float2bfloat16_rn(acc * inv);
    }
}

}  // namespace

cudaError_t launch_combine(const AttnParams &p, int dtype, cudaStream_t st)
{
    dim3 grid(p.B * p.Hkv, (p.M + 7) / 8);
    if (dtype == ORTHRUS_FP32) combine_kernel<float><<<grid, 256, 0, st>>>(p);
    else combine_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace orthrus
