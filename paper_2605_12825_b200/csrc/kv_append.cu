// KV commit: copy the first n_commit[b] AR-view block rows of every KV head to the end
// of sequence b's prefix in the shared cache (16-byte vector copies), then grow the
// prefix length.  One CTA per sequence so the length update is ordered after the copy.
#include "common.cuh"

namespace orthrus {
namespace {

__global__ void __launch_bounds__(256) kv_append_kernel(
    uint4 *k_cache, uint4 *v_cache, int32_t *cache_len, const uint4 *k_blk, const uint4 *v_blk,
    const int32_t *n_commit, int K, int Hkv, int row_vecs, long long capacity, int update_len,
    int32_t *status)
{
    const int b = blockIdx.x;
    const int P = cache_len[b];
    const int n = n_commit[b];
    if (n < 0 || n > K || P < 0 || (long long)P + n > capacity) {
        if (status && threadIdx.x == 0) atomicOr(status, ORTHRUS_DEV_APPEND_OVERFLOW);
        return;
    }
    const int total = n * Hkv * row_vecs;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int c = e % row_vecs;
        const int h = (e / row_vecs) % Hkv;
        const int i = e / (row_vecs * Hkv);
        const long long src = (((long long)b * K + i) * Hkv + h) * row_vecs + c;
        const long long dst = (((long long)b * Hkv + h) * capacity + P + i) * row_vecs + c;
        k_cache[dst] = k_blk[src];
        v_cache[dst] = v_blk[src];
    }
    __syncthreads();
    if (update_len && threadIdx.x == 0) cache_len[b] = P + n;
}

// Several layers in one launch.  CTA (b, l, h) copies the accepted rows of KV head h of layer
// l of sequence b; the lengths are left alone, so every CTA sees the same P_b whatever the
// order they run in.
constexpr int kLayersPerLaunch = 64;
struct AppendBatch { AppendLayer layer[kLayersPerLaunch]; };

__global__ void __launch_bounds__(128) kv_append_layers_kernel(
    const __grid_constant__ AppendBatch batch, const int32_t *n_commit, int K, int Hkv, int row_vecs,
    long long capacity, int32_t *status)
{
    const int b = blockIdx.x, h = blockIdx.z;
    const AppendLayer &L = batch.layer[blockIdx.y];
    const int P = L.cache_len[b];
    const int n = n_commit[b];
    if (n < 0 || n > K || P < 0 || (long long)P + n > capacity) {
        if (status && threadIdx.x == 0 && h == 0) atomicOr(status, ORTHRUS_DEV_APPEND_OVERFLOW);
        return;
    }
    uint4 *kc = static_cast<uint4 *>(L.k_cache), *vc = static_cast<uint4 *>(L.v_cache);
    const uint4 *kb = static_cast<const uint4 *>(L.k_blk), *vb = static_cast<const uint4 *>(L.v_blk);
    // the n destination rows of this head are contiguous: [P, P + n) x row_vecs vectors
    const long long dst0 = (((long long)b * Hkv + h) * capacity + P) * row_vecs;
    const int total = n * row_vecs;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int i = e / row_vecs, c = e - i * row_vecs;
        const long long src = (((long long)b * K + i) * Hkv + h) * row_vecs + c;
        kc[dst0 + e] = kb[src];
        vc[dst0 + e] = vb[src];
    }
}

// Runs after the copies: grows every distinct length array once, under the same validity
// rule the copy applied.
struct LenBatch { int32_t *len[128]; };

__global__ void kv_append_bump_kernel(const __grid_constant__ LenBatch lens, int n_lens,
                                      const int32_t *n_commit, int B, int K, long long capacity)
{
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < B * n_lens; e += gridDim.x * blockDim.x) {
        const int b = e % B;
        int32_t *len = lens.len[e / B];
        const int P = len[b], n = n_commit[b];
        if (n >= 0 && n <= K && P >= 0 && (long long)P + n <= capacity) len[b] = P + n;
    }
}

}  // namespace

cudaError_t launch_kv_append_layers(const orthrus_layer_t &shape, const AppendLayer *layers, int n_layers,
                                    int32_t *const *len_arrays, int n_len_arrays,
                                    const int32_t *n_commit, int32_t *status, cudaStream_t st)
{
    const int es = shape.dtype == ORTHRUS_FP32 ? 4 : 2;
    const int row_vecs = shape.head_dim * es / 16;
    for (int l0 = 0; l0 < n_layers; l0 += kLayersPerLaunch) {
        AppendBatch batch;
        const int n = n_layers - l0 < kLayersPerLaunch ? n_layers - l0 : kLayersPerLaunch;
        for (int l = 0; l < n; ++l) batch.layer[l] = layers[l0 + l];
        for (int l = n; l < kLayersPerLaunch; ++l) batch.layer[l] = layers[l0];
        kv_append_layers_kernel<<<dim3(shape.batch, n, shape.n_kv_heads), 128, 0, st>>>(
            batch, n_commit, shape.block, shape.n_kv_heads, row_vecs, shape.capacity, status);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (n_len_arrays > 0) {
        LenBatch lb;
        for (int j = 0; j < 128; ++j) lb.len[j] = len_arrays[j < n_len_arrays ? j : 0];
        const int total = shape.batch * n_len_arrays;
        const int blocks = (total + 255) / 256 < 64 ? (total + 255) / 256 : 64;
        kv_append_bump_kernel<<<blocks, 256, 0, st>>>(lb, n_len_arrays, n_commit, shape.batch, shape.block,
                                                      shape.capacity);
        count_launch();
        return cudaGetLastError();
    }
    return cudaSuccess;
}

cudaError_t launch_kv_append(const orthrus_layer_t &L, const void *k_blk, const void *v_blk,
                             const int32_t *n_commit, int update_len, int32_t *status,
                             cudaStream_t st)
{
    const int es = L.dtype == ORTHRUS_FP32 ? 4 : 2;
    const int row_vecs = L.head_dim * es / 16;
    kv_append_kernel<<<L.batch, 256, 0, st>>>(
        static_cast<uint4 *>(L.k_cache), static_cast<uint4 *>(L.v_cache), L.cache_len,
        static_cast<const uint4 *>(k_blk), static_cast<const uint4 *>(v_blk), n_commit, L.block,
        L.n_kv_heads, row_vecs, L.capacity, update_len, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace orthrus
