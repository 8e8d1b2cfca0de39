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

}  // namespace

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
