// The write-then-truncate form of the KV commit and the step in front of it.
//   block_kv_write        every pass puts the K/V rows of its whole block behind the prefix of the
//                         shared cache (rows [P, P + K) of every KV head); the length is left alone,
//                         so those rows are dead until the consensus confirms some of them
//   commit_len            the consensus result only grows the length: len += n_commit
//   rope_block_kv_write   the same write fused with the rotary embedding of the block's queries and
//                         keys (row i of sequence b sits at position P_b + i), so that the projection
//                         outputs go straight to their places: rotated Q to the query tensor the
//                         attention reads, rotated K and V into the cache
// All are copies or a few flops per element: latency-bound launches of a few microseconds.
#include "common.cuh"

namespace orthrus {
namespace {

// grid (B, Hkv): the K destination rows of one KV head are contiguous
__global__ void __launch_bounds__(128) block_kv_write_kernel(
    uint4 *k_cache, uint4 *v_cache, const int32_t *cache_len, const uint4 *k_blk, const uint4 *v_blk,
    int K, int Hkv, int row_vecs, long long capacity, int32_t *status)
{
    const int b = blockIdx.x, h = blockIdx.y;
    const int P = cache_len[b];
    if (P < 0 || (long long)P + K > capacity) {
        if (status && threadIdx.x == 0 && h == 0) atomicOr(status, ORTHRUS_DEV_APPEND_OVERFLOW);
        return;
    }
    const long long dst0 = (((long long)b * Hkv + h) * capacity + P) * row_vecs;
    const int total = K * row_vecs;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int i = e / row_vecs, c = e - i * row_vecs;
        const long long src = (((long long)b * K + i) * Hkv + h) * row_vecs + c;
        k_cache[dst0 + e] = k_blk[src];
        v_cache[dst0 + e] = v_blk[src];
    }
}

__global__ void commit_len_kernel(int32_t *cache_len, const int32_t *n_commit, int B, int K,
                                  long long capacity, int32_t *status)
{
    for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x) {
        const int P = cache_len[b], n = n_commit[b];
        if (n >= 0 && n <= K && P >= 0 && (long long)P + n <= capacity) cache_len[b] = P + n;
        else if (status) atomicOr(status, ORTHRUS_DEV_APPEND_OVERFLOW);
    }
}

__device__ inline float load_f(const float *p) { return *p; }
__device__ inline float load_f(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
__device__ inline void store_f(float *p, double x) { *p = (float)x; }
__device__ inline void store_f(__nv_bfloat16 *p, double x) { *p = __float2bfloat16_rn((float)x); }

// grid (K, B): one CTA per block row.  The d/2 angles of the row are taken once, in double
// (pos * theta^(-2c/d) reaches tens of thousands of radians at long contexts, where a float
// angle would be off by more than the output's rounding), then every head is rotated with them.
template <typename T>
__global__ void __launch_bounds__(256) rope_block_kv_write_kernel(
    const T *q, const T *k_blk, const T *v_blk, T *q_out, T *k_cache, T *v_cache, const int32_t *cache_len,
    int K, int Hq, int Hkv, int d, long long capacity, double log2_theta, int32_t *status)
{
    extern __shared__ double cs[];             // [d/2] cosines, [d/2] sines
    const int i = blockIdx.x, b = blockIdx.y;
    const int half = d >> 1;
    const int P = cache_len[b];
    const bool room = P >= 0 && (long long)P + K <= capacity;
    if (!room && status && threadIdx.x == 0 && i == 0) atomicOr(status, ORTHRUS_DEV_APPEND_OVERFLOW);
    const int pos = (P < 0 ? 0 : P) + i;       // (a sequence without room is not written; its
                                               //  queries are still rotated, for a defined output)
    for (int c = threadIdx.x; c < half; c += blockDim.x) {
        const double ang = (double)pos * exp2(-2.0 * (double)c / (double)d * log2_theta);
        double s, co;
        sincos(ang, &s, &co);
        cs[c] = co; cs[half + c] = s;
    }
    __syncthreads();
    const long long row = (long long)b * K + i;
    // queries
    for (int e = threadIdx.x; e < Hq * half; e += blockDim.x) {
        const int hq = e / half, c = e - hq * half;
        const long long off = (row * Hq + hq) * d + c;
        const double x0 = load_f(q + off), x1 = load_f(q + off + half);
        store_f(q_out + off, x0 * cs[c] - x1 * cs[half + c]);
        store_f(q_out + off + half, x1 * cs[c] + x0 * cs[half + c]);
    }
    if (!room) return;
    // keys (rotated) and values (copied) into the cache row P + i of every KV head
    for (int e = threadIdx.x; e < Hkv * half; e += blockDim.x) {
        const int h = e / half, c = e - h * half;
        const long long src = (row * Hkv + h) * d + c;
        const long long dst = (((long long)b * Hkv + h) * capacity + P + i) * d + c;
        const double x0 = load_f(k_blk + src), x1 = load_f(k_blk + src + half);
        store_f(k_cache + dst, x0 * cs[c] - x1 * cs[half + c]);
        store_f(k_cache + dst + half, x1 * cs[c] + x0 * cs[half + c]);
        v_cache[dst] = v_blk[src];
        v_cache[dst + half] = v_blk[src + half];
    }
}

}  // namespace

cudaError_t launch_block_kv_write(const orthrus_layer_t &L, const void *k_blk, const void *v_blk,
                                  int32_t *status, cudaStream_t st)
{
    const int es = L.dtype == ORTHRUS_FP32 ? 4 : 2;
    const int row_vecs = L.head_dim * es / 16;
    block_kv_write_kernel<<<dim3(L.batch, L.n_kv_heads), 128, 0, st>>>(
        static_cast<uint4 *>(L.k_cache), static_cast<uint4 *>(L.v_cache), L.cache_len,
        static_cast<const uint4 *>(k_blk), static_cast<const uint4 *>(v_blk), L.block, L.n_kv_heads,
        row_vecs, L.capacity, status);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_commit_len(const orthrus_layer_t &L, const int32_t *n_commit, int32_t *status,
                              cudaStream_t st)
{
    const int blocks = (L.batch + 255) / 256 < 64 ? (L.batch + 255) / 256 : 64;
    commit_len_kernel<<<blocks, 256, 0, st>>>(L.cache_len, n_commit, L.batch, L.block, L.capacity, status);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_rope_block_kv_write(const orthrus_layer_t &L, const void *q, const void *k_blk,
                                       const void *v_blk, double theta, void *q_out, int32_t *status,
                                       cudaStream_t st)
{
    const dim3 grid(L.block, L.batch);
    const size_t smem = (size_t)L.head_dim * sizeof(double);
    const double log2_theta = log2(theta);
    if (L.dtype == ORTHRUS_FP32)
        rope_block_kv_write_kernel<float><<<grid, 256, smem, st>>>(
            static_cast<const float *>(q), static_cast<const float *>(k_blk), static_cast<const float *>(v_blk),
            static_cast<float *>(q_out), static_cast<float *>(L.k_cache), static_cast<float *>(L.v_cache),
            L.cache_len, L.block, L.n_q_heads, L.n_kv_heads, L.head_dim, L.capacity, log2_theta, status);
    else
        rope_block_kv_write_kernel<__nv_bfloat16><<<grid, 256, smem, st>>>(
            static_cast<const __nv_bfloat16 *>(q), static_cast<const __nv_bfloat16 *>(k_blk),
            static_cast<const __nv_bfloat16 *>(v_blk), static_cast<__nv_bfloat16 *>(q_out),
            static_cast<__nv_bfloat16 *>(L.k_cache), static_cast<__nv_bfloat16 *>(L.v_cache), L.cache_len,
            L.block, L.n_q_heads, L.n_kv_heads, L.head_dim, L.capacity, log2_theta, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace orthrus
