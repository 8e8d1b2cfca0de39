// Greedy consensus: a streaming per-row argmax of the AR logits (16-byte loads, one
// (value, index) pair per thread, warp-shuffle then shared-memory reduction with the
// lowest index winning ties), followed by the sequential accept rule per sequence.
#include <mutex>
#include "common.cuh"

namespace orthrus {
namespace {

__device__ inline bool better(float v, int i, float bv, int bi) {
    return v > bv || (v == bv && i < bi);
}

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void unpack(const uint4 &u, float (&x)[8]) {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            x[2 * k] = __uint_as_float(w[k] << 16);
            x[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
        }
    }
    __device__ static float scalar(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
};
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ static void unpack(const uint4 &u, float (&x)[4]) {
        x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y);
        x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
    }
    __device__ static float scalar(const float *p) { return *p; }
};

// grid (n_seg, rows): CTA (seg, row) scans logits[row][seg*seg_len .. ) and writes one
// (value, index) pair.  Indices are visited in increasing order by every thread, so a
// strict '>' keeps the lowest index among equal values; reductions compare (value, index).
template <typename T>
__global__ void __launch_bounds__(256) argmax_partial_kernel(const T *logits, int V, int seg_len,
                                                             ArgPart *parts)
{
    constexpr int N = Vec<T>::N;
    const int row = blockIdx.y, seg = blockIdx.x;
    const int start = seg * seg_len;
    const int end = min(V, start + seg_len);
    const T *rowp = logits + (long long)row * V;
    float bv = -INFINITY;
    int bi = 0x7fffffff;

    if (start < end) {
        const uintptr_t addr = reinterpret_cast<uintptr_t>(rowp + start);
        int head = (int)(((16 - (addr & 15)) & 15) / sizeof(T));
        head = min(head, end - start);
        const int body0 = start + head;
        const int n_vec = (end - body0) / N;
        const int tail0 = body0 + n_vec * N;
        // ragged head and tail (at most N-1 elements each): one element per thread
        if ((int)threadIdx.x < head) {
            const int i = start + threadIdx.x;
            const float x = Vec<T>::scalar(rowp + i);
            if (x > bv) { bv = x; bi = i; }      // strict, like the body: -inf and NaN never replace the sentinel
        }
        const uint4 *vp = reinterpret_cast<const uint4 *>(rowp + body0);
        int v = threadIdx.x;
        for (; v + 3 * 256 < n_vec; v += 4 * 256) {
            uint4 u[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) u[k] = __ldg(vp + v + k * 256);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float x[N];
                Vec<T>::unpack(u[k], x);
                const int i0 = body0 + (v + k * 256) * N;
#pragma unroll
                for (int e = 0; e < N; ++e)
                    if (x[e] > bv) { bv = x[e]; bi = i0 + e; }
            }
        }
        for (; v < n_vec; v += 256) {
            float x[N];
            Vec<T>::unpack(__ldg(vp + v), x);
            const int i0 = body0 + v * N;
#pragma unroll
            for (int e = 0; e < N; ++e)
                if (x[e] > bv) { bv = x[e]; bi = i0 + e; }
        }
        if ((int)threadIdx.x < end - tail0) {
            const int i = tail0 + threadIdx.x;
            const float x = Vec<T>::scalar(rowp + i);
            if (x > bv) { bv = x; bi = i; }      // strict, like the body: -inf and NaN never replace the sentinel
        }
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    __shared__ float sv[8];
    __shared__ int si[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
    __syncthreads();
    if (warp == 0) {
        bv = lane < 8 ? sv[lane] : -INFINITY;
        bi = lane < 8 ? si[lane] : 0x7fffffff;
#pragma unroll
        for (int off = 4; off; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) parts[(long long)row * gridDim.x + seg] = ArgPart{bv, bi};
    }
}

// One CTA per sequence: thread i folds the segment partials of row i, then thread 0
// walks the block left to right: drafts are kept while they equal the greedy token,
// the first disagreeing position contributes the correction token, a fully agreeing
// block commits K tokens.
__global__ void consensus_finalize_kernel(const ArgPart *parts, int n_seg, const int32_t *draft,
                                          int K, int32_t *n_commit, int32_t *committed,
                                          int32_t *ar_argmax, int32_t *next_anchor)
{
    extern __shared__ int g[];
    const int b = blockIdx.x;
    for (int i = threadIdx.x; i < K; i += blockDim.x) {
        const ArgPart *pp = parts + ((long long)b * K + i) * n_seg;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int s = 0; s < n_seg; ++s)
            if (better(pp[s].v, pp[s].idx, bv, bi)) { bv = pp[s].v; bi = pp[s].idx; }
        if (bi == 0x7fffffff) bi = 0;            // a row with no comparable value
        g[i] = bi;
        ar_argmax[(long long)b * K + i] = bi;
    }
    __syncthreads();
    __shared__ int n_sh;
    if (threadIdx.x == 0) {
        int m = 0;
        while (m < K && draft[(long long)b * K + m] == g[m]) ++m;
        const int n = m + 1 < K ? m + 1 : K;
        n_sh = n;
        n_commit[b] = n;
        next_anchor[b] = g[n - 1];
    }
    __syncthreads();
    const int n = n_sh;
    for (int i = threadIdx.x; i < K; i += blockDim.x)
        committed[(long long)b * K + i] = i < n ? g[i] : -1;
}

// The same with many partials per row (one per vocabulary tile of the fused LM head): a warp
// per row folds them, lanes striding over the tiles.
__global__ void __launch_bounds__(256) consensus_finalize_wide_kernel(
        const ArgPart *parts, int n_seg, const int32_t *draft, int K, int32_t *n_commit,
        int32_t *committed, int32_t *ar_argmax, int32_t *next_anchor)
{
    extern __shared__ int g[];
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // launched early (programmatic dependent launch): the pairs are complete once the kernel
    // that writes them has finished
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int i = warp; i < K; i += 8) {
        const ArgPart *pp = parts + ((long long)b * K + i) * n_seg;
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int s = lane; s < n_seg; s += 32) {
            const ArgPart a = pp[s];
            if (better(a.v, a.idx, bv, bi)) { bv = a.v; bi = a.idx; }
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (bi == 0x7fffffff) bi = 0;            // a row with no comparable value
        if (lane == 0) { g[i] = bi; ar_argmax[(long long)b * K + i] = bi; }
    }
    __syncthreads();
    __shared__ int n_sh;
    if (threadIdx.x == 0) {
        int m = 0;
        while (m < K && draft[(long long)b * K + m] == g[m]) ++m;
        const int n = m + 1 < K ? m + 1 : K;
        n_sh = n;
        n_commit[b] = n;
        next_anchor[b] = g[n - 1];
    }
    __syncthreads();
    const int n = n_sh;
    for (int i = threadIdx.x; i < K; i += blockDim.x)
        committed[(long long)b * K + i] = i < n ? g[i] : -1;
}

}  // namespace

cudaError_t launch_consensus_finalize_wide(const ArgPart *parts, int n_seg, const int32_t *draft, int B,
                                           int K, int32_t *n_commit, int32_t *committed,
                                           int32_t *ar_argmax, int32_t *next_anchor, cudaStream_t st)
{
    // programmatic dependent launch: the CTAs are placed while the producer of `parts` is still
    // running and wait for it on the device
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(B);
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = K * sizeof(int);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, consensus_finalize_wide_kernel, parts, n_seg, draft, K, n_commit,
                                       committed, ar_argmax, next_anchor);
    count_launch();
    return e;
}

int consensus_segments(int B, int K, int V)
{
    const long long rows = (long long)B * K;
    long long want = (4LL * num_sms() + rows - 1) / rows;          // enough CTAs to fill the GPU
    const long long max_by_len = (V + 2047) / 2048;              // at least 2048 logits each
    if (want > max_by_len) want = max_by_len;
    if (want < 1) want = 1;
    return (int)want;
}

cudaError_t launch_consensus(const void *logits, int dtype, const int32_t *draft, int B, int K,
                             int V, int32_t *n_commit, int32_t *committed, int32_t *ar_argmax,
                             int32_t *next_anchor, void *partials, int n_seg, cudaStream_t st)
{
    int seg_len = (V + n_seg - 1) / n_seg;
    seg_len = (seg_len + 7) / 8 * 8;
    dim3 grid(n_seg, B * K);
    ArgPart *parts = static_cast<ArgPart *>(partials);
    if (dtype == ORTHRUS_FP32)
        argmax_partial_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float *>(logits), V,
                                                          seg_len, parts);
    else
        argmax_partial_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(
            static_cast<const __nv_bfloat16 *>(logits), V, seg_len, parts);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int threads = K <= 32 ? 32 : ((K + 31) / 32 * 32 > 256 ? 256 : (K + 31) / 32 * 32);
    consensus_finalize_kernel<<<B, threads, K * sizeof(int), st>>>(parts, n_seg, draft, K, n_commit,
                                                                    committed, ar_argmax, next_anchor);
    count_launch(2);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- consensus without a workspace
//
// Scratch for orthrus_consensus_accept_static: the per-segment (value, index) pairs of the
// streaming argmax.  It is part of the library image, so every GPU that loads the library
// holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = ORTHRUS_STATIC_CONSENSUS_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_consensus_scratch[kStaticScratchBytes];

// In host code `g_consensus_scratch` only names the symbol; the address a kernel can use is
// looked up once per device (with that device current) and remembered.
static cudaError_t static_scratch_address(void **out)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void *addr[kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_consensus_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        addr[dev] = ptr;
    }
    *out = addr[dev];
    return cudaSuccess;
}

size_t static_consensus_scratch_needed(int B, int K, int V)
{
    return (size_t)B * K * consensus_segments(B, K, V) * sizeof(ArgPart);
}

cudaError_t launch_consensus_static(const void *logits, int dtype, const int32_t *draft, int B, int K,
                                    int V, int32_t *n_commit, int32_t *committed, int32_t *ar_argmax,
                                    int32_t *next_anchor, cudaStream_t st)
{
    void *scratch = nullptr;
    cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return e;
    // every (row, segment) pair the second kernel reads is written by the first one in the
    // same call, so nothing in the array has to start at zero
    return launch_consensus(logits, dtype, draft, B, K, V, n_commit, committed, ar_argmax, next_anchor,
                            scratch, consensus_segments(B, K, V), st);
}

}  // namespace orthrus
