// Sampled consensus for temperature T > 0: the rejection-sampling rule of Section 3.3.
//
// With p = softmax(ar_logits / T) and q = softmax(diff_logits / T) per block position, the
// drafts are visited left to right; draft y_k is kept iff u_accept * q_k(y_k) <= p_k(y_k);
// the first position that fails gets a correction token drawn from max(0, p_k - q_k) by
// inverting its running sum with u_resample.  Four kernels, all streaming:
//   1. sample_stats      grid (segments, rows): one online pass over BOTH logit rows
//                        giving, per segment, an integer reference at or above the maximum
//                        and the sum of exponentials relative to it (16-byte loads, exp2 with the 1/T and
//                        log2(e) factors folded into one multiply);
//   2. sample_decide     one CTA per sequence: folds the segments (in order), evaluates
//                        the K accept tests, finds the first failure;
//   3. sample_residual   grid (segments, sequences): for the failing row only, the
//                        per-segment sums of max(0, p - q) and of p;
//   4. sample_pick       one CTA per sequence: walks the segment sums in order to the
//                        segment that contains u * total, then scans that segment.
// Exponentials are fp32; every sum is carried in double and taken in a fixed order, and
// references are integers so that rescaling is exact: the result is reproducible run to run
// and departs from an exact evaluation only by the rounding of the individual exponentials.
#include <cstdlib>
#include "common.cuh"

namespace orthrus {
namespace {

constexpr int kThreads = 256;
constexpr int kPickSegMax = 4096;       // elements one CTA scans in sample_pick: 256 threads x 16

__device__ inline float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T> struct Elem;
template <> struct Elem<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void unpack(const uint4 &u, float (&x)[8]) {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            x[2 * k] = __uint_as_float(w[k] << 16);
            x[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
        }
    }
    __device__ static float load(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
};
template <> struct Elem<float> {
    static constexpr int N = 4;
    __device__ static void unpack(const uint4 &u, float (&x)[4]) {
        x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y);
        x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
    }
    __device__ static float load(const float *p) { return *p; }
};

// Running (reference, sum of 2^(x - reference)).  The reference is an INTEGER at or above the
// largest value seen (in the log2 domain), so that moving it rescales the sum by an exact
// power of two: partial results of different threads and segments then combine without any
// rounding beyond that of the additions, which are carried in double.
struct RefSum { float m; double s; };
__device__ inline float pow2i(float k) {                 // 2^k for integer-valued k <= 0 (0 below the normal range)
    const int e = (int)k + 127;
    return e > 0 ? __int_as_float(e << 23) : 0.f;
}
__device__ inline RefSum combine(const RefSum &a, const RefSum &b) {
    if (b.m == -INFINITY) return a;
    if (a.m == -INFINITY) return b;
    const float M = fmaxf(a.m, b.m);
    return RefSum{M, a.s * (double)pow2i(a.m - M) + b.s * (double)pow2i(b.m - M)};
}
template <int N>
__device__ inline void absorb_vec(RefSum &a, const float (&x)[N], float c) {
    float y[N], mx = -INFINITY;
#pragma unroll
    for (int e = 0; e < N; ++e) { y[e] = x[e] * c; mx = fmaxf(mx, y[e]); }
    if (mx == -INFINITY) return;
    if (mx > a.m) {
        const float m_new = ceilf(mx);
        if (a.m > -INFINITY) a.s *= (double)pow2i(a.m - m_new);
        a.m = m_new;
    }
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < N; ++e) s += ex2f(y[e] - a.m);
    a.s += (double)s;
}
__device__ inline void absorb(RefSum &a, float x) {
    const float v[1] = {x};
    absorb_vec<1>(a, v, 1.f);
}
__device__ inline RefSum shfl_down(const RefSum &v, int off) {
    return RefSum{__shfl_down_sync(0xffffffffu, v.m, off), __shfl_down_sync(0xffffffffu, v.s, off)};
}
// block-wide fold of one RefSum per thread, in a fixed order; the result is valid in thread 0
__device__ inline RefSum block_fold(RefSum v, RefSum *sh) {
#pragma unroll
    for (int off = 16; off; off >>= 1) v = combine(v, shfl_down(v, off));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) sh[warp] = v;
    __syncthreads();
    if (warp == 0) {
        v = lane < kThreads / 32 ? sh[lane] : RefSum{-INFINITY, 0.0};
#pragma unroll
        for (int off = 4; off; off >>= 1) v = combine(v, shfl_down(v, off));
    }
    __syncthreads();
    return v;
}

// true when rows of V elements starting at `base` can be read with 16-byte loads
template <typename T> __host__ __device__ inline bool vector_ok(const void *base, int V) {
    return V % Elem<T>::N == 0 && (reinterpret_cast<uintptr_t>(base) & 15) == 0;
}

struct StatPart { float ma, md; double sa, sd; };       // per (row, segment)
struct Sum2 { double x, y; };                           // (residual mass, AR mass) of a segment

// 1. per (row, segment): (reference, sum) of both logit rows, in the log2 domain scaled by c = log2(e) / T.
// The launch covers block positions [k0, k1) of every sequence; with `fail` given, sequences
// whose first rejection is already known (fail[b] < K) are skipped: verification halts at the
// first rejected draft, so their later rows are never looked at.
template <typename T>
__global__ void __launch_bounds__(kThreads) sample_stats_kernel(const T *la, const T *ld, int V, int seg_len,
                                                                float c, StatPart *parts, int vec, int K, int k0,
                                                                int k1, const int *fail)
{
    constexpr int N = Elem<T>::N;
    __shared__ RefSum sh[kThreads / 32];
    const int seq = blockIdx.y / (k1 - k0), seg = blockIdx.x;
    if (fail != nullptr && fail[seq] < K) return;
    const int row = seq * K + k0 + blockIdx.y % (k1 - k0);
    const int start = seg * seg_len, end = min(V, start + seg_len);
    const T *ra = la + (long long)row * V, *rd = ld + (long long)row * V;
    RefSum a{-INFINITY, 0.0}, d{-INFINITY, 0.0};
    if (vec) {                                  // seg_len and V are multiples of N, rows are 16-byte aligned
        const uint4 *va = reinterpret_cast<const uint4 *>(ra + start), *vd = reinterpret_cast<const uint4 *>(rd + start);
        const int n_vec = (end - start) / N;
        for (int v = threadIdx.x; v < n_vec; v += 4 * kThreads) {     // up to 8 loads in flight per thread
            uint4 av[4], dv[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int w = min(v + k * kThreads, n_vec - 1);
                av[k] = __ldg(va + w); dv[k] = __ldg(vd + w);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (v + k * kThreads < n_vec) {
                    float x[N];
                    Elem<T>::unpack(av[k], x); absorb_vec<N>(a, x, c);
                    Elem<T>::unpack(dv[k], x); absorb_vec<N>(d, x, c);
                }
            }
        }
    } else {
        for (int i = start + threadIdx.x; i < end; i += kThreads) {
            absorb(a, Elem<T>::load(ra + i) * c);
            absorb(d, Elem<T>::load(rd + i) * c);
        }
    }
    a = block_fold(a, sh);
    d = block_fold(d, sh);
    if (threadIdx.x == 0) parts[(long long)row * gridDim.x + seg] = StatPart{a.m, d.m, a.s, d.s};
}

struct RowStat { float ma, md; double inv_za, inv_zd; int row; int pad; };   // of the first rejected row (1 / sums); row = -1: none

// 2. per sequence: fold the segments, take the accept tests, find the first failure
template <typename T>
// for block positions [k0, k1); fail[b] carries the outcome between the stages (K: no rejection
// so far).  A sequence's results are written by the stage that settles it: the one that finds
// its first rejection, or the last one.
__global__ void sample_decide_kernel(const T *la, const T *ld, const StatPart *parts, int n_seg, int K, int V,
                                     float c, const int32_t *draft, const float *u_accept,
                                     int32_t *n_commit, int32_t *committed, int32_t *next_anchor,
                                     RowStat *stat, int k0, int k1, int *fail)
{
    extern __shared__ StatPart folded[];        // [K]
    __shared__ int first_fail;
    const int b = blockIdx.x;
    if (k0 > 0 && fail[b] < K) return;          // settled by an earlier stage
    if (threadIdx.x == 0) first_fail = K;
    __syncthreads();
    for (int i = k0 + threadIdx.x; i < k1; i += blockDim.x) {
        const long long row = (long long)b * K + i;
        RefSum a{-INFINITY, 0.0}, d{-INFINITY, 0.0};
        for (int s = 0; s < n_seg; ++s) {
            const StatPart t = parts[row * n_seg + s];
            a = combine(a, RefSum{t.ma, t.sa});
            d = combine(d, RefSum{t.md, t.sd});
        }
        folded[i] = StatPart{a.m, d.m, a.s, d.s};
        int y = draft[row];
        y = min(max(y, 0), V - 1);              // an out-of-range draft id is clamped, not dereferenced
        const double py = (double)ex2f(Elem<T>::load(la + row * V + y) * c - a.m) / a.s;
        const double qy = (double)ex2f(Elem<T>::load(ld + row * V + y) * c - d.m) / d.s;
        if (!((double)u_accept[row] * qy <= py)) atomicMin(&first_fail, i);
    }
    __syncthreads();
    const int j = first_fail;                   // K: every draft so far kept
    if (threadIdx.x == 0) fail[b] = j;
    if (j >= K && k1 < K) return;               // still open: the next stage goes on
    const int n = j < K ? j + 1 : K;
    for (int i = threadIdx.x; i < K; i += blockDim.x)
        committed[(long long)b * K + i] = i < min(j, K) ? draft[(long long)b * K + i] : -1;
    if (threadIdx.x == 0) {
        n_commit[b] = n;
        RowStat st;
        st.row = j < K ? j : -1;
        const StatPart f = j < K ? folded[j] : StatPart{0.f, 0.f, 1.0, 1.0};
        st.ma = f.ma; st.inv_za = 1.0 / f.sa; st.md = f.md; st.inv_zd = 1.0 / f.sd;
        st.pad = 0;
        stat[b] = st;
        if (j >= K) next_anchor[b] = draft[(long long)b * K + K - 1];
    }
}

__device__ inline void residual_of(float xa, float xd, float c, const RowStat &st, double &r, double &p) {
    p = (double)ex2f(xa * c - st.ma) * st.inv_za;
    const double q = (double)ex2f(xd * c - st.md) * st.inv_zd;
    r = fmax(p - q, 0.0);
}

// 3. per (sequence, segment) of the rejected row: sum of max(0, p - q) and of p
template <typename T>
__global__ void __launch_bounds__(kThreads) sample_residual_kernel(const T *la, const T *ld, int K, int V,
                                                                   int seg_len, float c, const RowStat *stat,
                                                                   Sum2 *seg_sums)
{
    __shared__ Sum2 sh[kThreads];
    const int b = blockIdx.y, seg = blockIdx.x;
    const RowStat st = stat[b];
    if (st.row < 0) return;
    const long long row = (long long)b * K + st.row;
    const int start = seg * seg_len, end = min(V, start + seg_len);
    // every thread owns a contiguous run of the segment; the runs are added up in order
    const int per = (seg_len + kThreads - 1) / kThreads;
    const int i0 = start + threadIdx.x * per, i1 = min(end, i0 + per);
    double sr = 0.0, sp = 0.0;
    for (int i = i0; i < i1; ++i) {
        double r, p;
        residual_of(Elem<T>::load(la + row * V + i), Elem<T>::load(ld + row * V + i), c, st, r, p);
        sr += r; sp += p;
    }
    sh[threadIdx.x] = Sum2{sr, sp};
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, p = 0.0;
        for (int t = 0; t < kThreads; ++t) { a += sh[t].x; p += sh[t].y; }
        seg_sums[(long long)b * gridDim.x + seg] = Sum2{a, p};
    }
}

// 4. per sequence: invert the running sum of the residual (of p itself if the residual is empty)
template <typename T>
__global__ void __launch_bounds__(kThreads) sample_pick_kernel(const T *la, const T *ld, int K, int V, int seg_len,
                                                               int n_seg, float c, const RowStat *stat,
                                                               const Sum2 *seg_sums, const float *u_resample,
                                                               int32_t *committed, int32_t *next_anchor)
{
    __shared__ double run_sh[kThreads];
    __shared__ int seg_sh, use_p_sh;
    __shared__ double before_sh, target_sh;
    const int b = blockIdx.x;
    const RowStat st = stat[b];
    if (st.row < 0) return;
    const long long row = (long long)b * K + st.row;
    if (threadIdx.x == 0) {
        double tot_r = 0.0, tot_p = 0.0;
        for (int s = 0; s < n_seg; ++s) { tot_r += seg_sums[(long long)b * n_seg + s].x; tot_p += seg_sums[(long long)b * n_seg + s].y; }
        const int use_p = !(tot_r > 0.0);
        const double total = use_p ? tot_p : tot_r;
        const double target = (double)u_resample[row] * total;
        // the first segment whose running sum exceeds the target (the last non-empty one otherwise)
        double run = 0.0, before = 0.0;
        int pick = -1, last = 0;
        for (int s = 0; s < n_seg; ++s) {
            const Sum2 t = seg_sums[(long long)b * n_seg + s];
            const double v = use_p ? t.y : t.x;
            if (v > 0.0) {
                last = s;
                if (pick < 0 && run + v > target) { pick = s; before = run; }
                run += v;
            }
        }
        if (pick < 0) { pick = last; before = run; }      // rounding: the target is at or past the total
        seg_sh = pick; use_p_sh = use_p; before_sh = before; target_sh = target;
    }
    __syncthreads();
    const int seg = seg_sh, use_p = use_p_sh;
    const double before = before_sh, target = target_sh;
    const int start = seg * seg_len, end = min(V, start + seg_len);
    const int per = (seg_len + kThreads - 1) / kThreads;
    const int i0 = start + threadIdx.x * per, i1 = min(end, i0 + per);
    double mine = 0.0;
    for (int i = i0; i < i1; ++i) {
        double r, p;
        residual_of(Elem<T>::load(la + row * V + i), Elem<T>::load(ld + row * V + i), c, st, r, p);
        mine += use_p ? p : r;
    }
    run_sh[threadIdx.x] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        // walk the threads' runs in order, then the elements of the run that contains the target
        double run = before;
        int t_pick = -1, t_last = -1;
        for (int t = 0; t < kThreads; ++t) {
            if (run_sh[t] > 0.0) {
                t_last = t;
                if (run + run_sh[t] > target) { t_pick = t; break; }
                run += run_sh[t];
            }
        }
        const bool past_end = t_pick < 0;                // rounding again: take the last positive element
        if (past_end) t_pick = t_last;
        int z = -1, z_last = -1;
        if (t_pick >= 0) {
            const int j0 = start + t_pick * per, j1 = min(end, j0 + per);
            double acc = run;
            for (int i = j0; i < j1; ++i) {
                double r, p;
                residual_of(Elem<T>::load(la + row * V + i), Elem<T>::load(ld + row * V + i), c, st, r, p);
                const double v = use_p ? p : r;
                if (v > 0.0) {
                    z_last = i;
                    if (!past_end) { acc += v; if (acc > target) { z = i; break; } }
                }
            }
        }
        if (z < 0) z = z_last >= 0 ? z_last : 0;
        committed[(long long)b * K + st.row] = z;
        next_anchor[b] = z;
    }
}

}  // namespace

int sample_stat_segments(int B, int K, int V)
{
    const long long rows = (long long)B * K;
    long long want = (8LL * num_sms() + rows - 1) / rows;           // more CTAs than fit at once, for balance
    const long long max_by_len = (V + 4095) / 4096;
    if (want > max_by_len) want = max_by_len;
    return (int)(want < 1 ? 1 : want);
}

int sample_pick_segments(int V) { return (V + kPickSegMax - 1) / kPickSegMax; }

size_t sample_workspace_bytes(int B, int K, int V)
{
    return (size_t)B * K * sample_stat_segments(B, K, V) * sizeof(StatPart) + (size_t)B * sizeof(RowStat) +
           (size_t)B * sample_pick_segments(V) * sizeof(Sum2) + (size_t)B * sizeof(int);
}

// Block positions verified by the first statistics pass.  Verification halts at the first
// rejected draft, so rows behind it need not be looked at: when the two logit tensors are
// large enough for the pass to be bound by throughput, the first pass covers a quarter of the
// block (at least 4 positions) and a second pass the rest, for the sequences still open only.
// More stages were measured slower (each costs two dependent launches), and small problems
// are bound by launch latency and take one pass.  ORTHRUS_SAMPLE_FIRST_STAGE overrides.
int sample_first_stage(int B, int K, int V)
{
    const long long bytes = 2LL * B * K * V * 2;
    static const int forced = [] { const char *e = getenv("ORTHRUS_SAMPLE_FIRST_STAGE"); return e ? atoi(e) : 0; }();
    if (forced > 0) return forced < K ? forced : K;
    if (K <= 4 || bytes < (64LL << 20)) return K;
    const int k1 = (K + 3) / 4;
    return k1 < 4 ? 4 : k1;
}

template <typename T>
static cudaError_t launch_sample_t(const void *ar_logits, const void *diff_logits, const int32_t *draft,
                                   const float *u_accept, const float *u_resample, float temperature, int B, int K,
                                   int V, int32_t *n_commit, int32_t *committed, int32_t *next_anchor,
                                   unsigned char *ws, cudaStream_t st)
{
    constexpr int N = Elem<T>::N;
    const T *la = static_cast<const T *>(ar_logits), *ld = static_cast<const T *>(diff_logits);
    const float c = 1.4426950408889634f / temperature;
    const int n_seg = sample_stat_segments(B, K, V);
    int seg_len = (V + n_seg - 1) / n_seg;
    seg_len = (seg_len + N - 1) / N * N;
    const int vec = vector_ok<T>(la, V) && vector_ok<T>(ld, V);
    StatPart *parts = reinterpret_cast<StatPart *>(ws);
    RowStat *stat = reinterpret_cast<RowStat *>(ws + (size_t)B * K * n_seg * sizeof(StatPart));
    const int n_seg2 = sample_pick_segments(V);
    Sum2 *seg_sums = reinterpret_cast<Sum2 *>(reinterpret_cast<unsigned char *>(stat) + (size_t)B * sizeof(RowStat));
    int *fail = reinterpret_cast<int *>(reinterpret_cast<unsigned char *>(seg_sums) + (size_t)B * n_seg2 * sizeof(Sum2));
    const int threads = K <= 32 ? 32 : ((K + 31) / 32 * 32 > 256 ? 256 : (K + 31) / 32 * 32);
    const int k_first = sample_first_stage(B, K, V);
    cudaError_t e = cudaSuccess;
    int launches = 2;
    for (int k0 = 0, k1 = k_first; k0 < K; k0 = k1, k1 = K) {
        sample_stats_kernel<T><<<dim3(n_seg, B * (k1 - k0)), kThreads, 0, st>>>(la, ld, V, seg_len, c, parts, vec, K,
                                                                               k0, k1, k0 > 0 ? fail : nullptr);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        sample_decide_kernel<T><<<B, threads, K * sizeof(StatPart), st>>>(la, ld, parts, n_seg, K, V, c, draft,
                                                                      u_accept, n_commit, committed, next_anchor,
                                                                      stat, k0, k1, fail);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        launches += 2;
    }
    sample_residual_kernel<T><<<dim3(n_seg2, B), kThreads, 0, st>>>(la, ld, K, V, kPickSegMax, c, stat, seg_sums);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    sample_pick_kernel<T><<<B, kThreads, 0, st>>>(la, ld, K, V, kPickSegMax, n_seg2, c, stat, seg_sums, u_resample,
                                                  committed, next_anchor);
    count_launch(launches);
    return cudaGetLastError();
}

cudaError_t launch_consensus_sample(const void *ar_logits, const void *diff_logits, int dtype, const int32_t *draft,
                                    const float *u_accept, const float *u_resample, float temperature, int B, int K,
                                    int V, int32_t *n_commit, int32_t *committed, int32_t *next_anchor, void *ws,
                                    cudaStream_t st)
{
    unsigned char *w = static_cast<unsigned char *>(ws);
    if (dtype == ORTHRUS_FP32)
        return launch_sample_t<float>(ar_logits, diff_logits, draft, u_accept, u_resample, temperature, B, K, V,
                                      n_commit, committed, next_anchor, w, st);
    return launch_sample_t<__nv_bfloat16>(ar_logits, diff_logits, draft, u_accept, u_resample, temperature, B, K, V,
                                          n_commit, committed, next_anchor, w, st);
}

}  // namespace orthrus
