/*
 * CPU oracle for the Orthrus generation-step hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, fp64 statement of
 * what the path computes, written from the paper.  It shares no code with the
 * CUDA library and must never be called from the product path; only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Every function takes HOST pointers.  Tensors may be given as bf16 (raw
 * 16-bit patterns), fp32 or fp64; each element is widened exactly to double
 * before any arithmetic, and all sums are carried in double.
 *
 * Layouts (row-major):
 *   q, out        [B][K][Hq][d]
 *   k_blk, v_blk  [B][K][Hkv][d]
 *   k_cache, v_cache [B][Hkv][capacity][d]
 *   cache_len     [B] int32   (P_b = number of valid prefix positions)
 *   logits        [B][K][V];  draft, committed, ar_argmax [B][K] int32
 *
 * Parity status: every function here is pinned by tests/test_oracle_pins.py and
 * tests/test_oracle_sampling_pins.py (brute-force mask-matrix softmax, closed forms,
 * K=1 reduction, permutation invariances, sequential greedy decoding of a toy
 * model, byte-level append checks; for the sampled consensus: the committed token
 * follows the AR distribution, acceptance rate 1 - total variation, reduction to
 * the greedy rule at low temperature, library inverse-CDF on the degenerate
 * cases) and tests/test_oracle_lm_head_pins.py (planted maxima, exact-integer
 * logits against the logits-based rule, the library matrix product, ties, a
 * transposition trap), tests/test_oracle_truncate_rope_pins.py (the in-cache block
 * against the library attention over one concatenated key sequence with an explicit
 * mask; write + length bump against the append, byte for byte; the rotation against
 * the transformers library's rotary embedding, its norm and relative-position
 * properties) and tests/test_oracle_multiblock_pins.py.  Nothing is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_BF16 = 0, ORACLE_FP32 = 1, ORACLE_FP64 = 2 };
enum { ORACLE_VIEW_DIFFUSION = 0, ORACLE_VIEW_AR = 1 };

typedef struct {
    int32_t batch, block, n_q_heads, n_kv_heads, head_dim;
    int32_t dtype;          /* element type of q, k_blk, v_blk, k_cache, v_cache */
    int64_t capacity;
    const void *q, *k_blk, *v_blk, *k_cache, *v_cache;
    const int32_t *cache_len;
    double scale;           /* <= 0 selects 1/sqrt(head_dim), the scale of Eq. 4 */
} oracle_attn_t;

static double load_elem(const void *p, int dtype, int64_t idx)
{
    if (dtype == ORACLE_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t *)p)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    if (dtype == ORACLE_FP32)
        return (double)((const float *)p)[idx];
    return ((const double *)p)[idx];
}

static size_t elem_size(int dtype)
{
    return dtype == ORACLE_BF16 ? 2 : dtype == ORACLE_FP32 ? 4 : 8;
}

/*
 * One query row of the dual-view attention.
 *
 * Diffusion view (Eq. 4): the query of block position i, head hq, takes a softmax
 * over the concatenation [K_AR || K_diff] = all P_b prefix rows of the shared
 * cache followed by all K rows of the diffusion block (bidirectional inside the
 * block, Section 3.2 rule (ii)), scaled by 1/sqrt(d_head), and averages
 * [V_AR || V_diff] with those weights.
 *
 * AR view (Section 3.3, "Intra-Model Distribution Matching"): the block is fed
 * through the ordinary causal model, so query i sees the whole prefix and block
 * rows 0..i only.
 *
 * Grouped-query mapping: query head hq reads KV head hq / (Hq / Hkv).
 *
 * out_row: d doubles.  w_row: optional, P_b + K doubles (weights of masked block
 * keys are written as exact zeros).  Returns 0, or -1 on allocation failure.
 */
static int attend_row(const oracle_attn_t *a, int view, int b, int hq, int i,
                      double *out_row, double *w_row)
{
    const int d = a->head_dim, K = a->block, Hq = a->n_q_heads, Hkv = a->n_kv_heads;
    const int G = Hq / Hkv;
    const int h = hq / G;
    const int64_t P = a->cache_len[b];
    const int n_blk = (view == ORACLE_VIEW_DIFFUSION) ? K : i + 1;
    const int64_t n = P + n_blk;
    const double scale = a->scale > 0.0 ? a->scale : 1.0 / sqrt((double)d);
    /* k_blk == NULL: the block's K/V rows are the cache rows [P_b, P_b + K) themselves
     * (the pass wrote them there before attending; last paragraph of Section 3.3) */
    const int in_cache = a->k_blk == NULL;

    double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    double *qv = (double *)malloc(sizeof(double) * (size_t)d);
    if (!s || !qv) { free(s); free(qv); return -1; }

    const int64_t q_off = (((int64_t)b * K + i) * Hq + hq) * d;
    for (int c = 0; c < d; ++c) qv[c] = load_elem(a->q, a->dtype, q_off + c);

    /* scores against the prefix cache rows */
    const int64_t cache_base = ((int64_t)b * Hkv + h) * a->capacity * d;
    for (int64_t j = 0; j < P; ++j) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
            acc += qv[c] * load_elem(a->k_cache, a->dtype, cache_base + j * d + c);
        s[j] = acc * scale;
    }
    /* scores against the visible block rows */
    for (int ip = 0; ip < n_blk; ++ip) {
        const int64_t off = in_cache ? cache_base + (P + ip) * d : (((int64_t)b * K + ip) * Hkv + h) * d;
        const void *src = in_cache ? a->k_cache : a->k_blk;
        double acc = 0.0;
        for (int c = 0; c < d; ++c)
            acc += qv[c] * load_elem(src, a->dtype, off + c);
        s[P + ip] = acc * scale;
    }

    /* softmax */
    double mx = -INFINITY;
    for (int64_t j = 0; j < n; ++j) if (s[j] > mx) mx = s[j];
    double den = 0.0;
    for (int64_t j = 0; j < n; ++j) { s[j] = exp(s[j] - mx); den += s[j]; }
    for (int64_t j = 0; j < n; ++j) s[j] /= den;

    /* weighted average of the value rows */
    for (int c = 0; c < d; ++c) out_row[c] = 0.0;
    for (int64_t j = 0; j < P; ++j)
        for (int c = 0; c < d; ++c)
            out_row[c] += s[j] * load_elem(a->v_cache, a->dtype, cache_base + j * d + c);
    for (int ip = 0; ip < n_blk; ++ip) {
        const int64_t off = in_cache ? cache_base + (P + ip) * d : (((int64_t)b * K + ip) * Hkv + h) * d;
        const void *src = in_cache ? a->v_cache : a->v_blk;
        for (int c = 0; c < d; ++c)
            out_row[c] += s[P + ip] * load_elem(src, a->dtype, off + c);
    }

    if (w_row) {
        for (int64_t j = 0; j < n; ++j) w_row[j] = s[j];
        for (int64_t j = n; j < P + K; ++j) w_row[j] = 0.0;
    }
    free(s);
    free(qv);
    return 0;
}

/*
 * Whole-tensor dual-view attention: out [B][K][Hq][d] doubles.
 * weights (optional): [B][K][Hq][w_stride] doubles with w_stride >= max_b P_b + K;
 * row (b,i,hq) holds its P_b + K weights followed by untouched slack.
 */
int oracle_block_attend(const oracle_attn_t *a, int view, double *out,
                        double *weights, int64_t w_stride)
{
    const int B = a->batch, K = a->block, Hq = a->n_q_heads, d = a->head_dim;
    if (a->n_kv_heads <= 0 || Hq % a->n_kv_heads != 0) return -2;
    int rc = 0;
    const int64_t rows = (int64_t)B * K * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
        const int hq = (int)(r % Hq);
        const int i = (int)((r / Hq) % K);
        const int b = (int)(r / ((int64_t)Hq * K));
        double *w = weights ? weights + r * w_stride : NULL;
        if (attend_row(a, view, b, hq, i, out + r * d, w) != 0) {
#pragma omp atomic write
            rc = -1;
        }
    }
    return rc;
}

/*
 * Sampled rows of the same attention, for sizes at which the whole tensor would
 * take too long: rows[3*s + {0,1,2}] = (b, i, hq); out [n_rows][d] doubles.
 */
int oracle_block_attend_rows(const oracle_attn_t *a, int view, const int32_t *rows,
                             int64_t n_rows, double *out)
{
    const int d = a->head_dim;
    if (a->n_kv_heads <= 0 || a->n_q_heads % a->n_kv_heads != 0) return -2;
    int rc = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t s = 0; s < n_rows; ++s) {
        if (attend_row(a, view, rows[3 * s], rows[3 * s + 2], rows[3 * s + 1],
                       out + s * d, NULL) != 0) {
#pragma omp atomic write
            rc = -1;
        }
    }
    return rc;
}

/*
 * Multi-block diffusion-view attention, the training-time mask of Eq. 6 (Section 3.2).
 *
 * One clean sequence of L = cache_len[s] positions lives in the cache (the frozen AR
 * view's K/V); NB blocks of K diffusion rows each are concatenated behind it, block j
 * anchored at position a_j = anchors[s][j].  With q the row index among the NB*K
 * diffusion rows and k the key index among the L + NB*K keys, Eq. 6 permits
 *     k < L  and  k <= a_j - 1               (clean context before the block's anchor), or
 *     k >= L and  floor(q / K) == floor((k - L) / K)   (the rows of the same block).
 * The predicate is evaluated for every (q, k) exactly as printed; permitted keys enter
 * one softmax with scale 1/sqrt(d).  q: [S][NB][K][Hq][d]; k_blk, v_blk: [S][NB][K][Hkv][d]
 * (a->block = K, a->batch = S); out: [S][NB][K][Hq][d] doubles.
 */
int oracle_multi_block_attend(const oracle_attn_t *a, int32_t NB, const int32_t *anchors, double *out)
{
    const int S = a->batch, K = a->block, Hq = a->n_q_heads, Hkv = a->n_kv_heads, d = a->head_dim;
    if (Hkv <= 0 || Hq % Hkv != 0 || NB <= 0) return -2;
    const int G = Hq / Hkv;
    const double scale = a->scale > 0.0 ? a->scale : 1.0 / sqrt((double)d);
    int rc = 0;
    const int64_t rows = (int64_t)S * NB * K * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
        const int hq = (int)(r % Hq);
        const int64_t q = (r / Hq) % ((int64_t)NB * K);      /* row among the diffusion rows */
        const int s = (int)(r / ((int64_t)Hq * NB * K));
        const int h = hq / G;
        const int64_t L = a->cache_len[s];
        const int64_t n_keys = L + (int64_t)NB * K;
        const int64_t anchor = anchors[(int64_t)s * NB + q / K];
        double *w = (double *)malloc(sizeof(double) * (size_t)(n_keys > 0 ? n_keys : 1));
        if (!w) {
#pragma omp atomic write
            rc = -1;
            continue;
        }
        const int64_t q_off = r * d;
        const int64_t cache_base = ((int64_t)s * Hkv + h) * a->capacity * d;
        double mx = -INFINITY;
        for (int64_t k = 0; k < n_keys; ++k) {
            const int allowed = (k < L && k <= anchor - 1) || (k >= L && q / K == (k - L) / K);
            if (!allowed) { w[k] = -INFINITY; continue; }
            double acc = 0.0;
            if (k < L) {
                for (int c = 0; c < d; ++c)
                    acc += load_elem(a->q, a->dtype, q_off + c) *
                           load_elem(a->k_cache, a->dtype, cache_base + k * d + c);
            } else {
                const int64_t off = ((((int64_t)s * NB * K) + (k - L)) * Hkv + h) * d;
                for (int c = 0; c < d; ++c)
                    acc += load_elem(a->q, a->dtype, q_off + c) * load_elem(a->k_blk, a->dtype, off + c);
            }
            w[k] = acc * scale;
            if (w[k] > mx) mx = w[k];
        }
        double den = 0.0;
        for (int64_t k = 0; k < n_keys; ++k) { w[k] = exp(w[k] - mx); den += w[k]; }   /* exp(-inf) = 0 */
        double *o = out + r * d;
        for (int c = 0; c < d; ++c) o[c] = 0.0;
        for (int64_t k = 0; k < n_keys; ++k) {
            if (w[k] == 0.0) continue;
            const double p = w[k] / den;
            if (k < L) {
                for (int c = 0; c < d; ++c)
                    o[c] += p * load_elem(a->v_cache, a->dtype, cache_base + k * d + c);
            } else {
                const int64_t off = ((((int64_t)s * NB * K) + (k - L)) * Hkv + h) * d;
                for (int c = 0; c < d; ++c) o[c] += p * load_elem(a->v_blk, a->dtype, off + c);
            }
        }
        free(w);
    }
    return rc;
}

/*
 * Greedy consensus (Eq. 8 and the halt/commit rule of Section 3.3).
 *
 * Row i of the AR logits is conditioned on the anchor and drafts 0..i-1; its
 * greedy token is g_i = argmax_v logits[b][i][v] (softmax is monotone, so the
 * argmax of p_AR is the argmax of the logits; the smallest id wins ties; a NaN
 * never wins).  Draft i is retained iff draft[i] == g_i.  Verification stops at
 * the first mismatch; with m retained drafts the cycle commits those m tokens
 * plus, when m < K, the correction token g_m.  When all K drafts agree there is
 * no further verified row, so K tokens are committed.  Hence
 *     n = min(m + 1, K),  committed = g_0..g_{n-1},  next anchor = g_{n-1},
 * and 1 <= n <= K (at least one token per cycle, Section 4.2).
 *
 * Outputs: n_commit [B], committed [B][K] (-1 beyond n), ar_argmax [B][K],
 * next_anchor [B].
 */
int oracle_consensus_accept(const void *logits, int dtype, const int32_t *draft,
                            int32_t B, int32_t K, int32_t V,
                            int32_t *n_commit, int32_t *committed,
                            int32_t *ar_argmax, int32_t *next_anchor)
{
    if (B < 0 || K <= 0 || V <= 0) return -2;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < (int64_t)B * K; ++r) {
        double best = -INFINITY;
        int32_t arg = 0;
        for (int32_t v = 0; v < V; ++v) {
            const double x = load_elem(logits, dtype, r * V + v);
            if (x > best) { best = x; arg = v; }
        }
        ar_argmax[r] = arg;
    }
    for (int32_t b = 0; b < B; ++b) {
        const int32_t *g = ar_argmax + (int64_t)b * K;
        const int32_t *y = draft + (int64_t)b * K;
        int32_t m = 0;
        while (m < K && y[m] == g[m]) ++m;
        const int32_t n = (m + 1 < K) ? m + 1 : K;
        n_commit[b] = n;
        for (int32_t i = 0; i < K; ++i)
            committed[(int64_t)b * K + i] = (i < n) ? g[i] : -1;
        next_anchor[b] = g[n - 1];
    }
    return 0;
}

/*
 * Greedy tokens straight from the last hidden states (the step that produces the
 * logits Eq. 8 takes the argmax of: logits[r][v] = sum_c hidden[r][c] * lm_head[v][c],
 * the shared LM head of Section 3.1 applied to row r of the AR view's final hidden
 * states).  Every product and sum is carried in double; nothing is rounded to a
 * storage type before the comparison.
 *
 * rows == NULL: all n_rows rows 0..n_rows-1; otherwise rows[j] names the row of
 * `hidden` that output j is computed from (for sampled checks at full size).
 * Outputs per listed row: arg (smallest id attaining the maximum; a NaN never
 * wins) and top2 = (largest logit, largest logit among the other ids; -inf when
 * V == 1), from which a caller judges how close the decision was.
 */
int oracle_lm_head_argmax(const void *hidden, const void *lm_head, int dtype,
                          const int32_t *rows, int32_t n_rows, int32_t V, int32_t H,
                          int32_t *arg, double *top2)
{
    if (n_rows < 0 || V <= 0 || H <= 0) return -2;
    int rc = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t j = 0; j < n_rows; ++j) {
        const int64_t r = rows ? rows[j] : j;
        double *x = (double *)malloc((size_t)H * sizeof(double));
        if (!x) {
#pragma omp critical
            rc = -4;
            continue;
        }
        for (int32_t c = 0; c < H; ++c) x[c] = load_elem(hidden, dtype, r * H + c);
        double best = -INFINITY, second = -INFINITY;
        int32_t a = 0;
        for (int32_t v = 0; v < V; ++v) {
            double s = 0.0;
            for (int32_t c = 0; c < H; ++c) s += x[c] * load_elem(lm_head, dtype, (int64_t)v * H + c);
            if (s > best) { second = best; best = s; a = v; }
            else if (s > second) second = s;
        }
        arg[j] = a;
        top2[2 * j] = best;
        top2[2 * j + 1] = second;
        free(x);
    }
    return rc;
}

/*
 * The accept rule of oracle_consensus_accept applied to given greedy tokens g [B][K]
 * (Eq. 8 and the halt/commit rule of Section 3.3): n = min(m + 1, K) with m the number
 * of leading drafts equal to g, committed = g_0..g_{n-1} (-1 beyond), next anchor g_{n-1}.
 */
int oracle_accept_rule(const int32_t *g_all, const int32_t *draft, int32_t B, int32_t K,
                       int32_t *n_commit, int32_t *committed, int32_t *next_anchor)
{
    if (B < 0 || K <= 0) return -2;
    for (int32_t b = 0; b < B; ++b) {
        const int32_t *g = g_all + (int64_t)b * K;
        const int32_t *y = draft + (int64_t)b * K;
        int32_t m = 0;
        while (m < K && y[m] == g[m]) ++m;
        const int32_t n = (m + 1 < K) ? m + 1 : K;
        n_commit[b] = n;
        for (int32_t i = 0; i < K; ++i)
            committed[(int64_t)b * K + i] = (i < n) ? g[i] : -1;
        next_anchor[b] = g[n - 1];
    }
    return 0;
}

/*
 * Sampled consensus for temperature T > 0 (Section 3.3: "exact rejection sampling",
 * the speculative-sampling rule of the work it cites, which keeps the committed
 * tokens distributed exactly as the AR view would have sampled them).
 *
 * With p_k = softmax(ar_logits[b][k] / T) and q_k = softmax(diff_logits[b][k] / T),
 * the drafts are visited left to right.  Draft y_k (drawn from q_k by the caller) is
 * kept iff  u_accept[b][k] * q_k(y_k) <= p_k(y_k),  i.e. with probability
 * min(1, p_k(y_k) / q_k(y_k)).  At the first k that fails, verification halts and the
 * correction token is drawn from the residual distribution
 *     r(v) = max(0, p_k(v) - q_k(v)) / sum_w max(0, p_k(w) - q_k(w))
 * by inverting its running sum with u_resample[b][k]: the smallest v whose running
 * sum exceeds u * total.  (If the residual is identically zero, which exact
 * arithmetic allows only when nothing can be rejected, p_k itself is inverted.)
 * n = kept drafts + 1 correction token, or K when every draft is kept (there is no
 * further verified row: the same reading as in the greedy rule).
 *
 * u_accept, u_resample: [B][K] doubles in [0, 1), supplied by the caller.
 * Outputs: n_commit [B], committed [B][K] (-1 beyond n), next_anchor [B], and
 * margin [B][2] (optional): how far the decisions of sequence b were from flipping.
 * margin[b][0] = min over the accept tests taken of |u*q(y) - p(y)| / max(p(y), u*q(y));
 * margin[b][1] = if a token was resampled, the distance of u*total to the nearer of the
 * two running sums that bracket it, as a fraction of the chosen token's own residual
 * mass (0.5 = dead centre), else infinity.
 */
int oracle_consensus_sample(const void *ar_logits, const void *diff_logits, int dtype,
                            const int32_t *draft, const double *u_accept,
                            const double *u_resample, double temperature,
                            int32_t B, int32_t K, int32_t V,
                            int32_t *n_commit, int32_t *committed, int32_t *next_anchor,
                            double *margin)
{
    if (B < 0 || K <= 0 || V <= 0 || !(temperature > 0.0)) return -2;
    int rc = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b) {
        double *p = (double *)malloc(sizeof(double) * (size_t)V);
        double *q = (double *)malloc(sizeof(double) * (size_t)V);
        if (!p || !q) {
            free(p); free(q);
#pragma omp atomic write
            rc = -1;
            continue;
        }
        double worst = INFINITY, worst_pick = INFINITY;
        int32_t n = 0;
        for (int32_t k = 0; k < K; ++k) {
            const int64_t row = ((int64_t)b * K + k) * V;
            double mp = -INFINITY, mq = -INFINITY;
            for (int32_t v = 0; v < V; ++v) {
                p[v] = load_elem(ar_logits, dtype, row + v) / temperature;
                q[v] = load_elem(diff_logits, dtype, row + v) / temperature;
                if (p[v] > mp) mp = p[v];
                if (q[v] > mq) mq = q[v];
            }
            double zp = 0.0, zq = 0.0;
            for (int32_t v = 0; v < V; ++v) {
                p[v] = exp(p[v] - mp); zp += p[v];
                q[v] = exp(q[v] - mq); zq += q[v];
            }
            for (int32_t v = 0; v < V; ++v) { p[v] /= zp; q[v] /= zq; }

            const int32_t y = draft[(int64_t)b * K + k];
            const double lhs = u_accept[(int64_t)b * K + k] * q[y], rhs = p[y];
            const double big = lhs > rhs ? lhs : rhs;
            const double m1 = big > 0.0 ? fabs(lhs - rhs) / big : INFINITY;
            if (m1 < worst) worst = m1;
            if (lhs <= rhs) {                       /* draft kept */
                committed[(int64_t)b * K + n] = y;
                ++n;
                continue;
            }
            /* first rejection: draw the correction token from the residual */
            double total = 0.0;
            for (int32_t v = 0; v < V; ++v) { const double r = p[v] - q[v]; if (r > 0.0) total += r; }
            const int use_p = !(total > 0.0);
            if (use_p) total = 1.0;
            const double target = u_resample[(int64_t)b * K + k] * total;
            double run = 0.0, prev = 0.0;
            int32_t z = -1;
            for (int32_t v = 0; v < V; ++v) {
                const double r = use_p ? p[v] : (p[v] - q[v] > 0.0 ? p[v] - q[v] : 0.0);
                if (r > 0.0) {
                    prev = run;
                    run += r;
                    if (run > target) { z = v; break; }
                }
            }
            if (z < 0) {                            /* rounding left the last sum at or below target */
                for (int32_t v = V - 1; v >= 0; --v) {
                    const double r = use_p ? p[v] : p[v] - q[v];
                    if (r > 0.0) { z = v; break; }
                }
                if (z < 0) z = 0;
                prev = run;
            }
            {
                const double width = run - prev;
                const double lo = fabs(target - prev), hi = fabs(run - target);
                worst_pick = width > 0.0 ? (lo < hi ? lo : hi) / width : 0.0;
            }
            committed[(int64_t)b * K + n] = z;
            ++n;
            break;
        }
        n_commit[b] = n;
        for (int32_t i = n; i < K; ++i) committed[(int64_t)b * K + i] = -1;
        next_anchor[b] = committed[(int64_t)b * K + n - 1];
        if (margin) { margin[2 * b] = worst; margin[2 * b + 1] = worst_pick; }
        free(p); free(q);
    }
    return rc;
}

/*
 * KV commit (Figure 2(b) and the last paragraph of Section 3.3): the AR-view
 * K/V rows of the first n_b block positions join the shared cache right after
 * the current prefix, for every KV head; the prefix grows by n_b.  Everything
 * else in the cache is left byte-for-byte as it was.  The diffusion view's
 * block KV is never stored.  Caches and block tensors are raw bytes of the
 * given element type.  Returns -3 if a sequence would exceed its capacity
 * (nothing is written for that sequence).
 */
int oracle_kv_append(int32_t B, int32_t K, int32_t Hkv, int32_t d, int64_t capacity,
                     int dtype, void *k_cache, void *v_cache, int32_t *cache_len,
                     const void *k_blk, const void *v_blk, const int32_t *n_commit,
                     int update_len)
{
    const size_t es = elem_size(dtype);
    const size_t row = (size_t)d * es;
    int rc = 0;
    for (int32_t b = 0; b < B; ++b) {
        const int64_t P = cache_len[b];
        const int32_t n = n_commit[b];
        if (n < 0 || n > K || P < 0 || P + n > capacity) { rc = -3; continue; }
        for (int32_t i = 0; i < n; ++i)
            for (int32_t h = 0; h < Hkv; ++h) {
                const size_t src = ((((size_t)b * K + i) * Hkv) + h) * row;
                const size_t dst = ((((size_t)b * Hkv + h) * (size_t)capacity) + (size_t)(P + i)) * row;
                memcpy((char *)k_cache + dst, (const char *)k_blk + src, row);
                memcpy((char *)v_cache + dst, (const char *)v_blk + src, row);
            }
        if (update_len) cache_len[b] = (int32_t)(P + n);
    }
    return rc;
}

/*
 * Write-then-truncate form of the commit (last paragraph of Section 3.3: after the
 * consensus the model "truncates the shared KV cache" to the accepted length).
 *
 * Step 1, oracle_block_kv_write: a pass writes the K/V rows of all K block positions
 * behind the prefix, cache[b][h][P_b + i] = blk[b][i][h] for i < K, and leaves the
 * length alone: rows at or beyond the length are dead, so the cache still denotes the
 * same prefix.  The diffusion pass may park its transient block there, the AR pass
 * overwrites it.  Returns -3 if a sequence has no room for K rows (it is skipped).
 *
 * Step 2, oracle_commit_len: the length grows by n_b; the rows beyond it, drafts the
 * AR view did not confirm, are dead again.  Returns -3 for an n_b outside [0, K] or a
 * length that would pass the capacity (that sequence keeps its length).
 *
 * Together, with the AR-view block written last, they leave rows [0, P_b + n_b) and
 * the length exactly as oracle_kv_append does.
 */
int oracle_block_kv_write(int32_t B, int32_t K, int32_t Hkv, int32_t d, int64_t capacity,
                          int dtype, void *k_cache, void *v_cache, const int32_t *cache_len,
                          const void *k_blk, const void *v_blk)
{
    const size_t row = (size_t)d * elem_size(dtype);
    int rc = 0;
    for (int32_t b = 0; b < B; ++b) {
        const int64_t P = cache_len[b];
        if (P < 0 || P + K > capacity) { rc = -3; continue; }
        for (int32_t i = 0; i < K; ++i)
            for (int32_t h = 0; h < Hkv; ++h) {
                const size_t src = ((((size_t)b * K + i) * Hkv) + h) * row;
                const size_t dst = ((((size_t)b * Hkv + h) * (size_t)capacity) + (size_t)(P + i)) * row;
                memcpy((char *)k_cache + dst, (const char *)k_blk + src, row);
                memcpy((char *)v_cache + dst, (const char *)v_blk + src, row);
            }
    }
    return rc;
}

int oracle_commit_len(int32_t B, int32_t K, int64_t capacity, int32_t *cache_len,
                      const int32_t *n_commit)
{
    int rc = 0;
    for (int32_t b = 0; b < B; ++b) {
        const int64_t P = cache_len[b];
        const int32_t n = n_commit[b];
        if (n < 0 || n > K || P < 0 || P + n > capacity) { rc = -3; continue; }
        cache_len[b] = (int32_t)(P + n);
    }
    return rc;
}

/*
 * Rotary position embedding of a block, the step between the Q/K/V projections of a
 * view (Section 3.1) and its attention: block row i of sequence b sits at position
 * pos = P_b + i.  Head vectors are rotated pairwise in the half-split convention of
 * the Qwen / Llama family the paper builds on (Section 4.1): for c < d/2,
 *   angle = pos * theta^(-2c/d),
 *   y[c]       = x[c] * cos(angle) - x[c + d/2] * sin(angle),
 *   y[c + d/2] = x[c + d/2] * cos(angle) + x[c] * sin(angle).
 * x: [B][K][H][d] of `dtype`; y: the same shape in double (the caller rounds).
 */
int oracle_rope_block(const void *x, int dtype, int32_t B, int32_t K, int32_t H, int32_t d,
                      const int32_t *cache_len, double theta, double *y)
{
    if (d <= 0 || (d & 1) || theta <= 0.0) return -2;
    const int half = d / 2;
    for (int32_t b = 0; b < B; ++b)
        for (int32_t i = 0; i < K; ++i) {
            const double pos = (double)cache_len[b] + (double)i;
            for (int32_t h = 0; h < H; ++h) {
                const int64_t off = (((int64_t)b * K + i) * H + h) * d;
                for (int c = 0; c < half; ++c) {
                    const double ang = pos * pow(theta, -2.0 * (double)c / (double)d);
                    const double cs = cos(ang), sn = sin(ang);
                    const double x0 = load_elem(x, dtype, off + c);
                    const double x1 = load_elem(x, dtype, off + c + half);
                    y[off + c] = x0 * cs - x1 * sn;
                    y[off + c + half] = x1 * cs + x0 * sn;
                }
            }
        }
    return 0;
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
