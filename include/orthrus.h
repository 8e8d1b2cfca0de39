/*
 * orthrus.h — C ABI of the B200 (sm_100a) hot path of the Orthrus generation step.
 *
 * One generation cycle (Section 3.3 of the paper) is, per transformer layer,
 *   1. the diffusion view attending from a block of K positions to the shared
 *      prefix KV cache and, bidirectionally, to the block itself   (Eq. 4),
 *   2. the AR view verifying the same block causally over the same cache,
 * then once per cycle
 *   3. the greedy consensus between drafts and AR logits            (Eq. 8),
 *   4. the commit of the accepted AR-view KV rows to the cache (Figure 2(b)).
 * This library implements exactly those four operations as CUDA kernels.
 *
 * Conventions shared by every call
 *   - Every data pointer is a DEVICE pointer owned by the caller, 16-byte
 *     aligned, valid until the stream has passed the call.  Descriptors
 *     (orthrus_layer_t) are HOST structs read during the call only.
 *   - `stream` is a cudaStream_t passed as an opaque pointer (NULL = legacy
 *     default stream).  Calls only enqueue work: they never synchronise, never
 *     allocate, and keep no device state between calls.
 *   - Problems the host can see (null or misaligned pointers, unsupported
 *     shapes, a workspace that is too small) return an error code before
 *     anything is launched.  Problems only the device can see (a cache_len
 *     outside [0, capacity - K], an append past the capacity, a hardware wait
 *     that ran out) never trap: the offending sequence is clamped or skipped
 *     and a code is OR-ed into the status word at the start of the workspace,
 *     which orthrus_read_status() fetches.
 *   - Tensors are row-major, innermost dimension last:
 *       q_*, out           [B][K][Hq][d]
 *       k_*_blk, v_*_blk   [B][K][Hkv][d]
 *       k_cache, v_cache   [B][Hkv][capacity][d]
 *       ar_logits          [B][K][V]
 *       draft, committed, ar_argmax  [B][K] int32;  n_commit, next_anchor, cache_len [B] int32
 *     Query head hq reads KV head hq / (Hq / Hkv).
 *   - dtype ORTHRUS_BF16: bf16 inputs/outputs, fp32 softmax and accumulation.
 *     dtype ORTHRUS_FP32: fp32 everywhere (a slow test mode).
 */
#ifndef ORTHRUS_H_
#define ORTHRUS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ORTHRUS_OK = 0,
    ORTHRUS_ERR_INVALID_ARG = 1,  /* null/misaligned pointer, bad size            */
    ORTHRUS_ERR_UNSUPPORTED = 2,  /* shape or dtype outside the supported set     */
    ORTHRUS_ERR_CAPACITY = 3,     /* max_len_hint + block exceeds capacity        */
    ORTHRUS_ERR_WORKSPACE = 4,    /* workspace smaller than *_workspace_bytes()   */
    ORTHRUS_ERR_CUDA = 5,         /* a CUDA runtime call failed                   */
    ORTHRUS_ERR_TIMEOUT = 6       /* orthrus_read_status only: the status word has
                                     ORTHRUS_DEV_WAIT_TIMEOUT set                  */
} orthrus_status_t;

/* bits of the device status word (first int32 of the workspace) */
enum {
    ORTHRUS_DEV_BAD_CACHE_LEN = 1,   /* cache_len[b] outside [0, capacity-K], or above a
                                        max_len_hint the launch was sized for: clamped      */
    ORTHRUS_DEV_APPEND_OVERFLOW = 2, /* cache_len[b]+n_commit[b] > capacity, or n_commit[b]
                                        outside [0,K]: that sequence was not appended       */
    ORTHRUS_DEV_WAIT_TIMEOUT = 4     /* a bounded hardware wait expired; outputs undefined  */
};

typedef enum { ORTHRUS_BF16 = 0, ORTHRUS_FP32 = 1 } orthrus_dtype_t;

/* One layer's shared KV cache plus the shape of the block attending to it. */
typedef struct {
    int32_t batch;          /* B >= 1                                               */
    int32_t n_q_heads;      /* Hq, a multiple of n_kv_heads                         */
    int32_t n_kv_heads;     /* Hkv                                                  */
    int32_t head_dim;       /* d in {32, 64, 128, 256}; tensor-core paths: 64, 128  */
    int32_t block;          /* K, 1..64                                             */
    int32_t dtype;          /* orthrus_dtype_t of q, out, block KV and cache        */
    int64_t capacity;       /* positions per (sequence, KV head) in the cache       */
    void *k_cache;          /* device [B][Hkv][capacity][d]                         */
    void *v_cache;          /* device [B][Hkv][capacity][d]                         */
    int32_t *cache_len;     /* device [B]: prefix length P_b, 0 <= P_b <= cap - K   */
    int32_t max_len_hint;   /* host upper bound on every P_b; sizes the split-KV
                               grid.  0 means capacity - block.  A P_b above the
                               hint may be clamped to what the grid covers (then
                               ORTHRUS_DEV_BAD_CACHE_LEN is raised)                 */
    float softmax_scale;    /* 0 selects 1/sqrt(head_dim), the scale of Eq. 4       */
    uint32_t flags;         /* OR of ORTHRUS_LAYER_* bits, 0 for none               */
} orthrus_layer_t;

/*
 * orthrus_layer_t.flags
 *
 * ORTHRUS_LAYER_CACHE_QUIESCENT: a promise by the caller that the kernel enqueued
 * immediately before this call on the same stream writes neither cache_len nor any
 * cache row below cache_len (in a generation loop that kernel is the projection that
 * produced q and the block KV; the cache was last written by the previous cycle's
 * commit).  The attention kernels are launched with programmatic stream
 * serialisation: they may start while the preceding kernel is still running and wait
 * for it on the device before touching anything it may have produced.  With this
 * flag they request the first prefix K/V tiles before that wait.  Without it nothing
 * is read early and any caller is safe.
 *
 * ORTHRUS_LAYER_NO_EARLY_LAUNCH: launch with ordinary stream order only.
 *
 * ORTHRUS_LAYER_BLOCK_IN_CACHE (attention calls only): the K/V rows of the block are not
 * passed as tensors but already sit in the cache, at rows [P_b, P_b + K) of every KV
 * head, where orthrus_block_kv_write or orthrus_rope_block_kv_write put them; the
 * k_*_blk / v_*_blk arguments are ignored and may be NULL.  The masks are unchanged
 * (diffusion view: all K rows; AR view: row i sees block rows 0..i).  Rows from P_b + K
 * on are never read.  Compatible with ORTHRUS_LAYER_CACHE_QUIESCENT: the writing call
 * touches only rows at or beyond cache_len.
 */
enum {
    ORTHRUS_LAYER_CACHE_QUIESCENT = 1,
    ORTHRUS_LAYER_NO_EARLY_LAUNCH = 2,
    ORTHRUS_LAYER_BLOCK_IN_CACHE = 4
};

/*
 * Bytes of workspace the two attention calls (and orthrus_kv_append) need for
 * this layer shape: a 256-byte header holding the status word, followed by the
 * split-KV partial results (written and read back inside one call; they are meant
 * to stay in L2).  Sizes depend on the device (its SM count shapes the split plan):
 * ask with the device current that will run the calls.  A workspace serves one stream at a time: calls on the same stream
 * may share it, calls that can overlap on the GPU (different streams) need their own.
 * Returns 0 for an invalid descriptor.
 */
size_t orthrus_attend_workspace_bytes(const orthrus_layer_t *layer);

/*
 * Zeroes the workspace: the status word in its header, and the arrival counters the
 * attention kernels keep in it (they return to zero at the end of every call that
 * completes).  Call once after allocating a workspace, whenever the status word should
 * be cleared, and after a call that reported ORTHRUS_DEV_WAIT_TIMEOUT.
 */
orthrus_status_t orthrus_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/*
 * Diffusion-view block attention, Eq. 4: for every sequence b, query head hq and
 * block position i,
 *   out[b][i][hq] = softmax_j( q_diff[b][i][hq] . key_j * scale ) applied to value_j,
 * where j runs over the P_b cache rows of KV head hq/(Hq/Hkv) followed by ALL K
 * rows of the diffusion block (k_diff_blk, v_diff_blk): the block is
 * bidirectional (Section 3.2, viewing rule (ii)).  The block KV is transient: it
 * is read here and never stored.
 */
orthrus_status_t orthrus_diffusion_block_attend(const orthrus_layer_t *layer,
        const void *q_diff, const void *k_diff_blk, const void *v_diff_blk, void *out,
        void *workspace, size_t workspace_bytes, void *stream);

/*
 * AR-view verify attention (Section 3.3, "Intra-Model Distribution Matching"):
 * the same as above with the AR-view block tensors, except that the block is
 * causal: position i sees the P_b cache rows and block rows 0..i only, which is
 * what the frozen causal model computes for the materialised block.
 */
orthrus_status_t orthrus_ar_verify_attend(const orthrus_layer_t *layer,
        const void *q_ar, const void *k_ar_blk, const void *v_ar_blk, void *out,
        void *workspace, size_t workspace_bytes, void *stream);

/*
 * Diffusion-view attention under the multi-block mask of Eq. 6 (Section 3.2, the
 * training-time form; inference is its single-block case): n_blocks blocks of K rows per
 * sequence, block j of sequence s anchored at position anchors[s][j], all reading the one
 * clean cache of their sequence.  Row i of block j attends to the cache rows
 * [0, anchors[s][j]) of KV head hq/(Hq/Hkv) (rule (i): the clean context before its anchor)
 * and to all K rows of its own block (rule (ii)), and to nothing else: not to other
 * blocks, not to the context at or after its anchor.
 *   q_diff, out            [S][n_blocks][K][Hq][d]
 *   k_diff_blk, v_diff_blk [S][n_blocks][K][Hkv][d]
 *   anchors                device int32 [S][n_blocks], 0 <= anchor <= capacity - K (values
 *                          outside are clamped and flagged like a bad cache_len); the caller
 *                          keeps them at or below the sequence's clean length
 * layer describes the S sequences (batch = S; cache_len is not read; max_len_hint bounds
 * the anchors).  On the tcgen05 path, when at least two blocks fit the 128 rows of a query
 * tile (2 * K * Hq/Hkv <= 128), consecutive blocks of a sequence share query tiles: the
 * prefix is streamed once per tile, up to the largest anchor among its blocks, each row
 * masked at its own anchor and to its own block's keys.  Otherwise every block is a unit
 * of work of its own, scheduled longest prefix first.
 * Workspace: orthrus_multi_block_workspace_bytes(layer, n_blocks).
 */
size_t orthrus_multi_block_workspace_bytes(const orthrus_layer_t *layer, int32_t n_blocks);
orthrus_status_t orthrus_multi_block_attend(const orthrus_layer_t *layer, int32_t n_blocks,
        const int32_t *anchors, const void *q_diff, const void *k_diff_blk, const void *v_diff_blk,
        void *out, void *workspace, size_t workspace_bytes, void *stream);

/* Workspace bytes for orthrus_consensus_accept (header + per-row partial maxima). */
size_t orthrus_consensus_workspace_bytes(int32_t batch, int32_t block, int32_t vocab);

/*
 * Greedy consensus, Eq. 8 with the halt/commit rule of Section 3.3.
 *   ar_argmax[b][i] = smallest v maximising ar_logits[b][i][v]   (NaN never wins)
 *   m_b       = number of leading positions with draft[b][i] == ar_argmax[b][i]
 *   n_commit[b] = min(m_b + 1, K)   (agreeing drafts plus the correction token;
 *                                    K when the whole block agrees; always >= 1)
 *   committed[b][i] = ar_argmax[b][i] for i < n_commit[b], else -1
 *   next_anchor[b]  = ar_argmax[b][n_commit[b] - 1]
 * `dtype` is the element type of ar_logits.  All outputs are bit-exact.
 */
orthrus_status_t orthrus_consensus_accept(const void *ar_logits, int32_t dtype,
        const int32_t *draft, int32_t batch, int32_t block, int32_t vocab,
        int32_t *n_commit, int32_t *committed, int32_t *ar_argmax, int32_t *next_anchor,
        void *workspace, size_t workspace_bytes, void *stream);

/*
 * Sampled consensus for temperature T > 0: the exact rejection sampling of Section 3.3
 * (the speculative-sampling rule of the work cited there), which keeps the committed
 * tokens distributed as the AR view alone would have sampled them.
 *   p_k = softmax(ar_logits[b][k] / T),  q_k = softmax(diff_logits[b][k] / T);
 *   draft[b][k] (drawn from q_k by the caller) is kept iff
 *       u_accept[b][k] * q_k(draft) <= p_k(draft)      (probability min(1, p/q));
 *   at the first k that fails, committed[b][k] is drawn from max(0, p_k - q_k),
 *   normalised, by inverting its running sum over the vocabulary with u_resample[b][k]
 *   (from p_k itself if that residual is empty), and verification halts;
 *   n_commit[b] = kept drafts + 1, or K when every draft is kept;
 *   committed[b][i] = -1 for i >= n_commit[b];  next_anchor[b] = last committed token.
 * ar_logits, diff_logits: [B][K][V] of `dtype`; draft int32 [B][K]; u_accept, u_resample:
 * float32 [B][K] in [0, 1), drawn by the caller (the library draws no random numbers);
 * temperature > 0.  Softmax sums are taken in fp32 in a fixed order: results are
 * reproducible, and differ from an exact evaluation only where a comparison is within
 * rounding of a tie.  The commit of the accepted KV rows is orthrus_kv_append as before.
 */
size_t orthrus_consensus_sample_workspace_bytes(int32_t batch, int32_t block, int32_t vocab);
orthrus_status_t orthrus_consensus_sample(const void *ar_logits, const void *diff_logits, int32_t dtype,
        const int32_t *draft, const float *u_accept, const float *u_resample, float temperature,
        int32_t batch, int32_t block, int32_t vocab,
        int32_t *n_commit, int32_t *committed, int32_t *next_anchor,
        void *workspace, size_t workspace_bytes, void *stream);

/*
 * The greedy consensus for callers that cannot hand over a workspace.  (The paper has no
 * counterpart to this entry point; it exists for the embedding, not for the method.)
 *
 * Who needs it: code that runs where device memory may not be allocated - a plugin that
 * is given its input and output buffers by a host runtime and is forbidden to call
 * cudaMalloc (or any allocator built on it, a framework's caching allocator included),
 * or a serving loop whose memory budget is fixed before it starts.  Such a caller can
 * supply the logits, the drafts and the four result arrays, but has nowhere to get the
 * scratch that the streaming argmax needs between its two kernels.
 *
 * Here that scratch is an array compiled into the library
 * (ORTHRUS_STATIC_CONSENSUS_SCRATCH_BYTES of device memory on every GPU that loads the
 * library, held until the process exits).  The call allocates nothing and frees nothing.
 *   - Limit: batch * block * segments * 8 bytes must fit in the array, where segments is
 *     the split of the vocabulary the library chooses (at most about 600 / (batch*block),
 *     at least 1): in practice batch * block <= 8192 rows.  A larger problem returns
 *     ORTHRUS_ERR_WORKSPACE and launches nothing; use orthrus_consensus_accept then.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside of any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the previous call
 *     left in it.  Nothing has to be cleared (each call overwrites every entry it later
 *     reads), but two calls that overlap on the GPU - different streams, or different
 *     host threads - race on it and may both return wrong tokens.  Serialise them.
 * Arguments, results and errors are otherwise those of orthrus_consensus_accept.
 */
#define ORTHRUS_STATIC_CONSENSUS_SCRATCH_BYTES 65536
orthrus_status_t orthrus_consensus_accept_static(const void *ar_logits, int32_t dtype,
        const int32_t *draft, int32_t batch, int32_t block, int32_t vocab,
        int32_t *n_commit, int32_t *committed, int32_t *ar_argmax, int32_t *next_anchor,
        void *stream);

/*
 * Greedy consensus straight from the AR view's last hidden states (the step before Eq. 8
 * fused into it): with the shared LM head of Section 3.1,
 *   logits[b][i][v] = sum_c hidden[b][i][c] * lm_head[v][c],
 * the greedy tokens g[b][i] = argmax_v logits[b][i][v] (smallest id on ties, a NaN never
 * wins) and then the accept rule of orthrus_consensus_accept on g.  The logits are never
 * written to memory.  Products of the bf16 operands are accumulated in fp32 on the tensor
 * cores and compared as fp32 sums (they are not rounded to bf16 first, so a near-tie can
 * resolve differently from the two-step path that stores bf16 logits).
 *
 * hidden   device [batch][block][hidden_dim] bf16 (final-norm output of the AR view)
 * lm_head  device [vocab][hidden_dim] bf16, one row per vocabulary entry
 * Both 16-byte aligned; hidden_dim a multiple of 8.  draft and the four outputs as for
 * orthrus_consensus_accept.  Only ORTHRUS_BF16 is supported (anything else, or a driver
 * without tensor-map support: ORTHRUS_ERR_UNSUPPORTED).  `workspace`: at least
 * orthrus_lm_head_consensus_workspace_bytes(batch, block, vocab) bytes, 16-byte aligned,
 * header initialised by orthrus_workspace_init; a wait inside the kernel that does not end
 * reports ORTHRUS_DEV_WAIT_TIMEOUT through orthrus_read_status and leaves the outputs of
 * that call undefined.  Two launches; nothing is allocated and the stream is not synchronised.
 * The first call on each device sets kernel attributes and builds the tensor maps of its
 * operands (cached by pointer and shape): make that call outside of any stream capture; later
 * calls with the same buffers can be captured into a CUDA graph.
 */
size_t orthrus_lm_head_consensus_workspace_bytes(int32_t batch, int32_t block, int32_t vocab);
orthrus_status_t orthrus_lm_head_consensus(const void *hidden, const void *lm_head, int32_t dtype,
        int32_t hidden_dim, const int32_t *draft, int32_t batch, int32_t block, int32_t vocab,
        int32_t *n_commit, int32_t *committed, int32_t *ar_argmax, int32_t *next_anchor,
        void *workspace, size_t workspace_bytes, void *stream);

/*
 * KV commit (Figure 2(b); last paragraph of Section 3.3): for every sequence b,
 * KV head h and i < n_commit[b],
 *   k_cache[b][h][P_b + i] = k_ar_blk[b][i][h]   (likewise v),
 * a byte copy; with update_len != 0, cache_len[b] += n_commit[b] afterwards.
 * update_len = 0 lets several layers that share one cache_len array be appended
 * before the length is bumped by the last of them.  Rows outside
 * [P_b, P_b + n_commit[b]) are not touched.  `workspace` may be NULL; if given,
 * overflow is reported through its status word.
 */
orthrus_status_t orthrus_kv_append(const orthrus_layer_t *layer, const void *k_ar_blk,
        const void *v_ar_blk, const int32_t *n_commit, int32_t update_len,
        void *workspace, size_t workspace_bytes, void *stream);

/*
 * The commit in its write-then-truncate form (last paragraph of Section 3.3: the model
 * "truncates the shared KV cache" to the accepted length).  Instead of copying accepted
 * rows after the consensus, every pass writes its whole block behind the prefix first:
 *
 * orthrus_block_kv_write: for every sequence b, KV head h and i < K,
 *   k_cache[b][h][P_b + i] = k_blk[b][i][h]   (likewise v), a byte copy; cache_len is
 *   not changed, so the rows are dead until a length says otherwise.  The diffusion pass
 *   may park its transient block there; the AR pass of the same layer overwrites it.
 *   A sequence with P_b + K > capacity is skipped (ORTHRUS_DEV_APPEND_OVERFLOW).
 *
 * orthrus_commit_len: cache_len[b] += n_commit[b] for the layer's length array (layers
 * that share one array need one call).  An n_commit[b] outside [0, K] or a length that
 * would pass the capacity leaves that length alone (ORTHRUS_DEV_APPEND_OVERFLOW).
 * With the AR-view rows written last, rows [0, P_b + n) and the length end up exactly as
 * orthrus_kv_append leaves them; the unconfirmed rows beyond are dead again.
 *
 * orthrus_rope_block_kv_write: the write fused with the rotary position embedding that
 * sits between the projections (Section 3.1) and the attention.  Block row i of
 * sequence b has position P_b + i; with the half-split pairing (c, c + d/2) and
 *   angle = (P_b + i) * rope_theta^(-2c/d),
 *   y[c] = x[c] cos(angle) - x[c + d/2] sin(angle),  y[c + d/2] = x[c + d/2] cos(angle) + x[c] sin(angle),
 * q_out[b][i][hq] = rotate(q[b][i][hq]) (q_out may be q: in place), k_cache[b][h][P_b + i]
 * = rotate(k_blk[b][i][h]), v_cache[b][h][P_b + i] = v_blk[b][i][h].  Angles are formed in
 * double precision, results are rounded once to the layer's dtype.  q, q_out:
 * [B][K][Hq][d]; k_blk, v_blk: [B][K][Hkv][d], straight from the projections (not rotated).
 *
 * `workspace` may be NULL in all three; if given, problems are reported through its status
 * word.  One launch each.
 */
orthrus_status_t orthrus_block_kv_write(const orthrus_layer_t *layer, const void *k_blk, const void *v_blk,
        void *workspace, size_t workspace_bytes, void *stream);
orthrus_status_t orthrus_commit_len(const orthrus_layer_t *layer, const int32_t *n_commit,
        void *workspace, size_t workspace_bytes, void *stream);
orthrus_status_t orthrus_rope_block_kv_write(const orthrus_layer_t *layer, const void *q, const void *k_blk,
        const void *v_blk, float rope_theta, void *q_out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The same commit for n_layers layers in one launch: the cycle's verify pass has
 * produced the AR-view block KV of every layer by the time the consensus is known, so
 * one kernel moves all of it.  layers[l] is the l-th layer's descriptor (a HOST array;
 * all layers must agree in batch, n_kv_heads, head_dim, block, dtype and capacity);
 * k_ar_blks[l] / v_ar_blks[l] are HOST arrays of DEVICE pointers to that layer's
 * [B][K][Hkv][d] block tensors.  With update_len != 0 every DISTINCT cache_len array
 * among the layers grows by n_commit once, after all of its layers have been copied
 * (layers sharing one array are bumped once).  1 <= n_layers <= 128.
 */
orthrus_status_t orthrus_kv_append_layers(const orthrus_layer_t *layers, int32_t n_layers,
        const void *const *k_ar_blks, const void *const *v_ar_blks, const int32_t *n_commit,
        int32_t update_len, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Copies the device status word to *host_status and waits for the stream (the
 * only call here that synchronises).  0 means no device-side problem so far.
 * Returns ORTHRUS_ERR_TIMEOUT (with *host_status filled in) if the word has
 * ORTHRUS_DEV_WAIT_TIMEOUT set: the outputs of the calls since the word was last
 * cleared are undefined; the other bits are advisory and return ORTHRUS_OK.
 */
orthrus_status_t orthrus_read_status(const void *workspace, void *stream, int32_t *host_status);

/*
 * Kernel-path selection for measurements: "auto" (default), "simt", "mma" or
 * "tcgen05".  A path that does not support the shape falls back to the next
 * more general one.  Returns ORTHRUS_ERR_INVALID_ARG for an unknown name.
 * Also settable through the environment variable ORTHRUS_FORCE_PATH.
 */
orthrus_status_t orthrus_set_path(const char *name);

/* Name of the kernel path the last attention call on this thread took. */
const char *orthrus_last_path(void);

/* Number of kernels launched by this library in this process so far. */
int64_t orthrus_launch_count(void);

const char *orthrus_status_string(orthrus_status_t status);
int32_t orthrus_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ORTHRUS_H_ */
