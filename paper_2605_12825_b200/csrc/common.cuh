// Shared declarations of the Orthrus CUDA library: kernel parameter blocks,
// workspace layout and the launchers each translation unit exports.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "orthrus.h"

namespace orthrus {

constexpr int kHeaderBytes = 256;       // workspace header; int32 status word at offset 0
constexpr int kMaxSplits = 64;
constexpr int kDefaultSMs = 148;      // a full B200; used only when no device can be asked

// Streaming multiprocessors of the current device (asked once per device; kDefaultSMs when
// there is no device, so that size queries still work on a host without a GPU).
int num_sms();

// Parameters common to every attention kernel.  Rows of one (sequence, KV head)
// unit are ordered r = i * G + g  (block position i, head g within the group), so
// that the G query heads sharing a KV head and all K block positions form one tile
// of M = G * K rows.
struct AttnParams {
    const void *q, *k_blk, *v_blk, *k_cache, *v_cache;
    const int32_t *cache_len;
    void *out;
    float *part_o;      // [unit][split][M][d]   unnormalised partial outputs
    float *part_ml;     // [unit][split][M][2]   running max (log2 domain), running sum
    int32_t *status;    // device status word
    int B, K, Hq, Hkv, G, M, d;
    long long capacity;
    int chunk;          // prefix positions per split
    int n_splits;       // grid extent along the split axis
    int causal;         // 0: diffusion view (bidirectional block), 1: AR view (causal block)
    int blk_in_cache;   // the block's K/V rows are the cache rows [P, P + K) (k_blk / v_blk unused)
    int nb;             // blocks per sequence: batch entry b reads the cache of sequence b / nb
                        // (1 except for the multi-block mask of Eq. 6, where B counts blocks)
    int kb_width;       // packed form of Eq. 6 (0 otherwise): B counts sequences, K = nb * kb_width
                        // positions hold the nb blocks back to back, cache_len is [B][nb]
    long long len_cap;  // largest admissible prefix length: capacity - block width
    float scale_log2;   // softmax scale times log2(e)
};

// split s of a unit covers prefix positions [s*chunk, min((s+1)*chunk, P)); the split
// that holds the last prefix position (split 0 for an empty prefix) also takes the
// block keys.  Splits beyond it do nothing.
__host__ __device__ inline int last_split(int P, int chunk) {
    return P <= 0 ? 0 : (P - 1) / chunk;
}

// Largest prefix length a launch can serve: the capacity left beside the block, and (split-KV
// grids of the SIMT / mma paths, sized from max_len_hint) what the planned splits cover.
__host__ __device__ inline long long max_served_len(const AttnParams &p) {
    const long long hi = p.len_cap;
    const long long planned = (long long)p.n_splits * p.chunk;
    return planned < hi ? planned : hi;
}

__device__ inline int clamp_cache_len(const AttnParams &p, int b) {
    int P = p.cache_len[b];
    const long long hi = max_served_len(p);
    if (P < 0 || P > hi) {
        if (p.status) atomicOr(p.status, ORTHRUS_DEV_BAD_CACHE_LEN);
        P = P < 0 ? 0 : (int)hi;
    }
    return P;
}

// launchers (each returns the cudaError of its launches)
cudaError_t launch_attend_simt(const AttnParams &p, int dtype, cudaStream_t st);
bool mma_path_supports(const AttnParams &p, int dtype);
cudaError_t launch_attend_mma(const AttnParams &p, cudaStream_t st);
int mma_tile_positions();
bool tc_driver_ok();                    // the driver offers cuTensorMapEncodeTiled
cudaError_t launch_attend_tc(const AttnParams &p, int flags, cudaStream_t st);   // n_splits = cluster size
cudaError_t launch_attend_tc_packed(const AttnParams &p, int flags, cudaStream_t st);   // p.kb_width > 0
int tc_row_tiles(int G, int K);          // 128-row query tiles per unit (0: group too wide)
int tc_tiles_per_cta(int G, int K);      // query tiles that share one K/V ring in a CTA (1 or 2)
int tc_cta_groups(int G, int K);         // CTAs along the query-tile axis: ceil(row tiles / tiles per CTA)
int tc_ctas_per_sm(int nt);              // resident CTAs per SM of the shape with nt query tiles
int tc_max_cluster(int nt);              // largest cluster the device can co-schedule (<= 16)
int tc_tile_positions();
bool tc_stream_shape(int B, int G, int K);                  // the persistent kernel serves this shape
size_t tc_stream_workspace_bytes(int B, int Hkv, int n_ctas);
cudaError_t launch_attend_tc_stream(const AttnParams &p, int n_ctas, void *ws_body, int flags, cudaStream_t st);
cudaError_t launch_combine(const AttnParams &p, int dtype, cudaStream_t st);

cudaError_t launch_consensus(const void *logits, int dtype, const int32_t *draft, int B, int K,
                             int V, int32_t *n_commit, int32_t *committed, int32_t *ar_argmax,
                             int32_t *next_anchor, void *partials, int n_seg, cudaStream_t st);
int consensus_segments(int B, int K, int V);
struct ArgPart { float v; int idx; };    // the best (value, id) of one stretch of a row
cudaError_t launch_consensus_finalize_wide(const ArgPart *parts, int n_seg, const int32_t *draft, int B,
                                           int K, int32_t *n_commit, int32_t *committed,
                                           int32_t *ar_argmax, int32_t *next_anchor, cudaStream_t st);
int lm_head_vocab_tiles(int R, int V);     // (value, id) pairs per row for R rows, vocabulary V
int lm_head_max_vocab_tiles(int V);        // the most any row count needs
bool lm_head_supported();
cudaError_t launch_lm_head_argmax(const void *hidden, const void *lm_head, int R, int V, int H,
                                  ArgPart *parts, int32_t *status, cudaStream_t st);
size_t static_consensus_scratch_needed(int B, int K, int V);
cudaError_t launch_consensus_static(const void *logits, int dtype, const int32_t *draft, int B, int K,
                                    int V, int32_t *n_commit, int32_t *committed, int32_t *ar_argmax,
                                    int32_t *next_anchor, cudaStream_t st);

cudaError_t launch_kv_append(const orthrus_layer_t &L, const void *k_blk, const void *v_blk,
                             const int32_t *n_commit, int update_len, int32_t *status,
                             cudaStream_t st);
cudaError_t launch_block_kv_write(const orthrus_layer_t &L, const void *k_blk, const void *v_blk,
                                  int32_t *status, cudaStream_t st);
cudaError_t launch_commit_len(const orthrus_layer_t &L, const int32_t *n_commit, int32_t *status,
                              cudaStream_t st);
cudaError_t launch_rope_block_kv_write(const orthrus_layer_t &L, const void *q, const void *k_blk,
                                       const void *v_blk, double theta, void *q_out, int32_t *status,
                                       cudaStream_t st);

size_t sample_workspace_bytes(int B, int K, int V);
cudaError_t launch_consensus_sample(const void *ar_logits, const void *diff_logits, int dtype, const int32_t *draft,
                                    const float *u_accept, const float *u_resample, float temperature, int B, int K,
                                    int V, int32_t *n_commit, int32_t *committed, int32_t *next_anchor, void *ws,
                                    cudaStream_t st);

struct AppendLayer { void *k_cache, *v_cache; const void *k_blk, *v_blk; int32_t *cache_len; };
cudaError_t launch_kv_append_layers(const orthrus_layer_t &shape, const AppendLayer *layers, int n_layers,
                                    int32_t *const *len_arrays, int n_len_arrays,
                                    const int32_t *n_commit, int32_t *status, cudaStream_t st);

void count_launch(int n = 1);

}  // namespace orthrus
