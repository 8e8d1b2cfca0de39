// C-ABI entry points: argument validation, split-KV planning, kernel-path dispatch.
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include "common.cuh"

namespace orthrus {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

enum Path { PATH_AUTO = 0, PATH_SIMT, PATH_MMA, PATH_TCGEN05 };
static std::atomic<int> g_path{-1};
static thread_local const char *t_last_path = "none";

static int parse_path(const char *s)
{
    if (!s || !*s || !strcmp(s, "auto")) return PATH_AUTO;
    if (!strcmp(s, "simt")) return PATH_SIMT;
    if (!strcmp(s, "mma")) return PATH_MMA;
    if (!strcmp(s, "tcgen05")) return PATH_TCGEN05;
    return -1;
}

static int current_path()
{
    int v = g_path.load();
    if (v < 0) {
        v = parse_path(getenv("ORTHRUS_FORCE_PATH"));
        if (v < 0) v = PATH_AUTO;
        g_path.store(v);
    }
    return v;
}

static int env_int(const char *name, int dflt)
{
    const char *s = getenv(name);
    if (!s || !*s) return dflt;
    const int v = atoi(s);
    return v > 0 ? v : dflt;
}

}  // namespace orthrus

int orthrus::num_sms()
{
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cached[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return kDefaultSMs;
    }
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        return kDefaultSMs;
    }
    cached[dev].store(n, std::memory_order_relaxed);
    return n;
}

namespace orthrus {

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

static orthrus_status_t check_layer(const orthrus_layer_t *L)
{
    if (!L) return ORTHRUS_ERR_INVALID_ARG;
    if (L->batch < 1 || L->n_q_heads < 1 || L->n_kv_heads < 1 || L->block < 1 || L->capacity < 1)
        return ORTHRUS_ERR_INVALID_ARG;
    if (L->n_q_heads % L->n_kv_heads != 0) return ORTHRUS_ERR_INVALID_ARG;
    if (L->dtype != ORTHRUS_BF16 && L->dtype != ORTHRUS_FP32) return ORTHRUS_ERR_UNSUPPORTED;
    if (L->head_dim != 32 && L->head_dim != 64 && L->head_dim != 128 && L->head_dim != 256)
        return ORTHRUS_ERR_UNSUPPORTED;
    if (L->block > 64) return ORTHRUS_ERR_UNSUPPORTED;
    if (L->max_len_hint < 0 || !(L->softmax_scale >= 0.f) || std::isinf(L->softmax_scale))
        return ORTHRUS_ERR_INVALID_ARG;
    if (L->block > L->capacity) return ORTHRUS_ERR_CAPACITY;
    if (L->capacity > 0x7fffffffLL) return ORTHRUS_ERR_UNSUPPORTED;
    if ((long long)L->max_len_hint + L->block > L->capacity) return ORTHRUS_ERR_CAPACITY;
    if (L->flags & ~(uint32_t)(ORTHRUS_LAYER_CACHE_QUIESCENT | ORTHRUS_LAYER_NO_EARLY_LAUNCH |
                               ORTHRUS_LAYER_BLOCK_IN_CACHE))
        return ORTHRUS_ERR_INVALID_ARG;
    return ORTHRUS_OK;
}

static int max_len_of(const orthrus_layer_t *L)
{
    return L->max_len_hint > 0 ? L->max_len_hint : (int)(L->capacity - L->block);
}

// Split-KV plan: a pure function of the descriptor, the kernel path and a few tuning
// variables read from the environment, so that the workspace query and the launch agree.
struct Plan { int chunk, n_splits, tile; };

static bool tc_shape(const orthrus_layer_t *L)
{
    return L->dtype == ORTHRUS_BF16 && L->head_dim == 128 && L->block <= 64 &&
           tc_row_tiles(L->n_q_heads / L->n_kv_heads, L->block) > 0;
}

// The tcgen05 path as a whole: the shape, the row count a 2-D tensor map can index and a
// driver that offers the tensor-map encoder.  Anything else plans and launches on mma / SIMT.
static bool tc_usable(const orthrus_layer_t *L)
{
    if (!tc_shape(L)) return false;
    const unsigned long long rows = (unsigned long long)L->batch * L->n_kv_heads * (unsigned long long)L->capacity;
    return rows < 0x7fffffffull && tc_driver_ok();
}

// ORTHRUS_TC_SCHEDULE=stream (read at every call) selects the persistent kernel, which cuts the
// work by tiles instead of by units, for the shapes it serves; it was measured slower than the
// cluster kernel and is a measurement knob.  A forced split count keeps the cluster kernel.
static bool tc_use_stream(const orthrus_layer_t *L)
{
    if (!tc_usable(L)) return false;
    const int G = L->n_q_heads / L->n_kv_heads;
    if (!tc_stream_shape(L->batch, G, L->block) || env_int("ORTHRUS_SPLITS", 0) > 0) return false;
    const char *e = getenv("ORTHRUS_TC_SCHEDULE");
    return e && !strcmp(e, "stream");
}
static int tc_stream_ctas() { return tc_ctas_per_sm(1) * num_sms(); }

static Plan make_plan(const orthrus_layer_t *L, bool tc)
{
    const int max_len = max_len_of(L);
    const int forced = env_int("ORTHRUS_SPLITS", 0);
    Plan pl;
    if (tc) {
        // The splits of a unit are the CTAs of one thread-block cluster (<= 16).  Few units:
        // as many splits as still fit on the GPU in one wave.  Many units: just enough CTAs
        // to fill every slot once; sequences of unequal length are handed out longest first.
        const int tn = tc_tile_positions();
        const int G = L->n_q_heads / L->n_kv_heads, nt = tc_tiles_per_cta(G, L->block);
        const int units = L->batch * L->n_kv_heads * tc_cta_groups(G, L->block);
        const int slots = tc_ctas_per_sm(nt) * num_sms();
        const int tiles = max_len > 0 ? (max_len + tn - 1) / tn : 1;
        int S = 1;
        if (forced > 0) {
            S = forced;
        } else if (units * 2 <= slots) {
            const int min_tiles = env_int("ORTHRUS_MIN_CHUNK_TILES", 2);
            while (S < 16 && units * S * 2 <= slots && tiles / (S * 2) >= min_tiles) S *= 2;
        } else {
            // (a lone CTA streams slower than an SM's share of HBM, so the longest unit is
            //  still split; many small CTAs would spend their time starting and merging)
            while (S < 16 && units * S < slots && tiles / (S * 2) >= 8) S *= 2;
        }
        const int max_cluster = tc_max_cluster(nt);
        if (S > max_cluster) S = max_cluster;
        if (S > tiles) S = tiles;
        if (S < 1) S = 1;
        pl.n_splits = S;
        pl.chunk = ((tiles + S - 1) / S) * tn;
        pl.tile = tn;
        return pl;
    }
    const int granule = 128;
    const int units = L->batch * L->n_kv_heads;
    const int tiles = max_len > 0 ? (max_len + granule - 1) / granule : 1;
    const int target = env_int("ORTHRUS_TARGET_CTAS", 2 * num_sms());
    const int min_chunk_tiles = env_int("ORTHRUS_MIN_CHUNK_TILES", 2);
    int splits = (target + units - 1) / units;
    if (forced > 0) splits = forced;
    int max_splits = forced > 0 ? tiles : tiles / min_chunk_tiles;
    if (max_splits < 1) max_splits = 1;
    if (max_splits > kMaxSplits) max_splits = kMaxSplits;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    const int chunk_tiles = (tiles + splits - 1) / splits;
    pl.chunk = chunk_tiles * granule;
    pl.n_splits = max_len > 0 ? (max_len + pl.chunk - 1) / pl.chunk : 1;
    pl.tile = granule;
    return pl;
}

static size_t partial_bytes(const orthrus_layer_t *L, const Plan &pl, size_t *ml_off, bool tc = false)
{
    if (ml_off) *ml_off = 0;
    if (pl.n_splits == 1) return 0;
    // the tcgen05 path keeps one 128-row partial tile per CTA
    const size_t units = (size_t)L->batch * L->n_kv_heads *
                         (tc ? tc_row_tiles(L->n_q_heads / L->n_kv_heads, L->block) : 1);
    const size_t M = tc ? 128 : (size_t)(L->n_q_heads / L->n_kv_heads) * L->block;
    const size_t o_bytes = units * pl.n_splits * M * L->head_dim * sizeof(float);
    const size_t ml_bytes = units * pl.n_splits * M * 2 * sizeof(float);
    if (ml_off) *ml_off = o_bytes;
    return o_bytes + ml_bytes;
}

// nb: blocks per sequence (the batch of *L then counts blocks, and batch entry b reads the cache
// of sequence b / nb)
static orthrus_status_t attend(const orthrus_layer_t *L, int causal, const void *q,
                               const void *k_blk, const void *v_blk, void *out, void *ws,
                               size_t ws_bytes, void *stream, int nb = 1)
{
    orthrus_status_t st = check_layer(L);
    if (st != ORTHRUS_OK) return st;
    const bool in_cache = (L->flags & ORTHRUS_LAYER_BLOCK_IN_CACHE) != 0;
    if (in_cache) k_blk = v_blk = nullptr;    // not read in this mode
    if (!q || (!in_cache && (!k_blk || !v_blk)) || !out || !ws || !L->k_cache || !L->v_cache || !L->cache_len)
        return ORTHRUS_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out) ||
        !aligned16(ws) || !aligned16(L->k_cache) || !aligned16(L->v_cache) ||
        (reinterpret_cast<uintptr_t>(L->cache_len) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    const int want = current_path();
    const bool tc = (want == PATH_AUTO || want == PATH_TCGEN05) && tc_usable(L);
    const bool stream_k = tc && tc_use_stream(L);
    Plan pl = make_plan(L, tc);
    if (stream_k) pl.n_splits = 1;
    size_t ml_off = 0;
    const size_t need = kHeaderBytes + (stream_k ? tc_stream_workspace_bytes(L->batch, L->n_kv_heads, tc_stream_ctas())
                                                 : partial_bytes(L, pl, &ml_off, tc));
    if (ws_bytes < need) return ORTHRUS_ERR_WORKSPACE;

    AttnParams p;
    p.q = q; p.k_blk = k_blk; p.v_blk = v_blk; p.k_cache = L->k_cache; p.v_cache = L->v_cache;
    p.cache_len = L->cache_len; p.out = out;
    unsigned char *base = static_cast<unsigned char *>(ws);
    p.status = reinterpret_cast<int32_t *>(base);
    p.part_o = reinterpret_cast<float *>(base + kHeaderBytes);
    p.part_ml = reinterpret_cast<float *>(base + kHeaderBytes + ml_off);
    p.B = L->batch; p.K = L->block; p.Hq = L->n_q_heads; p.Hkv = L->n_kv_heads;
    p.G = p.Hq / p.Hkv; p.M = p.G * p.K; p.d = L->head_dim; p.capacity = L->capacity;
    p.chunk = pl.chunk; p.n_splits = pl.n_splits; p.causal = causal;
    p.blk_in_cache = in_cache ? 1 : 0;
    p.nb = nb; p.kb_width = 0; p.len_cap = L->capacity - L->block;
    const float scale = L->softmax_scale > 0.f ? L->softmax_scale : 1.f / sqrtf((float)p.d);
    p.scale_log2 = scale * 1.4426950408889634f;

    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    bool merge_kernel = pl.n_splits > 1;
    if (tc) {
        t_last_path = "tcgen05";
        int flags = (int)(L->flags & (ORTHRUS_LAYER_CACHE_QUIESCENT | ORTHRUS_LAYER_NO_EARLY_LAUNCH));
        if (env_int("ORTHRUS_NO_EARLY_LAUNCH", 0)) flags |= ORTHRUS_LAYER_NO_EARLY_LAUNCH;
        if (stream_k) e = launch_attend_tc_stream(p, tc_stream_ctas(), base + kHeaderBytes, flags, cs);
        else e = launch_attend_tc(p, flags, cs);
        merge_kernel = false;
    } else if (want != PATH_SIMT && mma_path_supports(p, L->dtype)) {
        t_last_path = "mma";
        e = launch_attend_mma(p, cs);
    } else {
        t_last_path = "simt";
        e = launch_attend_simt(p, L->dtype, cs);
    }
    if (e != cudaSuccess) return ORTHRUS_ERR_CUDA;
    if (merge_kernel) {
        e = launch_combine(p, L->dtype, cs);
        if (e != cudaSuccess) return ORTHRUS_ERR_CUDA;
    }
    return ORTHRUS_OK;
}

}  // namespace orthrus

using namespace orthrus;

extern "C" {

size_t orthrus_attend_workspace_bytes(const orthrus_layer_t *layer)
{
    if (check_layer(layer) != ORTHRUS_OK) return 0;
    // enough for whichever kernel path a later call resolves to
    size_t need = partial_bytes(layer, make_plan(layer, false), nullptr, false);
    if (tc_usable(layer)) {
        const size_t n2 = partial_bytes(layer, make_plan(layer, true), nullptr, true);
        if (n2 > need) need = n2;
        if (tc_use_stream(layer)) {
            const size_t n3 = tc_stream_workspace_bytes(layer->batch, layer->n_kv_heads, tc_stream_ctas());
            if (n3 > need) need = n3;
        }
    }
    return kHeaderBytes + need;
}

orthrus_status_t orthrus_workspace_init(void *workspace, size_t workspace_bytes, void *stream)
{
    if (!workspace || workspace_bytes < (size_t)kHeaderBytes) return ORTHRUS_ERR_INVALID_ARG;
    // all of it: besides the status word, the arrival counters some kernels keep there must start at zero
    return cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

orthrus_status_t orthrus_diffusion_block_attend(const orthrus_layer_t *layer, const void *q_diff,
        const void *k_diff_blk, const void *v_diff_blk, void *out, void *workspace,
        size_t workspace_bytes, void *stream)
{
    return attend(layer, 0, q_diff, k_diff_blk, v_diff_blk, out, workspace, workspace_bytes, stream);
}

orthrus_status_t orthrus_ar_verify_attend(const orthrus_layer_t *layer, const void *q_ar,
        const void *k_ar_blk, const void *v_ar_blk, void *out, void *workspace,
        size_t workspace_bytes, void *stream)
{
    return attend(layer, 1, q_ar, k_ar_blk, v_ar_blk, out, workspace, workspace_bytes, stream);
}

// Eq. 6 as a batch of blocks: the descriptor of S sequences becomes one of S * n_blocks batch
// entries whose prefix lengths are the anchors; entry b reads the cache of sequence b / n_blocks.
static bool multi_block_layer(const orthrus_layer_t *layer, int32_t n_blocks, const int32_t *anchors,
                              orthrus_layer_t *out)
{
    if (!layer || n_blocks < 1 || layer->batch < 1 || (long long)layer->batch * n_blocks > 0x7fffffffLL) return false;
    *out = *layer;
    out->batch = layer->batch * n_blocks;
    out->cache_len = const_cast<int32_t *>(anchors);
    out->flags = layer->flags & ~(uint32_t)ORTHRUS_LAYER_BLOCK_IN_CACHE;
    return true;
}

// The packed form of Eq. 6 (tcgen05 path): the blocks of a sequence share 128-row query tiles, so
// the prefix is streamed once per tile instead of once per block.  Taken when at least two blocks
// fit one tile; ORTHRUS_MULTI_BLOCK_PACK=0 keeps the one-unit-per-block form (a measurement knob).
static bool multi_block_packed(const orthrus_layer_t *layer, int32_t n_blocks)
{
    if (n_blocks < 2 || check_layer(layer) != ORTHRUS_OK || !tc_usable(layer)) return false;
    const int want = current_path();
    if (want != PATH_AUTO && want != PATH_TCGEN05) return false;
    if (2 * (layer->n_q_heads / layer->n_kv_heads) * layer->block > 128) return false;
    if ((long long)n_blocks * layer->block > (1 << 20)) return false;
    const char *e = getenv("ORTHRUS_MULTI_BLOCK_PACK");
    return !(e && e[0] == '0');
}

// the descriptor the packed form plans with: one "block" of n_blocks * K positions per sequence
static orthrus_layer_t packed_layer(const orthrus_layer_t *layer, int32_t n_blocks)
{
    orthrus_layer_t L = *layer;
    L.max_len_hint = max_len_of(layer);
    L.block = n_blocks * layer->block;
    L.flags = layer->flags & ~(uint32_t)ORTHRUS_LAYER_BLOCK_IN_CACHE;
    return L;
}

static orthrus_status_t attend_packed(const orthrus_layer_t *layer, int32_t n_blocks, const int32_t *anchors,
                                      const void *q, const void *k_blk, const void *v_blk, void *out,
                                      void *ws, size_t ws_bytes, void *stream)
{
    if (!q || !k_blk || !v_blk || !out || !ws || !layer->k_cache || !layer->v_cache) return ORTHRUS_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out) || !aligned16(ws) ||
        !aligned16(layer->k_cache) || !aligned16(layer->v_cache) || (reinterpret_cast<uintptr_t>(anchors) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    const orthrus_layer_t L = packed_layer(layer, n_blocks);
    const Plan pl = make_plan(&L, true);
    size_t ml_off = 0;
    if (ws_bytes < kHeaderBytes + partial_bytes(&L, pl, &ml_off, true)) return ORTHRUS_ERR_WORKSPACE;

    AttnParams p;
    p.q = q; p.k_blk = k_blk; p.v_blk = v_blk; p.k_cache = layer->k_cache; p.v_cache = layer->v_cache;
    p.cache_len = anchors; p.out = out;
    unsigned char *base = static_cast<unsigned char *>(ws);
    p.status = reinterpret_cast<int32_t *>(base);
    p.part_o = reinterpret_cast<float *>(base + kHeaderBytes);
    p.part_ml = reinterpret_cast<float *>(base + kHeaderBytes + ml_off);
    p.B = layer->batch; p.K = L.block; p.Hq = layer->n_q_heads; p.Hkv = layer->n_kv_heads;
    p.G = p.Hq / p.Hkv; p.M = p.G * p.K; p.d = layer->head_dim; p.capacity = layer->capacity;
    p.chunk = pl.chunk; p.n_splits = pl.n_splits; p.causal = 0; p.blk_in_cache = 0;
    p.nb = n_blocks; p.kb_width = layer->block; p.len_cap = layer->capacity - layer->block;
    const float scale = layer->softmax_scale > 0.f ? layer->softmax_scale : 1.f / sqrtf((float)p.d);
    p.scale_log2 = scale * 1.4426950408889634f;
    t_last_path = "tcgen05";
    int flags = (int)(layer->flags & (ORTHRUS_LAYER_CACHE_QUIESCENT | ORTHRUS_LAYER_NO_EARLY_LAUNCH));
    if (env_int("ORTHRUS_NO_EARLY_LAUNCH", 0)) flags |= ORTHRUS_LAYER_NO_EARLY_LAUNCH;
    return launch_attend_tc_packed(p, flags, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

size_t orthrus_multi_block_workspace_bytes(const orthrus_layer_t *layer, int32_t n_blocks)
{
    orthrus_layer_t L;
    if (!multi_block_layer(layer, n_blocks, nullptr, &L)) return 0;
    // enough for either form
    size_t need = orthrus_attend_workspace_bytes(&L);
    if (need && check_layer(layer) == ORTHRUS_OK && tc_usable(layer) && n_blocks >= 2 &&
        (long long)n_blocks * layer->block <= (1 << 20)) {
        const orthrus_layer_t Lp = packed_layer(layer, n_blocks);
        const size_t n2 = kHeaderBytes + partial_bytes(&Lp, make_plan(&Lp, true), nullptr, true);
        if (n2 > need) need = n2;
    }
    return need;
}

orthrus_status_t orthrus_multi_block_attend(const orthrus_layer_t *layer, int32_t n_blocks,
        const int32_t *anchors, const void *q_diff, const void *k_diff_blk, const void *v_diff_blk,
        void *out, void *workspace, size_t workspace_bytes, void *stream)
{
    orthrus_layer_t L;
    if (!anchors || !multi_block_layer(layer, n_blocks, anchors, &L)) return ORTHRUS_ERR_INVALID_ARG;
    if (layer->flags & ORTHRUS_LAYER_BLOCK_IN_CACHE) return ORTHRUS_ERR_INVALID_ARG;
    if (multi_block_packed(layer, n_blocks))
        return attend_packed(layer, n_blocks, anchors, q_diff, k_diff_blk, v_diff_blk, out, workspace,
                             workspace_bytes, stream);
    return attend(&L, 0, q_diff, k_diff_blk, v_diff_blk, out, workspace, workspace_bytes, stream, n_blocks);
}

size_t orthrus_consensus_workspace_bytes(int32_t batch, int32_t block, int32_t vocab)
{
    if (batch < 1 || block < 1 || vocab < 1) return 0;
    return kHeaderBytes + (size_t)batch * block * consensus_segments(batch, block, vocab) * 8;
}

orthrus_status_t orthrus_consensus_accept(const void *ar_logits, int32_t dtype, const int32_t *draft,
        int32_t batch, int32_t block, int32_t vocab, int32_t *n_commit, int32_t *committed,
        int32_t *ar_argmax, int32_t *next_anchor, void *workspace, size_t workspace_bytes,
        void *stream)
{
    if (batch < 1 || block < 1 || vocab < 1) return ORTHRUS_ERR_INVALID_ARG;
    if (dtype != ORTHRUS_BF16 && dtype != ORTHRUS_FP32) return ORTHRUS_ERR_UNSUPPORTED;
    if (block > 1024 || (long long)batch * block > 65535) return ORTHRUS_ERR_UNSUPPORTED;
    if (!ar_logits || !draft || !n_commit || !committed || !ar_argmax || !next_anchor || !workspace)
        return ORTHRUS_ERR_INVALID_ARG;
    const size_t es = dtype == ORTHRUS_FP32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(ar_logits) & (es - 1)) || !aligned16(workspace) ||
        ((reinterpret_cast<uintptr_t>(draft) | reinterpret_cast<uintptr_t>(n_commit) |
          reinterpret_cast<uintptr_t>(committed) | reinterpret_cast<uintptr_t>(ar_argmax) |
          reinterpret_cast<uintptr_t>(next_anchor)) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    if (workspace_bytes < orthrus_consensus_workspace_bytes(batch, block, vocab))
        return ORTHRUS_ERR_WORKSPACE;
    const int n_seg = consensus_segments(batch, block, vocab);
    cudaError_t e = launch_consensus(ar_logits, dtype, draft, batch, block, vocab, n_commit, committed,
                                     ar_argmax, next_anchor,
                                     static_cast<unsigned char *>(workspace) + kHeaderBytes, n_seg,
                                     static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

size_t orthrus_consensus_sample_workspace_bytes(int32_t batch, int32_t block, int32_t vocab)
{
    if (batch < 1 || block < 1 || vocab < 1) return 0;
    return kHeaderBytes + sample_workspace_bytes(batch, block, vocab);
}

orthrus_status_t orthrus_consensus_sample(const void *ar_logits, const void *diff_logits, int32_t dtype,
        const int32_t *draft, const float *u_accept, const float *u_resample, float temperature,
        int32_t batch, int32_t block, int32_t vocab, int32_t *n_commit, int32_t *committed,
        int32_t *next_anchor, void *workspace, size_t workspace_bytes, void *stream)
{
    if (batch < 1 || block < 1 || vocab < 1 || !(temperature > 0.f) || std::isinf(temperature))
        return ORTHRUS_ERR_INVALID_ARG;
    if (dtype != ORTHRUS_BF16 && dtype != ORTHRUS_FP32) return ORTHRUS_ERR_UNSUPPORTED;
    if (block > 1024 || (long long)batch * block > 65535) return ORTHRUS_ERR_UNSUPPORTED;
    if (!ar_logits || !diff_logits || !draft || !u_accept || !u_resample || !n_commit || !committed ||
        !next_anchor || !workspace)
        return ORTHRUS_ERR_INVALID_ARG;
    const size_t es = dtype == ORTHRUS_FP32 ? 4 : 2;
    if (((reinterpret_cast<uintptr_t>(ar_logits) | reinterpret_cast<uintptr_t>(diff_logits)) & (es - 1)) ||
        !aligned16(workspace) ||
        ((reinterpret_cast<uintptr_t>(draft) | reinterpret_cast<uintptr_t>(u_accept) |
          reinterpret_cast<uintptr_t>(u_resample) | reinterpret_cast<uintptr_t>(n_commit) |
          reinterpret_cast<uintptr_t>(committed) | reinterpret_cast<uintptr_t>(next_anchor)) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    if (workspace_bytes < orthrus_consensus_sample_workspace_bytes(batch, block, vocab))
        return ORTHRUS_ERR_WORKSPACE;
    cudaError_t e = launch_consensus_sample(ar_logits, diff_logits, dtype, draft, u_accept, u_resample,
                                            temperature, batch, block, vocab, n_commit, committed, next_anchor,
                                            static_cast<unsigned char *>(workspace) + kHeaderBytes,
                                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

orthrus_status_t orthrus_consensus_accept_static(const void *ar_logits, int32_t dtype,
        const int32_t *draft, int32_t batch, int32_t block, int32_t vocab, int32_t *n_commit,
        int32_t *committed, int32_t *ar_argmax, int32_t *next_anchor, void *stream)
{
    if (batch < 1 || block < 1 || vocab < 1) return ORTHRUS_ERR_INVALID_ARG;
    if (dtype != ORTHRUS_BF16 && dtype != ORTHRUS_FP32) return ORTHRUS_ERR_UNSUPPORTED;
    if (block > 1024 || (long long)batch * block > 65535) return ORTHRUS_ERR_UNSUPPORTED;
    if (!ar_logits || !draft || !n_commit || !committed || !ar_argmax || !next_anchor)
        return ORTHRUS_ERR_INVALID_ARG;
    const size_t es = dtype == ORTHRUS_FP32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(ar_logits) & (es - 1)) ||
        ((reinterpret_cast<uintptr_t>(draft) | reinterpret_cast<uintptr_t>(n_commit) |
          reinterpret_cast<uintptr_t>(committed) | reinterpret_cast<uintptr_t>(ar_argmax) |
          reinterpret_cast<uintptr_t>(next_anchor)) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    // the built-in scratch has a fixed size: larger problems need the workspace variant
    if (static_consensus_scratch_needed(batch, block, vocab) > (size_t)ORTHRUS_STATIC_CONSENSUS_SCRATCH_BYTES)
        return ORTHRUS_ERR_WORKSPACE;
    cudaError_t e = launch_consensus_static(ar_logits, dtype, draft, batch, block, vocab, n_commit,
                                            committed, ar_argmax, next_anchor,
                                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

size_t orthrus_lm_head_consensus_workspace_bytes(int32_t batch, int32_t block, int32_t vocab)
{
    if (batch < 1 || block < 1 || vocab < 1) return 0;
    return kHeaderBytes + (size_t)batch * block * lm_head_max_vocab_tiles(vocab) * sizeof(ArgPart);
}

orthrus_status_t orthrus_lm_head_consensus(const void *hidden, const void *lm_head, int32_t dtype,
        int32_t hidden_dim, const int32_t *draft, int32_t batch, int32_t block, int32_t vocab,
        int32_t *n_commit, int32_t *committed, int32_t *ar_argmax, int32_t *next_anchor,
        void *workspace, size_t workspace_bytes, void *stream)
{
    if (batch < 1 || block < 1 || vocab < 1 || hidden_dim < 1) return ORTHRUS_ERR_INVALID_ARG;
    if (dtype != ORTHRUS_BF16) return ORTHRUS_ERR_UNSUPPORTED;
    if (block > 1024 || (long long)batch * block > 65535 || vocab > (1 << 24) || (hidden_dim & 7))
        return ORTHRUS_ERR_UNSUPPORTED;
    if (!hidden || !lm_head || !draft || !n_commit || !committed || !ar_argmax || !next_anchor || !workspace)
        return ORTHRUS_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(lm_head) || !aligned16(workspace) ||
        ((reinterpret_cast<uintptr_t>(draft) | reinterpret_cast<uintptr_t>(n_commit) |
          reinterpret_cast<uintptr_t>(committed) | reinterpret_cast<uintptr_t>(ar_argmax) |
          reinterpret_cast<uintptr_t>(next_anchor)) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    if (workspace_bytes < orthrus_lm_head_consensus_workspace_bytes(batch, block, vocab))
        return ORTHRUS_ERR_WORKSPACE;
    if (!lm_head_supported()) return ORTHRUS_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    ArgPart *parts = reinterpret_cast<ArgPart *>(static_cast<unsigned char *>(workspace) + kHeaderBytes);
    cudaError_t e = launch_lm_head_argmax(hidden, lm_head, batch * block, vocab, hidden_dim, parts,
                                          static_cast<int32_t *>(workspace), st);
    if (e == cudaErrorNotSupported) return ORTHRUS_ERR_UNSUPPORTED;
    if (e == cudaSuccess)
        e = launch_consensus_finalize_wide(parts, lm_head_vocab_tiles(batch * block, vocab), draft, batch, block, n_commit,
                                           committed, ar_argmax, next_anchor, st);
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

orthrus_status_t orthrus_kv_append(const orthrus_layer_t *layer, const void *k_ar_blk,
        const void *v_ar_blk, const int32_t *n_commit, int32_t update_len, void *workspace,
        size_t workspace_bytes, void *stream)
{
    orthrus_status_t st = check_layer(layer);
    if (st != ORTHRUS_OK) return st;
    if (!k_ar_blk || !v_ar_blk || !n_commit || !layer->k_cache || !layer->v_cache || !layer->cache_len)
        return ORTHRUS_ERR_INVALID_ARG;
    if (!aligned16(k_ar_blk) || !aligned16(v_ar_blk) || !aligned16(layer->k_cache) ||
        !aligned16(layer->v_cache) || (reinterpret_cast<uintptr_t>(n_commit) & 3) ||
        (reinterpret_cast<uintptr_t>(layer->cache_len) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    if (workspace && (workspace_bytes < (size_t)kHeaderBytes || !aligned16(workspace)))
        return ORTHRUS_ERR_WORKSPACE;
    cudaError_t e = launch_kv_append(*layer, k_ar_blk, v_ar_blk, n_commit, update_len,
                                     static_cast<int32_t *>(workspace),
                                     static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

static orthrus_status_t check_block_call(const orthrus_layer_t *layer, void *workspace, size_t workspace_bytes)
{
    const orthrus_status_t st = check_layer(layer);
    if (st != ORTHRUS_OK) return st;
    if (!layer->k_cache || !layer->v_cache || !layer->cache_len) return ORTHRUS_ERR_INVALID_ARG;
    if (!aligned16(layer->k_cache) || !aligned16(layer->v_cache) ||
        (reinterpret_cast<uintptr_t>(layer->cache_len) & 3))
        return ORTHRUS_ERR_INVALID_ARG;
    if (workspace && (workspace_bytes < (size_t)kHeaderBytes || !aligned16(workspace)))
        return ORTHRUS_ERR_WORKSPACE;
    return ORTHRUS_OK;
}

orthrus_status_t orthrus_block_kv_write(const orthrus_layer_t *layer, const void *k_blk, const void *v_blk,
        void *workspace, size_t workspace_bytes, void *stream)
{
    const orthrus_status_t st = check_block_call(layer, workspace, workspace_bytes);
    if (st != ORTHRUS_OK) return st;
    if (!k_blk || !v_blk || !aligned16(k_blk) || !aligned16(v_blk)) return ORTHRUS_ERR_INVALID_ARG;
    cudaError_t e = launch_block_kv_write(*layer, k_blk, v_blk, static_cast<int32_t *>(workspace),
                                          static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

orthrus_status_t orthrus_commit_len(const orthrus_layer_t *layer, const int32_t *n_commit,
        void *workspace, size_t workspace_bytes, void *stream)
{
    const orthrus_status_t st = check_block_call(layer, workspace, workspace_bytes);
    if (st != ORTHRUS_OK) return st;
    if (!n_commit || (reinterpret_cast<uintptr_t>(n_commit) & 3)) return ORTHRUS_ERR_INVALID_ARG;
    cudaError_t e = launch_commit_len(*layer, n_commit, static_cast<int32_t *>(workspace),
                                      static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

orthrus_status_t orthrus_rope_block_kv_write(const orthrus_layer_t *layer, const void *q, const void *k_blk,
        const void *v_blk, float rope_theta, void *q_out, void *workspace, size_t workspace_bytes, void *stream)
{
    const orthrus_status_t st = check_block_call(layer, workspace, workspace_bytes);
    if (st != ORTHRUS_OK) return st;
    if (!q || !k_blk || !v_blk || !q_out || !aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) ||
        !aligned16(q_out) || !(rope_theta > 0.f) || std::isinf(rope_theta))
        return ORTHRUS_ERR_INVALID_ARG;
    cudaError_t e = launch_rope_block_kv_write(*layer, q, k_blk, v_blk, (double)rope_theta, q_out,
                                               static_cast<int32_t *>(workspace),
                                               static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

orthrus_status_t orthrus_kv_append_layers(const orthrus_layer_t *layers, int32_t n_layers,
        const void *const *k_ar_blks, const void *const *v_ar_blks, const int32_t *n_commit,
        int32_t update_len, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!layers || !k_ar_blks || !v_ar_blks || !n_commit || n_layers < 1 || n_layers > 128)
        return ORTHRUS_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(n_commit) & 3) return ORTHRUS_ERR_INVALID_ARG;
    if (workspace && (workspace_bytes < (size_t)kHeaderBytes || !aligned16(workspace)))
        return ORTHRUS_ERR_WORKSPACE;
    AppendLayer al[128];
    int32_t *lens[128];
    int n_lens = 0;
    const orthrus_layer_t &L0 = layers[0];
    for (int l = 0; l < n_layers; ++l) {
        const orthrus_layer_t &L = layers[l];
        const orthrus_status_t st = check_layer(&L);
        if (st != ORTHRUS_OK) return st;
        if (L.batch != L0.batch || L.n_kv_heads != L0.n_kv_heads || L.head_dim != L0.head_dim ||
            L.block != L0.block || L.dtype != L0.dtype || L.capacity != L0.capacity)
            return ORTHRUS_ERR_INVALID_ARG;
        if (!k_ar_blks[l] || !v_ar_blks[l] || !L.k_cache || !L.v_cache || !L.cache_len)
            return ORTHRUS_ERR_INVALID_ARG;
        if (!aligned16(k_ar_blks[l]) || !aligned16(v_ar_blks[l]) || !aligned16(L.k_cache) ||
            !aligned16(L.v_cache) || (reinterpret_cast<uintptr_t>(L.cache_len) & 3))
            return ORTHRUS_ERR_INVALID_ARG;
        al[l] = AppendLayer{L.k_cache, L.v_cache, k_ar_blks[l], v_ar_blks[l], L.cache_len};
        bool seen = false;
        for (int j = 0; j < n_lens; ++j) seen |= lens[j] == L.cache_len;
        if (!seen) lens[n_lens++] = L.cache_len;
    }
    cudaError_t e = launch_kv_append_layers(L0, al, n_layers, lens, update_len ? n_lens : 0, n_commit,
                                            static_cast<int32_t *>(workspace),
                                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? ORTHRUS_OK : ORTHRUS_ERR_CUDA;
}

orthrus_status_t orthrus_read_status(const void *workspace, void *stream, int32_t *host_status)
{
    if (!workspace || !host_status) return ORTHRUS_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(host_status, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, cs) != cudaSuccess)
        return ORTHRUS_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return ORTHRUS_ERR_CUDA;
    return (*host_status & ORTHRUS_DEV_WAIT_TIMEOUT) ? ORTHRUS_ERR_TIMEOUT : ORTHRUS_OK;
}

orthrus_status_t orthrus_set_path(const char *name)
{
    const int v = parse_path(name);
    if (v < 0) return ORTHRUS_ERR_INVALID_ARG;
    g_path.store(v);
    return ORTHRUS_OK;
}

const char *orthrus_last_path(void) { return t_last_path; }

int64_t orthrus_launch_count(void) { return g_launches.load(); }

const char *orthrus_status_string(orthrus_status_t status)
{
    switch (status) {
    case ORTHRUS_OK: return "ok";
    case ORTHRUS_ERR_INVALID_ARG: return "invalid argument";
    case ORTHRUS_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case ORTHRUS_ERR_CAPACITY: return "block does not fit in the cache capacity";
    case ORTHRUS_ERR_WORKSPACE: return "workspace too small";
    case ORTHRUS_ERR_CUDA: return "CUDA runtime error";
    case ORTHRUS_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    }
    return "unknown status";
}

int32_t orthrus_version(void) { return 200; }

}  // extern "C"
