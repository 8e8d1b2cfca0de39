// Persistent form of the tcgen05 block-attention kernel for batches of many units (included
// by attend_tc.cu inside its unnamed namespace; it uses that file's Shape<1>, constants and
// PTX wrappers).
//
// Why.  With more units than CTA slots the cluster kernel runs in waves: 512 CTAs on 296 slots
// leave the second wave three quarters full, and a ragged batch finishes unevenly on top of
// that.  Here the grid is one CTA per slot and the work is cut by tiles, not by units: the
// units' 64-position tiles (prefix tiles, then the block tile), units ordered longest sequence
// first, form one sequence of T tiles, and CTA c of G takes tiles [c*T/G, (c+1)*T/G).  A CTA
// walks its range as a list of pieces (unit, first tile, last tile): at most two of them are cut
// (the first and the last), the ones in between are whole units.
//
// Status: parity-tested, but measured slower than the cluster kernel on the ragged serving batch
// it was written for (122 us against 109 us per call in one run: what the even cut wins is lost
// again to the refill of the pipeline at every piece boundary and to the merges, each done by one
// CTA alone), and far slower for few long units, whose many pieces one CTA merges.  It is therefore
// selected only by ORTHRUS_TC_SCHEDULE=stream.
//
// A whole unit is normalised and written straight from TMEM.  A cut piece is stored as a partial
// result (max, sum, unnormalised O; chunk-major, as in the cluster kernel) into one of the CTA's
// two slots of the workspace, then the CTA counts itself in on the unit's counter; the CTA that
// arrives last merges all pieces of the unit (they belong to consecutive CTAs) and clears the
// counter.  Nobody waits for anybody: no cluster, no spinning.  While the softmax warps of the last
// arriver merge, the producer and the MMA warp already work on the CTA's next piece.
//
// Barriers carry running counts across pieces: ring items and key tiles are numbered through the
// whole CTA, so slot and phase of every wait follow from one counter.  Per piece there are three
// more hand-overs: QFULL (the piece's query rows have landed), QFREE (the last QK^T of the piece
// has retired: the query area may be overwritten) and OFREE (the softmax threads have read the
// piece's output accumulator: the first P.V of the next piece may clear it).
//
// Restrictions (the host falls back to the cluster kernel otherwise): one 128-row query tile per
// unit, at most 128 batch entries (their lengths are ranked in shared memory).

constexpr int STREAM_MAX_B = 128;
// extra barriers of the persistent kernel, behind those of Shape<1>
constexpr int SBAR_QFREE = Shape<1>::NUM_BARS, SBAR_OFREE = SBAR_QFREE + 1, SBAR_NUM = SBAR_OFREE + 1;
static_assert(SBAR_NUM <= 24, "the barrier area's last 128 bytes hold the ranking");
// Two CTAs per SM leave 640 bytes beside Shape<1>'s map: the ranked sequences go into the unused
// end of the barrier area, the flag into the spare words next to the TMEM address, the tile
// counts behind the map.
constexpr int SOFF_SEQ = Shape<1>::OFF_BAR + 24 * 8;             // uint8 [128]: sequence of rank r
constexpr int SOFF_FLAG = Shape<1>::OFF_MISC + 24;               // int: "this CTA arrived last"
constexpr int SOFF_CUM = Shape<1>::SMEM_BYTES;                   // int [129]: tiles per KV head before rank r
constexpr int STREAM_SMEM_BYTES = SOFF_CUM + ((STREAM_MAX_B + 1) * 4 + 15) / 16 * 16;
static_assert(SOFF_SEQ + STREAM_MAX_B <= Shape<1>::OFF_MISC, "ranking inside the barrier area");
static_assert(2 * (STREAM_SMEM_BYTES + 1024) <= 228 * 1024, "two CTAs per SM");

struct StreamArgs {
    float4 *part_o;        // [G][2] partial tiles, each [32 chunks][128 rows] of 16 bytes
    float2 *part_ml;       // [G][2][128] (max, sum)
    int32_t *counters;     // [B * Hkv] arrivals per unit; zero between calls
};

// first global tile of CTA c when T tiles are cut into G ranges
__device__ inline long long stream_range_start(long long c, long long T, long long G) { return c * T / G; }
// the CTA whose range holds global tile x
__device__ inline int stream_cta_of(long long x, long long T, long long G)
{
    long long c = x * G / T;
    while (c + 1 < G && stream_range_start(c + 1, T, G) <= x) ++c;
    while (c > 0 && stream_range_start(c, T, G) > x) --c;
    return (int)c;
}

// one piece of a CTA's range: tiles [tl0, tl1) of the unit (b, h), whose n tiles start at global
// tile U0; tile n - 1 is the block tile
struct StreamPiece { int b, h, P, tl0, tl1, n, unit; long long U0; };

// Merge of all pieces of one unit by the CTA that arrived last (its softmax warps): tasks of
// (32-row group, 16-byte column chunk), lane = row, contributors folded four at a time with a
// running reference.  Contributor u is CTA c_first + u when every CTA has tiles (T >= G: the CTAs of
// a unit are consecutive), else the CTA of the unit's tile u (fewer tiles than CTAs: one tile each).
// The first contributor's piece starts at the unit's first tile and sits in its slot 1, every
// other piece starts at its CTA's range start and sits in slot 0.  (The 64-bit divisions behind
// stream_cta_of are kept out of the dense case: they would dominate the merge.)
__device__ __noinline__ void stream_merge_unit(const StreamArgs sa, const StreamPiece pc, long long T, long long G,
                                               int c_first, int n_contrib, int rows_here, int warp, int lane,
                                               int n_warps, __nv_bfloat16 *out_tile, int Gq, int Hq)
{
    const bool dense = T >= G;
    const int n_tasks = ((rows_here + 31) >> 5) * (HD / 4);
    for (int task = warp; task < n_tasks; task += n_warps) {
        const int R = (task / (HD / 4)) * 32 + lane, c = task % (HD / 4);
        if (R >= rows_here) continue;
        float m_ref = -INFINITY, L = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int u0 = 0; u0 < n_contrib; u0 += 4) {
            float2 ml[4];
            float4 o[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (u0 + u < n_contrib) {
                    const int cc = dense ? c_first + u0 + u : stream_cta_of(pc.U0 + u0 + u, T, G);
                    const long long slot = (long long)cc * 2 + (u0 + u == 0 ? 1 : 0);
                    ml[u] = __ldcg(sa.part_ml + slot * MROWS + R);
                    o[u] = __ldcg(sa.part_o + slot * (MROWS * HD / 4) + c * MROWS + R);
                }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (u0 + u < n_contrib && ml[u].y > 0.f) {
                    const float m_new = fmaxf(m_ref, ml[u].x);
                    const float a = ex2(m_ref - m_new), w = ex2(ml[u].x - m_new);   // ex2(-inf) = 0
                    L = fmaf(w, ml[u].y, L * a);
                    acc.x = fmaf(w, o[u].x, acc.x * a); acc.y = fmaf(w, o[u].y, acc.y * a);
                    acc.z = fmaf(w, o[u].z, acc.z * a); acc.w = fmaf(w, o[u].w, acc.w * a);
                    m_ref = m_new;
                }
        }
        const float inv = 1.f / L;
        __nv_bfloat16 *row = out_tile + ((long long)(R / Gq) * Hq + R % Gq) * HD;
        reinterpret_cast<uint2 *>(row)[c] =
            make_uint2(pack_bf16(acc.x * inv, acc.y * inv), pack_bf16(acc.z * inv, acc.w * inv));
    }
}

__global__ void __launch_bounds__(Shape<1>::NTHREADS, 2)
attend_tc_stream_kernel(const AttnParams p, const __grid_constant__ TcMaps tm, const StreamArgs sa)
{
    using C = Shape<1>;
    constexpr int W = TN, NSLOT = C::NSLOT, NTHREADS = C::NTHREADS;
    constexpr int OFF_Q = C::OFF_Q, OFF_RING = C::OFF_RING, OFF_BAR = C::OFF_BAR, OFF_MISC = C::OFF_MISC;
    constexpr int BAR_FULL = C::BAR_FULL, BAR_EMPTY = C::BAR_EMPTY, BAR_QFULL = C::BAR_QFULL;
    constexpr int BAR_SFULL = C::BAR_SFULL, BAR_PFULL = C::BAR_PFULL, BAR_PVDONE = C::BAR_PVDONE,
                  BAR_ALLDONE = C::BAR_ALLDONE;
    constexpr uint32_t TM_O = C::tm_o(0);
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t sbase = smem_u32(smem);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + OFF_MISC + 8);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + OFF_MISC);
    unsigned char *s_seq = smem + SOFF_SEQ;
    int *s_cum = reinterpret_cast<int *>(smem + SOFF_CUM);
    volatile int *s_flag = reinterpret_cast<volatile int *>(smem + SOFF_FLAG);
    auto bar = [&](int i) { return sbase + OFF_BAR + i * 8; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rows_here = p.K * p.G;                          // one query tile per unit
    const int n_act = (rows_here + 31) >> 5;                  // softmax warps with rows
    const bool aligned = (sbase & 1023u) == 0;                // swizzled tiles need 1 KB alignment

    // ------------------------------------------------------------------ prologue
    if (tid == 0) *abort_flag = aligned ? 0 : 1;
    if (warp == C::PRODUCER_WARP && lane == 0) {
        for (int i = 0; i < 2 * NSLOT; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(BAR_QFULL), 1);
        for (int sb = 0; sb < 2; ++sb) {
            mbar_init(bar(BAR_SFULL + sb), 1);
            mbar_init(bar(BAR_PFULL + sb), n_act);
        }
        mbar_init(bar(BAR_PVDONE), 1);
        mbar_init(bar(BAR_ALLDONE), 1);
        mbar_init(bar(SBAR_QFREE), 1);
        mbar_init(bar(SBAR_OFREE), n_act);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
        prefetch_map(&tm.k); prefetch_map(&tm.v); prefetch_map(&tm.q);
        prefetch_map(&tm.kb); prefetch_map(&tm.vb);
    } else if (warp == C::MMA_WARP) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_slot)), "r"(C::TM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Nothing written by earlier work of the stream is read before this wait.
    griddep_wait();
    griddep_launch();

    // ------------------------------------------------------------------ the tile sequence
    // sequences ranked longest prefix first (ties by index); per rank its tiles per KV head
    const int len_hi = (int)p.len_cap;
    for (int i = tid; i < p.B; i += NTHREADS) {
        const int raw = p.cache_len[i];
        if ((raw < 0 || raw > len_hi) && blockIdx.x == 0 && p.status) atomicOr(p.status, ORTHRUS_DEV_BAD_CACHE_LEN);
        const int Pi = min(max(raw, 0), len_hi);
        int before = 0;
        for (int j = 0; j < p.B; ++j) {
            const int Pj = min(max(__ldg(p.cache_len + j), 0), len_hi);
            before += (Pj > Pi) || (Pj == Pi && j < i);
        }
        s_seq[before] = (unsigned char)i;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (tid == 0) {
        int cum = 0;
        for (int r = 0; r < p.B; ++r) {
            const int Pr = min(max(p.cache_len[s_seq[r]], 0), len_hi);
            s_cum[r] = cum;
            cum += (Pr + TN - 1) / TN + 1;
        }
        s_cum[p.B] = cum;
    }
    __syncthreads();
    const long long T = (long long)p.Hkv * s_cum[p.B], G = gridDim.x;
    const long long g_begin = stream_range_start(blockIdx.x, T, G), g_end = stream_range_start(blockIdx.x + 1, T, G);
    // every role walks the same pieces with its own cursor (g, r)
    auto next_piece = [&](long long &g, int &r, StreamPiece &pc) -> bool {
        if (g >= g_end) return false;
        while ((long long)p.Hkv * s_cum[r + 1] <= g) ++r;
        const int n = s_cum[r + 1] - s_cum[r];
        const long long within = g - (long long)p.Hkv * s_cum[r];
        pc.n = n; pc.h = (int)(within / n); pc.tl0 = (int)(within % n);
        pc.tl1 = (int)min((long long)n, pc.tl0 + (g_end - g));
        pc.b = s_seq[r]; pc.P = min(max(__ldg(p.cache_len + pc.b), 0), len_hi); pc.unit = r * p.Hkv + pc.h;
        pc.U0 = (long long)p.Hkv * s_cum[r] + (long long)pc.h * n;
        g += pc.tl1 - pc.tl0;
        return true;
    };
    auto item_of_k = [](int t) { return t == 0 ? 0 : 2 * t - 1; };
    const bool active = aligned && g_end > g_begin;

    if (warp < 4) {
        // ------------------------------------------------------------------ softmax, thread = query row
        const int r = tid;
        const bool valid = r < rows_here;
        const bool warp_active = warp * 32 < rows_here;
        const int i_row = r / p.G;
        const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
        const float sc = p.scale_log2;
        const float2 sc2 = make_float2(sc, sc);
        long long g = g_begin;
        int rk = 0, tg0 = 0, pcidx = 0;
        StreamPiece pc;
        bool ok = active && warp_active;
        while (ok && next_piece(g, rk, pc)) {
            const int nt = pc.tl1 - pc.tl0;
            float m_run = -INFINITY, l_run = 0.f;
            for (int t = 0; t < nt; ++t) {
                const int tg = tg0 + t, sb = tg & 1;
                ok = mbar_wait_warp(bar(BAR_SFULL + sb), (tg >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t TM_S = C::tm_s(0, sb);
                uint32_t s[W];
#pragma unroll
                for (int c = 0; c < W / 32; ++c) tmem_ld32(lane_base + TM_S + c * 32, s + c * 32);
                tmem_ld_wait();
                // visible columns of this row in this tile
                const int ut = pc.tl0 + t;                    // tile of the unit
                int lim;
                if (ut < pc.n - 1) lim = min(TN, pc.P - ut * TN);
                else lim = p.causal ? min(p.K, i_row + 1) : p.K;
                lim = valid ? lim : 0;
                float mx;
                if (lim == W) {
                    float m4[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        m4[q] = max3(__uint_as_float(s[q]), __uint_as_float(s[q + 4]), __uint_as_float(s[q + 8]));
#pragma unroll
                    for (int j = 12; j + 8 <= W; j += 8)
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            m4[q] = max3(m4[q], __uint_as_float(s[j + q]), __uint_as_float(s[j + q + 4]));
#pragma unroll
                    for (int q = 0; q < 4; ++q) m4[q] = fmaxf(m4[q], __uint_as_float(s[W - 4 + q]));
                    mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                } else {
                    mx = -INFINITY;
#pragma unroll
                    for (int c = 0; c < W; c += 16) {
                        if (c < lim) {
#pragma unroll
                            for (int j = c; j < c + 16; ++j) if (j < lim) mx = fmaxf(mx, __uint_as_float(s[j]));
                        }
                    }
                }
                const float m_new = fmaxf(m_run, mx * sc);
                const bool need = m_new > m_run + RESCALE_THRESHOLD;   // also the first finite maximum
                if (__any_sync(0xffffffffu, need)) {
                    const float alpha = need ? ex2(m_run - m_new) : 1.f;
                    if (need) { m_run = m_new; l_run *= alpha; }
                    if (t > 0) {
                        // O holds the products of the piece's tiles 0..t-1 and nothing is adding to it now
                        ok = mbar_wait_warp(bar(BAR_PVDONE), (tg - 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll 1
                        for (int c4 = 0; c4 < HD / 32; ++c4) {
                            uint32_t o[32];
                            tmem_ld32(lane_base + TM_O + c4 * 32, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                            tmem_st32(lane_base + TM_O + c4 * 32, o);
                        }
                    }
                }
                const float neg_m = (m_run == -INFINITY) ? 0.f : -m_run;
                const float2 nm2 = make_float2(neg_m, neg_m);
                uint32_t pk[W / 2];
                float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
                if (lim == W) {
#pragma unroll
                    for (int j = 0; j < W; j += 4) {
                        float2 a = __ffma2_rn(make_float2(__uint_as_float(s[j]), __uint_as_float(s[j + 1])), sc2, nm2);
                        float2 c = __ffma2_rn(make_float2(__uint_as_float(s[j + 2]), __uint_as_float(s[j + 3])), sc2, nm2);
                        a.x = ex2(a.x); a.y = ex2(a.y); c.x = ex2(c.x); c.y = ex2(c.y);
                        acc0 = __fadd2_rn(acc0, a);
                        acc1 = __fadd2_rn(acc1, c);
                        pk[j >> 1] = pack_bf16(a.x, a.y);
                        pk[(j >> 1) + 1] = pack_bf16(c.x, c.y);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < W; c += 16) {
                        if (c < lim) {
#pragma unroll
                            for (int j = c; j < c + 16; j += 2) {
                                float p0 = ex2(fmaf(__uint_as_float(s[j]), sc, neg_m));
                                float p1 = ex2(fmaf(__uint_as_float(s[j + 1]), sc, neg_m));
                                if (j >= lim) p0 = 0.f;
                                if (j + 1 >= lim) p1 = 0.f;
                                acc0.x += p0; acc0.y += p1;
                                pk[j >> 1] = pack_bf16(p0, p1);
                            }
                        } else {
#pragma unroll
                            for (int j = c; j < c + 16; j += 2) pk[j >> 1] = 0u;
                        }
                    }
                }
                l_run += (acc0.x + acc0.y) + (acc1.x + acc1.y);
                tmem_st32(lane_base + TM_S, pk);
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_PFULL + sb));
            }
            if (ok) ok = mbar_wait_warp(bar(BAR_ALLDONE), pcidx & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // the piece's accumulator row into registers; then the MMA warp may clear the accumulator
            uint32_t o[HD];
#pragma unroll
            for (int c4 = 0; c4 < HD / 32; ++c4) tmem_ld32(lane_base + TM_O + c4 * 32, o + c4 * 32);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(SBAR_OFREE));
            __nv_bfloat16 *out_tile = static_cast<__nv_bfloat16 *>(p.out) +
                                      ((long long)pc.b * p.K * p.Hq + pc.h * p.G) * HD;
            if (pc.tl0 == 0 && pc.tl1 == pc.n) {
                // the whole unit was here: normalise and write the final row
                if (valid) {
                    const float inv = 1.f / l_run;
                    uint4 *dst = reinterpret_cast<uint4 *>(out_tile + ((long long)i_row * p.Hq + r % p.G) * HD);
#pragma unroll
                    for (int c = 0; c < HD / 8; ++c) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(o[c * 8 + 0]) * inv, __uint_as_float(o[c * 8 + 1]) * inv);
                        w.y = pack_bf16(__uint_as_float(o[c * 8 + 2]) * inv, __uint_as_float(o[c * 8 + 3]) * inv);
                        w.z = pack_bf16(__uint_as_float(o[c * 8 + 4]) * inv, __uint_as_float(o[c * 8 + 5]) * inv);
                        w.w = pack_bf16(__uint_as_float(o[c * 8 + 6]) * inv, __uint_as_float(o[c * 8 + 7]) * inv);
                        dst[c] = w;
                    }
                }
            } else {
                // a cut piece: partial row to this CTA's slot, chunk-major (a warp stores 512 contiguous bytes)
                const long long slot = (long long)blockIdx.x * 2 + (pc.tl0 > 0 ? 0 : 1);
                if (valid) {
                    float4 *my_o = sa.part_o + slot * (MROWS * HD / 4);
#pragma unroll
                    for (int c = 0; c < HD / 4; ++c)
                        __stcg(my_o + c * MROWS + r,
                               make_float4(__uint_as_float(o[c * 4]), __uint_as_float(o[c * 4 + 1]),
                                           __uint_as_float(o[c * 4 + 2]), __uint_as_float(o[c * 4 + 3])));
                    __stcg(sa.part_ml + slot * MROWS + r, make_float2(m_run, l_run));
                }
                __threadfence();                              // this thread's stores before the arrival below
                named_bar_sync(1, n_act * 32);
                if (tid == 0) {
                    // CTAs that hold tiles of this unit: consecutive ones when every CTA has tiles, else
                    // one per tile
                    const int c_first = stream_cta_of(pc.U0, T, G);
                    const int n_contrib = T >= G ? stream_cta_of(pc.U0 + pc.n - 1, T, G) - c_first + 1 : pc.n;
                    const int old = atomicAdd(sa.counters + pc.unit, 1);
                    s_flag[0] = (old == n_contrib - 1);
                    s_flag[1] = c_first;
                    s_flag[2] = n_contrib;
                }
                named_bar_sync(1, n_act * 32);
                if (s_flag[0]) {
                    // every other piece of the unit is in place: merge, write, leave the counter at zero
                    __threadfence();
                    stream_merge_unit(sa, pc, T, G, s_flag[1], s_flag[2], rows_here, warp, lane, n_act, out_tile,
                                      p.G, p.Hq);
                    if (tid == 0) sa.counters[pc.unit] = 0;
                }
                named_bar_sync(1, n_act * 32);                // (the flag is rewritten by the next cut piece)
            }
            tg0 += nt;
            ++pcidx;
        }
        tc_fence_before();
    } else if (warp == C::PRODUCER_WARP) {
        // ------------------------------------------------------------------ producer
        if (active && lane == 0) {
            const uint64_t stream_policy = policy_evict_first();
            long long g = g_begin;
            int rk = 0, jg = 0, pcidx = 0;
            StreamPiece pc;
            bool ok = true;
            while (ok && next_piece(g, rk, pc)) {
                const int nt = pc.tl1 - pc.tl0, n_items = 2 * nt;
                const int row_base = (int)(((long long)(pc.b / p.nb) * p.Hkv + pc.h) * p.capacity);
                bool q_loaded = false;
                auto load_q = [&]() {
                    // the query rows of the unit: box = 64 columns x G heads x K positions
                    mbar_expect_tx(bar(BAR_QFULL), (uint32_t)(2 * 128 * p.G * p.K));
                    tma_load_4d(sbase + OFF_Q, &tm.q, 0, pc.h * p.G, 0, pc.b, bar(BAR_QFULL));
                    tma_load_4d(sbase + OFF_Q + QSUB_BYTES, &tm.q, 64, pc.h * p.G, 0, pc.b, bar(BAR_QFULL));
                    q_loaded = true;
                };
                for (int jl = 0; jl < n_items && ok; ++jl, ++jg) {
                    // the query area is free once the previous piece's last QK^T has retired; until
                    // then the ring is filled ahead
                    if (!q_loaded && (pcidx == 0 || mbar_try(bar(SBAR_QFREE), (pcidx - 1) & 1))) load_q();
                    const int slot = jg % NSLOT, use = jg / NSLOT;
                    if (use > 0) ok = mbar_wait(bar(BAR_EMPTY + slot), (use - 1) & 1, abort_flag);
                    if (!ok) break;
                    // item jl of the piece, in the order the MMAs consume them: K0, K1, V0, K2, V1, ...
                    const bool is_v = jl == n_items - 1 || (jl > 0 && (jl & 1) == 0);
                    const int t = is_v ? (jl == n_items - 1 ? nt - 1 : jl / 2 - 1) : (jl + 1) / 2;
                    const int ut = pc.tl0 + t;
                    const uint32_t dst = sbase + OFF_RING + slot * SLOT_BYTES;
                    const uint32_t fb = bar(BAR_FULL + slot);
                    mbar_expect_tx(fb, SLOT_BYTES);
                    if (ut < pc.n - 1) {
                        const CUtensorMap *m = is_v ? &tm.v : &tm.k;
                        tma_load_2d(dst, m, 0, row_base + ut * TN, fb, stream_policy);
                        tma_load_2d(dst + SUB_BYTES, m, 64, row_base + ut * TN, fb, stream_policy);
                    } else if (p.blk_in_cache) {
                        const CUtensorMap *m = is_v ? &tm.v : &tm.k;
                        tma_load_2d(dst, m, 0, row_base + pc.P, fb, stream_policy);
                        tma_load_2d(dst + SUB_BYTES, m, 64, row_base + pc.P, fb, stream_policy);
                    } else {              // block tile: rows >= K are out of bounds and arrive as zeros
                        const CUtensorMap *m = is_v ? &tm.vb : &tm.kb;
                        tma_load_4d(dst, m, 0, pc.h, 0, pc.b, fb);
                        tma_load_4d(dst + SUB_BYTES, m, 64, pc.h, 0, pc.b, fb);
                    }
                }
                if (ok && !q_loaded) {
                    ok = pcidx == 0 || mbar_wait(bar(SBAR_QFREE), (pcidx - 1) & 1, abort_flag);
                    if (ok) load_q();
                }
                ++pcidx;
            }
            if (*abort_flag) {
                // give the copies that were armed a bounded time to land before smem is released
                for (int j = max(0, jg - NSLOT); j < jg; ++j) {
                    int dummy = 0;
                    mbar_wait(bar(BAR_FULL + j % NSLOT), (j / NSLOT) & 1, &dummy);
                }
            }
        }
    } else if (active) {
        // ------------------------------------------------------------------ MMA issue
        constexpr uint32_t IDESC_QK = make_idesc(TN, 0);      // A = Q, B = K tile, both K-major
        constexpr uint32_t IDESC_PV = make_idesc(HD, 1);      // A = P (TMEM), B = V tile (MN-major)
        const uint32_t q_addr = sbase + OFF_Q;
        long long g = g_begin;
        int rk = 0, jg0 = 0, tg0 = 0, pcidx = 0;
        StreamPiece pc;
        bool ok = true;
        while (ok && next_piece(g, rk, pc)) {
            const int nt = pc.tl1 - pc.tl0;
            auto issue_qk = [&](int t) -> bool {
                const int j = jg0 + item_of_k(t), slot = j % NSLOT, tg = tg0 + t;
                if (!mbar_wait_warp(bar(BAR_FULL + slot), (j / NSLOT) & 1, abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t k_addr = sbase + OFF_RING + slot * SLOT_BYTES;
#pragma unroll
                    for (int kk = 0; kk < HD / 16; ++kk) {    // 16 head-dim columns per MMA
                        umma_ss(tmem + C::tm_s(0, tg & 1),
                                make_desc(q_addr + (kk >> 2) * QSUB_BYTES + (kk & 3) * 32, 16, 1024),
                                make_desc(k_addr + (kk >> 2) * SUB_BYTES + (kk & 3) * 32, 16, 1024),
                                IDESC_QK, kk > 0);
                    }
                    umma_commit(bar(BAR_EMPTY + slot));
                    umma_commit(bar(BAR_SFULL + (tg & 1)));
                    if (t == nt - 1) umma_commit(bar(SBAR_QFREE));   // the query rows have served this piece
                }
                __syncwarp();
                return true;
            };
            auto issue_pv = [&](int t) -> bool {
                const int j = jg0 + min(2 * t + 2, 2 * nt - 1), slot = j % NSLOT, tg = tg0 + t;
                if (!mbar_wait_warp(bar(BAR_FULL + slot), (j / NSLOT) & 1, abort_flag)) return false;
                // V rows past the prefix (or past the block) may hold anything, and 0 * NaN would poison
                // the product: they are cleared before the MMA reads them
                const int ut = pc.tl0 + t;
                const int nv = ut < pc.n - 1 ? min(TN, pc.P - ut * TN) : (p.blk_in_cache ? p.K : TN);
                if (nv < TN) {
                    unsigned char *vt = smem + OFF_RING + slot * SLOT_BYTES;
                    for (int e = lane; e < (TN - nv) * 16; e += 32) {
                        const int rr = nv + (e >> 4), c = e & 15;
                        *reinterpret_cast<uint4 *>(vt + sw_off(rr, c, SUB_BYTES)) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async();
                    __syncwarp();
                }
                // the first product of a piece clears the accumulator: the previous piece's must have been read
                if (t == 0 && pcidx > 0 && !mbar_wait_warp(bar(SBAR_OFREE), (pcidx - 1) & 1, abort_flag)) return false;
                if (!mbar_wait_warp(bar(BAR_PFULL + (tg & 1)), (tg >> 1) & 1, abort_flag)) return false;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t v_addr = sbase + OFF_RING + slot * SLOT_BYTES;
#pragma unroll
                    for (int kk = 0; kk < TN / 16; ++kk) {    // 16 key positions per MMA
                        umma_ts(tmem + TM_O, tmem + C::tm_s(0, tg & 1) + kk * 8,
                                make_desc(v_addr + kk * 2048, SUB_BYTES, 1024), IDESC_PV, (t > 0) || (kk > 0));
                    }
                    umma_commit(bar(BAR_EMPTY + slot));
                    umma_commit(bar(BAR_PVDONE));
                    if (t == nt - 1) umma_commit(bar(BAR_ALLDONE));
                }
                __syncwarp();
                return true;
            };
            ok = mbar_wait_warp(bar(BAR_QFULL), pcidx & 1, abort_flag);
            if (ok) { tc_fence_after(); ok = issue_qk(0); }
            for (int t = 0; t < nt && ok; ++t) {
                if (t + 1 < nt) ok = issue_qk(t + 1);
                if (ok) ok = issue_pv(t);
            }
            jg0 += 2 * nt;
            tg0 += nt;
            ++pcidx;
        }
        // every MMA must have retired before TMEM is freed
        if (ok && pcidx > 0) mbar_wait_warp(bar(BAR_ALLDONE), (pcidx - 1) & 1, abort_flag);
        tc_fence_before();
    }

    __syncthreads();
    tc_fence_after();
    if (warp == C::MMA_WARP)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TM_COLS) : "memory");
    if (tid == 0 && *abort_flag && p.status) atomicOr(p.status, ORTHRUS_DEV_WAIT_TIMEOUT);
}
