// Block scoring (Eq. 9 / ScoreBlock of Algorithm 1) and exact, ordered top-k selection of
// eviction victims (Evict of Algorithm 1) and prefetch candidates (BetweenStep, Eq. 10-11).
//
// Every kernel that walks the block index reads the SoA metadata in 512-entry warp tiles
// (contiguous 128-, 64- and 32-bit loads; 16 entries per thread and iteration) and the select
// path never materialises the score.
// A positive fp32 score orders like its bit pattern, so each eligible entry has a 96-bit
// integer key (primary, secondary, id) and "the k best in order" is "the k smallest keys in
// ascending order":
//   victims : primary = score bits,                      secondary = last_access
//   prefetch: primary = (not a*)<<31 | ~score bits[30:0], secondary = ~last_access
//
// This file holds the multi-launch path, used for indexes above 262,144 entries (smaller ones take
// the single-launch cluster kernel of cs_select_cluster.cu).  Six launches, none of which waits
// on another CTA:
//   0 fast pass : one scan against the threshold bin remembered from the last call of this kind; when the k
//                 winners lie within it (the usual case) the candidates are complete and launches 1 and 2
//                 return at once.  Its last CTA searches the threshold and sorts the splitter sample side by side.
//   1 histogram : 4096-bin histogram of the top 12 primary bits; the last CTA to finish finds
//                 the threshold bin b0 (first bin whose running count reaches k).
//   2 collect   : every eligible entry whose bin <= b0 is appended to the candidate buffer
//                 (c >= min(k, eligible) keys); the last CTA samples <= 1024 candidates,
//                 sorts them in shared memory and publishes <= 255 splitters.
//   3 bucket    : each candidate finds its bucket by a search over the splitters and takes a slot in it; with few
//                 candidates the key goes straight into the bucket's own fixed-size region.
//   4 scatter   : otherwise the candidates of the needed buckets are grouped by bucket (every CTA derives the
//                 bucket offsets from the 256 counters itself).
//   5 rank      : every needed bucket is sorted by one CTA in a shared-memory tile; bucket offset
//                 + position in the bucket is the position in the output list.
// Keys are unique (the id is part of the key), so the order is total and the output does not
// depend on the order in which atomics were served.
#include "cs_common.cuh"

#include "cs_select_common.cuh"

// ---------------------------------------------------------------------------------------------
// ScoreBlock for every entry (cs_score_blocks).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SEL_THREADS) cs_score_kernel(SelArgs a, cs_workspace ws, float *__restrict__ out)
{
    extern __shared__ float smem[];
    resolve_now(a);
    Tables T;
    load_tables(a, ws, smem, T, false);
    __syncthreads();
    const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    const uint32_t lane = threadIdx.x & 31, n_tiles = a.n / TILE;
    for (uint32_t t = gtid >> 5; t < n_tiles; t += nth >> 5) {
        Group G;
        load_group<false, false>(a, t, lane, G);            // the score needs agent, last_access and size only
        float s[GRP];
#pragma unroll
        for (int j = 0; j < GRP; ++j) {
            const uint32_t ag = grp_u16(G.ag0, G.ag1, j);
            const uint32_t tok = a.ntok ? grp_u8(G.tk, j) : a.block_tokens;
            if (ag < a.A) s[j] = score_of(a, T, ag, grp_u32(G, j), tok);
            else { s[j] = 0.0f; atomicOr(&ws.sc->status, CS_ST_BAD_AGENT); }
        }
        float4 *o = (float4 *)out + t * 128u + lane;         // quad q of this lane: coalesced 512 B per warp store
#pragma unroll
        for (int q = 0; q < 4; ++q) __stcs(o + 32 * q, make_float4(s[4 * q], s[4 * q + 1], s[4 * q + 2], s[4 * q + 3]));
    }
    const uint32_t t0 = n_tiles * TILE;
    if (gtid < a.n - t0) {
        const uint32_t i = t0 + gtid;
        const uint32_t ag = a.agent[i];
        const uint32_t tok = a.ntok ? a.ntok[i] : a.block_tokens;
        if (ag < a.A) out[i] = score_of(a, T, ag, a.la[i], tok);
        else { out[i] = 0.0f; atomicOr(&ws.sc->status, CS_ST_BAD_AGENT); }
    }
}

// ---------------------------------------------------------------------------------------------
// Sample sort set-up, run by one CTA (or half of one) once every candidate is in the buffer: sort P <= 1024 sampled
// keys in shared memory, publish <= 255 splitters, clear the bucket counters, and decide where the buckets will
// live.  When the candidates are few for the size of the sort region (8 c <= its capacity), every bucket gets a
// fixed region of `cap` keys -- at least eight times the mean bucket -- that the bucket launch fills directly.
// P: power of two, 64 <= P <= min(CS_SAMPLE, 2 * threads of the group).
// ---------------------------------------------------------------------------------------------
#define RANK_TILE 2048u                 // keys of the shared-memory tile a bucket is sorted in
#define CS_SPLIT_SAMPLE_MAX 32768u      // up to this many candidates half a CTA sorts a 512-key sample (fast pass)
__device__ __forceinline__ void publish_splitters(const cs_workspace &ws, unsigned long long *s_km, uint32_t *s_id,
                                                  uint32_t c, uint32_t sort_cap, uint32_t region_cap_max, uint32_t P,
                                                  const CtaPart &cp)
{
    const uint32_t n_samp = c < P ? c : P;
    {
        // a group sorts two keys per thread: both are fetched before either is stored
        const uint32_t i0 = cp.t, i1 = cp.t + cp.n;
        unsigned long long k0 = ~0ull, k1 = ~0ull;
        uint32_t d0 = 0xFFFFFFFFu, d1 = 0xFFFFFFFFu;
        if (i0 < n_samp) {
            const uint32_t pos = (uint32_t)(((unsigned long long)i0 * c) / n_samp);
            k0 = __ldcg(&ws.cand_km[pos]);
            d0 = __ldcg(&ws.cand_id[pos]);
        }
        if (i1 < n_samp) {
            const uint32_t pos = (uint32_t)(((unsigned long long)i1 * c) / n_samp);
            k1 = __ldcg(&ws.cand_km[pos]);
            d1 = __ldcg(&ws.cand_id[pos]);
        }
        if (i0 < P) { s_km[i0] = k0; s_id[i0] = d0; }
        if (i1 < P) { s_km[i1] = k1; s_id[i1] = d1; }
    }
    part_sync(cp);
    bitonic_sort_fast(s_km, s_id, P, cp);
    uint32_t n_spl = c / 64;
    if (n_spl > CS_MAX_SPLITTERS) n_spl = CS_MAX_SPLITTERS;
    for (uint32_t j = cp.t; j <= CS_MAX_SPLITTERS; j += cp.n) {
        if (j < n_spl) {
            const uint32_t q = (uint32_t)(((unsigned long long)(j + 1) * n_samp) / (n_spl + 1));
            ws.spl_km[j] = s_km[q];
            ws.spl_id[j] = s_id[q];
        }
        CS_BCOUNT(ws, j) = 0;
    }
    if (cp.t == 0) {
        uint32_t cap = sort_cap / (n_spl + 1u);
        if (cap > RANK_TILE) cap = RANK_TILE;
        if (region_cap_max && cap > region_cap_max) cap = region_cap_max;
        ws.sel->n_spl = n_spl;
        ws.sel->placed = (c && 8ull * c <= sort_cap) ? 1u : 0u;
        ws.sel->cap = cap;
        ws.sel->overflow = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// 0 fast pass (remembered threshold)
//
// The threshold bin moves little from one call to the next, so each kind of call (GPU victims, host
// victims, prefetch) remembers a bin H at or a little above the one it ended with.  With H known, almost
// every eligible entry can be dismissed without its key, in two steps:
//   a  by age alone.  For victims (low scores = old blocks) an entry younger than a cut A_c cannot reach
//      H whatever its agent and size: fl(f_min * g(age)) is already on the far side of the largest per-size
//      threshold X (build_x_thresholds), g never increases with age, and IEEE products are monotone.  That is
//      ONE integer compare on last_access per entry.  For prefetch candidates (high scores = young blocks)
//      the same holds with the roles swapped, for entries of agents other than a*.
//   b  what is left (a few per cent) is queued per warp as entry ids and worked off with all 32 lanes
//      busy: two table look-ups, one multiply and one compare against X decide exactly whether the entry's
//      first key digit is <= H; only then is the key built, binned and appended to the candidate buffer.
// Dismissed entries are only counted.  The last CTA has the exact histogram of bins <= H plus the number
// of entries above: if the k-th smallest key lies within H the candidates are complete, the sample sort is
// set up right here, and the index has been read ONCE at a fraction of the instructions of a full-key
// scan.  Otherwise (the threshold rose above H, or nothing is remembered yet) the pass reports a miss and
// the full histogram and collect passes below run.  The result never depends on H.
// ---------------------------------------------------------------------------------------------
#define FQ_CAP 544u                 // per-warp queue: at most 31 left over + the 512 entries of one warp tile

// Largest value of every 16-bit half over eight packed words.
__device__ __forceinline__ uint32_t max_halves(const uint4 &a, const uint4 &b)
{
    const uint32_t m0 = __vmaxu2(__vmaxu2(a.x, a.y), __vmaxu2(a.z, a.w)), m1 = __vmaxu2(__vmaxu2(b.x, b.y), __vmaxu2(b.z, b.w));
    const uint32_t m = __vmaxu2(m0, m1);
    return max(m & 0xFFFFu, m >> 16);
}

template <bool PF>
__global__ void __launch_bounds__(SEL_THREADS) cs_sel_fast_kernel(SelArgs a, cs_workspace ws)
{
    extern __shared__ float smem[];                 // tables, then the per-warp queues (reused by the epilogue)
    __shared__ __align__(16) uint32_t s_hist[CS_HIST_BINS];   // bins of the candidates (the threshold bin is dense: global
                                                              // atomics on one address per candidate would serialise)
    __shared__ uint32_t s_xt[2 * XT_TOK];
    __shared__ uint32_t s_part[SEL_THREADS];
    __shared__ uint32_t s_b0, s_ahead, s_above;
    __shared__ bool s_flag;
    constexpr int PS = PF ? 8 : 0;                  // phase-stamp slots of this kind of scan (profiling builds)
    CS_STAMP(ws, CS_PS_SCAN_ENTRY + PS, blockIdx.x == 0 && threadIdx.x == 0);
    cs_release_successor();
    // Before waiting for the predecessor grid: everything that depends only on the context's constants and on the
    // remembered bin (a stale bin would cost time, never correctness: the result does not depend on H).
    const uint32_t H = ws.sc->sel_hint[a.hint_slot];        // ~0: nothing remembered
    Tables T;
    const size_t table_words = ((size_t)(a.A + a.gtab_len) * 4 + (size_t)a.A * 2 + 15) / 16 * 4;
    uint32_t *queues = (uint32_t *)smem + table_words;
    const size_t cut_off_words = table_words + (size_t)(SEL_THREADS / 32) * (FQ_CAP + STAGE_CAP * 3) + 4;     // after queues and staging
    if (H != 0xFFFFFFFFu) {
        load_tables_static(a, ws, smem, T);
        build_x_thresholds<PF>(a, H, s_xt);
        for (uint32_t i = threadIdx.x; i < CS_HIST_BINS; i += blockDim.x) s_hist[i] = 0;
        if (threadIdx.x == 0) s_above = 0;
    }
    CS_STAMP(ws, CS_PS_SCAN_SETUP + PS, blockIdx.x == 0 && threadIdx.x == 0);
    cs_wait_for_predecessor();
    CS_STAMP(ws, CS_PS_SCAN_WAITED + PS, blockIdx.x == 0 && threadIdx.x == 0);
    if (H == 0xFFFFFFFFu) {                                   // every CTA sees the same word
        if (blockIdx.x == 0 && threadIdx.x == 0) ws.sel->spec = 0;
        return;
    }
    resolve_now(a);
    load_tables_dynamic(a, ws, T, PF && a.anchor);
    __syncthreads();
    CS_STAMP(ws, CS_PS_SCAN_TABLES + PS / 2, blockIdx.x == 0 && threadIdx.x == 0);
    // ---- the age cuts, one per agent, for blocks of the common size ----------------------------------------
    // victims: s_cut[agent] = number of ages (0, 1, ..) that are dismissed, i.e. for which fl(f g(age)) >= X;
    // prefetch: s_cut[agent] = first age that is dismissed, i.e. fl(f g(age)) < X of the agents other than a*.
    // Both rely on g never increasing with age (checked when the table was built) and on the table covering every
    // unsaturated age; otherwise nothing is dismissed by age and every eligible entry takes the exact test.
    const uint32_t Tb = a.block_tokens;
    uint32_t *s_cut = (uint32_t *)smem + cut_off_words;
    {
        const bool usable = ws.sc->gtab_monotone && a.gtab_len == a.age_sat;
        const uint32_t X = s_xt[(PF ? XT_TOK : 0u) + Tb];
        for (uint32_t e = threadIdx.x; e < a.A; e += blockDim.x) {
            const float f = T.fsurv[e];
            auto dismissed = [&](uint32_t age) {
                const uint32_t xb = __float_as_uint(__fmul_rn(f, recency_of_age(a, T, age)));
                return PF ? (xb < X) : (xb >= X);
            };
            uint32_t cut;
            if (!PF) {
                cut = 0;                                            // none
                if (usable && X != XT_NONE && dismissed(0)) {
                    if (dismissed(a.age_sat)) cut = 0xFFFFFFFFu;    // every age
                    else {
                        uint32_t lo = 0, hi = a.age_sat;            // largest dismissed age
                        while (lo < hi) {
                            const uint32_t mid = lo + ((hi - lo + 1) >> 1);
                            if (dismissed(mid)) lo = mid;
                            else hi = mid - 1;
                        }
                        cut = lo + 1;
                    }
                }
            } else {
                cut = 0xFFFFFFFFu;                                  // none
                if (usable && (X == XT_NONE || dismissed(0))) cut = 0;          // every age
                else if (usable && dismissed(a.age_sat)) {
                    uint32_t lo = 0, hi = a.age_sat;                // smallest dismissed age
                    while (lo < hi) {
                        const uint32_t mid = lo + ((hi - lo) >> 1);
                        if (dismissed(mid)) hi = mid;
                        else lo = mid + 1;
                    }
                    cut = lo;
                }
            }
            s_cut[e] = cut;
        }
    }
    __syncthreads();
    CS_STAMP(ws, CS_PS_SCAN_CUTS + PS / 2, blockIdx.x == 0 && threadIdx.x == 0);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t *q = queues + warp * FQ_CAP;
    uint32_t qn = 0;                                           // queued ids of this warp (same value in every lane)
    WarpStage st;
    {
        unsigned long long *stage_km = (unsigned long long *)(((uintptr_t)(queues + (SEL_THREADS / 32) * FQ_CAP) + 7) & ~(uintptr_t)7);
        stage_init(st, stage_km, (uint32_t *)(stage_km + (SEL_THREADS / 32) * STAGE_CAP));
    }
    uint32_t n_above = 0;
    const bool enabled = !PF || prefetch_enabled(ws, a.A);

    // Works off whole rounds of 32 queued entries (all of them when `all`), every lane busy.
    auto drain = [&](bool all) {
        const uint32_t rounds = all ? (qn + 31u) / 32u : qn / 32u;
        for (uint32_t r = 0; r < rounds; ++r) {
            const uint32_t i = r * 32u + lane;
            bool cand = false;
            uint32_t id = 0, ag = 0, la = 0, tok = a.block_tokens, dp = 0, fl = 0;
            if (i < qn) {
                id = q[i];
                ag = __ldg(a.agent + id);
                la = __ldg(a.la + id);
                fl = __ldg(a.flags + id);                        // (needed by the key of a candidate: one round trip, not two)
                if (a.ntok) tok = __ldg(a.ntok + id);
                if (PF && a.anchor) dp = __ldg(a.depth + id);
                bool elig = true;
                if (ag >= a.A) { atomicOr(&ws.sc->status, CS_ST_BAD_AGENT); elig = false; }
                else if (PF && a.anchor && !(dp < T.anchor[ag])) elig = false;
                if (elig) {
                    const uint32_t age = la <= a.now ? a.now - la : 0u;
                    const uint32_t xb = __float_as_uint(__fmul_rn(T.fsurv[ag], recency_of_age(a, T, age)));
                    const uint32_t X = s_xt[((PF && ag != T.a_star) ? XT_TOK : 0u) + tok];
                    cand = PF ? (xb >= X) : (xb < X);
                    if (!cand) ++n_above;
                }
            }
            uint32_t pr = 0, se = 0;
            if (cand) {
                entry_key_rest<PF>(a, T, &ws.sc->status, ag, dp, fl, la, tok, pr, se);
                atomicAdd(&s_hist[pr >> 20], 1u);
            }
            // candidates gather in the warp's slice of shared memory and leave it 32 or more at a time
            stage_push(st, cand, pr, se, id, &ws.sel->c_spec, ws.cand_km, ws.cand_id);
        }
        if (!all) {
            const uint32_t done = rounds * 32u, left = qn - done;        // < 32
            __syncwarp();
            const uint32_t v = lane < left ? q[done + lane] : 0u;
            __syncwarp();
            if (lane < left) q[lane] = v;
            __syncwarp();
            qn = left;
        } else {
            qn = 0;
        }
    };

    if (enabled) {
        const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
        const uint32_t n_tiles = a.n / TILE, n_warps = nth >> 5;
        const uint32_t n_iter = (n_tiles + n_warps - 1) / n_warps;     // whole warps stay in the shuffles
        for (uint32_t it = 0; it < n_iter; ++it) {
            const uint32_t t = it * n_warps + (gtid >> 5);
            uint32_t rem = 0;                                          // entries that need the exact test
            if (t < n_tiles) {
                Group G;
                load_group<PF>(a, t, lane, G);
                const uint32_t em = group_elig<PF>(a, G);
                if (!PF) {
                    uint32_t dm = 0;                                   // dismissed by age: young, of the common size
                    if (max_halves(G.ag0, G.ag1) < a.A) {              // (a bad agent id anywhere: everything takes the exact test)
#pragma unroll
                        for (int j = 0; j < GRP; ++j) {
                            const uint32_t la = grp_u32(G, j), age = max(a.now, la) - la;
                            dm |= (age < s_cut[grp_u16(G.ag0, G.ag1, j)] ? 1u : 0u) << j;
                        }
                        if (a.ntok) {
                            uint32_t same = 0;
#pragma unroll
                            for (int w = 0; w < 4; ++w)
                                same |= nibble_of_flags(zero_bytes(u4_word(G.tk, w) ^ (0x01010101u * Tb))) << (4 * w);
                            dm &= same;
                        }
                    }
                    n_above += __popc(em & dm);
                    rem = em & ~dm;
                } else {
#pragma unroll
                    for (int j = 0; j < GRP; ++j) {
                        if (!((em >> j) & 1u)) continue;
                        const uint32_t ag = grp_u16(G.ag0, G.ag1, j);
                        const uint32_t tok = a.ntok ? grp_u8(G.tk, j) : Tb;
                        if (ag >= a.A || ag == T.a_star || tok != Tb) { rem |= 1u << j; continue; }
                        if (a.anchor && !(grp_u16(G.dp0, G.dp1, j) < T.anchor[ag])) continue;      // not eligible
                        const uint32_t la = grp_u32(G, j), age = max(a.now, la) - la;
                        if (age >= s_cut[ag]) ++n_above;
                        else rem |= 1u << j;
                    }
                }
            }
            // queue the remaining entries of the warp (ids only), then work off whole rounds
            const uint32_t cnt = __popc(rem);
            uint32_t incl = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d) incl += v;
            }
            const uint32_t total = __shfl_sync(0xFFFFFFFFu, incl, 31);
            if (total == 0) continue;
            uint32_t pos = qn + incl - cnt;
            while (rem) {
                const int j = __ffs(rem) - 1;
                rem &= rem - 1;
                q[pos++] = grp_id(t, lane, j);
            }
            qn += total;
            __syncwarp();
            if (qn >= 32u) drain(false);
        }
        CS_STAMP(ws, CS_PS_SCAN_WALKED + PS / 2, blockIdx.x == 0 && threadIdx.x == 0);
        drain(true);
        stage_flush(st, &ws.sel->c_spec, ws.cand_km, ws.cand_id);
        CS_STAMP(ws, CS_PS_SCAN_READ + PS, blockIdx.x == 0 && threadIdx.x == 0);
        const uint32_t t0 = n_tiles * TILE;
        if (gtid < a.n - t0) {                                // ragged tail, one entry per thread, through the key
            const uint32_t i = t0 + gtid;
            uint32_t pr, se;
            const uint32_t tok = a.ntok ? a.ntok[i] : a.block_tokens;
            if (entry_key<PF>(a, T, &ws.sc->status, a.agent[i], a.depth[i], a.ref[i], a.flags[i], a.la[i], tok, pr, se)) {
                if ((pr >> 20) <= H) {
                    atomicAdd(&s_hist[pr >> 20], 1u);
                    const uint32_t pos = atomicAdd(&ws.sel->c_spec, 1u);
                    ws.cand_km[pos] = ((unsigned long long)pr << 32) | se;
                    ws.cand_id[pos] = i;
                } else {
                    ++n_above;
                }
            }
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) n_above += __shfl_xor_sync(0xFFFFFFFFu, n_above, d);
    if (lane == 0 && n_above) atomicAdd(&s_above, n_above);
    __syncthreads();
    {
        const uint32_t h_end = H < CS_HIST_BINS ? H + 1u : CS_HIST_BINS;          // bins above H stay empty
        for (uint32_t i = threadIdx.x; i < h_end; i += blockDim.x) {
            const uint32_t v = s_hist[i];
            if (v) atomicAdd(&ws.hist[i], v);
        }
    }
    if (threadIdx.x == 0 && s_above) atomicAdd(&ws.sel->n_above, s_above);
    CS_STAMP(ws, CS_PS_SCAN_FLUSHED + PS, blockIdx.x == 0 && threadIdx.x == 0);
    if (!last_cta_done(&ws.sel->ticket[0], &s_flag)) return;
    CS_STAMP(ws, CS_PS_SCAN_LAST_CTA + PS, threadIdx.x == 0);

    // ---- last CTA -----------------------------------------------------------------------------------------
    // Two things are left and neither needs the other: whether the k-th smallest key lies within the remembered
    // bin (a scan of the histogram), and the splitters for ordering the candidates (a sort of a sample of them).
    // With few candidates half of the CTA is enough for the sample, so the two halves do one each, side by side;
    // the sample sort is then wasted on a miss, which costs nothing on the critical path.
    constexpr uint32_t HALF = SEL_THREADS / 2;
    const uint32_t c_spec = __ldcg(&ws.sel->c_spec);
    const uint32_t c_use = a.k ? c_spec : 0u;
    const bool small = c_use <= CS_SPLIT_SAMPLE_MAX;
    unsigned long long *s_km = (unsigned long long *)(((uintptr_t)queues + 7) & ~(uintptr_t)7);   // the queues are idle now
    uint32_t *s_id = (uint32_t *)(s_km + CS_SAMPLE);
    if (threadIdx.x >= HALF) {
        if (small) {
            // a sample of at least twice the splitters (c / 64 of them): 128, 256 or 512 keys
            const uint32_t P = c_use <= 4096u ? 128u : (c_use <= 8192u ? 256u : CS_SAMPLE / 2);
            publish_splitters(ws, s_km, s_id, c_use, a.sort_cap, a.region_cap_max, P, CtaPart{threadIdx.x - HALF, HALF, 2u});
        }
    } else {
        const CtaPart cp{threadIdx.x, HALF, 1u};
        constexpr uint32_t PER = CS_HIST_BINS / HALF;
        uint32_t loc[PER], sum = 0;
        {
            uint4 *h4 = (uint4 *)(ws.hist + threadIdx.x * PER);
#pragma unroll
            for (uint32_t qq = 0; qq < PER / 4; ++qq) {
                const uint4 v = __ldcg(h4 + qq);
                h4[qq] = make_uint4(0u, 0u, 0u, 0u);             // ready for the next pass or call
                loc[4 * qq] = v.x; loc[4 * qq + 1] = v.y; loc[4 * qq + 2] = v.z; loc[4 * qq + 3] = v.w;
                sum += v.x + v.y + v.z + v.w;
            }
        }
        if (threadIdx.x == 0) s_b0 = 0xFFFFFFFFu;
        uint32_t below;                                          // eligible entries at or below H
        const uint32_t before = sel_block_scan(sum, s_part, below, cp);
        const uint32_t total = below + __ldcg(&ws.sel->n_above);
        if (a.k && below >= a.k && before < a.k && a.k <= before + sum) {
            uint32_t run = before;
#pragma unroll
            for (uint32_t qq = 0; qq < PER; ++qq) {
                run += loc[qq];
                if (run >= a.k) { s_b0 = threadIdx.x * PER + qq; break; }
            }
        }
        part_sync(cp);
        // complete when the k winners lie at or below H, when fewer than k entries are eligible and all of them do, or when k = 0
        const bool hit = a.k == 0 || below >= a.k || below == total;
        const uint32_t b0 = a.k == 0 ? 0xFFFFFFFFu : (s_b0 != 0xFFFFFFFFu ? s_b0 : (H < CS_HIST_BINS ? H : CS_HIST_BINS - 1));
        uint32_t ahead = 0;
        const bool have_b0 = a.k && below >= a.k;
        if (hit && have_b0) {
            ahead = collect_ahead_limit<PER>(loc, threadIdx.x * PER, before, a.k, b0, &s_ahead, cp);
            if (ahead > H) ahead = H;                             // nothing is known about the bins above H
        }
        if (threadIdx.x == 0) {
            s_flag = hit;
            if (hit) {
                ws.sel->b0 = b0;
                ws.sel->n_elig = total;
                ws.sel->n_out = total < a.k ? total : a.k;
                ws.sel->c = c_use;
                count_select(ws, a.kind, total, total < a.k ? total : a.k);
                count_candidates(ws, a.kind, c_use, true);
                // fewer eligible entries than k: keep H; otherwise tighten it to what the histogram allows
                if (have_b0) remember_threshold(ws.sc, a.hint_slot, true, ahead);
            }
        }
    }
    __syncthreads();
    const bool hit = s_flag;
    if (hit && !small) publish_splitters(ws, s_km, s_id, c_use, a.sort_cap, a.region_cap_max, CS_SAMPLE, whole_cta());
    if (threadIdx.x == 0) {
        ws.sel->spec = hit ? 1u : 0u;
        ws.sel->c_spec = 0;
        ws.sel->n_above = 0;
        ws.sel->ticket[0] = 0;
    }
    CS_STAMP(ws, CS_PS_SCAN_TAIL_DONE + PS, threadIdx.x == 0);
}

// ---------------------------------------------------------------------------------------------
// 1 histogram (runs when the fast pass missed or had nothing to go by)
//
// Full keys of all eligible entries into a 4096-bin histogram; the last CTA finds the threshold bin and
// chooses how far ahead of it the next call of this kind may look.
// ---------------------------------------------------------------------------------------------
template <bool PF>
__global__ void __launch_bounds__(SEL_THREADS) cs_sel_hist_kernel(SelArgs a, cs_workspace ws)
{
    extern __shared__ float smem[];
    __shared__ __align__(16) uint32_t s_hist[CS_HIST_BINS];
    __shared__ uint32_t s_part[SEL_THREADS];
    __shared__ uint32_t s_b0, s_ahead;
    __shared__ bool s_flag;
    cs_wait_for_predecessor();
    cs_release_successor();
    if (ws.sel->spec) return;          // the fast pass already has the candidates
    resolve_now(a);
    Tables T;
    load_tables(a, ws, smem, T, PF && a.anchor);
    for (uint32_t i = threadIdx.x; i < CS_HIST_BINS; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
    if (!PF || prefetch_enabled(ws, a.A)) {
        uint32_t run_bin = 0xFFFFFFFFu, run_cnt = 0;                    // adjacent entries often share a bin
        for_each_eligible<PF>(a, T, &ws.sc->status, [&](uint32_t, uint32_t pr, uint32_t) {
            const uint32_t bin = pr >> 20;
            if (bin == run_bin) { ++run_cnt; return; }
            if (run_cnt) atomicAdd(&s_hist[run_bin], run_cnt);
            run_bin = bin;
            run_cnt = 1;
        });
        if (run_cnt) atomicAdd(&s_hist[run_bin], run_cnt);
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < CS_HIST_BINS; i += blockDim.x) {
        const uint32_t v = s_hist[i];
        if (v) atomicAdd(&ws.hist[i], v);
    }
    if (!last_cta_done(&ws.sel->ticket[1], &s_flag)) return;

    // ---- last CTA: threshold bin = first bin whose inclusive running count reaches k ------------
    constexpr uint32_t PER = CS_HIST_BINS / SEL_THREADS;
    uint32_t loc[PER], sum = 0;
#pragma unroll
    for (uint32_t q = 0; q < PER; ++q) {
        loc[q] = __ldcg(&ws.hist[threadIdx.x * PER + q]);
        ws.hist[threadIdx.x * PER + q] = 0;                 // ready for the next call
        sum += loc[q];
    }
    s_part[threadIdx.x] = sum;
    if (threadIdx.x == 0) s_b0 = (a.k == 0) ? 0xFFFFFFFFu : CS_HIST_BINS - 1;   // k = 0: nothing; k > eligible: everything
    __syncthreads();
    for (uint32_t d = 1; d < SEL_THREADS; d <<= 1) {         // inclusive scan
        const uint32_t v = threadIdx.x >= d ? s_part[threadIdx.x - d] : 0;
        __syncthreads();
        s_part[threadIdx.x] += v;
        __syncthreads();
    }
    const uint32_t total = s_part[SEL_THREADS - 1];
    const uint32_t before = s_part[threadIdx.x] - sum;
    if (a.k && total >= a.k && before < a.k && a.k <= before + sum) {
        uint32_t run = before;
#pragma unroll
        for (uint32_t q = 0; q < PER; ++q) {
            run += loc[q];
            if (run >= a.k) { s_b0 = threadIdx.x * PER + q; break; }
        }
    }
    __syncthreads();
    const uint32_t b0 = s_b0;
    const bool have_b0 = a.k && total >= a.k;
    const uint32_t ahead = have_b0 ? collect_ahead_limit<PER>(loc, threadIdx.x * PER, before, a.k, b0, &s_ahead, whole_cta()) : 0u;
    if (threadIdx.x == 0) {
        ws.sel->b0 = b0;
        ws.sel->n_elig = total;
        ws.sel->n_out = total < a.k ? total : a.k;
        count_select(ws, a.kind, total, total < a.k ? total : a.k);
        ws.sel->c = 0;
        remember_threshold(ws.sc, a.hint_slot, have_b0, ahead);
        ws.sel->ticket[1] = 0;
    }
}

// ---------------------------------------------------------------------------------------------
// 2 collect (+ splitters)
// ---------------------------------------------------------------------------------------------
// Age limits.  For a fixed agent and block size the score never increases with age (the recency
// table is checked to be monotone, IEEE multiplication is), so "first digit <= b0" is an interval
// of ages: victims  age >= lim (low scores are old blocks), prefetch  age + 1 <= lim (high scores
// are young blocks).  One limit per (agent, size) found by binary search lets the scan of a large
// index decide with one table look-up per entry; the full key is computed for candidates only.
#define AGE_LIM_MAX 8192u
#define AGE_CLAMP 0xFFFFFFFEu

template <bool PF>
__device__ __forceinline__ uint32_t age_limit_of(const SelArgs &a, const Tables &T, uint32_t agent, uint32_t tok,
                                                 uint32_t b0)
{
    const uint32_t n_age = a.age_sat;                        // ages >= age_sat all score like age_sat
    if (!PF) {
        // candidate <=> score bits < lim_bits, i.e. (bits [<< 1 | copy bit]) >> 20 <= b0
        const unsigned long long lim_bits = (unsigned long long)(b0 + 1u) << (a.prefer_copy ? 19 : 20);
        uint32_t lo = 0, hi = n_age + 1;                      // first age with bits < lim_bits; n_age + 1 = none
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            const unsigned long long bits = __float_as_uint(score_from_age(a, T, agent, mid, tok));
            if (bits < lim_bits) hi = mid;
            else lo = mid + 1;
        }
        return lo > n_age ? 0xFFFFFFFFu : lo;                 // 0xFFFFFFFF: no age qualifies (ages are clamped below it)
    } else {
        const bool star = agent == T.a_star;
        if (!star && b0 < 2048u) return 0u;                   // the whole non-a* class lies above the threshold bin
        if (star && b0 >= 2048u) return 0xFFFFFFFFu;          // every a* entry is a candidate
        const uint32_t x = star ? b0 : b0 - 2048u;            // (~bits & 0x7FFFFFFF) >> 20 <= x  <=>  bits >= lim_bits
        const uint32_t lim_bits = (0x7FFu - x) << 20;
        uint32_t lo = 0, hi = n_age + 1;                      // first age with bits < lim_bits
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (__float_as_uint(score_from_age(a, T, agent, mid, tok)) < lim_bits) hi = mid;
            else lo = mid + 1;
        }
        return lo > n_age ? 0xFFFFFFFFu : lo;                 // candidate <=> age + 1 <= lo  (lo = 0: none)
    }
}

template <bool PF>
__global__ void __launch_bounds__(SEL_THREADS) cs_sel_collect_kernel(SelArgs a, cs_workspace ws)
{
    extern __shared__ float smem[];
    __shared__ unsigned long long s_km[CS_SAMPLE];
    __shared__ uint32_t s_id[CS_SAMPLE];
    __shared__ bool s_flag;
    cs_wait_for_predecessor();
    cs_release_successor();
    if (ws.sel->spec) return;          // the histogram pass already collected the candidates
    resolve_now(a);
    Tables T;
    load_tables(a, ws, smem, T, PF && a.anchor);
    __syncthreads();
    const uint32_t b0 = ws.sel->b0;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t n_cls = a.ntok ? a.block_tokens : 1u;     // size classes: tok = 1 .. block_tokens (or the constant)
    const bool limits = a.use_age_limits && ws.sc->gtab_monotone && b0 != 0xFFFFFFFFu;
    uint32_t *s_lim = (uint32_t *)(smem + a.A + a.gtab_len) + (a.A + 1) / 2;      // after the tables (and the anchor table)
    if (limits) {
        for (uint32_t e = threadIdx.x; e < a.A * n_cls; e += blockDim.x) {
            const uint32_t agent = e / n_cls, tok = a.ntok ? (e - agent * n_cls) + 1u : a.block_tokens;
            s_lim[e] = age_limit_of<PF>(a, T, agent, tok, b0);
        }
        __syncthreads();
    }
    if (b0 != 0xFFFFFFFFu && (!PF || prefetch_enabled(ws, a.A))) {
        // Whole groups: count this thread's candidates, reserve a range with one atomic per warp,
        // then write.  The loop bound is rounded up so that whole warps stay in the shuffles.
        const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
        const uint32_t n_tiles = a.n / TILE, n_warps = nth >> 5;
        const uint32_t n_iter = (n_tiles + n_warps - 1) / n_warps;
        for (uint32_t it = 0; it < n_iter; ++it) {
            const uint32_t t = it * n_warps + (gtid >> 5);
            uint32_t mask = 0;               // keys are recomputed for the (few) candidates instead of kept in registers
            Group G;
            if (t < n_tiles) {
                load_group<PF>(a, t, lane, G);
                const uint32_t em = group_elig<PF>(a, G);
#pragma unroll
                for (int j = 0; j < GRP; ++j) {
                    if (!((em >> j) & 1u)) continue;
                    uint32_t se;
                    const uint32_t tok = a.ntok ? grp_u8(G.tk, j) : a.block_tokens;
                    const uint32_t dp = (PF && a.anchor) ? grp_u16(G.dp0, G.dp1, j) : 0u;
                    const uint32_t ag = grp_u16(G.ag0, G.ag1, j);
                    if (limits && ag < a.A && tok - 1u < n_cls) {
                        // prefilter: one look-up; exact, so the key is only needed when the entry is written
                        const uint32_t la = grp_u32(G, j);
                        uint32_t age = la <= a.now ? a.now - la : 0u;
                        age = age < AGE_CLAMP ? age : AGE_CLAMP;
                        const uint32_t lim = s_lim[ag * n_cls + (a.ntok ? tok - 1u : 0u)];
                        const bool in = PF ? (age + 1u <= lim) : (age >= lim);
                        if (in && !(PF && a.anchor && !(dp < T.anchor[ag]))) mask |= 1u << j;
                        continue;
                    }
                    uint32_t prj;
                    if (entry_key_rest<PF>(a, T, &ws.sc->status, ag, dp, grp_u8(G.fl, j), grp_u32(G, j), tok, prj, se) &&
                        (prj >> 20) <= b0)
                        mask |= 1u << j;
                }
            }
            if (!__any_sync(0xFFFFFFFFu, mask != 0)) continue;      // most warps hold no candidate at all
            const uint32_t cnt = __popc(mask);
            uint32_t incl = cnt;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
                if (lane >= d) incl += v;
            }
            uint32_t base = 0;
            if (lane == 31 && incl) base = atomicAdd(&ws.sel->c, incl);
            base = __shfl_sync(0xFFFFFFFFu, base, 31);
            uint32_t pos = base + incl - cnt;
#pragma unroll
            for (int j = 0; j < GRP; ++j) {
                if (mask & (1u << j)) {
                    uint32_t prj, se;
                    const uint32_t tok = a.ntok ? grp_u8(G.tk, j) : a.block_tokens;
                    const uint32_t dp = (PF && a.anchor) ? grp_u16(G.dp0, G.dp1, j) : 0u;
                    const bool ok = entry_key_rest<PF>(a, T, &ws.sc->status, grp_u16(G.ag0, G.ag1, j), dp, grp_u8(G.fl, j),
                                                       grp_u32(G, j), tok, prj, se) && (prj >> 20) <= b0;
                    // (a slot was reserved from the prefilter's verdict; should the exact key ever disagree,
                    //  the slot gets a key that sorts behind every real candidate and is never emitted)
                    ws.cand_km[pos] = ok ? (((unsigned long long)prj << 32) | se) : ~0ull;
                    ws.cand_id[pos] = ok ? grp_id(t, lane, j) : CS_ID_NONE;
                    ++pos;
                }
            }
        }
        const uint32_t t0 = n_tiles * TILE;
        if (gtid < a.n - t0) {
            const uint32_t i = t0 + gtid;
            uint32_t p, se;
            const uint32_t tok = a.ntok ? a.ntok[i] : a.block_tokens;
            if (entry_key<PF>(a, T, &ws.sc->status, a.agent[i], a.depth[i], a.ref[i], a.flags[i], a.la[i], tok, p, se) &&
                (p >> 20) <= b0) {
                const uint32_t pos = atomicAdd(&ws.sel->c, 1u);
                ws.cand_km[pos] = ((unsigned long long)p << 32) | se;
                ws.cand_id[pos] = i;
            }
        }
    }
    if (!last_cta_done(&ws.sel->ticket[2], &s_flag)) return;

    // ---- last CTA: sample, sort the sample (bitonic, shared memory), publish splitters -----------
    publish_splitters(ws, s_km, s_id, __ldcg(&ws.sel->c), a.sort_cap, a.region_cap_max, CS_SAMPLE, whole_cta());
    if (threadIdx.x == 0) { ws.sel->ticket[2] = 0; count_candidates(ws, a.kind, __ldcg(&ws.sel->c), false); }
}

// ---------------------------------------------------------------------------------------------
// Sorts the first m <= RANK_TILE keys of a shared-memory tile ascending (bitonic; m is padded to a power of two
// with keys that sort last).  Whole CTA.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void sort_tile(unsigned long long *t_km, uint32_t *t_id, uint32_t m)
{
    uint32_t P = 64;
    while (P < m) P <<= 1;
    for (uint32_t i = m + threadIdx.x; i < P; i += blockDim.x) { t_km[i] = ~0ull; t_id[i] = 0xFFFFFFFFu; }
    __syncthreads();
    if (P <= 2 * blockDim.x) {
        bitonic_sort_fast(t_km, t_id, P, whole_cta());
        return;
    }
    for (uint32_t size = 2; size <= P; size <<= 1) {
        for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
            for (uint32_t t = threadIdx.x; t < P / 2; t += blockDim.x) {
                const uint32_t lo = 2 * t - (t & (stride - 1));
                const uint32_t hi = lo + stride;
                const bool up = (lo & size) == 0;
                const unsigned long long ka = t_km[lo], kb = t_km[hi];
                const uint32_t ia = t_id[lo], ib = t_id[hi];
                if (key_less(kb, ib, ka, ia) == up) {
                    t_km[lo] = kb; t_id[lo] = ib;
                    t_km[hi] = ka; t_id[hi] = ia;
                }
            }
            __syncthreads();
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Exclusive prefix sum of the bucket sizes, computed by every CTA that needs it (256 counters, L2-resident):
// s_off[b] = first output position of bucket b, s_off[256] = candidates in all buckets.  Also returns the last
// bucket that holds one of the n_out winners (0 when n_out = 0).  Whole CTA of 256 threads.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t bucket_offsets(const cs_workspace &ws, uint32_t n_spl, uint32_t n_out, uint32_t *s_off,
                                                   uint32_t *s_tmp)
{
    const uint32_t t = threadIdx.x, lane = t & 31, warp = t >> 5;
    const uint32_t mine = t <= n_spl ? __ldcg(&CS_BCOUNT(ws, t)) : 0u;
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += v;
    }
    if (t == 0) s_tmp[8] = 0;
    if (lane == 31) s_tmp[warp] = incl;
    __syncthreads();
    uint32_t before = 0;
#pragma unroll
    for (uint32_t w = 0; w < 8; ++w) before += w < warp ? s_tmp[w] : 0u;
    const uint32_t excl = before + incl - mine;
    s_off[t] = excl;
    if (t == 255) s_off[256] = excl + mine;
    if (n_out && mine && excl <= n_out - 1 && n_out - 1 < excl + mine) s_tmp[8] = t;
    __syncthreads();
    return s_tmp[8];
}

// ---------------------------------------------------------------------------------------------
// 3 bucket
//
// Each candidate finds its bucket by binary search over the splitters and takes a slot in it.
// Roomy case (few candidates for the size of the sort region): the slot comes straight from one atomic on the
// bucket's counter and the key is written to slot `slot` of the bucket's own fixed-size region, so that the
// buckets are ready for the rank launch and the scatter launch has nothing to do.  A bucket that outgrows its
// region sets `overflow`: bucket and slot of every candidate are recorded as well, and the scatter and rank
// launches then take the general route.
// General case: per round a CTA takes 1024 candidates, counts them per bucket in shared memory and reserves the
// CTA's range in each non-empty bucket with one global atomic; bucket and slot are recorded for the scatter launch.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) cs_sel_bucket_kernel(cs_workspace ws, uint32_t sort_cap, uint32_t kind)
{
    __shared__ unsigned long long s_km[CS_MAX_SPLITTERS + 1];
    __shared__ uint32_t s_id[CS_MAX_SPLITTERS + 1];
    __shared__ uint32_t s_cnt[CS_MAX_SPLITTERS + 1], s_base[CS_MAX_SPLITTERS + 1];
    constexpr int ITEMS = 4;                                  // candidates per thread and round
    const int PS = kind == 2 ? 8 : 0;                         // phase-stamp slots (profiling builds)
    cs_wait_for_predecessor();
    CS_STAMP(ws, CS_PS_BUCKET_WAITED + PS, blockIdx.x == 0 && threadIdx.x == 0);
    cs_release_successor();
    // Everything the first round needs is asked for at once -- the select's state, the splitters and the round's keys
    // (addresses bounded by the capacity of the buffers; what lies beyond the live counts is ignored below) -- so that
    // the launch starts with one trip to L2 instead of three.
    unsigned long long km[ITEMS];
    uint32_t id[ITEMS], bkt[ITEMS], loc[ITEMS];
    // Item u of a round lies one grid-wide sweep (sweep = 256 keys per CTA) after item u - 1, so that few candidates
    // spread over all CTAs with one live key per thread instead of filling a few CTAs with four.
    const uint32_t sweep = gridDim.x * 256u, lane0 = blockIdx.x * 256u + threadIdx.x;
    const uint4 st = cs_ld_cg_pinned((const uint4 *)&ws.sel->c);          // c, n_spl, placed, cap
#pragma unroll
    for (int u = 0; u < ITEMS; ++u) {
        const uint32_t i = u * sweep + lane0, ii = i < sort_cap ? i : 0u;
        km[u] = cs_ld_cg_pinned(ws.cand_km + ii);
        id[u] = cs_ld_cg_pinned(ws.cand_id + ii);
    }
    const unsigned long long my_spl_km = cs_ld_cg_pinned(ws.spl_km + threadIdx.x);
    const uint32_t my_spl_id = cs_ld_cg_pinned(ws.spl_id + threadIdx.x);
    const uint32_t c = st.x, n_spl = st.y, placed = st.z, cap = st.w;
    // splitters past the last one sort behind every key, so that the search below always takes eight steps
    s_km[threadIdx.x] = threadIdx.x < n_spl ? my_spl_km : ~0ull;
    s_id[threadIdx.x] = threadIdx.x < n_spl ? my_spl_id : 0xFFFFFFFFu;
    s_cnt[threadIdx.x] = 0;
    __syncthreads();
    CS_STAMP(ws, CS_PS_BUCKET_STAGED + PS, blockIdx.x == 0 && threadIdx.x == 0);
    for (uint32_t base = 0; base < c; base += sweep * ITEMS) {
        if (base != 0) {
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {                 // all of the round's keys are fetched before any is used
                const uint32_t i = base + u * sweep + lane0, ii = i < c ? i : 0u;
                km[u] = cs_ld_cg_pinned(ws.cand_km + ii);
                id[u] = cs_ld_cg_pinned(ws.cand_id + ii);
            }
        }
        // bucket = number of splitters <= key: a branch-free descent over the 255 (padded) splitters, the round's four
        // keys side by side
        uint32_t pos[ITEMS];
#pragma unroll
        for (int u = 0; u < ITEMS; ++u) pos[u] = 0;
#pragma unroll 1
        for (uint32_t step = 128; step > 0; step >>= 1) {
            unsigned long long sk[ITEMS];
            uint32_t si[ITEMS];
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {                 // the step's eight loads first, ...
                const uint32_t probe = pos[u] + step - 1u;
                sk[u] = s_km[probe];
                si[u] = s_id[probe];
            }
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {                 // ... then the compares, with no short-circuit branch
                const bool lt = (km[u] < sk[u]) | ((km[u] == sk[u]) & (id[u] < si[u]));
                pos[u] += lt ? 0u : step;
            }
        }
#pragma unroll
        for (int u = 0; u < ITEMS; ++u) {
            const uint32_t i = base + u * sweep + lane0;
            bkt[u] = 0xFFFFFFFFu;
            if (i < c) {
                bkt[u] = pos[u] < n_spl ? pos[u] : n_spl;    // (a key equal to the padding stays in the last bucket)
                if (!placed) loc[u] = atomicAdd(&s_cnt[bkt[u]], 1u);
            }
        }
        CS_STAMP(ws, CS_PS_BUCKET_SEARCHED + PS, blockIdx.x == 0 && threadIdx.x == 0 && base == 0);
        if (placed) {
#pragma unroll
            for (int u = 0; u < ITEMS; ++u)                   // the round's atomics are in flight together
                if (bkt[u] != 0xFFFFFFFFu) loc[u] = atomicAdd(&CS_BCOUNT(ws, bkt[u]), 1u);
            CS_STAMP(ws, CS_PS_BUCKET_SLOTS + PS, blockIdx.x == 0 && threadIdx.x == 0 && base == 0 && loc[0] != 0xFFFFFFF1u);
#pragma unroll
            for (int u = 0; u < ITEMS; ++u) {
                const uint32_t i = base + u * sweep + lane0;
                if (bkt[u] == 0xFFFFFFFFu) continue;
                ws.cand_bkt[i] = bkt[u];
                ws.cand_slot[i] = loc[u];
                if (loc[u] < cap) {
                    ws.sort_km[(size_t)bkt[u] * cap + loc[u]] = km[u];
                    ws.sort_id[(size_t)bkt[u] * cap + loc[u]] = id[u];
                } else {
                    ws.sel->overflow = 1;
                }
            }
            continue;
        }
        __syncthreads();
        {
            const uint32_t n_b = s_cnt[threadIdx.x];
            if (n_b) s_base[threadIdx.x] = atomicAdd(&CS_BCOUNT(ws, threadIdx.x), n_b);
            s_cnt[threadIdx.x] = 0;
        }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < ITEMS; ++u) {
            const uint32_t i = base + u * sweep + lane0;
            if (bkt[u] != 0xFFFFFFFFu) {
                ws.cand_bkt[i] = bkt[u];
                ws.cand_slot[i] = s_base[bkt[u]] + loc[u];
            }
        }
        __syncthreads();
    }
    CS_STAMP(ws, CS_PS_BUCKET_DONE + PS, blockIdx.x == 0 && threadIdx.x == 0);
    (void)PS;
}

// ---------------------------------------------------------------------------------------------
// 4 scatter (general case only: candidates of the needed buckets are grouped by bucket)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) cs_sel_scatter_kernel(cs_workspace ws, uint32_t kind)
{
    __shared__ uint32_t s_off[CS_MAX_SPLITTERS + 2];
    __shared__ uint32_t s_tmp[16];
    cs_wait_for_predecessor();
    CS_STAMP(ws, CS_PS_SCATTER_WAITED + (kind == 2 ? 8 : 0), blockIdx.x == 0 && threadIdx.x == 0);
    (void)kind;
    cs_release_successor();
    if (ws.sel->placed && !ws.sel->overflow) return;         // the buckets are in their regions already
    const uint32_t c = ws.sel->c, n_out = ws.sel->n_out;
    if (n_out == 0) return;
    const uint32_t b_last = bucket_offsets(ws, ws.sel->n_spl, n_out, s_off, s_tmp);
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < c; i += gridDim.x * blockDim.x) {
        const uint32_t b = ws.cand_bkt[i];
        if (b > b_last) continue;
        const uint32_t pos = s_off[b] + ws.cand_slot[i];
        ws.sort_km[pos] = ws.cand_km[i];
        ws.sort_id[pos] = ws.cand_id[i];
    }
}

// ---------------------------------------------------------------------------------------------
// 5 rank and emit
// ---------------------------------------------------------------------------------------------
// Each needed bucket is ordered by one CTA: a bitonic sort of the bucket in a shared-memory tile
// (O(m log^2 m), so an unlucky large bucket costs little more than an average one), after which
// position i of the bucket is position offset + i of the output list.
__global__ void __launch_bounds__(256)
cs_sel_rank_kernel(cs_workspace ws, uint32_t k, uint32_t kind, uint32_t *__restrict__ ids_out, uint32_t *__restrict__ n_out_dev)
{
    __shared__ unsigned long long t_km[RANK_TILE];
    __shared__ uint32_t t_id[RANK_TILE];
    __shared__ uint32_t s_off[CS_MAX_SPLITTERS + 2];
    __shared__ uint32_t s_tmp[16];
    cs_wait_for_predecessor();
    CS_STAMP(ws, CS_PS_RANK_WAITED + (kind == 2 ? 8 : 0), blockIdx.x == 0 && threadIdx.x == 0);
    cs_release_successor();
    const uint32_t n_out = ws.sel->n_out, cap = ws.sel->cap;
    const bool in_regions = ws.sel->placed && !ws.sel->overflow;
    const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    for (uint32_t i = n_out + gtid; i < k; i += nth) ids_out[i] = CS_ID_NONE;
    if (gtid == 0) {
        *n_out_dev = n_out;
        if (ws.sel->placed && kind < 3) {                     // work counters: how the buckets got to their places
            atomicAdd((unsigned long long *)&ws.cnt->region_selects[kind], 1ull);
            if (ws.sel->overflow) atomicAdd((unsigned long long *)&ws.cnt->region_overflows[kind], 1ull);
        }
    }
    if (n_out == 0) return;
    const uint32_t b_last = bucket_offsets(ws, ws.sel->n_spl, n_out, s_off, s_tmp);
    CS_STAMP(ws, CS_PS_RANK_OFFSETS + (kind == 2 ? 8 : 0), blockIdx.x == 0 && threadIdx.x == 0);
    for (uint32_t b = blockIdx.x; b <= b_last; b += gridDim.x) {
        const uint32_t beg = s_off[b], end = s_off[b + 1], m = end - beg;
        const size_t src = in_regions ? (size_t)b * cap : (size_t)beg;      // where the bucket's keys are
        __syncthreads();
        if (m <= RANK_TILE) {
            for (uint32_t i = threadIdx.x; i < m; i += blockDim.x) {
                t_km[i] = ws.sort_km[src + i];
                t_id[i] = ws.sort_id[src + i];
            }
            CS_STAMP(ws, CS_PS_RANK_LOADED + (kind == 2 ? 8 : 0), blockIdx.x == 0 && threadIdx.x == 0 && t_km[0] != 1ull);
            sort_tile(t_km, t_id, m);
            CS_STAMP(ws, CS_PS_RANK_SORTED + (kind == 2 ? 8 : 0), blockIdx.x == 0 && threadIdx.x == 0);
            for (uint32_t i = threadIdx.x; i < m; i += blockDim.x)
                if (beg + i < n_out) ids_out[beg + i] = t_id[i];
        } else {                                              // larger than the tile: rank straight from global memory
            for (uint32_t i = threadIdx.x; i < m; i += blockDim.x) {
                const unsigned long long km = ws.sort_km[src + i];
                const uint32_t id = ws.sort_id[src + i];
                uint32_t rank = 0;
                for (uint32_t q = 0; q < m; ++q) rank += key_less(ws.sort_km[src + q], ws.sort_id[src + q], km, id) ? 1u : 0u;
                if (beg + rank < n_out) ids_out[beg + rank] = id;
            }
        }
    }
    CS_STAMP(ws, CS_PS_RANK_DONE + (kind == 2 ? 8 : 0), blockIdx.x == 0 && threadIdx.x == 0);
}

// ---------------------------------------------------------------------------------------------
void cs_fill_sel_args(const cs_ctx *ctx, const cs_block_index *idx, uint32_t now, const float *fsurv, SelArgs &a)
{
    a.agent = idx->agent;
    a.depth = idx->depth;
    a.ref = idx->ref_count;
    a.flags = idx->flags;
    a.la = idx->last_access;
    a.ntok = idx->n_tokens;
    a.anchor = idx->anchor_blocks;
    a.fsurv = fsurv;
    a.n = idx->n_blocks;
    a.now = now;
    a.A = ctx->p.n_agents;
    a.block_tokens = ctx->p.block_tokens;
    a.gtab_len = ctx->gtab_len;
    a.age_sat = ctx->age_sat;
    a.lambda = ctx->p.lambda;
    a.delta = ctx->p.delta;
    a.tier = 0;
    a.k = 0;
    a.prefer_copy = ctx->p.prefer_other_copy ? 1u : 0u;
    a.use_age_limits = 0;
    a.hint_slot = 0;
    a.kind = 0;
    a.now_dev = ctx->step_now_dev ? ctx->step_now_dev : ctx->clock_dev;
    a.sort_cap = 0;
    a.region_cap_max = ctx->region_cap_max;
}

uint32_t cs_scan_grid(const cs_ctx *ctx, uint32_t n, uint32_t per_cta, uint32_t ctas_per_sm)
{
    uint32_t g = (n + per_cta - 1) / per_cta;
    const uint32_t cap = ctas_per_sm * (uint32_t)ctx->sm_count;
    if (g > cap) g = cap;
    return g ? g : 1u;
}

size_t cs_table_smem(const cs_ctx *ctx)
{
    return (size_t)(ctx->p.n_agents + ctx->gtab_len) * sizeof(float) + (size_t)ctx->p.n_agents * sizeof(uint16_t) + 16;
}

int cs_launch_score(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, const float *fsurv, float *scores_out,
                    cudaStream_t s)
{
    SelArgs a;
    cs_fill_sel_args(ctx, idx, now, fsurv, a);
    a.anchor = nullptr;
    const uint32_t grid = cs_scan_grid(ctx, idx->n_blocks, SEL_THREADS * GRP);
    cs_score_kernel<<<grid, SEL_THREADS, cs_table_smem(ctx), s>>>(a, ctx->ws, scores_out);
    return cs_check_launch(ctx);
}

// Shared-memory opt-in of the scan kernels that keep age limits in shared memory: an attribute of the
// function on a device, set once per process and device to one fixed size.
#include <mutex>
#define SCAN_SMEM_OPT_IN (96 * 1024)
static std::mutex g_scan_mu;
static bool g_scan_opted[64];
static int scan_opt_in(cs_ctx *ctx)
{
    if (ctx->device < 0 || ctx->device >= 64) return CS_EINVAL;
    std::lock_guard<std::mutex> lock(g_scan_mu);
    if (g_scan_opted[ctx->device]) return CS_OK;
    cudaError_t e = cudaFuncSetAttribute(cs_sel_collect_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SCAN_SMEM_OPT_IN);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(cs_sel_collect_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SCAN_SMEM_OPT_IN);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(cs_sel_fast_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SCAN_SMEM_OPT_IN);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(cs_sel_fast_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SCAN_SMEM_OPT_IN);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    g_scan_opted[ctx->device] = true;
    return CS_OK;
}

// One select through the grid-wide kernels (or one single-launch cluster select), on the scratch of `job`.
static int launch_select_job(cs_ctx *ctx, int job, const cs_block_index *idx, uint32_t now, int prefetch, uint32_t tier,
                             uint32_t k, uint32_t *ids_out, uint32_t *n_out, cudaStream_t s)
{
    const cs_workspace &ws = job == 0 ? ctx->ws : ctx->ws_job[job - 1];
    SelArgs a;
    cs_fill_sel_args(ctx, idx, now, ctx->fsurv_override ? ctx->fsurv_override : ctx->ws.fsurv, a);
    a.tier = tier;
    a.k = k;
    a.hint_slot = ctx->no_speculation ? 3u : (prefetch ? 2u : tier);
    a.kind = prefetch ? 2u : tier;
    a.sort_cap = ctx->p.max_blocks;          // keys the sort region of this select holds
    if (ctx->select_path != CS_SELECT_MULTI && idx->n_blocks <= CS_SELECT_CLUSTER_MAX_BLOCKS) {
        const int rc1 = cs_launch_select_cluster(ctx, &a, &ws, prefetch, ids_out, n_out, s);
        if (rc1 != CS_ENOTIMPL) return rc1;          // no usable cluster on this device: fall through
    }
    const uint32_t grid = cs_scan_grid(ctx, idx->n_blocks, SEL_THREADS * GRP);
    const uint32_t grid_c = cs_scan_grid(ctx, idx->n_blocks, 256);
    const size_t sm = cs_table_smem(ctx);
    int rc;
    const size_t sm_fast = (sm + 15) / 16 * 16 + (size_t)(SEL_THREADS / 32) * (FQ_CAP * sizeof(uint32_t) + STAGE_CAP * 12) + 32 +
                           (size_t)ctx->p.n_agents * sizeof(uint32_t);   // tables, per-warp queues, per-warp candidate staging, age cuts
    if ((rc = scan_opt_in(ctx)) != CS_OK) return rc;
    if (prefetch) cs_launch_chained(cs_sel_fast_kernel<true>, grid, SEL_THREADS, sm_fast, s, a, ws);
    else cs_launch_chained(cs_sel_fast_kernel<false>, grid, SEL_THREADS, sm_fast, s, a, ws);
    if ((rc = cs_check_launch(ctx)) != CS_OK) return rc;
    if (prefetch) cs_launch_chained(cs_sel_hist_kernel<true>, grid, SEL_THREADS, sm, s, a, ws);
    else cs_launch_chained(cs_sel_hist_kernel<false>, grid, SEL_THREADS, sm, s, a, ws);
    if ((rc = cs_check_launch(ctx)) != CS_OK) return rc;
    // large indexes: the collect pass prefilters by age limits (one look-up per entry instead of the full key)
    const uint32_t n_cls = idx->n_tokens ? ctx->p.block_tokens : 1u;
    size_t sm_collect = sm;
    if (idx->n_blocks >= CS_AGE_LIMIT_MIN_BLOCKS && (size_t)ctx->p.n_agents * n_cls <= AGE_LIM_MAX) {
        a.use_age_limits = 1;
        sm_collect += (size_t)ctx->p.n_agents * n_cls * sizeof(uint32_t);
        const int rc_opt = scan_opt_in(ctx);
        if (rc_opt != CS_OK) return rc_opt;
    }
    if (prefetch) cs_launch_chained(cs_sel_collect_kernel<true>, grid, SEL_THREADS, sm_collect, s, a, ws);
    else cs_launch_chained(cs_sel_collect_kernel<false>, grid, SEL_THREADS, sm_collect, s, a, ws);
    if ((rc = cs_check_launch(ctx)) != CS_OK) return rc;
    cs_launch_chained(cs_sel_bucket_kernel, grid_c, 256, 0, s, ws, (uint32_t)ctx->p.max_blocks, a.kind);
    if ((rc = cs_check_launch(ctx)) != CS_OK) return rc;
    cs_launch_chained(cs_sel_scatter_kernel, grid_c, 256, 0, s, ws, a.kind);
    if ((rc = cs_check_launch(ctx)) != CS_OK) return rc;
    cs_launch_chained(cs_sel_rank_kernel, CS_MAX_SPLITTERS + 1, 256, 0, s, ws, k, a.kind, ids_out, n_out);
    return cs_check_launch(ctx);
}

int cs_launch_select(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, int prefetch, uint32_t tier, uint32_t k,
                     uint32_t *ids_out, uint32_t *n_out, cudaStream_t s)
{
    return launch_select_job(ctx, 0, idx, now, prefetch, tier, k, ids_out, n_out, s);
}

// The selects of a step side by side.  Select q (0 GPU-tier victims, 1 host-tier victims, 2 prefetch candidates)
// is skipped when its count pointer is NULL.  Where the single-launch select applies they are the clusters of ONE
// launch; otherwise every select is a chain of grid-wide kernels, the first on the caller's stream and the others
// on the context's two extra streams, forked from and joined back into the caller's stream with events (each has
// its own select state, histogram and candidate / sort regions).  Indexes beyond CS_CONCURRENT_MAX_BLOCKS entries
// have no private regions of that size: their selects run one after the other.
int cs_launch_select_step(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t k_victims, uint32_t k_prefetch,
                          uint32_t *gpu_victims, uint32_t *n_gpu, uint32_t *host_victims, uint32_t *n_host,
                          uint32_t *prefetch_ids, uint32_t *n_prefetch, cudaStream_t s)
{
    uint32_t *const ids[3] = {gpu_victims, host_victims, prefetch_ids};
    uint32_t *const cnt[3] = {n_gpu, n_host, n_prefetch};
    const uint32_t ks[3] = {k_victims, k_victims, k_prefetch};
    int jobs[3], n_jobs = 0;
    for (int q = 0; q < 3; ++q)
        if (cnt[q]) jobs[n_jobs++] = q;
    if (n_jobs == 0) return CS_OK;
    if (ctx->select_path != CS_SELECT_MULTI && idx->n_blocks <= CS_SELECT_CLUSTER_MAX_BLOCKS) {
        SelArgs a[3];
        uint32_t *j_ids[3], *j_cnt[3];
        uint32_t pf[3];
        for (int i = 0; i < n_jobs; ++i) {
            const int q = jobs[i];
            cs_fill_sel_args(ctx, idx, now, ctx->fsurv_override ? ctx->fsurv_override : ctx->ws.fsurv, a[i]);
            a[i].tier = q == 0 ? 0u : 1u;
            a[i].k = ks[q];
            a[i].hint_slot = ctx->no_speculation ? 3u : (uint32_t)q;
            a[i].kind = (uint32_t)q;
            j_ids[i] = ids[q];
            j_cnt[i] = cnt[q];
            pf[i] = q == 2 ? 1u : 0u;
        }
        const int rc = cs_launch_select_clusters(ctx, n_jobs, a, pf, j_ids, j_cnt, s);
        if (rc != CS_ENOTIMPL) return rc;
    }
    const bool side_by_side = ctx->concurrent_selects && n_jobs > 1;
    cudaError_t e = cudaSuccess;
    if (side_by_side) e = cudaEventRecord(ctx->ev_sel_fork, s);
    int rc = CS_OK;
    for (int i = 0; i < n_jobs && rc == CS_OK && e == cudaSuccess; ++i) {
        const int q = jobs[i];
        cudaStream_t sq = (side_by_side && i > 0) ? ctx->sel_stream[i - 1] : s;
        if (side_by_side && i > 0) e = cudaStreamWaitEvent(sq, ctx->ev_sel_fork, 0);
        if (e != cudaSuccess) break;
        rc = launch_select_job(ctx, side_by_side ? i : 0, idx, now, q == 2, q == 0 ? 0u : 1u, ks[q], ids[q], cnt[q], sq);
        if (rc == CS_OK && side_by_side && i > 0) {
            e = cudaEventRecord(ctx->ev_sel_join[i - 1], sq);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ctx->ev_sel_join[i - 1], 0);
        }
    }
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return rc;
}

// =============================================================================================
// Victim selection for callers that cannot allocate device memory.
//
// Some embedders of this library never get to call cudaMalloc: a serving engine that has handed
// the whole GPU to its own KV pool at start-up, a plug-in hook that runs while allocation is
// forbidden (inside a region where the host application has frozen its memory map), or a
// process whose memory budget is fixed by its launcher.  They can pass inputs and outputs they
// already own, but not a workspace.  For them the scratch of the select kernels (recency table,
// histogram, candidate keys, buckets, counters) lives in the file-scope array below, which
// every GPU that loads the library holds until the process exits.
//
// The array's name is only a host-side handle: the device address is obtained once per device
// with cudaGetSymbolAddress() and that pointer is what the kernels get.
// =============================================================================================
#define CS_STATIC_MAX_DEVICES 64
#define CS_STATIC_ALIGN(x) (((x) + 255u) / 256u * 256u)
// layout of the static scratch, byte offsets (every region 256-byte aligned)
#define CS_SO_SC 0u
#define CS_SO_SEL (CS_SO_SC + CS_STATIC_ALIGN(sizeof(cs_scalars)))
#define CS_SO_GTAB (CS_SO_SEL + CS_STATIC_ALIGN(sizeof(cs_sel_state)))
#define CS_SO_HIST (CS_SO_GTAB + CS_GTAB_MAX * 4u)
#define CS_SO_SPLKM (CS_SO_HIST + CS_HIST_BINS * 4u)
#define CS_SO_SPLID (CS_SO_SPLKM + CS_STATIC_ALIGN((CS_MAX_SPLITTERS + 1u) * 8u))
#define CS_SO_BCOUNT (CS_SO_SPLID + CS_STATIC_ALIGN((CS_MAX_SPLITTERS + 1u) * 4u))
#define CS_SO_CANDKM (CS_SO_BCOUNT + CS_STATIC_ALIGN((CS_MAX_SPLITTERS + 1u) * CS_BCOUNT_STRIDE * 4u))
#define CS_SO_SORTKM (CS_SO_CANDKM + CS_STATIC_MAX_BLOCKS * 8u)
#define CS_SO_CANDID (CS_SO_SORTKM + CS_STATIC_MAX_BLOCKS * 8u)
#define CS_SO_CANDBKT (CS_SO_CANDID + CS_STATIC_MAX_BLOCKS * 4u)
#define CS_SO_CANDSLOT (CS_SO_CANDBKT + CS_STATIC_MAX_BLOCKS * 4u)
#define CS_SO_SORTID (CS_SO_CANDSLOT + CS_STATIC_MAX_BLOCKS * 4u)
#define CS_SO_CNT (CS_SO_SORTID + CS_STATIC_MAX_BLOCKS * 4u)
#define CS_STATIC_BYTES (CS_SO_CNT + CS_STATIC_ALIGN(sizeof(cs_counters)))

static __device__ __align__(256) unsigned char cs_static_scratch[CS_STATIC_BYTES];   // 2 MiB + 40 KiB

static std::mutex g_static_mu;
static unsigned char *g_static_ptr[CS_STATIC_MAX_DEVICES];     // device address of the array, per device
static int g_static_sms[CS_STATIC_MAX_DEVICES];

// Everything the select kernels expect to find zeroed, and the recency table for this call's
// lambda / delta.  The array keeps the previous call's contents, so this runs on every call.
__global__ void cs_static_prepare_kernel(cs_workspace ws, uint32_t gtab_len, float lambda, float delta)
{
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    for (uint32_t i = tid; i < CS_HIST_BINS; i += nth) ws.hist[i] = 0;
    for (uint32_t i = tid; i <= CS_MAX_SPLITTERS; i += nth) CS_BCOUNT(ws, i) = 0;
    for (uint32_t i = tid; i < gtab_len; i += nth) ws.gtab[i] = cs_recency(lambda, delta, i);
    if (tid == 0) {
        cs_scalars z;
        memset(&z, 0, sizeof(z));
        z.last_agent = CS_AGENT_NONE;
        z.a_star = 0xFFFFFFFFu;
        z.sel_hint[0] = z.sel_hint[1] = z.sel_hint[2] = z.sel_hint[3] = 0xFFFFFFFFu;
        *ws.sc = z;
        cs_sel_state zs;
        memset(&zs, 0, sizeof(zs));
        *ws.sel = zs;
    }
}

extern "C" int cs_select_victims_static(const cs_params *p, const float *fsurv, const cs_block_index *idx,
                                        uint32_t now, uint32_t tier, uint32_t k, uint32_t *ids_out, uint32_t *n_out,
                                        cs_stream_t stream)
{
    int rc = cs_validate_params(p);
    if (rc != CS_OK) return rc;
    if (!idx || !fsurv || (((uintptr_t)fsurv) & 3u) || tier > 1) return CS_EINVAL;
    if (idx->n_blocks > CS_STATIC_MAX_BLOCKS || k > CS_STATIC_MAX_BLOCKS) return CS_ECAPACITY;
    if (!n_out || (((uintptr_t)n_out) & 3u)) return CS_EINVAL;
    if (k && (!ids_out || (((uintptr_t)ids_out) & 15u))) return CS_EINVAL;
    if (idx->n_blocks) {
        if (!idx->agent || !idx->depth || !idx->ref_count || !idx->flags || !idx->last_access) return CS_EINVAL;
        const uintptr_t any = (uintptr_t)idx->agent | (uintptr_t)idx->depth | (uintptr_t)idx->ref_count |
                              (uintptr_t)idx->flags | (uintptr_t)idx->last_access | (uintptr_t)idx->n_tokens;
        if (any & 15u) return CS_EINVAL;
    }
    // Memory the SMs cannot address (a pageable host array) would fault the GPU: every pointer the kernels
    // dereference is looked up first (a host-side query that allocates nothing); nothing is launched on failure.
    {
        const void *ptrs[10] = {fsurv, n_out, k ? ids_out : nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr};
        if (idx->n_blocks) {
            ptrs[3] = idx->agent; ptrs[4] = idx->depth; ptrs[5] = idx->ref_count; ptrs[6] = idx->flags;
            ptrs[7] = idx->last_access; ptrs[8] = idx->n_tokens;
        }
        for (int i = 0; i < 10; ++i)
            if (ptrs[i] && !cs_device_can_address(ptrs[i])) return CS_EINVAL;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= CS_STATIC_MAX_DEVICES) return CS_ECUDA;
    int stream_dev = dev;        // the array of the CURRENT device is used: a stream of another device is refused
    if (stream && cudaStreamGetDevice((cudaStream_t)stream, &stream_dev) == cudaSuccess && stream_dev != dev) return CS_EINVAL;
    (void)cudaGetLastError();
    {
        // first call on this device: resolve the device address of the array (once, with the device current)
        std::lock_guard<std::mutex> lock(g_static_mu);
        if (!g_static_ptr[dev]) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, cs_static_scratch) != cudaSuccess || !ptr) return CS_ECUDA;
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return CS_ECUDA;
            g_static_sms[dev] = sms;
            g_static_ptr[dev] = (unsigned char *)ptr;
        }
    }
    unsigned char *base;
    int sms;
    {
        std::lock_guard<std::mutex> lock(g_static_mu);
        base = g_static_ptr[dev];
        sms = g_static_sms[dev];
    }
    cs_ctx ctx;                                        // host-side descriptor only; nothing is allocated
    memset(&ctx, 0, sizeof(ctx));
    ctx.p = *p;
    ctx.p.max_blocks = CS_STATIC_MAX_BLOCKS;
    cs_recency_table_shape(p, &ctx.gtab_len, &ctx.age_sat);
    ctx.device = dev;
    ctx.sm_count = sms;
    cs_workspace &ws = ctx.ws;
    ws.sc = (cs_scalars *)(base + CS_SO_SC);
    ws.sel = (cs_sel_state *)(base + CS_SO_SEL);
    ws.gtab = (float *)(base + CS_SO_GTAB);
    ws.hist = (uint32_t *)(base + CS_SO_HIST);
    ws.spl_km = (unsigned long long *)(base + CS_SO_SPLKM);
    ws.spl_id = (uint32_t *)(base + CS_SO_SPLID);
    ws.bcount = (uint32_t *)(base + CS_SO_BCOUNT);
    ws.cand_km = (unsigned long long *)(base + CS_SO_CANDKM);
    ws.sort_km = (unsigned long long *)(base + CS_SO_SORTKM);
    ws.cand_id = (uint32_t *)(base + CS_SO_CANDID);
    ws.cand_bkt = (uint32_t *)(base + CS_SO_CANDBKT);
    ws.cand_slot = (uint32_t *)(base + CS_SO_CANDSLOT);
    ws.sort_id = (uint32_t *)(base + CS_SO_SORTID);
    ws.cnt = (cs_counters *)(base + CS_SO_CNT);
    ws.fsurv = const_cast<float *>(fsurv);             // input table, read only
    cudaStream_t s = (cudaStream_t)stream;
    cs_static_prepare_kernel<<<16, 256, 0, s>>>(ws, ctx.gtab_len, p->lambda, p->delta);
    if ((rc = cs_check_launch(&ctx)) != CS_OK) return rc;
    return cs_launch_select(&ctx, idx, now, 0, tier, k, ids_out, n_out, s);
}
