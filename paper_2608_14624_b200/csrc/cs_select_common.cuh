// Device helpers shared by the select kernels: the per-entry eligibility rules and 96-bit key
// (Algorithm 1, Evict / BetweenStep; Eq. 9), 128-bit loads of the SoA block index, small tables.
#pragma once
#include "cs_common.cuh"

#define SEL_THREADS 512
#define GRP 16                    // index entries per thread and iteration

struct SelArgs {
    const uint16_t *agent;
    const uint16_t *depth;
    const uint8_t *ref;
    const uint8_t *flags;
    const uint32_t *la;
    const uint8_t *ntok;
    const uint16_t *anchor;
    const float *fsurv;
    uint32_t n, now, A, block_tokens, gtab_len, age_sat;
    float lambda, delta;
    uint32_t tier, k, prefer_copy;
    uint32_t use_age_limits;      // collect pass may prefilter by per-(agent, size) age limits (large indexes)
    uint32_t hint_slot;           // which remembered threshold bin this call may speculate on
    uint32_t kind;                // 0 GPU-tier victims, 1 host-tier victims, 2 prefetch candidates (work counters)
    const uint32_t *now_dev;      // when set, the clock is read from device memory at execution time (graph replay)
    uint32_t sort_cap;            // keys the sort region holds (0: buckets never get fixed regions)
    uint32_t region_cap_max;      // cap on a bucket's own region (0: none)
};

// host helpers defined in cs_select.cu
void cs_fill_sel_args(const cs_ctx *ctx, const cs_block_index *idx, uint32_t now, const float *fsurv, SelArgs &a);
uint32_t cs_scan_grid(const cs_ctx *ctx, uint32_t n, uint32_t per_cta, uint32_t ctas_per_sm = 2);
size_t cs_table_smem(const cs_ctx *ctx);

// A group of whole warps of a CTA that synchronises on a barrier of its own, so that two halves of a CTA can work on
// different things at the same time: t = index of the calling thread within the group, n = its threads,
// bar = hardware barrier (0 = the one of __syncthreads(), for the whole CTA).
struct CtaPart { uint32_t t, n, bar; };
__device__ __forceinline__ CtaPart whole_cta() { return CtaPart{threadIdx.x, blockDim.x, 0u}; }
__device__ __forceinline__ void part_sync(const CtaPart &p)
{
    asm volatile("bar.sync %0, %1;" ::"r"(p.bar), "r"(p.n) : "memory");
}

// What the next call of this kind may collect ahead of its own threshold.  The threshold bin of consecutive
// calls moves little, so the next call's first scan appends every entry up to a remembered bin.  That bin is
// chosen from this call's exact histogram: the furthest bin whose cumulative population stays within
// 3 k + 1024 entries, at least the threshold bin itself and at most CS_SPEC_MAX_AHEAD bins beyond it.  Sparse
// bins (a prefetch list whose best entries leave the tier every call, so its threshold jumps) get several bins
// of slack for a few thousand extra candidates; dense bins get none.  Only the amount of work depends on this,
// never the result.  `loc` are the calling thread's bins [first, first + PER), `before` the population below
// them; every thread of the group calls; s_lim is a shared word.
#define CS_SPEC_MAX_AHEAD 8u
template <uint32_t PER>
__device__ __forceinline__ uint32_t collect_ahead_limit(const uint32_t (&loc)[PER], uint32_t first, uint32_t before,
                                                        uint32_t k, uint32_t b0, uint32_t *s_lim, const CtaPart &cp)
{
    if (cp.t == 0) *s_lim = 0;
    part_sync(cp);
    const unsigned long long cap = 3ull * k + 1024ull;
    unsigned long long run = before;
    uint32_t best = 0xFFFFFFFFu;
#pragma unroll
    for (uint32_t q = 0; q < PER; ++q) {
        run += loc[q];
        if (run <= cap) best = first + q;
    }
    if (best != 0xFFFFFFFFu) atomicMax(s_lim, best);
    part_sync(cp);
    uint32_t lim = *s_lim;
    if (lim < b0) lim = b0;
    if (lim > b0 + CS_SPEC_MAX_AHEAD) lim = b0 + CS_SPEC_MAX_AHEAD;
    return lim < CS_HIST_BINS ? lim : CS_HIST_BINS - 1;
}

__device__ __forceinline__ void remember_threshold(cs_scalars *sc, uint32_t slot, bool valid, uint32_t limit)
{
    if (slot < 3) sc->sel_hint[slot] = valid ? limit : 0xFFFFFFFFu;
}

// Work counters of one finished select (called by one thread).
__device__ __forceinline__ void count_select(const cs_workspace &ws, uint32_t kind, uint32_t n_elig, uint32_t n_out)
{
    if (kind > 2) return;
    atomicAdd((unsigned long long *)&ws.cnt->selects[kind], 1ull);
    atomicAdd((unsigned long long *)&ws.cnt->selected[kind], (unsigned long long)n_out);
    ws.cnt->eligible[kind] = n_elig;
}

__device__ __forceinline__ void count_candidates(const cs_workspace &ws, uint32_t kind, uint32_t c, bool fast_hit)
{
    if (kind > 2) return;
    ws.cnt->candidates[kind] = c;
    if (fast_hit) atomicAdd((unsigned long long *)&ws.cnt->fast_hits[kind], 1ull);
}

// The clock of a call: by value, or from device memory when the caller asked for that.
__device__ __forceinline__ void resolve_now(SelArgs &a)
{
    if (a.now_dev) a.now = __ldg(a.now_dev);
}

// Per-CTA copies of the small tables every entry looks up.
struct Tables {
    float *fsurv;       // [A]
    float *gtab;        // [gtab_len]
    uint16_t *anchor;   // [A] or unused
    float g_sat;
    uint32_t a_star;
};

// The recency table depends only on the context's constants (written when the context was created), so a kernel
// launched with programmatic dependent launch may copy it before it waits for its predecessor ...
__device__ __forceinline__ void load_tables_static(const SelArgs &a, const cs_workspace &ws, float *smem, Tables &T)
{
    T.fsurv = smem;
    T.gtab = smem + a.A;
    T.anchor = (uint16_t *)(smem + a.A + a.gtab_len);
    for (uint32_t i = threadIdx.x; i < a.gtab_len; i += blockDim.x) T.gtab[i] = ws.gtab[i];
    T.g_sat = cs_recency(a.lambda, a.delta, a.age_sat);
}
// ... while the survival table, the anchor lengths and a* may have been written by that predecessor.
__device__ __forceinline__ void load_tables_dynamic(const SelArgs &a, const cs_workspace &ws, Tables &T, bool want_anchor)
{
    for (uint32_t i = threadIdx.x; i < a.A; i += blockDim.x) T.fsurv[i] = a.fsurv[i];
    if (want_anchor)
        for (uint32_t i = threadIdx.x; i < a.A; i += blockDim.x) T.anchor[i] = a.anchor[i];
    T.a_star = ws.sc->a_star;           // arg-max successor of the current agent, kept by the learner refresh
}

__device__ __forceinline__ void load_tables(const SelArgs &a, const cs_workspace &ws, float *smem, Tables &T,
                                            bool want_anchor)
{
    load_tables_static(a, ws, smem, T);
    load_tables_dynamic(a, ws, T, want_anchor);
}

// Recency factor of Eq. 9 for an age: from the table, the saturated constant, or (a decay so slow that the
// table does not reach saturation) computed directly.
__device__ __forceinline__ float recency_of_age(const SelArgs &a, const Tables &T, uint32_t age)
{
    if (age < a.gtab_len) return T.gtab[age];
    if (age >= a.age_sat) return T.g_sat;
    return cs_recency(a.lambda, a.delta, age);
}

__device__ __forceinline__ float score_from_age(const SelArgs &a, const Tables &T, uint32_t agent, uint32_t age,
                                                uint32_t tok)
{
    return __fmul_rn(__fmul_rn(T.fsurv[agent], recency_of_age(a, T, age)), (float)tok);      // two roundings, never an FMA
}

// ---------------------------------------------------------------------------------------------
// Threshold test without the key.  The score is fl(fl(f * g) * |b|) and IEEE multiplication by a positive
// constant never decreases when its operand grows, so "the first key digit is at most H" is, for a fixed
// block size, an interval of x = fl(f * g): victims  x < X[|b|],  prefetch candidates  x >= X[class][|b|]
// (class 0: blocks of a*, class 1: the rest).  X is found once per CTA by binary search over the bit
// patterns of positive floats; an entry then costs two table look-ups, one multiply and one compare, and only
// the few entries that pass get a key.  Exact: it is the same product the key is made of.
// ---------------------------------------------------------------------------------------------
#define XT_TOK 256u                // |b| is a u8
#define XT_NONE 0x7F800001u        // above every finite pattern

// smallest bit pattern x in [0, +inf] with bits(fl(x * tok)) >= lim; XT_NONE when there is none
__device__ __forceinline__ uint32_t first_x_reaching(unsigned long long lim, uint32_t tok)
{
    uint32_t lo = 0, hi = 0x7F800001u;
    const float t = (float)tok;
    while (lo < hi) {
        const uint32_t mid = lo + ((hi - lo) >> 1);
        const unsigned long long bits = __float_as_uint(__fmul_rn(__uint_as_float(mid), t));
        if (bits >= lim) hi = mid;
        else lo = mid + 1;
    }
    return lo;
}

// Fills xt[2][XT_TOK] for the remembered bin H (every thread of the CTA calls; synchronise afterwards).
template <bool PF>
__device__ __forceinline__ void build_x_thresholds(const SelArgs &a, uint32_t H, uint32_t *xt)
{
    for (uint32_t e = threadIdx.x; e < 2 * XT_TOK; e += blockDim.x) {
        const uint32_t cls = e / XT_TOK, tok = e % XT_TOK;
        uint32_t x;
        if (!PF) {
            // bin = bits >> 20 (bits >> 19 with the copy-preference bit below the score): candidate <=> bits < lim
            const unsigned long long lim = (unsigned long long)(H + 1u) << (a.prefer_copy ? 19 : 20);
            x = first_x_reaching(lim, tok);                                  // candidate <=> x bits < this
        } else if (cls == 0) {
            // a*: bin = (0x7FFFFFFF - bits) >> 20 <= H  <=>  bits >= 0x80000000 - ((H + 1) << 20)
            x = H >= 2047u ? 0u : first_x_reaching(0x80000000ull - ((unsigned long long)(H + 1u) << 20), tok);
        } else {
            // the rest: bin = 2048 + ((0x7FFFFFFF - bits) >> 20)
            x = H < 2048u ? XT_NONE : (H >= 4095u ? 0u : first_x_reaching(0x80000000ull - ((unsigned long long)(H - 2047u) << 20), tok));
        }
        xt[e] = x;                                                           // prefetch: candidate <=> x bits >= this
    }
}

__device__ __forceinline__ float score_of(const SelArgs &a, const Tables &T, uint32_t agent, uint32_t la,
                                          uint32_t tok)
{
    const uint32_t age = la <= a.now ? a.now - la : 0u;
    float g;
    if (age < a.gtab_len) g = T.gtab[age];
    else if (age >= a.age_sat) g = T.g_sat;
    else g = cs_recency(a.lambda, a.delta, age);
    return __fmul_rn(__fmul_rn(T.fsurv[agent], g), (float)tok);      // two roundings, never an FMA
}

// Key of an entry already known to pass the flag / ref_count rules: the agent range check, the
// anchor-depth rule of the prefetch list, and the 96-bit key.
template <bool PF>
__device__ __forceinline__ bool entry_key_rest(const SelArgs &a, const Tables &T, uint32_t *status, uint32_t agent,
                                               uint32_t depth, uint32_t flags, uint32_t la, uint32_t tok,
                                               uint32_t &primary, uint32_t &secondary)
{
    if (agent >= a.A) { atomicOr(status, CS_ST_BAD_AGENT); return false; }
    if (PF && a.anchor && !(depth < T.anchor[agent])) return false;
    const uint32_t bits = __float_as_uint(score_of(a, T, agent, la, tok));
    if (PF) {
        primary = ((agent == T.a_star) ? 0u : 0x80000000u) | (~bits & 0x7FFFFFFFu);
        secondary = ~la;
    } else {
        // Optional preference (Sec. 4) for victims whose contents already exist on the other tier:
        // one extra key bit right below the score (a positive float leaves bit 31 free).
        primary = a.prefer_copy ? ((bits << 1) | ((flags & CS_FLAG_OTHER_COPY) ? 0u : 1u)) : bits;
        secondary = la;
    }
    return true;
}

// Eligibility and key of one entry.  PF = prefetch-candidate rules, else eviction-victim rules.
template <bool PF>
__device__ __forceinline__ bool entry_key(const SelArgs &a, const Tables &T, uint32_t *status, uint32_t agent,
                                          uint32_t depth, uint32_t ref, uint32_t flags, uint32_t la, uint32_t tok,
                                          uint32_t &primary, uint32_t &secondary)
{
    if (!(flags & CS_FLAG_VALID) || (flags & CS_FLAG_PINNED) || ref != 0) return false;
    if (PF) {
        if (!(flags & CS_FLAG_TIER_HOST) || (flags & CS_FLAG_OTHER_COPY)) return false;
    } else {
        if (((flags >> 2) & 1u) != a.tier) return false;
    }
    return entry_key_rest<PF>(a, T, status, agent, depth, flags, la, tok, primary, secondary);
}

// The index is walked in warp tiles of 512 entries.  In step q (0..3) lane L owns the four
// consecutive entries tile*512 + q*128 + 4L .. +3, so every load instruction of a warp covers one
// contiguous, fully used span: 512 B of last_access (128-bit loads), 256 B of agent / depth
// (64-bit), 128 B of flags / ref_count / n_tokens (32-bit).  A thread's 16 entries are numbered
// j = 4q + r locally; Group keeps them in the order the accessors below expect.
#define TILE 512u
struct Group {
    uint4 ag0, ag1, dp0, dp1, rf, fl, la0, la1, la2, la3, tk;
};

__device__ __forceinline__ uint32_t grp_id(uint32_t tile, uint32_t lane, int j)
{
    return tile * TILE + (uint32_t)(j >> 2) * 128u + 4u * lane + (uint32_t)(j & 3);
}

template <bool PF, bool FLAGS = true>
__device__ __forceinline__ void load_group(const SelArgs &a, uint32_t tile, uint32_t lane, Group &G)
{
    const uint32_t q0 = tile * 128u + lane;            // index of this lane's first quad, in units of 4 entries
    const uint4 *la = (const uint4 *)a.la + q0;
    G.la0 = __ldg(la);
    G.la1 = __ldg(la + 32);
    G.la2 = __ldg(la + 64);
    G.la3 = __ldg(la + 96);
    const uint2 *ag = (const uint2 *)a.agent + q0;
    const uint2 g0 = __ldg(ag), g1 = __ldg(ag + 32), g2 = __ldg(ag + 64), g3 = __ldg(ag + 96);
    G.ag0 = make_uint4(g0.x, g0.y, g1.x, g1.y);
    G.ag1 = make_uint4(g2.x, g2.y, g3.x, g3.y);
    if (FLAGS) {
        const uint32_t *rf = (const uint32_t *)a.ref + q0, *fl = (const uint32_t *)a.flags + q0;
        G.rf = make_uint4(__ldg(rf), __ldg(rf + 32), __ldg(rf + 64), __ldg(rf + 96));
        G.fl = make_uint4(__ldg(fl), __ldg(fl + 32), __ldg(fl + 64), __ldg(fl + 96));
    }
    if (a.ntok) {
        const uint32_t *tk = (const uint32_t *)a.ntok + q0;
        G.tk = make_uint4(__ldg(tk), __ldg(tk + 32), __ldg(tk + 64), __ldg(tk + 96));
    }
    if (PF && a.anchor) {
        const uint2 *dp = (const uint2 *)a.depth + q0;
        const uint2 d0 = __ldg(dp), d1 = __ldg(dp + 32), d2 = __ldg(dp + 64), d3 = __ldg(dp + 96);
        G.dp0 = make_uint4(d0.x, d0.y, d1.x, d1.y);
        G.dp1 = make_uint4(d2.x, d2.y, d3.x, d3.y);
    }
}

__device__ __forceinline__ uint32_t u4_word(const uint4 &v, int w)
{
    return w == 0 ? v.x : (w == 1 ? v.y : (w == 2 ? v.z : v.w));
}
__device__ __forceinline__ uint32_t grp_u16(const uint4 &lo, const uint4 &hi, int j)   // j in [0,16)
{
    const uint32_t w = u4_word(j < 8 ? lo : hi, (j & 7) >> 1);
    return (w >> ((j & 1) * 16)) & 0xFFFFu;
}
__device__ __forceinline__ uint32_t grp_u8(const uint4 &v, int j)
{
    return (u4_word(v, j >> 2) >> ((j & 3) * 8)) & 0xFFu;
}
__device__ __forceinline__ uint32_t grp_u32(const Group &G, int j)
{
    const uint4 &v = j < 4 ? G.la0 : (j < 8 ? G.la1 : (j < 12 ? G.la2 : G.la3));
    return u4_word(v, j & 3);
}

// Flag / ref_count rules for the 16 entries of a group at once, four entries per 32-bit word
// (byte-wise SIMD compares): bit j of the result is set when entry j is VALID, not PINNED, on the
// requested tier (prefetch: on the host tier without a GPU copy) and unreferenced.
// 0x80 in every byte of x that is zero (exact for all four bytes at once, plain integer operations).
__device__ __forceinline__ uint32_t zero_bytes(uint32_t x)
{
    return ~(((x & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | x | 0x7F7F7F7Fu);
}
// The four 0x80 flags of a word gathered into a nibble (bit i = byte i).
__device__ __forceinline__ uint32_t nibble_of_flags(uint32_t t)
{
    return (((t >> 7) * 0x01020408u) >> 24) & 0xFu;
}

template <bool PF>
__device__ __forceinline__ uint32_t group_elig(const SelArgs &a, const Group &G)
{
    const uint32_t fmask = PF ? 0x0F0F0F0Fu : 0x07070707u;
    const uint32_t fpat = PF ? 0x05050505u : (0x01010101u * (CS_FLAG_VALID | (a.tier << 2)));
    uint32_t out = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        // a byte of x is zero exactly when the entry's flags match the pattern and its ref_count is 0
        const uint32_t x = ((u4_word(G.fl, w) & fmask) ^ fpat) | u4_word(G.rf, w);
        out |= nibble_of_flags(zero_bytes(x)) << (4 * w);
    }
    return out;
}

// Calls f(id, primary, secondary) for every eligible entry this thread owns: whole warp tiles
// grid-strided, then the ragged tail (n % 512 entries) one entry per thread.
template <bool PF, typename F>
__device__ __forceinline__ void for_each_eligible(const SelArgs &a, const Tables &T, uint32_t *status, F f)
{
    const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    const uint32_t lane = threadIdx.x & 31, n_tiles = a.n / TILE;
    for (uint32_t t = gtid >> 5; t < n_tiles; t += nth >> 5) {
        Group G;
        load_group<PF>(a, t, lane, G);
        const uint32_t em = group_elig<PF>(a, G);
#pragma unroll
        for (int j = 0; j < GRP; ++j) {
            if (!((em >> j) & 1u)) continue;
            uint32_t pr, se;
            const uint32_t tok = a.ntok ? grp_u8(G.tk, j) : a.block_tokens;
            const uint32_t dp = (PF && a.anchor) ? grp_u16(G.dp0, G.dp1, j) : 0u;
            if (entry_key_rest<PF>(a, T, status, grp_u16(G.ag0, G.ag1, j), dp, grp_u8(G.fl, j), grp_u32(G, j), tok, pr, se))
                f(grp_id(t, lane, j), pr, se);
        }
    }
    const uint32_t t0 = n_tiles * TILE;
    if (gtid < a.n - t0) {
        const uint32_t i = t0 + gtid;
        uint32_t pr, se;
        const uint32_t tok = a.ntok ? a.ntok[i] : a.block_tokens;
        if (entry_key<PF>(a, T, status, a.agent[i], a.depth[i], a.ref[i], a.flags[i], a.la[i], tok, pr, se))
            f(i, pr, se);
    }
}

// Warp-private staging of candidates.  Inside the 16-entry loop of a scan every lane holds at most one
// candidate per step; a ballot gives each its slot in the warp's shared-memory slice, with no atomic and no
// second pass over the group.  A slice that is more than half full is appended to the global candidate
// buffer: one atomic per flush, coalesced writes.  Every call below is made by all 32 lanes of the warp.
#define STAGE_CAP 64u
struct WarpStage {
    unsigned long long *km;      // [STAGE_CAP]
    uint32_t *id;                // [STAGE_CAP]
    uint32_t n;                  // staged entries (same value in every lane)
};

__device__ __forceinline__ void stage_init(WarpStage &st, unsigned long long *km_all, uint32_t *id_all)
{
    const uint32_t warp = threadIdx.x >> 5;
    st.km = km_all + warp * STAGE_CAP;
    st.id = id_all + warp * STAGE_CAP;
    st.n = 0;
}

__device__ __forceinline__ void stage_flush(WarpStage &st, uint32_t *counter, unsigned long long *out_km, uint32_t *out_id)
{
    if (st.n == 0) return;
    const uint32_t lane = threadIdx.x & 31;
    __syncwarp();
    uint32_t base = 0;
    if (lane == 0) base = atomicAdd(counter, st.n);
    base = __shfl_sync(0xFFFFFFFFu, base, 0);
    for (uint32_t i = lane; i < st.n; i += 32) {
        out_km[base + i] = st.km[i];
        out_id[base + i] = st.id[i];
    }
    __syncwarp();
    st.n = 0;
}

__device__ __forceinline__ void stage_push(WarpStage &st, bool cand, uint32_t pr, uint32_t se, uint32_t id,
                                           uint32_t *counter, unsigned long long *out_km, uint32_t *out_id)
{
    const uint32_t b = __ballot_sync(0xFFFFFFFFu, cand);
    if (b == 0) return;
    if (cand) {
        const uint32_t pos = st.n + __popc(b & ((1u << (threadIdx.x & 31)) - 1u));
        st.km[pos] = ((unsigned long long)pr << 32) | se;
        st.id[pos] = id;
    }
    st.n += __popc(b);
    if (st.n > STAGE_CAP - 32u) stage_flush(st, counter, out_km, out_id);
}

// The prefetch list is empty unless the gate of Eq. 11 is open and a current agent exists.
__device__ __forceinline__ bool prefetch_enabled(const cs_workspace &ws, uint32_t A)
{
    return ws.sc->gate != 0 && ws.sc->last_agent < A;
}

__device__ __forceinline__ bool last_cta_done(uint32_t *ticket, bool *s_flag)
{
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *s_flag = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    const bool last = *s_flag;
    if (last) __threadfence();
    return last;
}

// Exclusive prefix sum of one value per thread over a group of warps (warp shuffles, three barriers); also returns
// the total.  s_part: at least 64 words.
__device__ __forceinline__ uint32_t sel_block_scan(uint32_t v, uint32_t *s_part, uint32_t &total, const CtaPart &cp)
{
    const uint32_t lane = cp.t & 31, warp = cp.t >> 5, n_warps = cp.n >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += t;
    }
    part_sync(cp);
    if (lane == 31) s_part[warp] = incl;
    part_sync(cp);
    if (warp == 0) {
        uint32_t w = lane < n_warps ? s_part[lane] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, w, d);
            if (lane >= d) w += t;
        }
        s_part[32 + lane] = w;                         // inclusive warp totals
    }
    part_sync(cp);
    total = s_part[32 + n_warps - 1];
    const uint32_t before = warp ? s_part[32 + warp - 1] : 0;
    return before + incl - v;
}

__device__ __forceinline__ bool key_less(unsigned long long km_a, uint32_t id_a, unsigned long long km_b,
                                         uint32_t id_b)
{
    return km_a < km_b || (km_a == km_b && id_a < id_b);
}



// ---------------------------------------------------------------------------------------------
// Bitonic sort of P keys (power of two, 64 <= P <= 2 * threads of the group) held in shared memory,
// ascending by (km, id).  Each thread keeps two neighbouring elements in registers; compare-
// exchange steps whose partner lies in the same warp (element distance <= 32) use shuffles and
// no barrier, only the longer distances go through shared memory.  Called by every thread of the group.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void cx_keep(unsigned long long &k, uint32_t &i, unsigned long long pk, uint32_t pi,
                                        bool keep_min)
{
    const bool partner_less = key_less(pk, pi, k, i);
    if (partner_less == keep_min) { k = pk; i = pi; }
}

__device__ __forceinline__ void bitonic_sort_fast(unsigned long long *km, uint32_t *id, uint32_t P, const CtaPart &cp)
{
    const uint32_t t = cp.t;
    const bool act = t < P / 2;                           // whole warps, because P >= 64
    unsigned long long k0 = 0, k1 = 0;
    uint32_t i0 = 0, i1 = 0;
    if (act) { k0 = km[2 * t]; k1 = km[2 * t + 1]; i0 = id[2 * t]; i1 = id[2 * t + 1]; }
    for (uint32_t size = 2; size <= P; size <<= 1) {
        const bool up = ((2 * t) & size) == 0;            // both of this thread's elements share the direction
        uint32_t stride = size >> 1;
        if (stride >= 64) {                               // partners in other warps: through shared memory
            if (act) { km[2 * t] = k0; km[2 * t + 1] = k1; id[2 * t] = i0; id[2 * t + 1] = i1; }
            part_sync(cp);
            for (; stride >= 64; stride >>= 1) {
                if (act) {
                    const uint32_t lo = 2 * t - (t & (stride - 1)), hi = lo + stride;
                    const bool up2 = (lo & size) == 0;
                    const unsigned long long ka = km[lo], kb = km[hi];
                    const uint32_t ia = id[lo], ib = id[hi];
                    if (key_less(kb, ib, ka, ia) == up2) { km[lo] = kb; id[lo] = ib; km[hi] = ka; id[hi] = ia; }
                }
                part_sync(cp);
            }
            if (act) { k0 = km[2 * t]; k1 = km[2 * t + 1]; i0 = id[2 * t]; i1 = id[2 * t + 1]; }
        }
        if (act) {
            for (; stride >= 2; stride >>= 1) {           // partner thread t ^ (stride / 2), same warp
                const uint32_t d = stride >> 1;
                const unsigned long long pk0 = __shfl_xor_sync(0xFFFFFFFFu, k0, d), pk1 = __shfl_xor_sync(0xFFFFFFFFu, k1, d);
                const uint32_t pi0 = __shfl_xor_sync(0xFFFFFFFFu, i0, d), pi1 = __shfl_xor_sync(0xFFFFFFFFu, i1, d);
                const bool keep_min = ((t & d) == 0) == up;
                cx_keep(k0, i0, pk0, pi0, keep_min);
                cx_keep(k1, i1, pk1, pi1, keep_min);
            }
            if (key_less(k1, i1, k0, i0) == up) {         // distance 1: this thread's own pair
                const unsigned long long tk = k0; k0 = k1; k1 = tk;
                const uint32_t ti = i0; i0 = i1; i1 = ti;
            }
        }
    }
    part_sync(cp);
    if (act) { km[2 * t] = k0; km[2 * t + 1] = k1; id[2 * t] = i0; id[2 * t + 1] = i1; }
    part_sync(cp);
}
