// Transition Learner and Survival Scorer state: transition counting (Algorithm 1,
// ObserveTouch), Eq. 3 normalisation with row arg-max (Eq. 5 / Eq. 10), predictability
// (Eq. 2) and gate (Eq. 11), threshold graph (Eq. 7), BFS hop table and survival scores
// (Eq. 8).  The model is tiny (A <= 1024), so these kernels are latency-bound: the design
// goal is few launches and no host round trip, not bandwidth.
#include "cs_common.cuh"

#define OBS_THREADS 1024
#define ROW_THREADS 256
#define OBS_FUSED_MAX 256u     // events up to which a batch is applied inside the refresh launch (one per thread)
static_assert(OBS_FUSED_MAX == ROW_THREADS, "the refresh kernel stages one event per thread");

// ---------------------------------------------------------------------------------------------
// Initial state of Algorithm 1: zero counts, no current agent; plus the recency table.
// ---------------------------------------------------------------------------------------------
__global__ void cs_init_kernel(cs_workspace ws, uint32_t A, uint32_t n_chains, uint32_t gtab_len, float lambda,
                               float delta)
{
    const uint32_t tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    for (uint32_t i = tid; i < A * A; i += nth) ws.C[i] = 0;
    for (uint32_t i = tid; i < A; i += nth) { ws.rowsum[i] = 0; ws.qfix[i] = 0; }
    for (uint32_t i = tid; i < n_chains; i += nth) ws.cur[i] = CS_AGENT_NONE;
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
    }
}

// The recency factor must not increase with age for the select's age-limit prefilter to be exact.
// exp() is monotone mathematically; this checks the table that was actually produced.
__global__ void cs_gtab_check_kernel(cs_workspace ws, uint32_t gtab_len, uint32_t age_sat, float lambda, float delta)
{
    __shared__ int s_bad;
    if (threadIdx.x == 0) s_bad = (gtab_len != age_sat) ? 1 : 0;
    __syncthreads();
    const float g_sat = cs_recency(lambda, delta, age_sat);
    for (uint32_t i = threadIdx.x; i < gtab_len; i += blockDim.x) {
        const float next = (i + 1 < gtab_len) ? ws.gtab[i + 1] : g_sat;
        if (next > ws.gtab[i]) s_bad = 1;
    }
    __syncthreads();
    if (threadIdx.x == 0) ws.sc->gtab_monotone = s_bad ? 0u : 1u;
}

// ---------------------------------------------------------------------------------------------
// Transition counting over one batch of events, one CTA.  The update is sequential per chain
// (each event's predecessor is the previous non-warmup event of the same chain, in this batch
// or carried in cur[]), but the counter increments commute, so every event is handled by its
// own thread: it looks its predecessor up in the shared-memory copy of the batch and adds 1
// atomically.  Integer adds make the result independent of the order the atomics land in.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(OBS_THREADS)
cs_observe_kernel(cs_workspace ws, uint32_t A, uint32_t n_chains, const uint32_t *__restrict__ chain,
                  const uint16_t *__restrict__ agent, const uint8_t *__restrict__ evflags, uint32_t n_events,
                  const uint32_t *__restrict__ n_events_dev)
{
    cs_wait_for_predecessor();
    cs_release_successor();
    if (n_events_dev) n_events = min(n_events, *n_events_dev);     // device-resident count (graph replay)
    __shared__ uint32_t s_chain[OBS_THREADS];
    __shared__ uint16_t s_agent[OBS_THREADS];     // CS_AGENT_NONE marks an event that is skipped
    __shared__ int s_last;
    const int tid = threadIdx.x;
    if (tid == 0) atomicAdd((unsigned long long *)&ws.cnt->events_seen, (unsigned long long)n_events);
    for (uint32_t base = 0; base < n_events; base += OBS_THREADS) {
        const uint32_t e = base + tid;
        uint32_t c = 0, a = CS_AGENT_NONE;
        if (tid == 0) s_last = -1;
        if (e < n_events) {
            c = chain[e];
            a = agent[e];
            const bool warm = evflags && (evflags[e] & CS_EV_WARMUP);
            uint32_t bad = 0;
            if (!warm && a >= A) bad |= CS_ST_BAD_AGENT;
            if (!warm && c >= n_chains) bad |= CS_ST_BAD_CHAIN;
            if (bad) atomicOr(&ws.sc->status, bad);
            if (warm || bad) {
                a = CS_AGENT_NONE;
                atomicAdd((unsigned long long *)&ws.cnt->events_skipped, 1ull);
            }
        }
        s_chain[tid] = c;
        s_agent[tid] = (uint16_t)a;
        __syncthreads();
        const bool live = a != CS_AGENT_NONE;
        uint32_t prev = CS_AGENT_NONE;
        bool last_of_chain = live;
        if (live) {
            int j = tid - 1;
            for (; j >= 0; --j)
                if (s_chain[j] == c && s_agent[j] != CS_AGENT_NONE) { prev = s_agent[j]; break; }
            if (j < 0) prev = ws.cur[c];
            const int lim = min((int)OBS_THREADS, (int)(n_events - base));
            for (int q = tid + 1; q < lim; ++q)
                if (s_chain[q] == c && s_agent[q] != CS_AGENT_NONE) { last_of_chain = false; break; }
            atomicMax(&s_last, tid);
        }
        __syncthreads();                       // every read of cur[] above precedes the writes below
        if (live) {
            if (prev != CS_AGENT_NONE && prev != a) {
                atomicAdd(&ws.C[prev * A + a], 1u);
                atomicAdd(&ws.rowsum[prev], 1u);
                atomicAdd(&ws.sc->n_transitions, 1u);
                atomicAdd((unsigned long long *)&ws.cnt->transitions_counted, 1ull);
            }
            if (last_of_chain) ws.cur[c] = (uint16_t)a;
            if (s_last == tid) ws.sc->last_agent = a;
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------
// BFS over the bit-matrix graph from a set of source bits, then Eq. 8.  Runs inside one CTA.
// s_front: 64 words (two frontiers, used in turn), s_visit / s_next: 32 words each, s_hops: one entry per agent.
//
// Up to one agent per thread the search PULLS: thread v holds row v of the TRANSPOSED adjacency matrix (the
// predecessors of v; kept up to date in global memory by the refresh, fetched ahead of time into registers) and at
// every level ANDs it with the frontier.  A level is then W broadcast loads and ANDs per node, all nodes in
// parallel, one ballot per warp for the next frontier and ONE barrier -- whatever the frontier size, with no
// atomics and no divergent loops.  (A push over the frontier's nodes by one warp was tried: lanes that walk
// different frontier words run one after the other, 80 cycles per node.  So was a transpose built in shared memory
// by this CTA: 3 us of shared-memory atomics.)
// More agents take the level-synchronous push from global memory: a node of the current frontier ORs its adjacency
// row into the next frontier (shared-memory atomics), two barriers per level.
// ---------------------------------------------------------------------------------------------
#define BFS_ROW_WORDS 8u                   // words of a row when the search pulls (one agent per thread: 256 agents)
struct BfsRow { uint32_t w[BFS_ROW_WORDS]; };
__device__ __forceinline__ bool cs_bfs_pulls(uint32_t A) { return A <= ROW_THREADS; }

// Row threadIdx.x of the transposed adjacency matrix, fetched so that the trip to global memory overlaps whatever
// the caller does in between (zero where the search will not pull, or for a thread without a node).
__device__ __forceinline__ void cs_bfs_load_row(const uint32_t *adjT, uint32_t A, uint32_t W, BfsRow &row)
{
    if (!cs_bfs_pulls(A)) {
#pragma unroll
        for (uint32_t w = 0; w < BFS_ROW_WORDS; ++w) row.w[w] = 0u;
        return;
    }
    const bool mine = threadIdx.x < A;
    const uint32_t *r = adjT + (mine ? threadIdx.x * W : 0u);          // (always a valid address; unused words are masked)
#pragma unroll
    for (uint32_t w = 0; w < BFS_ROW_WORDS; ++w) row.w[w] = cs_ld_cg_pinned(r + (w < W ? w : 0u));
#pragma unroll
    for (uint32_t w = 0; w < BFS_ROW_WORDS; ++w)
        if (!mine || w >= W) row.w[w] = 0u;
}

__device__ __forceinline__ void cs_bfs_survival(const uint32_t *__restrict__ adj, uint32_t A, uint32_t W, const BfsRow &rowT,
                                                uint32_t *s_front, uint32_t *s_visit, uint32_t *s_next, uint16_t *s_hops,
                                                uint16_t *hops, float *fsurv, uint32_t e_max, float delta)
{
    // on entry s_front[0 .. 32) holds the source bits and s_front[32 .. 64) zeroes (synchronised by the caller)
    const uint32_t tid = threadIdx.x;
    if (cs_bfs_pulls(A)) {
        const uint32_t v = tid;                                       // blockDim.x >= A
        bool seen = v >= A || ((s_front[v >> 5] >> (v & 31)) & 1u);
        uint32_t my_hops = (v < A && seen) ? 0u : CS_HOP_NONE;
        for (uint32_t level = 1; level <= A; ++level) {
            const uint32_t *cur = s_front + ((level & 1u) ? 0u : 32u);
            uint32_t *nxt = s_front + ((level & 1u) ? 32u : 0u);
            uint32_t hit = 0;
#pragma unroll
            for (uint32_t w = 0; w < BFS_ROW_WORDS; ++w) hit |= rowT.w[w] & cur[w];
            const bool fresh = hit != 0u && !seen;
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, fresh);
            if ((tid & 31u) == 0) nxt[tid >> 5] = word;
            if (fresh) { seen = true; my_hops = level; }
            if (!__syncthreads_or(fresh)) break;
        }
        if (v < A) s_hops[v] = (uint16_t)my_hops;
    } else {
        for (uint32_t a = tid; a < A; a += blockDim.x)
            s_hops[a] = ((s_front[a >> 5] >> (a & 31)) & 1u) ? 0 : CS_HOP_NONE;
        if (tid < W) { s_visit[tid] = s_front[tid]; s_next[tid] = 0; }
        __syncthreads();
        for (uint32_t level = 1; level <= A; ++level) {
            for (uint32_t node = tid; node < A; node += blockDim.x) {
                if ((s_front[node >> 5] >> (node & 31)) & 1u) {
                    for (uint32_t w = 0; w < W; ++w) {
                        const uint32_t v = __ldcg(&adj[node * W + w]);
                        if (v) atomicOr(&s_next[w], v);
                    }
                }
            }
            __syncthreads();
            uint32_t acc = 0;
            if (tid < W) {
                acc = s_next[tid] & ~s_visit[tid];
                s_next[tid] = 0;
                s_front[tid] = acc;
                s_visit[tid] |= acc;
                uint32_t bits = acc;
                while (bits) {
                    const uint32_t b2 = tid * 32 + (__ffs(bits) - 1);
                    bits &= bits - 1;
                    if (b2 < A) s_hops[b2] = (uint16_t)level;
                }
            }
            if (!__syncthreads_or(acc != 0)) break;
        }
    }
    __syncthreads();
    for (uint32_t a = tid; a < A; a += blockDim.x) {
        const uint32_t h = s_hops[a];
        const uint32_t m = h < e_max ? h : e_max;          // CS_HOP_NONE > e_max by construction
        const double ptilde = 1.0 - (double)m / (double)e_max;
        hops[a] = (uint16_t)h;
        fsurv[a] = (float)(ptilde + (double)delta);
    }
}

// Deterministic block reductions: a fixed butterfly inside each warp, then the warp sums added in warp order, so the
// result does not depend on scheduling.  s_red: one entry per warp (two for the pair form).
template <typename T>
__device__ T cs_block_sum(T v, T *s_red)
{
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    __syncthreads();                                       // an earlier result may still be being read
    if (lane == 0) s_red[warp] = v;
    __syncthreads();
    T r = s_red[0];
    for (uint32_t w = 1; w < n_warps; ++w) r += s_red[w];
    return r;
}

__device__ void cs_block_sum2(double &a, double &b, double *s_red)
{
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        a += __shfl_xor_sync(0xFFFFFFFFu, a, d);
        b += __shfl_xor_sync(0xFFFFFFFFu, b, d);
    }
    __syncthreads();
    if (lane == 0) { s_red[warp] = a; s_red[32 + warp] = b; }
    __syncthreads();
    a = s_red[0];
    b = s_red[32];
    for (uint32_t w = 1; w < n_warps; ++w) { a += s_red[w]; b += s_red[32 + w]; }
}

// ---------------------------------------------------------------------------------------------
// One CTA per row i: Eq. 3 in canonical fp32 (one rounding per operation, no FMA), the row's
// arg-max, its adjacency bits (Eq. 7) and its entropy term.  The last CTA to finish then
// computes Eq. 2 / Eq. 11 over all rows and refreshes the cached BFS / Eq. 8 tables.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(ROW_THREADS)
cs_normalise_kernel(cs_workspace ws, uint32_t A, uint32_t W, float eps, float tau, float r_min, uint32_t e_max,
                    float delta, uint32_t all_chains, uint32_t n_chains, const uint32_t *__restrict__ ev_chain,
                    const uint16_t *__restrict__ ev_agent, const uint8_t *__restrict__ ev_flags, uint32_t n_events,
                    const uint32_t *__restrict__ n_events_dev)
{
    __shared__ uint32_t s_evc[OBS_FUSED_MAX];        // the batch: chain of event e,
    __shared__ uint16_t s_eva[OBS_FUSED_MAX];        // its agent (CS_AGENT_NONE: skipped),
    __shared__ uint16_t s_evp[OBS_FUSED_MAX];        // and the agent it follows when that is a counted transition
    __shared__ uint8_t s_succ[OBS_FUSED_MAX];        // 1: a later live event of the batch has the same chain
    __shared__ uint32_t s_add[CS_MAX_AGENTS];        // what the batch adds to the row being worked on
    __shared__ int s_last_live;
    __shared__ double s_red[64];
    __shared__ float s_bestv[ROW_THREADS / 32];
    __shared__ uint32_t s_besti[ROW_THREADS / 32];
    __shared__ uint32_t s_front[64], s_visit[32], s_next[32];
    __shared__ uint16_t s_hops[CS_MAX_AGENTS];
    __shared__ bool s_is_last;
    const uint32_t tid = threadIdx.x;
    CS_STAMP(ws, CS_PS_REFRESH_ENTRY, blockIdx.x == 0 && tid == 0);
    cs_wait_for_predecessor();
    CS_STAMP(ws, CS_PS_REFRESH_WAITED, blockIdx.x == 0 && tid == 0);
    cs_release_successor();

    // ---- a small batch of events is applied here, by every CTA to the rows it owns, instead of by a launch of its
    // own: each CTA stages the batch, finds every event's predecessor (in the batch, else the chain's current agent)
    // exactly as cs_observe_kernel does, and adds the transitions that start at row i to row i.  What is shared --
    // cur[], the last agent, the totals and the counters -- is written by the last CTA, after every CTA has read it.
    if (n_events_dev) n_events = min(n_events, *n_events_dev);
    uint32_t n_new = 0, n_skipped = 0;
    if (n_events) {
        uint32_t c = 0, a = CS_AGENT_NONE;
        if (tid == 0) s_last_live = -1;
        if (tid < n_events) {
            c = ev_chain[tid];
            a = ev_agent[tid];
            const bool warm = ev_flags && (ev_flags[tid] & CS_EV_WARMUP);
            uint32_t bad = 0;
            if (!warm && a >= A) bad |= CS_ST_BAD_AGENT;
            if (!warm && c >= n_chains) bad |= CS_ST_BAD_CHAIN;
            if (bad && blockIdx.x == 0) atomicOr(&ws.sc->status, bad);
            if (warm || bad) a = CS_AGENT_NONE;
        }
        s_evc[tid] = c;
        s_eva[tid] = (uint16_t)a;
        s_succ[tid] = 0;
        __syncthreads();
        const bool live = tid < n_events && a != CS_AGENT_NONE;
        uint32_t prev = CS_AGENT_NONE;
        if (live) {
            int j = (int)tid - 1;
            for (; j >= 0; --j)
                if (s_evc[j] == c && s_eva[j] != CS_AGENT_NONE) { prev = s_eva[j]; break; }
            if (j < 0) prev = ws.cur[c];
            else s_succ[j] = 1;                                // event j is not the last of its chain in this batch
            atomicMax(&s_last_live, (int)tid);
        }
        const bool counted = live && prev != CS_AGENT_NONE && prev != a;
        s_evp[tid] = (uint16_t)(counted ? prev : CS_AGENT_NONE);
        n_new = (uint32_t)__syncthreads_count(counted);
        n_skipped = (uint32_t)__syncthreads_count(tid < n_events && a == CS_AGENT_NONE);
    }
    // Column sums q_j = sum_i pi_i P_ij of Eq. 2 are accumulated by the row CTAs in 2^-60 fixed
    // point with integer atomics: integer addition commutes, so the sum is bit-identical from run
    // to run whatever order the CTAs finish in (a float atomic would not be).
    const uint32_t n_total = ws.sc->n_transitions + n_new;
    const uint32_t fill = ws.sc->adjT_cur ^ 1u;              // every CTA reads this before the last one flips it
    uint32_t *adjT_fill = ws.adjT + (size_t)fill * A * W, *adjT_clear = ws.adjT + (size_t)(fill ^ 1u) * A * W;
    const double inv_total = n_total ? 1.0 / (double)n_total : 0.0;
    for (uint32_t i = blockIdx.x; i < A; i += gridDim.x) {
        uint32_t n_i = ws.rowsum[i];
        // transitions of the batch that start at agent i
        const bool mine = n_events && tid < n_events && s_evp[tid] == i;
        const uint32_t row_new = n_events ? (uint32_t)__syncthreads_count(mine) : 0u;
        if (row_new) {
            for (uint32_t j = tid; j < A; j += ROW_THREADS) s_add[j] = 0;
            __syncthreads();
            if (mine) atomicAdd(&s_add[s_eva[tid]], 1u);
            __syncthreads();
            n_i += row_new;
            if (tid == 0) ws.rowsum[i] = n_i;
        }
        const double pi_fix = (double)n_i * inv_total * 1152921504606846976.0;      // pi_i * 2^60
        const float den = __fadd_rn((float)n_i, __fmul_rn((float)A, eps));
        // Most entries of a row have a zero count and therefore the same P = eps / den: their contribution to the
        // column sums is one number per row, added once to a scalar instead of A times to A columns; a column with a
        // count gets the difference on top.  Integer arithmetic, so the sums are bit for bit what A atomics per row gave.
        const long long base_fix = __double2ll_rn(pi_fix * (double)__fdiv_rn(__fadd_rn(0.0f, eps), den));
        if (tid == 0 && n_i) atomicAdd(&ws.sc->qbase, (unsigned long long)base_fix);
        float bestv = -1.0f;
        uint32_t besti = 0xFFFFFFFFu;
        double h = 0.0;
        for (uint32_t j0 = 0; j0 < A; j0 += ROW_THREADS) {       // A is padded to whole warps for the ballot
            const uint32_t j = j0 + tid;
            bool edge = false;
            if (j < A) {
                uint32_t cij = ws.C[i * A + j];
                if (row_new && s_add[j]) { cij += s_add[j]; ws.C[i * A + j] = cij; }
                const float p = __fdiv_rn(__fadd_rn((float)cij, eps), den);
                ws.P[i * A + j] = p;
                if (p > bestv) { bestv = p; besti = j; }         // strict: the lowest j among equals stays
                const double pd = (double)p;
                h += pd * log(pd);
                edge = p >= tau;
                if (n_i && cij) atomicAdd(&ws.qfix[j], (unsigned long long)(__double2ll_rn(pi_fix * pd) - base_fix));
            }
            const uint32_t bits = __ballot_sync(0xFFFFFFFFu, edge);
            if ((tid & 31) == 0 && (j >> 5) < W) ws.adj[i * W + (j >> 5)] = bits;
            if (edge) atomicOr(&adjT_fill[j * W + (i >> 5)], 1u << (i & 31));      // the transpose: i precedes j
        }
        for (uint32_t w = tid; w < W; w += ROW_THREADS) adjT_clear[i * W + w] = 0;  // for the refresh after this one
        // arg-max (max value, then min index) and the entropy term: a butterfly inside each warp, then the warp results
        // combined in warp order by thread 0
        const uint32_t lane = tid & 31, warp = tid >> 5;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            const float v = __shfl_xor_sync(0xFFFFFFFFu, bestv, d);
            const uint32_t x = __shfl_xor_sync(0xFFFFFFFFu, besti, d);
            if (v > bestv || (v == bestv && x < besti)) { bestv = v; besti = x; }
            h += __shfl_xor_sync(0xFFFFFFFFu, h, d);
        }
        __syncthreads();                                         // the partials of the row before have been read
        if (lane == 0) { s_bestv[warp] = bestv; s_besti[warp] = besti; s_red[warp] = h; }
        __syncthreads();
        if (tid == 0) {
            float bv = s_bestv[0];
            uint32_t bi = s_besti[0];
            double hs = s_red[0];
            for (uint32_t w = 1; w < ROW_THREADS / 32; ++w) {
                if (s_bestv[w] > bv || (s_bestv[w] == bv && s_besti[w] < bi)) { bv = s_bestv[w]; bi = s_besti[w]; }
                hs += s_red[w];
            }
            ws.amax[i] = (uint16_t)bi;
            ws.rowH[i] = hs;
        }
    }

    CS_STAMP(ws, CS_PS_REFRESH_ROWS_DONE, blockIdx.x == 0 && tid == 0);
    // ---- last CTA done: global quantities ---------------------------------------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const uint32_t t = atomicAdd(&ws.sc->ticket0, 1u);
        s_is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    CS_STAMP(ws, CS_PS_REFRESH_LAST_CTA, tid == 0);

    BfsRow rowT;                                                         // in flight during the sums
    cs_bfs_load_row(adjT_fill, A, W, rowT);
    // the operands of Eq. 2 (the first ROW_THREADS of each array) travel with it, so that the sums below start on data
    // that has arrived instead of on a trip of their own
    const uint32_t t0_ = tid < A ? tid : 0u;
    const uint32_t pre_rowsum = cs_ld_cg_pinned(ws.rowsum + t0_);
    const unsigned long long pre_rowH = cs_ld_cg_pinned((const unsigned long long *)ws.rowH + t0_);
    const unsigned long long pre_qfix = cs_ld_cg_pinned(ws.qfix + t0_);
    const unsigned long long qbase = cs_ld_cg_pinned(&ws.sc->qbase);
    uint32_t la = cs_ld_cg_pinned(&ws.sc->last_agent);
    if (n_events) {
        // the batch's effect on what all CTAs share (every other CTA is done reading it)
        const uint32_t a = tid < n_events ? s_eva[tid] : CS_AGENT_NONE;
        if (a != CS_AGENT_NONE) {
            if (!s_succ[tid]) ws.cur[s_evc[tid]] = (uint16_t)a;       // the chain's last live event of the batch
        }
        if (all_chains) __threadfence();                      // (cur[] is read back below when every chain is a source)
        if (s_last_live >= 0) la = s_eva[s_last_live];
        if (tid == 0) {
            ws.sc->last_agent = la;
            ws.sc->n_transitions = n_total;
            atomicAdd((unsigned long long *)&ws.cnt->events_seen, (unsigned long long)n_events);
            if (n_skipped) atomicAdd((unsigned long long *)&ws.cnt->events_skipped, (unsigned long long)n_skipped);
            if (n_new) atomicAdd((unsigned long long *)&ws.cnt->transitions_counted, (unsigned long long)n_new);
        }
    }
    if (tid < 64) s_front[tid] = (tid < 32 && !all_chains && la < A && (la >> 5) == tid) ? (1u << (la & 31)) : 0u;
    // Eq. 10's arg-max successor of the (now final) last agent: asked for here, used by thread 0 after the sums
    const uint32_t a_star_pre = (tid == 0 && la < A) ? (uint32_t)cs_ld_cg_pinned(ws.amax + la) : 0xFFFFFFFFu;
    const uint32_t N = n_total;
    double Hc = 0.0, Hm = 0.0;
    if (N > 0) {
        const double invN = 1.0 / (double)N;
        for (uint32_t i = tid; i < A; i += ROW_THREADS) {
            const uint32_t rs = i == tid ? pre_rowsum : __ldcg(&ws.rowsum[i]);
            const double rh = i == tid ? __longlong_as_double((long long)pre_rowH) : __ldcg(&ws.rowH[i]);
            Hc -= ((double)rs * invN) * rh;
        }
        for (uint32_t j = tid; j < A; j += ROW_THREADS) {
            const unsigned long long qf = j == tid ? pre_qfix : __ldcg(&ws.qfix[j]);
            const double q = (double)(qf + qbase) * (1.0 / 1152921504606846976.0);
            if (q > 0.0) Hm -= q * log(q);
        }
    }
    for (uint32_t j = tid; j < A; j += ROW_THREADS) ws.qfix[j] = 0;      // ready for the next refresh
    __syncthreads();                                                     // (every thread has read qbase)
    if (tid == 0) ws.sc->qbase = 0;
    cs_block_sum2(Hc, Hm, s_red);
    CS_STAMP(ws, CS_PS_REFRESH_SUMS_DONE, tid == 0);                                        // (its barriers also order s_front's zeroes)
    if (tid == 0) {
        double R = 0.0;
        if (N > 0 && Hm > 0.0) R = 1.0 - Hc / Hm;
        const float Rf = (float)R;
        ws.sc->R = Rf;
        ws.sc->gate = (Rf >= r_min) ? 1u : 0u;
        ws.sc->a_star = a_star_pre;                           // Eq. 10, for the prefetch ranking
        ws.sc->adjT_cur = fill;
        ws.sc->ticket0 = 0;
    }
    if (all_chains) {
        // sources: the current agent of every chain that has one (all live sessions)
        for (uint32_t ch = tid; ch < n_chains; ch += ROW_THREADS) {
            const uint32_t a = __ldcg(&ws.cur[ch]);
            if (a < A) atomicOr(&s_front[a >> 5], 1u << (a & 31));
        }
    }
    __syncthreads();
    cs_bfs_survival(ws.adj, A, W, rowT, s_front, s_visit, s_next, s_hops, ws.hops, ws.fsurv, e_max, delta);
    CS_STAMP(ws, CS_PS_REFRESH_END, tid == 0);
}

// BFS + Eq. 8 from explicit sources into the temporary tables (cs_score_blocks with sources).
__global__ void __launch_bounds__(ROW_THREADS)
cs_survival_kernel(cs_workspace ws, uint32_t A, uint32_t W, const uint16_t *__restrict__ sources, uint32_t n_sources,
                   uint32_t e_max, float delta)
{
    __shared__ uint32_t s_front[64], s_visit[32], s_next[32];
    __shared__ uint16_t s_hops[CS_MAX_AGENTS];
    const uint32_t tid = threadIdx.x;
    BfsRow rowT;
    cs_bfs_load_row(ws.adjT + (size_t)ws.sc->adjT_cur * A * W, A, W, rowT);
    if (tid < 64) s_front[tid] = 0;
    __syncthreads();
    for (uint32_t s = tid; s < n_sources; s += ROW_THREADS) {
        const uint32_t a = sources[s];
        if (a < A) atomicOr(&s_front[a >> 5], 1u << (a & 31));
        else atomicOr(&ws.sc->status, CS_ST_BAD_SOURCE);
    }
    __syncthreads();
    cs_bfs_survival(ws.adj, A, W, rowT, s_front, s_visit, s_next, s_hops, ws.hops_tmp, ws.fsurv_tmp, e_max, delta);
}

// ---------------------------------------------------------------------------------------------
// Exact survival probability of Eq. 6 for every agent: one CTA per target agent a.  The unit
// mass at the current agent a0 is pushed through K steps of the chain with column a removed
// (mass that reaches a leaves the vector); what is left after K steps never visited a:
//     v_0 = e_{a0};  v_{t+1}[j] = sum_i v_t[i] P[i][j] (j != a), v_{t+1}[a] = 0;
//     p = sum_t sum_i v_t[i] P[i][a]  (= 1 - sum_j v_K[j]).
// fp64 accumulation over the canonical fp32 matrix, terms added in index order.  The paper
// treats this as too expensive for its per-request runtime and uses the hop proxy of Eq. 8;
// here it is an alternative scorer (A^3 K multiply-adds, off the critical path).
// ---------------------------------------------------------------------------------------------
#define XS_MAX_TARGETS 8
__global__ void __launch_bounds__(ROW_THREADS)
cs_exact_survival_kernel(cs_workspace ws, uint32_t A, uint32_t a0_arg, uint32_t K, uint32_t n_tgt, float delta,
                         float *__restrict__ psurv_out, float *__restrict__ fsurv_out)
{
    // A CTA advances n_tgt target agents together, so that every element of the matrix it reads
    // feeds n_tgt accumulators (the matrix is the only sizeable traffic: A^2 floats per step).
    extern __shared__ double s_vec[];                 // v[n_tgt][A], w[n_tgt][A]
    double *v = s_vec, *w = s_vec + (size_t)n_tgt * A;
    const uint32_t tid = threadIdx.x;
    const uint32_t a0 = a0_arg == CS_AGENT_NONE ? ws.sc->last_agent : a0_arg;
    for (uint32_t base = blockIdx.x * n_tgt; base < A; base += gridDim.x * n_tgt) {
        // The probability is accumulated as the mass absorbed at the target step by step (no 1 - x
        // cancellation, so small probabilities keep full relative accuracy).  Column (base + m) of
        // target m is owned by one thread, which does the adding for that target.
        double hit[XS_MAX_TARGETS];
#pragma unroll
        for (int m = 0; m < XS_MAX_TARGETS; ++m) hit[m] = 0.0;
        if (a0 < A && K > 0) {
            __syncthreads();
            // step 1: every target starts from the unit mass at a0, i.e. from row a0 of the matrix
            for (uint32_t j = tid; j < A; j += ROW_THREADS) {
                const double p = (double)ws.P[a0 * A + j];
#pragma unroll
                for (int m = 0; m < XS_MAX_TARGETS; ++m) {
                    if ((uint32_t)m < n_tgt) {
                        const bool own = (j == base + m);
                        if (own) hit[m] += p;
                        v[(size_t)m * A + j] = own ? 0.0 : p;
                    }
                }
            }
            __syncthreads();
            for (uint32_t t = 1; t < K; ++t) {
                for (uint32_t j = tid; j < A; j += ROW_THREADS) {
                    double s[XS_MAX_TARGETS];
#pragma unroll
                    for (int m = 0; m < XS_MAX_TARGETS; ++m) s[m] = 0.0;
                    for (uint32_t i = 0; i < A; ++i) {
                        const double p = (double)ws.P[i * A + j];
#pragma unroll
                        for (int m = 0; m < XS_MAX_TARGETS; ++m)
                            if ((uint32_t)m < n_tgt) s[m] = fma(v[(size_t)m * A + i], p, s[m]);
                    }
#pragma unroll
                    for (int m = 0; m < XS_MAX_TARGETS; ++m) {
                        if ((uint32_t)m < n_tgt) {
                            const bool own = (j == base + m);
                            if (own) hit[m] += s[m];
                            w[(size_t)m * A + j] = own ? 0.0 : s[m];
                        }
                    }
                }
                __syncthreads();
                double *tmp = v; v = w; w = tmp;
            }
        }
#pragma unroll
        for (int m = 0; m < XS_MAX_TARGETS; ++m) {
            const uint32_t a = base + m;
            if ((uint32_t)m < n_tgt && a < A && tid == (a % ROW_THREADS)) {
                if (psurv_out) psurv_out[a] = (float)hit[m];
                if (fsurv_out) fsurv_out[a] = (float)(hit[m] + (double)delta);
            }
        }
    }
}

int cs_launch_exact_survival(cs_ctx *ctx, uint32_t a0, uint32_t K, float *psurv_out, float *fsurv_out, cudaStream_t s)
{
    const cs_params &p = ctx->p;
    uint32_t n_tgt = 2048u / p.n_agents;               // 2 * n_tgt * A doubles of shared memory <= 32 KiB
    if (n_tgt > XS_MAX_TARGETS) n_tgt = XS_MAX_TARGETS;
    if (n_tgt < 1) n_tgt = 1;
    const uint32_t grid = (p.n_agents + n_tgt - 1) / n_tgt;
    cs_exact_survival_kernel<<<grid, ROW_THREADS, 2 * (size_t)n_tgt * p.n_agents * sizeof(double), s>>>(
        ctx->ws, p.n_agents, a0, K, n_tgt, p.delta, psurv_out, fsurv_out);
    return cs_check_launch(ctx);
}

// ---------------------------------------------------------------------------------------------
// Restores learner state saved with cs_get_model(): counts, per-chain current agents, last agent.
// Row sums and the transition total are recomputed from the counts (one CTA per row; integer
// atomics, so the total does not depend on arrival order).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(ROW_THREADS)
cs_import_kernel(cs_workspace ws, uint32_t A, uint32_t n_chains, const uint32_t *__restrict__ C_in,
                 const uint16_t *__restrict__ cur_in, uint32_t last_agent)
{
    __shared__ uint32_t s_red[ROW_THREADS];
    const uint32_t tid = threadIdx.x;
    if (blockIdx.x == 0) {
        if (tid == 0) { ws.sc->last_agent = last_agent < A ? last_agent : CS_AGENT_NONE; }
        for (uint32_t c = tid; c < n_chains; c += ROW_THREADS) {
            const uint32_t a = cur_in ? cur_in[c] : CS_AGENT_NONE;
            ws.cur[c] = (uint16_t)(a < A ? a : CS_AGENT_NONE);
        }
    }
    for (uint32_t i = blockIdx.x; i < A; i += gridDim.x) {
        uint32_t part = 0;
        for (uint32_t j = tid; j < A; j += ROW_THREADS) {
            const uint32_t v = (i == j) ? 0u : C_in[i * A + j];      // a self transition is never counted
            ws.C[i * A + j] = v;
            part += v;
        }
        const uint32_t n_i = cs_block_sum<uint32_t>(part, s_red);
        if (tid == 0) {
            ws.rowsum[i] = n_i;
            atomicAdd(&ws.sc->n_transitions, n_i);
        }
    }
}

int cs_launch_import(cs_ctx *ctx, const uint32_t *C_in, const uint16_t *cur_in, uint32_t last_agent, cudaStream_t s)
{
    const cs_params &p = ctx->p;
    cudaError_t e = cudaMemsetAsync(&ctx->ws.sc->n_transitions, 0, sizeof(uint32_t), s);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    const uint32_t grid = p.n_agents < 2u * (uint32_t)ctx->sm_count ? p.n_agents : 2u * (uint32_t)ctx->sm_count;
    cs_import_kernel<<<grid, ROW_THREADS, 0, s>>>(ctx->ws, p.n_agents, p.n_chains, C_in, cur_in, last_agent);
    int rc = cs_check_launch(ctx);
    if (rc != CS_OK) return rc;
    return cs_launch_observe(ctx, nullptr, nullptr, nullptr, 0, s);      // refresh everything derived from the counts
}

// ---------------------------------------------------------------------------------------------
int cs_launch_init(cs_ctx *ctx, cudaStream_t s)
{
    const cs_params &p = ctx->p;
    cs_init_kernel<<<64, 256, 0, s>>>(ctx->ws, p.n_agents, p.n_chains, ctx->gtab_len, p.lambda, p.delta);
    int rc = cs_check_launch(ctx);
    if (rc != CS_OK) return rc;
    cs_gtab_check_kernel<<<1, 256, 0, s>>>(ctx->ws, ctx->gtab_len, ctx->age_sat, p.lambda, p.delta);
    if ((rc = cs_check_launch(ctx)) != CS_OK) return rc;
    return cs_launch_observe(ctx, nullptr, nullptr, nullptr, 0, s);
}

int cs_launch_observe(cs_ctx *ctx, const uint32_t *chain, const uint16_t *agent, const uint8_t *evflags,
                      uint32_t n_events, cudaStream_t s)
{
    const cs_params &p = ctx->p;
    const bool fused = n_events <= OBS_FUSED_MAX;             // small batches ride along with the refresh
    if (n_events && !fused) {
        cs_launch_chained(cs_observe_kernel, 1, OBS_THREADS, 0, s, ctx->ws, p.n_agents, p.n_chains, chain, agent, evflags,
                          n_events, ctx->step_n_events_dev);
        int rc = cs_check_launch(ctx);
        if (rc != CS_OK) return rc;
    }
    const uint32_t grid = p.n_agents < 2u * (uint32_t)ctx->sm_count ? p.n_agents : 2u * (uint32_t)ctx->sm_count;
    cs_launch_chained(cs_normalise_kernel, grid, ROW_THREADS, 0, s, ctx->ws, p.n_agents, ctx->W, p.eps, p.tau, p.r_min,
                      p.e_max, p.delta, ctx->source_mode == CS_SOURCES_ALL_CHAINS ? 1u : 0u, p.n_chains,
                      fused ? chain : (const uint32_t *)nullptr, fused ? agent : (const uint16_t *)nullptr,
                      fused ? evflags : (const uint8_t *)nullptr, fused ? n_events : 0u,
                      fused ? (const uint32_t *)ctx->step_n_events_dev : (const uint32_t *)nullptr);
    return cs_check_launch(ctx);
}

int cs_launch_survival(cs_ctx *ctx, const uint16_t *sources, uint32_t n_sources, cudaStream_t s)
{
    const cs_params &p = ctx->p;
    cs_survival_kernel<<<1, ROW_THREADS, 0, s>>>(ctx->ws, p.n_agents, ctx->W, sources, n_sources, p.e_max, p.delta);
    return cs_check_launch(ctx);
}
