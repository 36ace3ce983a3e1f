/*
 * cs_oracle.c -- plain, slow CPU oracle of the agent-aware KV-cache management step
 * and of the paged-KV block mover.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may include, link, import or
 * call this file; it shares no code, header, table or constant generator with the CUDA
 * path.  Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Every function follows the paper's statement of the step, in its notation, one plain
 * loop per definition, no blocking, fusion or reordering.  Floating point is fp64.  Where
 * a floating-point value decides an integer (graph edge, arg-max, eviction order) the
 * decision is taken on the fp32 value the kernels are specified to produce ("canonical
 * fp32": one IEEE round-to-nearest operation per arithmetic step, no fused multiply-add);
 * the fp64 value is returned beside it so tests can bound the difference.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC cs_oracle.c -lm
 *
 * Parity pins: every function here is pinned by the CPU tests (brute force on tiny
 * inputs, closed forms, invariants, hand-derived worked examples); none is "unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_AGENT_NONE 0xFFFFu      /* "bottom": no current agent yet (Algorithm 1 state) */
#define ORC_ID_NONE 0xFFFFFFFFu     /* list padding */
#define ORC_INF 0xFFFFFFFFu         /* unreachable hop distance */

#define FLAG_VALID 1u
#define FLAG_PINNED 2u
#define FLAG_TIER_HOST 4u
#define FLAG_OTHER_COPY 8u
#define EV_WARMUP 1u

/* ------------------------------------------------------------------------------------
 * Transition counting.  Sec. 3.2 ("for every observed transition A_t = i -> A_{t+1} = j
 * the counter C_ij is incremented") and Algorithm 1, ObserveTouch: the counter moves only
 * when the agent differs from the current one and a current one exists; then the current
 * agent is replaced.  One "current agent" register per chain (n_chains = 1 is the paper's
 * single register).  Warmup-flagged events are excluded from learning (Sec. 4).
 * Events naming an agent >= A or a chain >= n_chains are skipped and counted in the
 * return value.
 * ------------------------------------------------------------------------------------ */
uint32_t orc_observe(uint32_t A, uint32_t n_chains, uint32_t *C /*[A*A]*/,
                     uint16_t *cur /*[n_chains]*/, uint16_t *last_agent,
                     const uint32_t *chain, const uint16_t *agent, const uint8_t *evflags,
                     uint32_t n_events)
{
    uint32_t bad = 0;
    for (uint32_t e = 0; e < n_events; ++e) {
        if (evflags && (evflags[e] & EV_WARMUP)) continue;
        uint32_t c = chain[e];
        uint32_t a = agent[e];
        if (a >= A || c >= n_chains) { ++bad; continue; }
        uint32_t a_t = cur[c];
        if (a != a_t) {
            if (a_t != ORC_AGENT_NONE) C[(size_t)a_t * A + a] += 1u;
            cur[c] = (uint16_t)a;
        }
        *last_agent = (uint16_t)a;
    }
    return bad;
}

/* ------------------------------------------------------------------------------------
 * Eq. 3: P_ij = (C_ij + eps) / sum_k (C_ik + eps), k over all A agent slots.
 * P64: the definition in fp64.  P32: canonical fp32,
 *   num = f32(C_ij) + eps ; den = f32(n_i) + (f32(A) * eps) ; P = num / den,
 * with n_i = sum_k C_ik as an integer.  Eq. 5 / Eq. 10: row arg-max on P32, lowest
 * index among equal maxima.
 * ------------------------------------------------------------------------------------ */
void orc_normalise(uint32_t A, const uint32_t *C, float eps, double *P64, float *P32,
                   uint16_t *amax)
{
    for (uint32_t i = 0; i < A; ++i) {
        double den64 = 0.0;
        uint32_t n_i = 0;
        for (uint32_t k = 0; k < A; ++k) {
            den64 += (double)C[(size_t)i * A + k] + (double)eps;
            n_i += C[(size_t)i * A + k];
        }
        volatile float a_eps = (float)A * eps;
        volatile float den32 = (float)n_i + a_eps;
        uint32_t best = 0;
        for (uint32_t j = 0; j < A; ++j) {
            P64[(size_t)i * A + j] = ((double)C[(size_t)i * A + j] + (double)eps) / den64;
            volatile float num32 = (float)C[(size_t)i * A + j] + eps;
            float p = num32 / den32;
            P32[(size_t)i * A + j] = p;
            if (p > P32[(size_t)i * A + best]) best = j;
        }
        amax[i] = (uint16_t)best;
    }
}

/* ------------------------------------------------------------------------------------
 * Eq. 2: R = 1 - H(A_{t+1} | A_t) / H(A_{t+1}).  The distribution of A_t is the empirical
 * one of the counted transitions, pi_i = n_i / N; the conditional is the smoothed row
 * P_i,: of Eq. 3; the marginal of the next agent is q_j = sum_i pi_i P_ij.  Natural log.
 * R = 0 when nothing has been counted or the marginal entropy is not positive.
 * ------------------------------------------------------------------------------------ */
double orc_predictability(uint32_t A, const uint32_t *C, const double *P64)
{
    double N = 0.0;
    for (size_t x = 0; x < (size_t)A * A; ++x) N += (double)C[x];
    if (N <= 0.0) return 0.0;
    double Hc = 0.0;
    double *q = (double *)calloc(A, sizeof(double));
    for (uint32_t i = 0; i < A; ++i) {
        double n_i = 0.0;
        for (uint32_t k = 0; k < A; ++k) n_i += (double)C[(size_t)i * A + k];
        double pi_i = n_i / N;
        double h = 0.0;
        for (uint32_t j = 0; j < A; ++j) {
            double p = P64[(size_t)i * A + j];
            if (p > 0.0) h -= p * log(p);
            q[j] += pi_i * p;
        }
        Hc += pi_i * h;
    }
    double Hm = 0.0;
    for (uint32_t j = 0; j < A; ++j)
        if (q[j] > 0.0) Hm -= q[j] * log(q[j]);
    free(q);
    if (!(Hm > 0.0)) return 0.0;
    return 1.0 - Hc / Hm;
}

/* Eq. 7: (a,b) in E  <=>  P(b|a) >= tau, inclusive, on the canonical fp32 matrix. */
void orc_threshold_graph(uint32_t A, const float *P32, float tau, uint8_t *adj /*[A*A]*/)
{
    for (uint32_t a = 0; a < A; ++a)
        for (uint32_t b = 0; b < A; ++b)
            adj[(size_t)a * A + b] = (P32[(size_t)a * A + b] >= tau) ? 1u : 0u;
}

/* Sec. 3.3: one breadth-first search from the current agent(s); E[a] = minimum number of
 * hops, ORC_INF when unreachable.  Sources >= A are ignored. */
void orc_bfs(uint32_t A, const uint8_t *adj, const uint16_t *sources, uint32_t n_sources,
             uint32_t *E /*[A]*/)
{
    uint32_t *queue = (uint32_t *)malloc((size_t)A * sizeof(uint32_t));
    uint32_t head = 0, tail = 0;
    for (uint32_t a = 0; a < A; ++a) E[a] = ORC_INF;
    for (uint32_t s = 0; s < n_sources; ++s) {
        uint32_t a = sources[s];
        if (a < A && E[a] == ORC_INF) { E[a] = 0; queue[tail++] = a; }
    }
    while (head < tail) {
        uint32_t a = queue[head++];
        for (uint32_t b = 0; b < A; ++b)
            if (adj[(size_t)a * A + b] && E[b] == ORC_INF) { E[b] = E[a] + 1; queue[tail++] = b; }
    }
    free(queue);
}

/* Eq. 8: p~(a) = 1 - min(E[a], E_max) / E_max, fp64.  fsurv32 is the first factor of
 * Eq. 9 as the kernels hold it: f32(p~ + delta), the sum taken in fp64. */
void orc_survival(uint32_t A, const uint32_t *E, uint32_t E_max, float delta,
                  double *ptilde /*[A]*/, float *fsurv32 /*[A]*/)
{
    for (uint32_t a = 0; a < A; ++a) {
        uint32_t m = E[a] < E_max ? E[a] : E_max;
        ptilde[a] = 1.0 - (double)m / (double)E_max;
        fsurv32[a] = (float)(ptilde[a] + (double)delta);
    }
}

/* ------------------------------------------------------------------------------------
 * Eq. 9 / ScoreBlock: Score(b) = (p~(a_b) + delta) (exp(-lambda age(b)) + delta) |b|,
 * age = now - last_access in scheduler steps (0 when last_access lies in the future),
 * |b| = tokens the block caches (block_tokens when no per-block table is given).
 * score64: fp64.  score32: canonical fp32 = (fsurv32[a] * g) * f32(|b|) with
 * g = f32(exp(-f64(lambda) age) + f64(delta)).  Blocks whose agent is >= A get 0.
 * ------------------------------------------------------------------------------------ */
void orc_scores(uint32_t n, uint32_t A, const uint16_t *agent, const uint32_t *last_access,
                const uint8_t *n_tokens, uint32_t block_tokens, uint32_t now, float lambda,
                float delta, const double *ptilde, const float *fsurv32, double *score64,
                float *score32)
{
    for (uint32_t b = 0; b < n; ++b) {
        uint32_t a = agent[b];
        if (a >= A) { score64[b] = 0.0; score32[b] = 0.0f; continue; }
        double age = (last_access[b] <= now) ? (double)(now - last_access[b]) : 0.0;
        double size = n_tokens ? (double)n_tokens[b] : (double)block_tokens;
        double rec = exp(-(double)lambda * age) + (double)delta;
        score64[b] = (ptilde[a] + (double)delta) * rec * size;
        volatile float g = (float)rec;
        volatile float t = fsurv32[a] * g;
        score32[b] = t * (float)size;
    }
}

/* ------------------------------------------------------------------------------------
 * Selections: the plain definition -- sort every eligible entry by the key, keep the
 * first k.  Keys use the bit pattern of the (positive) fp32 score, so equal scores are
 * exactly the equal floats.
 * ------------------------------------------------------------------------------------ */
typedef struct { uint32_t primary, tiebreak, secondary, id; } orc_key;

static int key_cmp(const void *x, const void *y)
{
    const orc_key *a = (const orc_key *)x, *b = (const orc_key *)y;
    if (a->primary != b->primary) return a->primary < b->primary ? -1 : 1;
    if (a->tiebreak != b->tiebreak) return a->tiebreak < b->tiebreak ? -1 : 1;
    if (a->secondary != b->secondary) return a->secondary < b->secondary ? -1 : 1;
    if (a->id != b->id) return a->id < b->id ? -1 : 1;
    return 0;
}

static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

/* Algorithm 1, Evict: arg-min of ScoreBlock over the evictable set, k times over: the k
 * lowest (score, last_access, id) among VALID, not PINNED, ref_count 0, on tier `tier`
 * (0 GPU, 1 host), agent < A.  ids_out padded with ORC_ID_NONE; returns n_out.
 * prefer_copy != 0 adds the preference of Sec. 4 for blocks whose contents already exist on the
 * other tier (no offload needed): among equal scores those go first, i.e. the order becomes
 * (score, has no copy, last_access, id). */
uint32_t orc_select_victims(uint32_t n, uint32_t A, const uint16_t *agent, const uint8_t *ref_count,
                            const uint8_t *flags, const uint32_t *last_access,
                            const float *score32, uint32_t tier, uint32_t k, int prefer_copy,
                            uint32_t *ids_out)
{
    orc_key *keys = (orc_key *)malloc(((size_t)n + 1) * sizeof(orc_key));
    uint32_t m = 0;
    for (uint32_t b = 0; b < n; ++b) {
        uint32_t f = flags[b];
        if (!(f & FLAG_VALID) || (f & FLAG_PINNED) || ref_count[b] != 0) continue;
        if (((f & FLAG_TIER_HOST) ? 1u : 0u) != tier) continue;
        if (agent[b] >= A) continue;
        keys[m].primary = f32_bits(score32[b]);
        keys[m].tiebreak = (prefer_copy && !(f & FLAG_OTHER_COPY)) ? 1u : 0u;
        keys[m].secondary = last_access[b];
        keys[m].id = b;
        ++m;
    }
    qsort(keys, m, sizeof(orc_key), key_cmp);
    uint32_t n_out = m < k ? m : k;
    for (uint32_t i = 0; i < k; ++i) ids_out[i] = i < n_out ? keys[i].id : ORC_ID_NONE;
    free(keys);
    return n_out;
}

/* Algorithm 1, BetweenStep with Eq. 10-11 at block level: nothing unless the gate is open
 * and a current agent exists; a* = argmax row of the current agent.  Eligible: VALID, not
 * PINNED, ref_count 0, on the host tier, no copy on the other tier, and (when the anchor
 * table is given) depth < anchor_blocks[agent].  Order: blocks of a* first, then score
 * descending, last_access descending, id ascending. */
uint32_t orc_select_prefetch(uint32_t n, uint32_t A, const uint16_t *agent, const uint16_t *depth,
                             const uint8_t *ref_count, const uint8_t *flags,
                             const uint32_t *last_access, const uint16_t *anchor_blocks,
                             const float *score32, int gate, uint16_t last_agent,
                             const uint16_t *amax, uint32_t k, uint32_t *ids_out)
{
    for (uint32_t i = 0; i < k; ++i) ids_out[i] = ORC_ID_NONE;
    if (!gate || last_agent == ORC_AGENT_NONE || last_agent >= A) return 0;
    uint32_t a_star = amax[last_agent];
    orc_key *keys = (orc_key *)malloc(((size_t)n + 1) * sizeof(orc_key));
    uint32_t m = 0;
    for (uint32_t b = 0; b < n; ++b) {
        uint32_t f = flags[b];
        if (!(f & FLAG_VALID) || (f & FLAG_PINNED) || ref_count[b] != 0) continue;
        if (!(f & FLAG_TIER_HOST) || (f & FLAG_OTHER_COPY)) continue;
        uint32_t a = agent[b];
        if (a >= A) continue;
        if (anchor_blocks && !(depth[b] < anchor_blocks[a])) continue;
        /* descending score / last_access as ascending complemented words; a* class first */
        keys[m].primary = ((a == a_star) ? 0u : 0x80000000u) | (~f32_bits(score32[b]) & 0x7FFFFFFFu);
        keys[m].tiebreak = 0u;
        keys[m].secondary = ~last_access[b];
        keys[m].id = b;
        ++m;
    }
    qsort(keys, m, sizeof(orc_key), key_cmp);
    uint32_t n_out = m < k ? m : k;
    for (uint32_t i = 0; i < n_out; ++i) ids_out[i] = keys[i].id;
    free(keys);
    return n_out;
}

/* ------------------------------------------------------------------------------------
 * Block mover: for every listed block, every layer and both planes, copy one chunk.
 * Address of chunk (layer l, plane p in {0 = K, 1 = V}, slot s):
 *   layer-major: ((l*2 + p) * n_slots + s) * chunk_bytes
 *   block-major: ((s*L + l) * 2 + p) * chunk_bytes
 * Entries whose source or destination slot is ORC_ID_NONE or out of range are skipped;
 * the number skipped for being out of range is returned.
 * ------------------------------------------------------------------------------------ */
static size_t chunk_off(uint32_t layout, uint32_t L, uint32_t n_slots, uint32_t l, uint32_t p,
                        uint32_t s, size_t chunk)
{
    if (layout == 0) return (((size_t)l * 2 + p) * n_slots + s) * chunk;
    return (((size_t)s * L + l) * 2 + p) * chunk;
}

uint32_t orc_move_blocks(const uint8_t *src, uint32_t src_layout, uint32_t src_slots_total,
                         uint8_t *dst, uint32_t dst_layout, uint32_t dst_slots_total,
                         uint32_t L, size_t chunk_bytes, const uint32_t *src_slots,
                         const uint32_t *dst_slots, uint32_t n)
{
    uint32_t bad = 0;
    for (uint32_t i = 0; i < n; ++i) {
        uint32_t s = src_slots[i], d = dst_slots[i];
        if (s == ORC_ID_NONE || d == ORC_ID_NONE) continue;
        if (s >= src_slots_total || d >= dst_slots_total) { ++bad; continue; }
        for (uint32_t l = 0; l < L; ++l)
            for (uint32_t p = 0; p < 2; ++p)
                memcpy(dst + chunk_off(dst_layout, L, dst_slots_total, l, p, d, chunk_bytes),
                       src + chunk_off(src_layout, L, src_slots_total, l, p, s, chunk_bytes),
                       chunk_bytes);
    }
    return bad;
}

/* ------------------------------------------------------------------------------------
 * Eq. 6: exact survival probability p_surv(a; a0, K) = Pr(exists k in [1, K]: A_{t+k} = a |
 * A_t = a0) under the first-order chain with matrix P.  Written out from the definition: make
 * a absorbing-and-removed (zero column a: mass that reaches a leaves the vector), push the unit
 * mass at a0 through K steps, and what is left never visited a:
 *     v_0 = e_{a0};  v_{t+1}[j] = sum_i v_t[i] P[i][j]  (j != a),  v_{t+1}[a] = 0;
 *     p_surv(a) = 1 - sum_j v_K[j].
 * The paper calls this prohibitively expensive for its runtime and approximates it with the
 * hop-distance proxy of Eq. 8; here it is the alternative scorer.  a0 >= A gives all zeros.
 * ------------------------------------------------------------------------------------ */
void orc_exact_survival(uint32_t A, const double *P64, uint32_t a0, uint32_t K, double *psurv /*[A]*/)
{
    double *v = (double *)malloc((size_t)A * sizeof(double));
    double *w = (double *)malloc((size_t)A * sizeof(double));
    for (uint32_t a = 0; a < A; ++a) {
        if (a0 >= A) { psurv[a] = 0.0; continue; }
        for (uint32_t j = 0; j < A; ++j) v[j] = 0.0;
        v[a0] = 1.0;
        for (uint32_t t = 0; t < K; ++t) {
            for (uint32_t j = 0; j < A; ++j) {
                double s = 0.0;
                if (j != a)
                    for (uint32_t i = 0; i < A; ++i) s += v[i] * P64[(size_t)i * A + j];
                w[j] = s;
            }
            double *tmp = v; v = w; w = tmp;
        }
        double left = 0.0;
        for (uint32_t j = 0; j < A; ++j) left += v[j];
        psurv[a] = 1.0 - left;
    }
    free(v);
    free(w);
}
