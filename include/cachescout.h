/*
 * cachescout.h -- C ABI of the B200 (sm_100a) hot path of an agent-aware KV-cache layer:
 * the batched cache-management step (online agent-transition model, per-block reuse score,
 * eviction-victim and prefetch-candidate selection) and the paged-KV block mover that
 * carries the decisions out between a paged GPU pool and a pinned host tier.
 *
 * General rules
 *  - Every function returns an int: CS_OK (0) or a negative CS_E* code.  Nothing throws,
 *    aborts or prints.
 *  - Calls ENQUEUE work on the given CUDA stream and return; outputs are valid once that
 *    stream has been synchronised.  Only cs_get_status() synchronises.
 *  - "dev" pointers are caller-owned device memory, "pinned" pointers caller-owned
 *    page-locked host memory that the device can address (cudaHostAlloc /
 *    cudaHostRegister; with unified addressing the host pointer is used as is).  The
 *    library never allocates or frees device or pinned memory; it owns only the small
 *    host-side cs_ctx, with a few CUDA events and two streams of its own (made by cs_create,
 *    released by cs_destroy; cs_step and cs_select_step fork onto them and join back, so callers
 *    see everything ordered on the streams they pass), plus five more streams and their events
 *    once cs_set_mover_staging() has been called.  All scratch lives in the workspace the
 *    caller hands to cs_create() (and, for the copy-engine transfers, in the ring handed to
 *    cs_set_mover_staging()).
 *  - Block-index arrays, score / id output arrays and pool bases must be 16-byte aligned (the
 *    kernels use 128-bit accesses); event arrays, slot lists and counts need only their natural
 *    alignment.  A violation is CS_EINVAL before anything is launched.
 *  - All calls on one cs_ctx except the mover calls (offload, prefetch, exchange, compact) share
 *    workspace scratch: issue them on one stream (or order them with events).  The mover calls
 *    touch no workspace scratch besides the status word and may run on a side stream concurrently.
 *  - Bad ids inside device arrays (agent >= n_agents, chain >= n_chains, slot >= n_slots)
 *    are detected in the kernels: the entry is skipped and a bit is set in the device
 *    status word (read with cs_get_status()).  Kernels never trap or spin unboundedly.
 */
#ifndef CACHESCOUT_H
#define CACHESCOUT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cs_ctx cs_ctx;
typedef struct CUstream_st *cs_stream_t;   /* the same type as cudaStream_t */

/* ---- return codes ---------------------------------------------------------------- */
#define CS_OK 0
#define CS_EINVAL (-1)          /* bad argument (NULL, misaligned, inconsistent sizes) */
#define CS_ECAPACITY (-2)       /* n_blocks or k beyond what the workspace was sized for */
#define CS_ENOTIMPL (-3)
#define CS_ECUDA (-4)           /* a CUDA runtime call failed; see cs_last_cuda_error() */
#define CS_EDEVICE_STATUS (-5)  /* cs_get_status(): the device status word was non-zero */
#define CS_ENOMEM (-6)          /* host allocation of the context failed */

/* ---- device status word bits (cs_get_status) ---------------------------------------- */
#define CS_ST_BAD_AGENT 1u      /* an event or index entry named an agent >= n_agents */
#define CS_ST_BAD_CHAIN 2u      /* an event named a chain >= n_chains */
#define CS_ST_BAD_SLOT 4u       /* a mover list entry named a slot >= n_slots */
#define CS_ST_BAD_SOURCE 8u     /* a BFS source >= n_agents */
#define CS_ST_TIMEOUT 16u       /* a bounded wait inside a kernel ran out; the transfer is incomplete */
#define CS_ST_LIST_CONFLICT 32u /* cs_validate_*_lists(): a slot is written twice, or written and read, by one transfer */
#define CS_ST_BAD_SELECTION 64u /* cs_validate_selection(): a list is not the ordered k best eligible entries */

/* ---- sentinels ---------------------------------------------------------------------------- */
#define CS_AGENT_NONE 0xFFFFu      /* "no current agent yet" (the initial state of Algorithm 1) */
#define CS_ID_NONE 0xFFFFFFFFu     /* padding of id lists; skipped by the mover */
#define CS_HOP_NONE 0xFFFFu        /* unreachable in the execution graph */

/* ---- block-index flag bits ------------------------------------------------------------------ */
#define CS_FLAG_VALID 1u
#define CS_FLAG_PINNED 2u
#define CS_FLAG_TIER_HOST 4u
#define CS_FLAG_OTHER_COPY 8u      /* the block's contents also exist on the other tier */

#define CS_EV_WARMUP 1u            /* event flag: warmup request, excluded from learning (Sec. 4) */

#define CS_LAYER_MAJOR 0u
#define CS_BLOCK_MAJOR 1u

#define CS_MAX_AGENTS 1024u

/* Constants of the method (Algorithm 1 state; Eq. 3, 7, 8, 9, 11).  The paper names them
 * without values; the defaults used by the tests are eps 0.01, tau 0.05, e_max 4,
 * lambda 0.01 per scheduler step, delta 0.01, r_min 0.3. */
typedef struct cs_params {
    uint32_t n_agents;      /* A: 1 .. CS_MAX_AGENTS; Eq. 3's sum runs over all A slots */
    uint32_t n_chains;      /* independent "current agent" registers; 1 = the paper's single a_t */
    uint32_t max_blocks;    /* largest n_blocks / k any select call will use */
    uint32_t block_tokens;  /* |b| of a full block (1..255), used when n_tokens is NULL */
    uint32_t e_max;         /* E_max of Eq. 8, >= 1 */
    float eps;              /* smoothing constant of Eq. 3, > 0 */
    float tau;              /* confidence threshold of Eq. 7 */
    float lambda;           /* recency decay rate of Eq. 9, >= 0 */
    float delta;            /* floor of Eq. 9, > 0 */
    float r_min;            /* prefetch gate of Eq. 11 */
    uint32_t prefer_other_copy; /* 0: victims ordered by (score, last_access, id).  1: among equal scores,
                                   blocks whose contents already exist on the other tier go first (no
                                   offload needed, Sec. 4): (score, has no copy, last_access, id) */
} cs_params;

/* Structure-of-arrays metadata of the cached blocks (all dev, each [n_blocks] unless
 * noted).  Entry i describes block id i. */
typedef struct cs_block_index {
    uint32_t n_blocks;
    const uint16_t *agent;          /* owning agent (agentOf[] of Algorithm 1) */
    const uint16_t *depth;          /* position of the block in its prompt */
    const uint8_t *ref_count;       /* in use by running requests when > 0 */
    const uint8_t *flags;           /* CS_FLAG_* */
    const uint32_t *last_access;    /* scheduler step of the last touch (lastAccess[]) */
    const uint8_t *n_tokens;        /* tokens cached per block, or NULL = block_tokens */
    const uint16_t *anchor_blocks;  /* [n_agents] length of each agent's fixed context in
                                       blocks, or NULL = no depth restriction on prefetch */
} cs_block_index;

/* A paged KV pool.  One chunk = block_tokens*n_kv_heads*head_dim*elem_bytes bytes holds one
 * layer, one of K/V, one block ([token][head][dim] inside).  Byte offset of the chunk of
 * layer l, plane p (0 = K, 1 = V), slot s:
 *   CS_LAYER_MAJOR: ((l*2 + p)*n_slots + s) * chunk_bytes
 *   CS_BLOCK_MAJOR: ((s*n_layers + l)*2 + p) * chunk_bytes
 * base is dev or pinned; chunk_bytes must be a multiple of 16.
 * Slot lists given to the mover hold block ids of the index; the pool's slot is
 * id - first_id (first_id = 0 when ids are slot numbers).  This lets the lists the select
 * calls emit drive the mover directly when the index numbers the GPU tier [0, G) and the host
 * tier [G, G + H).  Ids outside [first_id, first_id + n_slots) are out of range. */
typedef struct cs_kv_pool {
    void *base;
    uint32_t n_slots, layout, n_layers, n_kv_heads, head_dim, block_tokens, elem_bytes;
    uint32_t first_id;
} cs_kv_pool;

/* ---- life cycle -------------------------------------------------------------------------------- */

/* Bytes of device workspace cs_create() needs for these parameters (host call, no CUDA). */
int cs_workspace_bytes(const cs_params *p, size_t *dev_bytes);

/* Creates a context on the current device over caller-owned `dev_workspace` (256-byte
 * aligned, >= cs_workspace_bytes()).  Enqueues the initialisation on `init_stream`: zero
 * counts, no current agent, the uniform Eq. 3 matrix, the recency table of Eq. 9.
 * The workspace must outlive the context; cs_destroy() frees only the host struct. */
int cs_create(const cs_params *p, void *dev_workspace, size_t bytes, cs_stream_t init_stream,
              cs_ctx **out);
int cs_destroy(cs_ctx *ctx);

/* ---- cache-management step ----------------------------------------------------------------------- */

/* Transition Learner (Sec. 3.2; Algorithm 1, ObserveTouch).  For the events in order, per
 * chain c: if a current agent exists and differs from the event's agent, C[cur][agent] += 1;
 * then cur[c] = agent.  Events with CS_EV_WARMUP are ignored.  After the batch the call
 * refreshes everything derived from the counts: the smoothed matrix of Eq. 3, each row's
 * arg-max (Eq. 5 / Eq. 10, lowest index among equal maxima), the predictability R of Eq. 2
 * with the gate of Eq. 11, the threshold graph of Eq. 7, and -- from the agent of the last
 * non-warmup event -- the BFS hop table and the survival scores of Eq. 8.
 * chain, agent, evflags: dev [n_events]; evflags may be NULL.  n_events may be 0 (refresh only). */
int cs_observe_invocations(cs_ctx *ctx, const uint32_t *chain, const uint16_t *agent,
                           const uint8_t *evflags, uint32_t n_events, cs_stream_t stream);

/* ScoreBlock of Algorithm 1 / Eq. 9 for every index entry:
 *   score = (p~(agent) + delta) * (exp(-lambda * age) + delta) * |b|,  age = now - last_access
 * (0 when last_access > now).  fp32, each product rounded once.  sources == NULL uses the
 * survival table cached by the last cs_observe_invocations(); otherwise a BFS from the given
 * agents (dev [n_sources]) is run first and used for this call only.
 * scores_out: dev [n_blocks]; entries whose agent is out of range get 0. */
int cs_score_blocks(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, const uint16_t *sources,
                    uint32_t n_sources, float *scores_out, cs_stream_t stream);

/* Evict of Algorithm 1, k times over: the k eligible entries with the lowest
 * (score, last_access, id), in ascending order.  Eligible: VALID, not PINNED, ref_count 0,
 * TIER_HOST bit == tier (0 GPU, 1 host).  ids_out: dev [k], padded with CS_ID_NONE;
 * n_out: dev, = min(k, number eligible).  k <= max_blocks. */
int cs_select_victims(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t tier, uint32_t k,
                      uint32_t *ids_out, uint32_t *n_out, cs_stream_t stream);

/* BetweenStep of Algorithm 1 with Eq. 10-11, at block level: empty unless R >= r_min and a
 * current agent exists.  a* = arg-max row of the current agent.  Eligible: VALID, not
 * PINNED, ref_count 0, on the host tier, no copy on the GPU tier, and depth <
 * anchor_blocks[agent] when that table is given.  Order: blocks of a* first, then score
 * descending, last_access descending, id ascending.  Outputs as for cs_select_victims(). */
int cs_select_prefetch(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t k,
                       uint32_t *ids_out, uint32_t *n_out, cs_stream_t stream);

/* Victim selection for callers that cannot allocate device memory (no counterpart in the
 * paper: it exists for embedders, not for the method).  A serving engine that gave the whole
 * GPU to its KV pool at start-up, a hook that runs while the host application forbids
 * allocation, or a process with a fixed memory budget can own inputs and outputs but cannot
 * provide a workspace.  This call needs neither a cs_ctx nor a workspace: the scratch of the
 * select kernels lives in a static device array inside the library (2 MiB + 40 KiB on every
 * GPU that loads the library, held until the process exits), and the call itself allocates
 * nothing, on the host or on the device.
 *   p      : the method's constants (n_chains and max_blocks are ignored).
 *   fsurv  : dev [n_agents], the survival factor p~ + delta of every agent (Eq. 8 plus the floor
 *            of Eq. 9), e.g. the fsurv table cs_get_model() returned earlier.
 *   the rest as for cs_select_victims(), with the same eligibility, order, padding and n_out.
 * Limits: idx->n_blocks and k at most CS_STATIC_MAX_BLOCKS, else CS_ECAPACITY.  Entries whose
 * agent is out of range are skipped without a status report.
 * The first call on a device looks up the device address of the static array (with that device
 * current); make that first call outside any stream capture.  All calls share the one array,
 * which keeps the previous call's contents: every call re-initialises what must start at zero,
 * and two calls of one process that overlap on the same GPU (different streams or threads)
 * race.  Issue them on one stream, or order them with events. */
#define CS_STATIC_MAX_BLOCKS 65536u
int cs_select_victims_static(const cs_params *p, const float *fsurv, const cs_block_index *idx, uint32_t now,
                             uint32_t tier, uint32_t k, uint32_t *ids_out, uint32_t *n_out, cs_stream_t stream);

/* ---- block mover (the paper reuses the serving engine's offload path, Sec. 4; these calls
 *      are that path written for B200) ------------------------------------------------------------ */

/* For i < n (n = min(n_max, *n_dev) when n_dev != NULL, else n_max), every layer and both
 * planes: copy the chunk of src slot src_slots[i] to dst slot dst_slots[i].  Entries with
 * CS_ID_NONE on either side are skipped.  src_slots / dst_slots / n_dev: dev.  The two pools
 * must agree in everything but base, n_slots and layout.  A pool base the device cannot address (pageable
 * host memory that was neither allocated page-locked nor registered) is CS_EINVAL: nothing is launched.
 * Destination slots must be distinct;
 * when src and dst are the same pool the two slot sets must be disjoint (not checked). */
int cs_offload_blocks(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *src_slots,
                      const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t side);
int cs_prefetch_blocks(cs_ctx *ctx, const cs_kv_pool *host, const cs_kv_pool *gpu, const uint32_t *src_slots,
                       const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t side);
int cs_compact_blocks(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                      const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t stream);

/* Offload and prefetch of one step in a single launch (the paper runs its evictions and prefetches
 * through the serving engine's offload path side by side, Sec. 4; the fused launch is this library's
 * way of keeping the two directions of the host link in step).  Equivalent to
 *   cs_offload_blocks(ctx, gpu, host, off_gpu_slots, off_host_slots, n_off_max, n_off_dev, side) and
 *   cs_prefetch_blocks(ctx, host, gpu, pre_host_slots, pre_gpu_slots, n_pre_max, n_pre_dev, side)
 * when no slot is written by one transfer and read or written by the other (not checked; otherwise the
 * order of the conflicting copies is unspecified).  Every copy pipeline walks its share of both lists
 * interleaved in proportion to their lengths, so both transfers finish together.  All slot lists and
 * counts: dev, as for the calls above; either list may be empty (n_*_max == 0 with NULL pointers).
 * Always takes the bulk path; its width is the host-link width of cs_set_mover_ctas() (default 32 warp
 * pipelines). */
int cs_exchange_blocks(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *off_gpu_slots,
                       const uint32_t *off_host_slots, uint32_t n_off_max, const uint32_t *n_off_dev,
                       const uint32_t *pre_host_slots, const uint32_t *pre_gpu_slots, uint32_t n_pre_max,
                       const uint32_t *n_pre_dev, cs_stream_t side);

/* ---- the same transfers on the GPU's copy engines --------------------------------------------------------
 * (No counterpart in the paper, which leaves the transfer to its engine's offload connector, Sec. 4; this is
 * the alternative to the SM-issued path above for engines whose latency-bound kernels must not share the SMs'
 * memory system with host-memory traffic.)
 *
 * cs_set_mover_staging(): hands the context a caller-owned DEVICE ring (256-byte aligned; at least 4 blocks,
 * 64-256 MiB is a sensible size) through which staged transfers pass, or takes it away (dev_ring = NULL).
 * The first call also creates the five streams and the events the staged calls use (host objects, released by
 * cs_destroy).  The ring must stay alive and unused by others while staged transfers are in flight.
 *
 * cs_exchange_blocks_staged(): offload of n_off blocks and prefetch of n_pre blocks.  GPU-side lists
 * (off_gpu_slots, pre_gpu_slots) are dev arrays exactly as for cs_exchange_blocks().  HOST-side lists
 * (off_host_ids, pre_host_ids) are arrays in HOST memory, read by this call before it returns: the copy
 * engines need addresses the host knows.  Each part of the offload list is packed into the ring by the mover
 * kernel and carried to the host tier by cudaMemcpyAsync, one call per run of consecutive host ids (a list of
 * consecutive ids becomes a few large copies); the prefetch is the mirror image, ending in a scatter launch.
 * The two directions are independent pipelines (pack launches on `stream`; copies and scatter launches on five
 * streams of the context), forked from and joined back into `stream` by events, so to the caller everything
 * is ordered on `stream`; the host is never synchronised.
 * Requirements: the host pool is CS_BLOCK_MAJOR (a block is one run of bytes), both pools agree in geometry.
 * A host id out of range, CS_ID_NONE included, is CS_EINVAL and nothing is issued (drop such entries and their
 * GPU-side partners before the call).  CS_ID_NONE or an out-of-range slot in a GPU-side list skips the entry on
 * the device (status word as usual); for an offload the corresponding host slot then receives unspecified bytes.  Results otherwise equal
 * cs_exchange_blocks() with the same lists.  The work counters book the blocks as offloaded / prefetched.
 * cs_offload_blocks_staged() / cs_prefetch_blocks_staged() are the one-directional forms. */
int cs_set_mover_staging(cs_ctx *ctx, void *dev_ring, size_t bytes);
int cs_exchange_blocks_staged(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *off_gpu_slots,
                              const uint32_t *off_host_ids, uint32_t n_off, const uint32_t *pre_host_ids,
                              const uint32_t *pre_gpu_slots, uint32_t n_pre, cs_stream_t stream);
int cs_offload_blocks_staged(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *src_slots,
                             const uint32_t *host_ids, uint32_t n, cs_stream_t stream);
int cs_prefetch_blocks_staged(cs_ctx *ctx, const cs_kv_pool *host, const cs_kv_pool *gpu, const uint32_t *host_ids,
                              const uint32_t *dst_slots, uint32_t n, cs_stream_t stream);

/* The selections of a step at once: cs_select_victims(tier 0, k_victims), cs_select_victims(tier 1,
 * k_victims) and cs_select_prefetch(k_prefetch) over the same index and clock, with the same results, run
 * side by side.  A selection whose count pointer is NULL is left out.  For index sizes the single-launch
 * select covers (<= 262,144 entries) they are the thread-block clusters of ONE launch; for larger indexes
 * each is a chain of grid-wide kernels, the first on `stream` and the others on two streams the context owns,
 * forked from and joined back into `stream` with events, so that to the caller everything is ordered on
 * `stream` (beyond 4,194,304 entries the selections run one after the other: private scratch of that size
 * is not reserved).  Arguments as for the single calls. */
int cs_select_step(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t k_victims, uint32_t k_prefetch,
                   uint32_t *gpu_victims, uint32_t *n_gpu_victims, uint32_t *host_victims, uint32_t *n_host_victims,
                   uint32_t *prefetch_ids, uint32_t *n_prefetch, cs_stream_t stream);

/* ---- one whole step as one call ------------------------------------------------------------------------ */

/* The calls of one scheduler step in their order (Algorithm 1: ObserveTouch for the step's invocations,
 * Evict for both tiers, BetweenStep's prefetch ranking) followed by the transfers that carry the decisions
 * out, with every list and count staying on the device:
 *   main: cs_observe_invocations(chain, agent, evflags, n_events)
 *         cs_select_step(idx, now, k_victims, k_prefetch) -> gpu_victims, n_gpu_victims (tier 0),
 *                                                            host_victims, n_host_victims (tier 1),
 *                                                            prefetch_ids, n_prefetch
 *         every prefetch candidate whose host slot is one of this step's offload destinations is replaced
 *         by CS_ID_NONE in prefetch_ids (it would be read while it is overwritten); n_prefetch still counts it
 *         cs_compact_blocks(gpu -> stage, gpu_victims -> stage_slots)            (skipped when stage == NULL)
 *   side: cs_exchange_blocks(gpu, host; gpu_victims -> host_victims, count min(n_gpu_victims, n_max);
 *                            prefetch_ids -> free_gpu_slots)                     (after the calls above)
 * The number of blocks offloaded is *n_gpu_victims; when the host tier yields fewer victims than that, the
 * surplus entries of host_victims hold CS_ID_NONE and those blocks are skipped.  side may equal main; when
 * it differs, main does not wait for the transfers unless join_main != 0 (needed when the call is captured
 * into a CUDA graph from main: the side stream must rejoin before the capture ends).
 * now_dev / n_events_dev (dev, optional): when not NULL the clock and the event count (at most n_events) are
 * read from device memory when the kernels run, not when the call is made, so that a captured graph can be
 * replayed for later steps after the caller has updated those words and the event buffers.
 * All pointers in the struct: dev, except idx / gpu / host / stage (host structs).  The fork and join use two
 * CUDA events the context owns (host objects made by cs_create, released by cs_destroy).  Before capturing
 * the call into a graph, run each kind of call it contains once outside capture: the first launch of a
 * kernel family sets its shared-memory attributes and probes the cluster size. */
typedef struct cs_step_io {
    const uint32_t *chain;
    const uint16_t *agent;
    const uint8_t *evflags;
    uint32_t n_events;
    const uint32_t *n_events_dev;
    const cs_block_index *idx;
    uint32_t now;
    const uint32_t *now_dev;
    uint32_t k_victims, k_prefetch;
    uint32_t *gpu_victims, *n_gpu_victims;
    uint32_t *host_victims, *n_host_victims;
    uint32_t *prefetch_ids, *n_prefetch;
    const cs_kv_pool *gpu, *host, *stage;
    const uint32_t *stage_slots;       /* [k_victims] destination slots in the staging pool */
    const uint32_t *free_gpu_slots;    /* [k_prefetch] GPU slots that receive the prefetched blocks */
    uint32_t join_main;
} cs_step_io;
int cs_step(cs_ctx *ctx, const cs_step_io *io, cs_stream_t main, cs_stream_t side);

/* ---- inspection ------------------------------------------------------------------------------------ */

/* Copies the learner / scorer state into caller dev buffers (any may be NULL):
 * C [A*A] counts, P [A*A] Eq. 3, amax [A], hops [A] (CS_HOP_NONE = unreachable), fsurv [A]
 * (= p~ + delta), R [1], cur [n_chains], last_agent [1]. */
int cs_get_model(cs_ctx *ctx, uint32_t *C_out, float *P_out, uint16_t *amax_out, uint16_t *hops_out,
                 float *fsurv_out, float *R_out, uint16_t *cur_out, uint16_t *last_agent_out,
                 cs_stream_t stream);

/* Checkpoint / resume.  The learner's state is the counts, the per-chain current agents and the last
 * agent; cs_get_model() exports them (C_out, cur_out, last_agent_out) and this call restores them into
 * a context created with the same n_agents / n_chains, then refreshes everything derived from the
 * counts exactly as cs_observe_invocations() does.  C_in: dev [A*A] (the diagonal is ignored: self
 * transitions are never counted); cur_in: dev [n_chains] or NULL (= no current agent on any chain);
 * last_agent: CS_AGENT_NONE or an agent id. */
int cs_import_state(cs_ctx *ctx, const uint32_t *C_in, const uint16_t *cur_in, uint32_t last_agent,
                    cs_stream_t stream);

/* Returns the device status word in *device_status and clears it: one small kernel on `stream` swaps the
 * word with zero atomically, the call then synchronises `stream` and reads the swapped-out value.  Bits
 * that a kernel on another stream (a transfer on a side stream) sets after the swap stay for the next
 * call; for an exact report of a finished step, order the side stream before `stream` first.
 * Returns CS_EDEVICE_STATUS when the word was non-zero. */
int cs_get_status(cs_ctx *ctx, uint32_t *device_status, cs_stream_t stream);

/* Number of kernels this context has launched so far (host counter). */
int cs_launch_count(cs_ctx *ctx, uint64_t *n_launches);

/* Work counters kept in the workspace by the kernels themselves (the paper reports only hit rate and
 * latency, Sec. 5.1; these are this library's metrics).  All cumulative since cs_create() or the last
 * reset, except `eligible`, which describes the latest select of each kind.  Kinds: 0 GPU-tier victims,
 * 1 host-tier victims, 2 prefetch candidates; directions: 0 device-to-device, 1 offload, 2 prefetch. */
typedef struct cs_counters {
    uint64_t events_seen;           /* events handed to cs_observe_invocations() */
    uint64_t events_skipped;        /* of those: warmup-flagged, or agent / chain out of range */
    uint64_t transitions_counted;   /* increments of the transition counts (agent changes) */
    uint64_t selects[3];            /* selects completed, per kind */
    uint64_t eligible[3];           /* eligible entries the latest select of the kind saw */
    uint64_t selected[3];           /* ids emitted, per kind */
    uint64_t candidates[3];         /* keys the latest select of the kind had to order (k winners + ties of the threshold bin) */
    uint64_t fast_hits[3];          /* selects whose remembered threshold held: the index was read once, mostly without keys */
    uint64_t blocks_moved[3];       /* blocks copied, per direction */
    uint64_t bytes_moved[3];        /* their bytes (block_bytes each) */
    uint64_t blocks_skipped;        /* mover list entries skipped: CS_ID_NONE or slot out of range */
    uint64_t region_selects[3];     /* multi-launch selects whose sample-sort buckets were filled in place (cs_set_select_bucket_regions) */
    uint64_t region_overflows[3];   /* of those: a bucket outgrew its region and the buckets were grouped by a launch of their own */
} cs_counters;

/* Synchronises `stream` and copies the counters to *out (host memory); reset != 0 clears them afterwards. */
int cs_get_counters(cs_ctx *ctx, cs_counters *out, uint32_t reset, cs_stream_t stream);

/* ---- checkers (debugging aids; the paper has no counterpart) ------------------------------------------ */

/* Checks a select result on the device, independently of how it was produced: ids_out[0, n) name eligible
 * entries (same rules as cs_select_victims / cs_select_prefetch with these arguments), their keys are
 * strictly increasing (so the ids are unique), exactly n eligible entries have a key at or below the last
 * one, n = min(k, number eligible), and ids_out[n, k) hold CS_ID_NONE.  Any violation sets
 * CS_ST_BAD_SELECTION in the status word.  One scan of the index; run it on the stream of the select.
 * prefetch != 0 checks a cs_select_prefetch() list (tier is then ignored). */
int cs_validate_selection(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t prefetch, uint32_t tier,
                          uint32_t k, const uint32_t *ids_out, const uint32_t *n_out, cs_stream_t stream);

/* Checks the slot lists of a mover call before it is issued (arguments as for cs_compact_blocks /
 * cs_offload_blocks / cs_prefetch_blocks): two entries with the same destination slot, or -- when src and
 * dst are the same pool -- a slot that is both read and written, set CS_ST_LIST_CONFLICT.  Entries the
 * mover would skip (CS_ID_NONE on either side) are ignored.  Cost: n^2 id compares. */
int cs_validate_move_lists(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                           const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t stream);

/* The same for the two transfers of cs_exchange_blocks() (same arguments): each list on its own, plus
 * host slots written by the offload and read by the prefetch, and GPU slots read by the offload and written
 * by the prefetch. */
int cs_validate_exchange_lists(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host,
                               const uint32_t *off_gpu_slots, const uint32_t *off_host_slots, uint32_t n_off_max,
                               const uint32_t *n_off_dev, const uint32_t *pre_host_slots, const uint32_t *pre_gpu_slots,
                               uint32_t n_pre_max, const uint32_t *n_pre_dev, cs_stream_t stream);

/* Self-test of the mover's bounded wait (no counterpart in the paper).  Launches one warp that sets up a
 * transfer barrier, issues NO copy, and waits on the barrier with the mover's own wait routine limited to
 * `max_polls` polls (1 .. 1,000,000).  Nothing can complete the barrier, so the wait runs out, the kernel
 * sets CS_ST_TIMEOUT in the status word -- the path a stalled transfer would take -- and returns.  No data
 * is in flight, so nothing is left behind; the context stays usable. */
int cs_selftest_bounded_wait(cs_ctx *ctx, uint32_t max_polls, cs_stream_t stream);

/* Phase stamps of the latest calls (profiling builds only: a library compiled with -DCS_PHASE_STAMPS makes its kernels
 * store the GPU's global nanosecond timer at phase boundaries -- refresh: entry, dependency wait over, rows done, last
 * CTA starts, sums done, end; scans: entry, set-up done, wait over, index read, flushed, last CTA starts, tail done;
 * ordering: bucket wait over / done, scatter wait over, rank wait over / done -- slots as in the CS_PS_* list of
 * csrc/cs_common.cuh, the prefetch select's eight slots above the victims').  Synchronises the device and copies the
 * CS_PHASE_STAMP_SLOTS stamps to `out` (host).  An ordinary build returns CS_ENOTIMPL and stores nothing. */
#define CS_PHASE_STAMP_SLOTS 64
int cs_debug_phase_stamps(cs_ctx *ctx, uint64_t *out);

/* Width of the mover (0 keeps the default): for transfers that cross the host link and for
 * device-to-device moves.  Unit: warp pipelines on the bulk path (each keeps up to two loads and two
 * stores of 16 KiB in flight; defaults 8 offload / 24 prefetch / 2 per SM device-to-device), CTAs of
 * 256 threads on the load/store path.  Narrow host-link transfers disturb other kernels less. */
int cs_set_mover_ctas(cs_ctx *ctx, uint32_t host_link_ctas, uint32_t d2d_ctas);

/* Data path of the mover: CS_MOVER_AUTO (= bulk), CS_MOVER_LDST (128-bit loads and stores by
 * every thread), CS_MOVER_BULK (1-D bulk asynchronous copies staged through shared memory). */
#define CS_MOVER_AUTO 0u
#define CS_MOVER_LDST 1u
#define CS_MOVER_BULK 2u
int cs_set_mover_path(cs_ctx *ctx, uint32_t path);

/* Sources of the cached hop table (Eq. 8).  The paper's runtime serves one request at a time and starts
 * the BFS at that request's current agent (Sec. 3.3); CS_SOURCES_LAST_AGENT is that.  With many sessions
 * in flight, CS_SOURCES_ALL_CHAINS starts it at the current agent of EVERY chain that has one (all live
 * sessions): E[a] is then the hop distance from the nearest of them, and blocks of any agent that some live
 * session is about to reach are protected.  Prefetch ranking keeps using the successor of the last invoked
 * agent (Eq. 10).  The call refreshes the cached tables on `stream`; later cs_observe_invocations() calls
 * keep the mode. */
#define CS_SOURCES_LAST_AGENT 0u
#define CS_SOURCES_ALL_CHAINS 1u
int cs_set_survival_sources(cs_ctx *ctx, uint32_t mode, cs_stream_t stream);

/* ---- exact survival probability (the quantity Eq. 8 approximates) ---------------------------------- */

/* Eq. 6 for every agent a: p_surv(a; a0, K) = Pr(a is invoked within the next K dispatches | the
 * current agent is a0), computed exactly from the matrix of Eq. 3 by pushing the unit mass at a0
 * through K steps of the chain with state a removed.  a0 = CS_AGENT_NONE uses the current agent
 * (agent of the last observed event; all zeros while there is none).  n_steps = K <= 4096.
 * psurv_out: dev [n_agents] p_surv; fsurv_out: dev [n_agents] p_surv + delta, the first factor of
 * Eq. 9 (either may be NULL).  fp64 accumulation, fp32 results.  Cost n_agents^3 * K multiply-adds. */
int cs_exact_survival(cs_ctx *ctx, uint32_t a0, uint32_t n_steps, float *psurv_out, float *fsurv_out,
                      cs_stream_t stream);

/* Makes cs_score_blocks (without explicit sources), cs_select_victims and cs_select_prefetch use
 * the caller's survival table (dev [n_agents], e.g. fsurv_out above, which must stay alive) in place
 * of the hop-distance table of Eq. 8; NULL restores the default.  Host-side switch, no launch. */
int cs_use_survival_table(cs_ctx *ctx, const float *fsurv);

/* Implementation of the two select calls: CS_SELECT_AUTO (= the single-launch cluster kernel up
 * to 262,144 index entries, the multi-launch path above), CS_SELECT_CLUSTER, CS_SELECT_MULTI
 * (fast pass / histogram / collect / bucket / scatter / rank as six grid-wide launches).  Both give the
 * same lists. */
#define CS_SELECT_AUTO 0u
#define CS_SELECT_CLUSTER 1u
#define CS_SELECT_MULTI 2u
int cs_set_select_path(cs_ctx *ctx, uint32_t path);

/* The multi-launch select remembers the threshold bin each kind of call (GPU victims, host victims,
 * prefetch) ended with, and the next call of that kind collects candidates up to that bin while it
 * builds its histogram; when the new threshold is not above the remembered one the index is read
 * once instead of twice.  The result never depends on it.  enabled = 0 turns the speculation off. */
int cs_set_select_speculation(cs_ctx *ctx, uint32_t enabled);

/* The multi-launch select orders its candidates by a sample sort into <= 256 buckets.  When the candidates are few
 * for the size of the workspace (8 c <= max_blocks) every bucket owns a fixed region of the sort arrays --
 * max_blocks / (buckets) keys, at most 2048 -- which the bucket launch fills directly; a bucket that outgrows its
 * region makes the call fall back to grouping the buckets in a launch of its own.  max_keys caps that region
 * (0 = no cap, the default; 1 = every bucket with two keys or more takes the fallback).  The result never depends
 * on it: the setting exists so that both routes can be exercised and compared.  Host-side, takes effect from the
 * next select call. */
int cs_set_select_bucket_regions(cs_ctx *ctx, uint32_t max_keys);

/* Clock source for CUDA-graph replay (the paper's runtime reads now() when a block is touched, Algorithm 1;
 * a captured call would freeze its `now` argument).  While now_dev (dev, 4-byte aligned) is set, every
 * cs_score_blocks / cs_select_* call issued on this context reads the clock from that word WHEN ITS KERNELS
 * RUN and ignores its `now` argument, so one captured sequence serves later steps after the caller has
 * updated the word.  NULL restores the argument.  Host-side switch, no launch. */
int cs_set_device_clock(cs_ctx *ctx, const uint32_t *now_dev);

/* cudaError_t of the last failing CUDA call on this context (0 if none). */
int cs_last_cuda_error(cs_ctx *ctx);
const char *cs_strerror(int code);
int cs_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CACHESCOUT_H */
