// Internal declarations shared by the translation units of libcachescout (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "cachescout.h"

// NVTX ranges around the entry points that enqueue work: a timeline tool shows which library call a kernel belongs
// to.  Header-only (NVTX 3 loads the tool's injection library on first use; without a tool a range costs a few
// nanoseconds).  -DCS_NO_NVTX compiles the ranges out.
#ifndef CS_NO_NVTX
#include <nvtx3/nvToolsExt.h>
struct cs_nvtx_range {
    explicit cs_nvtx_range(const char *name) { nvtxRangePushA(name); }
    ~cs_nvtx_range() { nvtxRangePop(); }
};
#define CS_RANGE(name) cs_nvtx_range cs_range_guard_(name)
#else
#define CS_RANGE(name) do { } while (0)
#endif

#if defined(__CUDA_ARCH__) && (__CUDA_ARCH__ < 1000)
#error "libcachescout is written for sm_100a (B200) only"
#endif

#define CS_SELECT_CLUSTER_MAX_BLOCKS (1u << 18)   // above this the index is scanned by the whole grid instead

#define CS_CONCURRENT_MAX_BLOCKS (1u << 22)        // up to this index size every select of a step has full-size scratch of its own

#define CS_AGE_LIMIT_MIN_BLOCKS (1u << 21)        // index size from which the collect pass builds age limits

#define CS_MOVE_D2D 0
#define CS_MOVE_OFFLOAD 1
#define CS_MOVE_PREFETCH 2
#define CS_MOVE_STAGE 3            // pack / scatter launch of the copy-engine path: inside the device, deliberately narrow

#define CS_HIST_BINS 4096u        // first radix digit of the select: top 12 bits of the primary key
#define CS_MAX_SPLITTERS 255u     // bucket sort of the candidates: up to 256 buckets
#define CS_SAMPLE 1024u           // candidates sampled to choose the splitters
#define CS_GTAB_MAX 4096u          // largest recency table kept in shared memory (ages below saturation)

// Scalars the kernels share, one 256-byte line in the workspace.
#define CS_BCOUNT_STRIDE 8u                                      // words between bucket counters
#define CS_BCOUNT(ws, b) ((ws).bcount[(size_t)(b) * CS_BCOUNT_STRIDE])
// Phase stamps (builds with -DCS_PHASE_STAMPS only; cs_debug_phase_stamps() reads them).  A call's kernels are chains
// of dependent steps whose cost is latency, not work, so "where does the time go" is answered by the GPU's global
// nanosecond timer read at the boundaries: CS_STAMP(ws, slot, cond) stores it into slot `slot` when `cond` holds
// (one thread of one CTA).  In ordinary builds the macro is empty and the slots do not exist.
#define CS_N_PHASE_STAMPS 64
enum {
    CS_PS_REFRESH_ENTRY = 0, CS_PS_REFRESH_WAITED, CS_PS_REFRESH_ROWS_DONE, CS_PS_REFRESH_LAST_CTA, CS_PS_REFRESH_SUMS_DONE,
    CS_PS_REFRESH_END,
    CS_PS_SCAN_ENTRY = 8,       // + 8 for the prefetch select: entry, set-up done, waited, index read, flushed, last CTA, tail done
    CS_PS_SCAN_SETUP, CS_PS_SCAN_WAITED, CS_PS_SCAN_READ, CS_PS_SCAN_FLUSHED, CS_PS_SCAN_LAST_CTA, CS_PS_SCAN_TAIL_DONE,
    CS_PS_BUCKET_WAITED = 24,   // + 8 for the prefetch select: bucket waited / done, scatter waited, rank waited / done
    CS_PS_BUCKET_DONE, CS_PS_SCATTER_WAITED, CS_PS_RANK_WAITED, CS_PS_RANK_DONE, CS_PS_BUCKET_STAGED, CS_PS_BUCKET_SEARCHED,
    CS_PS_BUCKET_SLOTS,
    CS_PS_RANK_OFFSETS = 40,    // + 8 for the prefetch select: bucket offsets known, bucket in the tile, tile sorted (CTA 0)
    CS_PS_RANK_LOADED, CS_PS_RANK_SORTED,
    CS_PS_SCAN_TABLES = 56,     // + 4 for the prefetch select: per-call tables loaded, age cuts built, index tiles walked (CTA 0)
    CS_PS_SCAN_CUTS, CS_PS_SCAN_WALKED
};
#ifdef CS_PHASE_STAMPS
#define CS_STAMP(ws, slot, cond)                                                         \
    do {                                                                                 \
        if (cond) {                                                                      \
            unsigned long long cs_t_;                                                    \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(cs_t_)::"memory");          \
            (ws).sc->stamps[slot] = cs_t_;                                               \
        }                                                                                \
    } while (0)
#else
#define CS_STAMP(ws, slot, cond) do { } while (0)
#endif

struct cs_scalars {
    uint32_t status;        // CS_ST_* bits
    uint32_t last_agent;    // agent of the last non-warmup event, CS_AGENT_NONE initially
    uint32_t a_star;        // arg-max successor of last_agent (Eq. 10), ~0 while there is no current agent; kept by the refresh
    float R;                // Eq. 2
    uint32_t gate;          // Eq. 11: R >= r_min
    uint32_t n_transitions; // sum of all counts
    uint32_t ticket0;       // "last CTA done" counter of the learner refresh
    uint32_t gtab_monotone; // the recency table covers every unsaturated age and never increases with age
    uint32_t status_read;   // cs_get_status(): the value swapped out of `status`
    uint32_t val_le, val_elig, val_ticket;   // cs_validate_selection(): keys at or below the last one, eligible entries, ticket
    uint32_t adjT_cur;      // which copy of the transposed adjacency the last refresh filled
    uint32_t sel_hint[4];   // bin up to which the next select of each kind (GPU victims, host victims, prefetch)
                            // collects ahead of its own threshold, chosen from the previous call's histogram;
                            // ~0 = none; slot 3 is never written: calls that must not speculate read it
    unsigned long long qbase;   // Eq. 2 column sums: what every column gets from the rows' zero-count entries (see qfix)
#ifdef CS_PHASE_STAMPS
    unsigned long long stamps[CS_N_PHASE_STAMPS];   // %globaltimer at phase boundaries of the latest call (profiling builds)
#endif
};

// State of one select in flight, rewritten by every call.  The selects of a step that run side by side each
// have their own (with their own histogram, candidate and sort regions).
struct cs_sel_state {
    // what the bucket launch reads first, as one 16-byte word
    uint32_t c;             // candidates collected (first digit <= b0)
    uint32_t n_spl;         // splitters in use
    uint32_t placed;        // 1: every bucket has a fixed region of `cap` keys in the sort arrays, filled by the bucket launch
    uint32_t cap;           // keys per bucket region
    uint32_t n_out;         // min(k, eligible)
    uint32_t overflow;      // 1: a bucket outgrew its region; the scatter launch groups the buckets instead
    uint32_t b0;            // threshold bin of the first digit
    uint32_t n_elig;        // eligible entries
    uint32_t ticket[6];     // "last CTA done" counters, one per kernel that has an epilogue
    uint32_t c_spec;        // candidates appended by the fast pass; 0 between calls
    uint32_t n_above;       // eligible entries the fast pass found above the remembered bin; 0 between calls
    uint32_t spec;          // 1: the fast pass's candidates cover the k winners, the histogram and collect passes are skipped
    uint32_t cc[2];         // candidate counters of the cluster kernel: a call uses one and clears the other for the
                            // next call, so that the counter is zero on entry without a barrier
    uint32_t toggle;        // which of the two the next call uses; flipped by every call on the device, so that a
                            // captured sequence of calls stays consistent when it is replayed
};

// Device pointers into the caller's workspace.
struct cs_workspace {
    cs_scalars *sc;
    cs_counters *cnt;     // work counters (cs_get_counters)
    cs_sel_state *sel;    // this select's state (one per concurrent select)
    uint32_t *C;          // [A*A] transition counts
    uint32_t *rowsum;     // [A]
    uint16_t *cur;        // [n_chains]
    float *P;             // [A*A] Eq. 3
    uint16_t *amax;       // [A]
    double *rowH;         // [A] sum_j P_ij ln P_ij
    unsigned long long *qfix;   // [A] column sums of Eq. 2 in 2^-60 fixed point, WITHOUT the part that is the same for every
                                // column (sc->qbase); zero between refreshes
    uint32_t *adj;        // [A*W] Eq. 7 adjacency, one bit per edge, W = ceil(A/32)
    uint32_t *adjT;       // [2][A*W] its transpose (row v = the predecessors of v), two copies used in turn: a refresh
                          // fills one with atomics and clears the other for the refresh after it
    uint16_t *hops;       // [A]
    float *fsurv;         // [A] p~ + delta for the cached source
    uint16_t *hops_tmp;   // [A] same, for cs_score_blocks() with explicit sources
    float *fsurv_tmp;     // [A]
    float *gtab;          // [gtab_len] exp(-lambda*age)+delta for age < gtab_len
    uint32_t *hist;       // [CS_HIST_BINS]
    unsigned long long *cand_km;    // [max_blocks] (primary<<32 | secondary) of each candidate
    uint32_t *cand_id;    // [max_blocks]
    uint32_t *cand_bkt;   // [max_blocks]
    uint32_t *cand_slot;  // [max_blocks]
    unsigned long long *sort_km;    // [max_blocks] candidates grouped by bucket
    uint32_t *sort_id;    // [max_blocks]
    unsigned long long *spl_km;     // [CS_MAX_SPLITTERS+1]
    uint32_t *spl_id;     // [CS_MAX_SPLITTERS+1]
    uint32_t *bcount;     // bucket counters, one per 32-byte sector (CS_BCOUNT): atomics on counters that share a sector
                          // queue up behind one another in L2 (measured: 3.6 us for 16,000 of them on adjacent words,
                          // 0.8 us on separate sectors; separate 128-byte lines are no faster and cost the readers more)
};

struct cs_ctx {
    cs_params p;
    cs_workspace ws;
    cs_workspace ws_job[2];        // the same workspace with private candidate / sort regions: jobs 1 and 2 of a fused select
    size_t ws_bytes;
    uint32_t W;            // adjacency words per row
    uint32_t gtab_len;     // ages [0, gtab_len) come from the table
    uint32_t age_sat;      // ages >= age_sat all give g_sat
    int device;
    int sm_count;
    uint32_t host_link_ctas, d2d_ctas;
    uint32_t mover_path;   // CS_MOVER_*
    uint32_t select_path;  // CS_SELECT_*
    uint32_t no_speculation;       // 1: the histogram pass never collects ahead of the threshold
    uint32_t region_cap_max;       // cap on the keys of a bucket's own region in the sort arrays (0: none)
    uint32_t source_mode;          // CS_SOURCES_*: where the cached BFS of Eq. 8 starts
    const float *fsurv_override;   // caller's survival table for score / select, NULL = the BFS table of Eq. 8
    const uint32_t *clock_dev;           // cs_set_device_clock(): selects and scores read the clock from here when they run
    const uint32_t *step_now_dev;        // set only while cs_step() issues its calls: device-resident clock / event count
    const uint32_t *step_n_events_dev;
    cudaEvent_t ev_fork, ev_join;        // cs_step(): main -> side and side -> main
    cudaStream_t sel_stream[2];          // the second and third select of a step run here, beside the first
    cudaEvent_t ev_sel_fork, ev_sel_join[2];
    int concurrent_selects;              // the per-select scratch regions are full size
    // copy-engine path of the mover (cs_set_mover_staging): caller-owned device ring split into four sub-buffers
    // (two per direction, double-buffered), two streams of the context for the two DMA directions, and the events
    // that order packing / copying / scattering
    unsigned char *stage_ring;
    size_t stage_bytes;
    cudaStream_t copy_stream[4];         // 0, 1: device -> host; 2, 3: host -> device
    cudaStream_t scatter_stream;         // scatter launches of staged prefetches
    cudaEvent_t ev_stage_fork, ev_stage_join[2];
    cudaEvent_t ev_packed[2], ev_copied[4], ev_filled[4], ev_scattered[2];   // [ring buffer] or [2 * ring buffer + copy stream]
    uint64_t n_launches;
    int last_cuda_error;
};

// ---- workspace layout (host) -------------------------------------------------------------------
size_t cs_layout_workspace(const cs_params *p, uint32_t gtab_len, void *base, cs_workspace *ws, cs_workspace *ws_job);
int cs_validate_params(const cs_params *p);
void cs_recency_table_shape(const cs_params *p, uint32_t *gtab_len, uint32_t *age_sat);

// ---- launchers implemented in the kernel files ---------------------------------------------------
int cs_launch_init(cs_ctx *ctx, cudaStream_t s);
int cs_launch_observe(cs_ctx *ctx, const uint32_t *chain, const uint16_t *agent, const uint8_t *evflags,
                      uint32_t n_events, cudaStream_t s);
int cs_launch_import(cs_ctx *ctx, const uint32_t *C_in, const uint16_t *cur_in, uint32_t last_agent, cudaStream_t s);
int cs_launch_survival(cs_ctx *ctx, const uint16_t *sources, uint32_t n_sources, cudaStream_t s);
int cs_launch_exact_survival(cs_ctx *ctx, uint32_t a0, uint32_t K, float *psurv_out, float *fsurv_out, cudaStream_t s);
int cs_launch_score(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, const float *fsurv,
                    float *scores_out, cudaStream_t s);
int cs_launch_select(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, int prefetch, uint32_t tier,
                     uint32_t k, uint32_t *ids_out, uint32_t *n_out, cudaStream_t s);
int cs_launch_select_step(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t k_victims, uint32_t k_prefetch,
                          uint32_t *gpu_victims, uint32_t *n_gpu, uint32_t *host_victims, uint32_t *n_host,
                          uint32_t *prefetch_ids, uint32_t *n_prefetch, cudaStream_t s);
int cs_launch_select_clusters(cs_ctx *ctx, int n_jobs, const void *sel_args, const uint32_t *prefetch,
                              uint32_t *const *ids_out, uint32_t *const *n_out, cudaStream_t s);
int cs_launch_select_cluster(cs_ctx *ctx, const void *sel_args, const cs_workspace *ws, int prefetch, uint32_t *ids_out,
                             uint32_t *n_out, cudaStream_t s);
int cs_launch_mover(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                    const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, int kind,
                    cudaStream_t s);

int cs_launch_mover_as(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                       const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, int kind, int count_as,
                       cudaStream_t s);
int cs_launch_bounded_wait_selftest(cs_ctx *ctx, uint32_t max_polls, cudaStream_t s);
int cs_launch_validate_selection(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, int prefetch, uint32_t tier,
                                 uint32_t k, const uint32_t *ids, const uint32_t *n_out, cudaStream_t s);
int cs_launch_validate_lists(cs_ctx *ctx, const uint32_t *w_list, const uint32_t *w_partner, uint32_t nw_max,
                             const uint32_t *nw_dev, const uint32_t *x_list, const uint32_t *x_partner, uint32_t nx_max,
                             const uint32_t *nx_dev, int self, cudaStream_t s);
bool cs_device_can_address(const void *ptr);
void cs_release_staging(cs_ctx *ctx);

int cs_launch_exchange(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *off_gpu_slots,
                       const uint32_t *off_host_slots, uint32_t n_off_max, const uint32_t *n_off_dev,
                       const uint32_t *pre_host_slots, const uint32_t *pre_gpu_slots, uint32_t n_pre_max,
                       const uint32_t *n_pre_dev, cudaStream_t s);

static inline int cs_check_launch(cs_ctx *ctx)
{
    cudaError_t e = cudaGetLastError();
    ctx->n_launches++;
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return CS_OK;
}

#ifdef __CUDACC__
// Programmatic dependent launch.  The chains of small kernels (observe -> normalise; histogram -> collect ->
// bucket -> scatter -> rank) are bound by launch latency, so each kernel of a chain is launched with the
// programmatic-serialisation attribute: its launch overlaps the tail of its predecessor, and its first
// instruction waits until the predecessor grid has completed and its writes are visible.  A kernel launched
// without the attribute executes the wait as a no-op.
#ifndef CS_USE_PDL
#define CS_USE_PDL 1
#endif
// Loads that stay where they are written.  The compiler is free to sink an ordinary load to its first use, which
// turns "fetch sixteen words, then work on them" into sixteen round trips to L2, one after the other (measured:
// 950 cycles each).  These can neither be sunk nor reordered against each other or against other memory
// operations, so a run of them is in flight together and costs one round trip.
__device__ __forceinline__ uint32_t cs_ld_cg_pinned(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint2 cs_ld_cg_pinned(const uint2 *p)
{
    uint2 v;
    asm volatile("ld.global.cg.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint16_t cs_ld_cg_pinned(const uint16_t *p)
{
    uint16_t v;
    asm volatile("ld.global.cg.u16 %0, [%1];" : "=h"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long cs_ld_cg_pinned(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.global.cg.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint4 cs_ld_cg_pinned(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ ulonglong2 cs_ld_cg_pinned(const ulonglong2 *p)
{
    ulonglong2 v;
    asm volatile("ld.global.cg.v2.u64 {%0, %1}, [%2];" : "=l"(v.x), "=l"(v.y) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void cs_wait_for_predecessor()
{
#if CS_USE_PDL
    asm volatile("griddepcontrol.wait;" ::: "memory");
#endif
}
// Lets the successor's launch proceed; called once the calling CTA no longer competes for the SM.
__device__ __forceinline__ void cs_release_successor()
{
#if CS_USE_PDL
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#endif
}

template <class... KArgs, class... Args>
static inline void cs_launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = CS_USE_PDL;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    (void)cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);       // the caller reads the error with cs_check_launch()
}

// Recency factor of Eq. 9 as every kernel computes it: fp64 exp and add, rounded once to fp32.
__device__ __forceinline__ float cs_recency(float lambda, float delta, uint32_t age)
{
    return (float)(exp(-(double)lambda * (double)age) + (double)delta);
}
#endif
