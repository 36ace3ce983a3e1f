// C-ABI entry points: argument validation, workspace layout, context life cycle.
// All device work is in cs_model.cu, cs_select.cu and cs_mover.cu.
#include <math.h>
#include <new>
#include <string.h>

#include "cs_common.cuh"

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline bool aligned16(const void *p) { return (((uintptr_t)p) & 15u) == 0; }

int cs_validate_params(const cs_params *p)
{
    if (!p) return CS_EINVAL;
    if (p->n_agents < 1 || p->n_agents > CS_MAX_AGENTS) return CS_EINVAL;
    if (p->n_chains < 1 || p->n_chains > (1u << 24)) return CS_EINVAL;
    if (p->max_blocks < 1) return CS_EINVAL;
    if (p->block_tokens < 1 || p->block_tokens > 255) return CS_EINVAL;
    if (p->e_max < 1 || p->e_max > 0xFFFEu) return CS_EINVAL;
    if (!(p->eps > 0.0f) || !isfinite(p->eps)) return CS_EINVAL;       // Eq. 3 is 0/0 on a cold row otherwise
    if (!isfinite(p->tau)) return CS_EINVAL;
    if (!(p->lambda >= 0.0f) || !isfinite(p->lambda)) return CS_EINVAL;
    if (!(p->delta > 0.0f) || !isfinite(p->delta)) return CS_EINVAL;    // the floor keeps both factors positive
    if (!isfinite(p->r_min)) return CS_EINVAL;
    if (p->prefer_other_copy > 1) return CS_EINVAL;
    return CS_OK;
}

// exp(-lambda*age) <= delta * 2^-26 cannot change f32(exp(..) + delta): from that age on the
// recency factor is the constant f32(delta)-rounded value, so only younger ages need a table.
void cs_recency_table_shape(const cs_params *p, uint32_t *gtab_len, uint32_t *age_sat)
{
    double sat;
    if (p->lambda > 0.0f) sat = ceil((26.0 * log(2.0) - log((double)p->delta)) / (double)p->lambda) + 1.0;
    else sat = 1.0;                                   // lambda = 0: the factor is constant from age 0
    if (sat < 1.0) sat = 1.0;
    if (sat > 4294967295.0) sat = 4294967295.0;
    *age_sat = (uint32_t)sat;
    *gtab_len = *age_sat < CS_GTAB_MAX ? *age_sat : CS_GTAB_MAX;
}

size_t cs_layout_workspace(const cs_params *p, uint32_t gtab_len, void *base, cs_workspace *ws, cs_workspace *ws_job)
{
    const size_t A = p->n_agents, W = (A + 31) / 32, N = p->max_blocks;
    size_t off = 0;
    char *b = (char *)base;
#define TAKE(field, type, count)                                  \
    do {                                                          \
        if (ws) ws->field = (type *)(b + off);                    \
        off = align_up(off + sizeof(type) * (size_t)(count), 256); \
    } while (0)
    TAKE(sc, cs_scalars, 1);
    TAKE(cnt, cs_counters, 1);
    TAKE(sel, cs_sel_state, 1);
    TAKE(C, uint32_t, A * A);
    TAKE(rowsum, uint32_t, A);
    TAKE(cur, uint16_t, p->n_chains);
    TAKE(P, float, A * A);
    TAKE(amax, uint16_t, A);
    TAKE(rowH, double, A);
    TAKE(qfix, unsigned long long, A);
    TAKE(adj, uint32_t, A * W);
    TAKE(adjT, uint32_t, 2 * A * W);
    TAKE(hops, uint16_t, A);
    TAKE(fsurv, float, A);
    TAKE(hops_tmp, uint16_t, A);
    TAKE(fsurv_tmp, float, A);
    TAKE(gtab, float, gtab_len);
    TAKE(hist, uint32_t, CS_HIST_BINS);
    TAKE(cand_km, unsigned long long, N);
    TAKE(cand_id, uint32_t, N);
    TAKE(cand_bkt, uint32_t, N);
    TAKE(cand_slot, uint32_t, N);
    TAKE(sort_km, unsigned long long, N);
    TAKE(sort_id, uint32_t, N);
    TAKE(spl_km, unsigned long long, CS_MAX_SPLITTERS + 1);
    TAKE(spl_id, uint32_t, CS_MAX_SPLITTERS + 1);
    TAKE(bcount, uint32_t, (CS_MAX_SPLITTERS + 1) * CS_BCOUNT_STRIDE);
    // Private select state, histogram and candidate / sort regions for the second and third select of a step,
    // which run beside the first one.  Full size up to CS_CONCURRENT_MAX_BLOCKS entries; beyond that only the
    // single-launch cluster select (at most CS_SELECT_CLUSTER_MAX_BLOCKS entries) runs selects side by side.
    const size_t Nc = N <= CS_CONCURRENT_MAX_BLOCKS ? N : CS_SELECT_CLUSTER_MAX_BLOCKS;
    for (int j = 0; j < 2; ++j) {
        cs_workspace *const all = ws;
        cs_workspace *const mine = (all && ws_job) ? &ws_job[j] : nullptr;
        if (mine) *mine = *all;
        ws = mine;                             // TAKE fills `mine`, or only advances the offset
        TAKE(sel, cs_sel_state, 1);
        TAKE(hist, uint32_t, CS_HIST_BINS);
        TAKE(cand_km, unsigned long long, Nc);
        TAKE(cand_id, uint32_t, Nc);
        TAKE(cand_bkt, uint32_t, Nc);
        TAKE(cand_slot, uint32_t, Nc);
        TAKE(sort_km, unsigned long long, Nc);
        TAKE(sort_id, uint32_t, Nc);
        TAKE(spl_km, unsigned long long, CS_MAX_SPLITTERS + 1);
        TAKE(spl_id, uint32_t, CS_MAX_SPLITTERS + 1);
        TAKE(bcount, uint32_t, (CS_MAX_SPLITTERS + 1) * CS_BCOUNT_STRIDE);
            ws = all;
    }
#undef TAKE
    return off;
}

// cs_step(): a prefetch candidate whose host slot receives an offloaded block in the same step must not be
// read while it is being overwritten; its entry in the prefetch list becomes CS_ID_NONE (the mover skips it).
// One thread per candidate; the offload destinations pass through shared memory in chunks.
#define STEP_FILTER_THREADS 256
__global__ void __launch_bounds__(STEP_FILTER_THREADS)
cs_step_filter_kernel(uint32_t *__restrict__ prefetch_ids, const uint32_t *__restrict__ n_prefetch, uint32_t k_prefetch,
                      const uint32_t *__restrict__ host_victims, const uint32_t *__restrict__ n_gpu_victims,
                      uint32_t k_victims)
{
    __shared__ uint32_t s_dst[STEP_FILTER_THREADS];
    const uint32_t n_pf = min(k_prefetch, *n_prefetch), n_off = min(k_victims, *n_gpu_victims);
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t mine = i < n_pf ? prefetch_ids[i] : CS_ID_NONE;
    bool hit = false;
    for (uint32_t base = 0; base < n_off; base += STEP_FILTER_THREADS) {
        __syncthreads();
        s_dst[threadIdx.x] = base + threadIdx.x < n_off ? host_victims[base + threadIdx.x] : CS_ID_NONE;
        __syncthreads();
        if (mine != CS_ID_NONE) {
            const uint32_t lim = min((uint32_t)STEP_FILTER_THREADS, n_off - base);
            for (uint32_t q = 0; q < lim; ++q) hit |= s_dst[q] == mine;
        }
    }
    if (hit) prefetch_ids[i] = CS_ID_NONE;
}

// Memory the SMs cannot address (pageable host memory that was never registered) would fault the GPU, so pool
// bases and index arrays are looked up before every launch (a host-side query of about a microsecond): device memory,
// pinned / registered host memory and managed memory pass.
bool cs_device_can_address(const void *ptr)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, ptr) != cudaSuccess) { (void)cudaGetLastError(); return false; }
    return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeHost || at.type == cudaMemoryTypeManaged;
}

// cs_get_status(): read and clear in one atomic step, so that a bit another stream sets in between is kept.
__global__ void cs_status_swap_kernel(cs_scalars *sc)
{
    sc->status_read = atomicExch(&sc->status, 0u);
}

extern "C" {

int cs_version(void) { return 201; }

const char *cs_strerror(int code)
{
    switch (code) {
    case CS_OK: return "ok";
    case CS_EINVAL: return "invalid argument";
    case CS_ECAPACITY: return "size beyond the capacity the workspace was created for";
    case CS_ENOTIMPL: return "not implemented";
    case CS_ECUDA: return "CUDA runtime error";
    case CS_EDEVICE_STATUS: return "device status word set (bad ids skipped)";
    case CS_ENOMEM: return "out of host memory";
    default: return "unknown error";
    }
}

int cs_workspace_bytes(const cs_params *p, size_t *dev_bytes)
{
    int rc = cs_validate_params(p);
    if (rc != CS_OK) return rc;
    if (!dev_bytes) return CS_EINVAL;
    uint32_t gl, as;
    cs_recency_table_shape(p, &gl, &as);
    *dev_bytes = cs_layout_workspace(p, gl, nullptr, nullptr, nullptr);
    return CS_OK;
}

int cs_create(const cs_params *p, void *dev_workspace, size_t bytes, cs_stream_t init_stream, cs_ctx **out)
{
    int rc = cs_validate_params(p);
    if (rc != CS_OK) return rc;
    if (!out || !dev_workspace || (((uintptr_t)dev_workspace) & 255u)) return CS_EINVAL;
    uint32_t gl, as;
    cs_recency_table_shape(p, &gl, &as);
    size_t need = cs_layout_workspace(p, gl, nullptr, nullptr, nullptr);
    if (bytes < need) return CS_ECAPACITY;
    cs_ctx *ctx = new (std::nothrow) cs_ctx;
    if (!ctx) return CS_ENOMEM;
    memset(ctx, 0, sizeof(*ctx));
    ctx->p = *p;
    ctx->gtab_len = gl;
    ctx->age_sat = as;
    ctx->W = (p->n_agents + 31) / 32;
    ctx->ws_bytes = cs_layout_workspace(p, gl, dev_workspace, &ctx->ws, ctx->ws_job);
    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e != cudaSuccess) { delete ctx; return CS_ECUDA; }
    ctx->host_link_ctas = 0;
    ctx->d2d_ctas = 0;
    // fork / join events of cs_step() and the two extra streams (with their events) on which the second and third
    // select of a step run: host objects, created here so that the calls themselves create nothing
    e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_sel_fork, cudaEventDisableTiming);
    for (int j = 0; j < 2 && e == cudaSuccess; ++j) {
        e = cudaStreamCreateWithFlags(&ctx->sel_stream[j], cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_sel_join[j], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) { cs_destroy(ctx); return CS_ECUDA; }
    ctx->concurrent_selects = p->max_blocks <= CS_CONCURRENT_MAX_BLOCKS ? 1 : 0;
    // everything that must start at zero (tickets, counters, histograms of all three select states)
    e = cudaMemsetAsync(dev_workspace, 0, ctx->ws_bytes, (cudaStream_t)init_stream);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; cs_destroy(ctx); return CS_ECUDA; }
    rc = cs_launch_init(ctx, (cudaStream_t)init_stream);
    if (rc != CS_OK) { cs_destroy(ctx); return rc; }
    *out = ctx;
    return CS_OK;
}

int cs_destroy(cs_ctx *ctx)
{
    if (!ctx) return CS_EINVAL;
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->ev_sel_fork) cudaEventDestroy(ctx->ev_sel_fork);
    for (int j = 0; j < 2; ++j) {
        if (ctx->ev_sel_join[j]) cudaEventDestroy(ctx->ev_sel_join[j]);
        if (ctx->sel_stream[j]) cudaStreamDestroy(ctx->sel_stream[j]);
    }
    cs_release_staging(ctx);
    delete ctx;
    return CS_OK;
}

int cs_observe_invocations(cs_ctx *ctx, const uint32_t *chain, const uint16_t *agent, const uint8_t *evflags,
                           uint32_t n_events, cs_stream_t stream)
{
    CS_RANGE("cs_observe_invocations");
    if (!ctx) return CS_EINVAL;
    if (n_events && (!chain || !agent)) return CS_EINVAL;
    if ((((uintptr_t)chain) & 3u) || (((uintptr_t)agent) & 1u)) return CS_EINVAL;   // scalar loads: natural alignment
    return cs_launch_observe(ctx, chain, agent, evflags, n_events, (cudaStream_t)stream);
}

static int check_index(const cs_ctx *ctx, const cs_block_index *idx)
{
    if (!idx) return CS_EINVAL;
    if (idx->n_blocks > ctx->p.max_blocks) return CS_ECAPACITY;
    if (idx->n_blocks == 0) return CS_OK;
    if (!idx->agent || !idx->depth || !idx->ref_count || !idx->flags || !idx->last_access) return CS_EINVAL;
    if (!aligned16(idx->agent) || !aligned16(idx->depth) || !aligned16(idx->ref_count) ||
        !aligned16(idx->flags) || !aligned16(idx->last_access) || !aligned16(idx->n_tokens) ||
        !aligned16(idx->anchor_blocks))
        return CS_EINVAL;
    const void *arrays[7] = {idx->agent, idx->depth, idx->ref_count, idx->flags, idx->last_access, idx->n_tokens,
                             idx->anchor_blocks};
    for (int i = 0; i < 7; ++i)
        if (arrays[i] && !cs_device_can_address(arrays[i])) return CS_EINVAL;     // a host array would fault the kernels
    return CS_OK;
}

int cs_score_blocks(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, const uint16_t *sources,
                    uint32_t n_sources, float *scores_out, cs_stream_t stream)
{
    CS_RANGE("cs_score_blocks");
    if (!ctx) return CS_EINVAL;
    int rc = check_index(ctx, idx);
    if (rc != CS_OK) return rc;
    if (idx->n_blocks && (!scores_out || !aligned16(scores_out))) return CS_EINVAL;
    if (sources && !aligned16(sources)) return CS_EINVAL;
    const float *fsurv = ctx->fsurv_override ? ctx->fsurv_override : ctx->ws.fsurv;
    if (sources) {
        rc = cs_launch_survival(ctx, sources, n_sources, (cudaStream_t)stream);
        if (rc != CS_OK) return rc;
        fsurv = ctx->ws.fsurv_tmp;
    }
    if (idx->n_blocks == 0) return CS_OK;
    return cs_launch_score(ctx, idx, now, fsurv, scores_out, (cudaStream_t)stream);
}

static int select_common(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, int prefetch, uint32_t tier,
                         uint32_t k, uint32_t *ids_out, uint32_t *n_out, cs_stream_t stream)
{
    if (!ctx) return CS_EINVAL;
    int rc = check_index(ctx, idx);
    if (rc != CS_OK) return rc;
    if (k > ctx->p.max_blocks) return CS_ECAPACITY;
    if (!n_out || (((uintptr_t)n_out) & 3u)) return CS_EINVAL;
    if (k && (!ids_out || !aligned16(ids_out))) return CS_EINVAL;
    if (tier > 1) return CS_EINVAL;
    return cs_launch_select(ctx, idx, now, prefetch, tier, k, ids_out, n_out, (cudaStream_t)stream);
}

int cs_select_victims(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t tier, uint32_t k,
                      uint32_t *ids_out, uint32_t *n_out, cs_stream_t stream)
{
    CS_RANGE("cs_select_victims");
    return select_common(ctx, idx, now, 0, tier, k, ids_out, n_out, stream);
}

int cs_select_prefetch(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t k, uint32_t *ids_out,
                       uint32_t *n_out, cs_stream_t stream)
{
    CS_RANGE("cs_select_prefetch");
    return select_common(ctx, idx, now, 1, 1, k, ids_out, n_out, stream);
}

int cs_select_step(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t k_victims, uint32_t k_prefetch,
                   uint32_t *gpu_victims, uint32_t *n_gpu_victims, uint32_t *host_victims, uint32_t *n_host_victims,
                   uint32_t *prefetch_ids, uint32_t *n_prefetch, cs_stream_t stream)
{
    CS_RANGE("cs_select_step");
    if (!ctx) return CS_EINVAL;
    int rc = check_index(ctx, idx);
    if (rc != CS_OK) return rc;
    if (k_victims > ctx->p.max_blocks || k_prefetch > ctx->p.max_blocks) return CS_ECAPACITY;
    uint32_t *const cnt[3] = {n_gpu_victims, n_host_victims, n_prefetch};
    uint32_t *const ids[3] = {gpu_victims, host_victims, prefetch_ids};
    for (int q = 0; q < 3; ++q) {
        if (!cnt[q]) continue;                                   // this select is not wanted
        if (((uintptr_t)cnt[q]) & 3u) return CS_EINVAL;
        if ((q == 2 ? k_prefetch : k_victims) && (!ids[q] || !aligned16(ids[q]))) return CS_EINVAL;
    }
    return cs_launch_select_step(ctx, idx, now, k_victims, k_prefetch, gpu_victims, n_gpu_victims, host_victims,
                                 n_host_victims, prefetch_ids, n_prefetch, (cudaStream_t)stream);
}

static int check_pools(const cs_kv_pool *a, const cs_kv_pool *b)
{
    if (!a || !b || !a->base || !b->base) return CS_EINVAL;
    if (!aligned16(a->base) || !aligned16(b->base)) return CS_EINVAL;
    if (a->layout > 1 || b->layout > 1) return CS_EINVAL;
    if (a->n_layers != b->n_layers || a->n_kv_heads != b->n_kv_heads || a->head_dim != b->head_dim ||
        a->block_tokens != b->block_tokens || a->elem_bytes != b->elem_bytes)
        return CS_EINVAL;
    if (a->n_layers == 0 || a->n_slots == 0 || b->n_slots == 0) return CS_EINVAL;
    unsigned long long chunk = (unsigned long long)a->block_tokens * a->n_kv_heads * a->head_dim * a->elem_bytes;
    if (chunk == 0 || (chunk & 15u) || chunk > (1ull << 30)) return CS_EINVAL;
    return CS_OK;
}

static int mover_common(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                        const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, int host_link,
                        cs_stream_t s)
{
    if (!ctx) return CS_EINVAL;
    int rc = check_pools(src, dst);
    if (rc != CS_OK) return rc;
    if (!cs_device_can_address(src->base) || !cs_device_can_address(dst->base)) return CS_EINVAL;
    if (n_max == 0) return CS_OK;
    if (!src_slots || !dst_slots || (((uintptr_t)src_slots) & 3u) || (((uintptr_t)dst_slots) & 3u)) return CS_EINVAL;
    if (n_dev && (((uintptr_t)n_dev) & 3u)) return CS_EINVAL;
    return cs_launch_mover(ctx, src, dst, src_slots, dst_slots, n_max, n_dev, host_link, (cudaStream_t)s);
}

int cs_offload_blocks(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *src_slots,
                      const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t side)
{
    CS_RANGE("cs_offload_blocks");
    return mover_common(ctx, gpu, host, src_slots, dst_slots, n_max, n_dev, CS_MOVE_OFFLOAD, side);
}

int cs_prefetch_blocks(cs_ctx *ctx, const cs_kv_pool *host, const cs_kv_pool *gpu, const uint32_t *src_slots,
                       const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t side)
{
    CS_RANGE("cs_prefetch_blocks");
    return mover_common(ctx, host, gpu, src_slots, dst_slots, n_max, n_dev, CS_MOVE_PREFETCH, side);
}

int cs_compact_blocks(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                      const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t stream)
{
    CS_RANGE("cs_compact_blocks");
    return mover_common(ctx, src, dst, src_slots, dst_slots, n_max, n_dev, CS_MOVE_D2D, stream);
}

int cs_exchange_blocks(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *off_gpu_slots,
                       const uint32_t *off_host_slots, uint32_t n_off_max, const uint32_t *n_off_dev,
                       const uint32_t *pre_host_slots, const uint32_t *pre_gpu_slots, uint32_t n_pre_max,
                       const uint32_t *n_pre_dev, cs_stream_t side)
{
    CS_RANGE("cs_exchange_blocks");
    if (!ctx) return CS_EINVAL;
    int rc = check_pools(gpu, host);
    if (rc != CS_OK) return rc;
    if (!cs_device_can_address(gpu->base) || !cs_device_can_address(host->base)) return CS_EINVAL;
    if (n_off_max == 0 && n_pre_max == 0) return CS_OK;
    const uint32_t *lists[4] = {off_gpu_slots, off_host_slots, pre_host_slots, pre_gpu_slots};
    for (int i = 0; i < 4; ++i) {
        const uint32_t n = i < 2 ? n_off_max : n_pre_max;
        if (n && (!lists[i] || (((uintptr_t)lists[i]) & 3u))) return CS_EINVAL;
    }
    if ((n_off_dev && (((uintptr_t)n_off_dev) & 3u)) || (n_pre_dev && (((uintptr_t)n_pre_dev) & 3u))) return CS_EINVAL;
    return cs_launch_exchange(ctx, gpu, host, off_gpu_slots, off_host_slots, n_off_max, n_off_dev, pre_host_slots,
                              pre_gpu_slots, n_pre_max, n_pre_dev, (cudaStream_t)side);
}

int cs_step(cs_ctx *ctx, const cs_step_io *io, cs_stream_t main_, cs_stream_t side_)
{
    CS_RANGE("cs_step");
    if (!ctx || !io || !io->idx || !io->gpu || !io->host) return CS_EINVAL;
    if (!io->n_gpu_victims || !io->n_host_victims || !io->n_prefetch) return CS_EINVAL;
    if ((io->now_dev && (((uintptr_t)io->now_dev) & 3u)) || (io->n_events_dev && (((uintptr_t)io->n_events_dev) & 3u)))
        return CS_EINVAL;
    if (io->stage && !io->stage_slots) return CS_EINVAL;
    cudaStream_t main = (cudaStream_t)main_, side = (cudaStream_t)side_;
    const bool forked = side != main;
    ctx->step_now_dev = io->now_dev;
    ctx->step_n_events_dev = io->n_events_dev;
    int rc = cs_observe_invocations(ctx, io->chain, io->agent, io->evflags, io->n_events, main_);
    if (rc == CS_OK)
        rc = cs_select_step(ctx, io->idx, io->now, io->k_victims, io->k_prefetch, io->gpu_victims, io->n_gpu_victims,
                            io->host_victims, io->n_host_victims, io->prefetch_ids, io->n_prefetch, main_);
    ctx->step_now_dev = nullptr;
    ctx->step_n_events_dev = nullptr;
    if (rc != CS_OK) return rc;
    if (io->k_prefetch && io->k_victims) {
        const uint32_t grid = (io->k_prefetch + STEP_FILTER_THREADS - 1) / STEP_FILTER_THREADS;
        cs_step_filter_kernel<<<grid, STEP_FILTER_THREADS, 0, main>>>(io->prefetch_ids, io->n_prefetch, io->k_prefetch,
                                                                      io->host_victims, io->n_gpu_victims, io->k_victims);
        if ((rc = cs_check_launch(ctx)) != CS_OK) return rc;
    }
    if (io->stage) {
        rc = cs_compact_blocks(ctx, io->gpu, io->stage, io->gpu_victims, io->stage_slots, io->k_victims, io->n_gpu_victims, main_);
        if (rc != CS_OK) return rc;
    }
    cudaError_t e = cudaSuccess;
    if (forked) {
        e = cudaEventRecord(ctx->ev_fork, main);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(side, ctx->ev_fork, 0);
        if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    }
    rc = cs_exchange_blocks(ctx, io->gpu, io->host, io->gpu_victims, io->host_victims, io->k_victims, io->n_gpu_victims,
                            io->prefetch_ids, io->free_gpu_slots, io->k_prefetch, io->n_prefetch, side_);
    if (rc != CS_OK) return rc;
    if (forked && io->join_main) {
        e = cudaEventRecord(ctx->ev_join, side);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(main, ctx->ev_join, 0);
        if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    }
    return CS_OK;
}

int cs_get_model(cs_ctx *ctx, uint32_t *C_out, float *P_out, uint16_t *amax_out, uint16_t *hops_out,
                 float *fsurv_out, float *R_out, uint16_t *cur_out, uint16_t *last_agent_out, cs_stream_t stream)
{
    if (!ctx) return CS_EINVAL;
    const size_t A = ctx->p.n_agents;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaSuccess;
#define COPY(dst, src, bytes) \
    if (e == cudaSuccess && (dst)) e = cudaMemcpyAsync((dst), (src), (bytes), cudaMemcpyDeviceToDevice, s)
    COPY(C_out, ctx->ws.C, A * A * sizeof(uint32_t));
    COPY(P_out, ctx->ws.P, A * A * sizeof(float));
    COPY(amax_out, ctx->ws.amax, A * sizeof(uint16_t));
    COPY(hops_out, ctx->ws.hops, A * sizeof(uint16_t));
    COPY(fsurv_out, ctx->ws.fsurv, A * sizeof(float));
    COPY(R_out, &ctx->ws.sc->R, sizeof(float));
    COPY(cur_out, ctx->ws.cur, ctx->p.n_chains * sizeof(uint16_t));
    COPY(last_agent_out, &ctx->ws.sc->last_agent, sizeof(uint16_t));   // little endian: low half of the u32
#undef COPY
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return CS_OK;
}

int cs_import_state(cs_ctx *ctx, const uint32_t *C_in, const uint16_t *cur_in, uint32_t last_agent, cs_stream_t stream)
{
    CS_RANGE("cs_import_state");
    if (!ctx || !C_in || (((uintptr_t)C_in) & 3u) || (((uintptr_t)cur_in) & 1u)) return CS_EINVAL;
    return cs_launch_import(ctx, C_in, cur_in, last_agent, (cudaStream_t)stream);
}

int cs_get_status(cs_ctx *ctx, uint32_t *device_status, cs_stream_t stream)
{
    if (!ctx || !device_status) return CS_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    uint32_t st = 0;
    cs_status_swap_kernel<<<1, 1, 0, s>>>(ctx->ws.sc);
    int rc = cs_check_launch(ctx);
    if (rc != CS_OK) return rc;
    cudaError_t e = cudaMemcpyAsync(&st, &ctx->ws.sc->status_read, sizeof(st), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    *device_status = st;
    return st ? CS_EDEVICE_STATUS : CS_OK;
}

int cs_get_counters(cs_ctx *ctx, cs_counters *out, uint32_t reset, cs_stream_t stream)
{
    if (!ctx || !out) return CS_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaMemcpyAsync(out, ctx->ws.cnt, sizeof(*out), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && reset) e = cudaMemsetAsync(ctx->ws.cnt, 0, sizeof(*out), s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return CS_OK;
}

int cs_validate_selection(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, uint32_t prefetch, uint32_t tier,
                          uint32_t k, const uint32_t *ids_out, const uint32_t *n_out, cs_stream_t stream)
{
    CS_RANGE("cs_validate_selection");
    if (!ctx) return CS_EINVAL;
    int rc = check_index(ctx, idx);
    if (rc != CS_OK) return rc;
    if (!n_out || (((uintptr_t)n_out) & 3u) || (k && !ids_out) || (((uintptr_t)ids_out) & 3u) || tier > 1) return CS_EINVAL;
    return cs_launch_validate_selection(ctx, idx, now, prefetch ? 1 : 0, prefetch ? 1u : tier, k, ids_out, n_out,
                                        (cudaStream_t)stream);
}

static bool list_ok(const uint32_t *p, uint32_t n) { return n == 0 || (p && !(((uintptr_t)p) & 3u)); }

int cs_validate_move_lists(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                           const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, cs_stream_t stream)
{
    CS_RANGE("cs_validate_move_lists");
    if (!ctx) return CS_EINVAL;
    int rc = check_pools(src, dst);
    if (rc != CS_OK) return rc;
    if (!list_ok(src_slots, n_max) || !list_ok(dst_slots, n_max) || (((uintptr_t)n_dev) & 3u)) return CS_EINVAL;
    if (n_max == 0) return CS_OK;
    cudaStream_t s = (cudaStream_t)stream;
    // two entries with one destination
    rc = cs_launch_validate_lists(ctx, dst_slots, src_slots, n_max, n_dev, dst_slots, src_slots, n_max, n_dev, 1, s);
    // one pool: a slot that is read by one entry and written by another
    if (rc == CS_OK && src->base == dst->base)
        rc = cs_launch_validate_lists(ctx, dst_slots, src_slots, n_max, n_dev, src_slots, dst_slots, n_max, n_dev, 0, s);
    return rc;
}

int cs_validate_exchange_lists(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host,
                               const uint32_t *off_gpu_slots, const uint32_t *off_host_slots, uint32_t n_off_max,
                               const uint32_t *n_off_dev, const uint32_t *pre_host_slots, const uint32_t *pre_gpu_slots,
                               uint32_t n_pre_max, const uint32_t *n_pre_dev, cs_stream_t stream)
{
    CS_RANGE("cs_validate_exchange_lists");
    if (!ctx) return CS_EINVAL;
    int rc = check_pools(gpu, host);
    if (rc != CS_OK) return rc;
    if (!list_ok(off_gpu_slots, n_off_max) || !list_ok(off_host_slots, n_off_max) || !list_ok(pre_host_slots, n_pre_max) ||
        !list_ok(pre_gpu_slots, n_pre_max) || (((uintptr_t)n_off_dev) & 3u) || (((uintptr_t)n_pre_dev) & 3u))
        return CS_EINVAL;
    cudaStream_t s = (cudaStream_t)stream;
    if (n_off_max)        // two offloaded blocks into one host slot
        rc = cs_launch_validate_lists(ctx, off_host_slots, off_gpu_slots, n_off_max, n_off_dev, off_host_slots, off_gpu_slots,
                                      n_off_max, n_off_dev, 1, s);
    if (rc == CS_OK && n_pre_max)     // two prefetched blocks into one GPU slot
        rc = cs_launch_validate_lists(ctx, pre_gpu_slots, pre_host_slots, n_pre_max, n_pre_dev, pre_gpu_slots, pre_host_slots,
                                      n_pre_max, n_pre_dev, 1, s);
    if (rc == CS_OK && n_off_max && n_pre_max) {
        // a host slot the offload writes while the prefetch reads it; a GPU slot the prefetch writes while the offload reads it
        rc = cs_launch_validate_lists(ctx, off_host_slots, off_gpu_slots, n_off_max, n_off_dev, pre_host_slots, pre_gpu_slots,
                                      n_pre_max, n_pre_dev, 0, s);
        if (rc == CS_OK)
            rc = cs_launch_validate_lists(ctx, pre_gpu_slots, pre_host_slots, n_pre_max, n_pre_dev, off_gpu_slots,
                                          off_host_slots, n_off_max, n_off_dev, 0, s);
    }
    return rc;
}

int cs_selftest_bounded_wait(cs_ctx *ctx, uint32_t max_polls, cs_stream_t stream)
{
    if (!ctx || max_polls < 1 || max_polls > 1000000u) return CS_EINVAL;
    return cs_launch_bounded_wait_selftest(ctx, max_polls, (cudaStream_t)stream);
}

int cs_launch_count(cs_ctx *ctx, uint64_t *n)
{
    if (!ctx || !n) return CS_EINVAL;
    *n = ctx->n_launches;
    return CS_OK;
}

int cs_set_mover_ctas(cs_ctx *ctx, uint32_t host_link_ctas, uint32_t d2d_ctas)
{
    if (!ctx) return CS_EINVAL;
    ctx->host_link_ctas = host_link_ctas;
    ctx->d2d_ctas = d2d_ctas;
    return CS_OK;
}

int cs_set_survival_sources(cs_ctx *ctx, uint32_t mode, cs_stream_t stream)
{
    if (!ctx || mode > CS_SOURCES_ALL_CHAINS) return CS_EINVAL;
    ctx->source_mode = mode;
    return cs_launch_observe(ctx, nullptr, nullptr, nullptr, 0, (cudaStream_t)stream);   // refresh the cached tables
}

int cs_set_mover_path(cs_ctx *ctx, uint32_t path)
{
    if (!ctx || path > CS_MOVER_BULK) return CS_EINVAL;
    ctx->mover_path = path;
    return CS_OK;
}

int cs_exact_survival(cs_ctx *ctx, uint32_t a0, uint32_t n_steps, float *psurv_out, float *fsurv_out, cs_stream_t stream)
{
    CS_RANGE("cs_exact_survival");
    if (!ctx) return CS_EINVAL;
    if (a0 != CS_AGENT_NONE && a0 >= ctx->p.n_agents) return CS_EINVAL;
    if (n_steps > 4096) return CS_EINVAL;
    if ((((uintptr_t)psurv_out) & 3u) || (((uintptr_t)fsurv_out) & 3u)) return CS_EINVAL;
    if (!psurv_out && !fsurv_out) return CS_OK;
    return cs_launch_exact_survival(ctx, a0, n_steps, psurv_out, fsurv_out, (cudaStream_t)stream);
}

int cs_use_survival_table(cs_ctx *ctx, const float *fsurv)
{
    if (!ctx || (((uintptr_t)fsurv) & 3u)) return CS_EINVAL;
    ctx->fsurv_override = fsurv;
    return CS_OK;
}

int cs_set_device_clock(cs_ctx *ctx, const uint32_t *now_dev)
{
    if (!ctx || (((uintptr_t)now_dev) & 3u)) return CS_EINVAL;
    if (now_dev && !cs_device_can_address(now_dev)) return CS_EINVAL;
    ctx->clock_dev = now_dev;
    return CS_OK;
}

int cs_set_select_path(cs_ctx *ctx, uint32_t path)
{
    if (!ctx || path > CS_SELECT_MULTI) return CS_EINVAL;
    ctx->select_path = path;
    return CS_OK;
}

int cs_set_select_speculation(cs_ctx *ctx, uint32_t enabled)
{
    if (!ctx) return CS_EINVAL;
    ctx->no_speculation = enabled ? 0u : 1u;
    return CS_OK;
}

int cs_set_select_bucket_regions(cs_ctx *ctx, uint32_t max_keys)
{
    if (!ctx) return CS_EINVAL;
    ctx->region_cap_max = max_keys;
    return CS_OK;
}

int cs_debug_phase_stamps(cs_ctx *ctx, uint64_t *out)
{
    if (!ctx || !out) return CS_EINVAL;
#ifdef CS_PHASE_STAMPS
    static_assert(CS_PHASE_STAMP_SLOTS == CS_N_PHASE_STAMPS, "header and kernels disagree on the number of stamps");
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(out, ctx->ws.sc->stamps, sizeof(uint64_t) * CS_N_PHASE_STAMPS, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return CS_OK;
#else
    return CS_ENOTIMPL;
#endif
}

int cs_last_cuda_error(cs_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

} // extern "C"
