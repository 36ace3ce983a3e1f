// Copy-engine path of the block mover.  The default path lets the SMs address pinned host memory directly,
// which keeps both slot lists device-resident but puts host-memory round trips into the SMs' memory system,
// where latency-bound kernels of the serving engine feel them.  Here the bytes cross the host link on the
// GPU's copy engines instead: an offload is PACKED by the mover kernel (HBM -> a device ring, at HBM speed) and
// carried to the host tier by plain cudaMemcpyAsync calls, one per run of consecutive host slots, while the
// next part of the list is being packed; a prefetch is the mirror image (copies into the ring, then a SCATTER
// launch).  The price: the host must know the host-tier slots, so those lists are host arrays here (an engine
// reads the few KB of a select result back, or assigns host slots itself as consecutive runs, which turns a
// whole transfer into a handful of large copies).  The GPU-side lists stay on the device.
//
// Ring: caller-owned device memory (cs_set_mover_staging), split into four sub-buffers, two per direction,
// so that packing / scattering one part overlaps the copies of the other.  All ordering is by events between
// the caller's stream (pack launches) and five streams of the context (two per DMA direction, one for the
// scatter launches); nothing synchronises with the host.
#include "cs_common.cuh"

void cs_release_staging(cs_ctx *ctx)
{
    if (ctx->scatter_stream) cudaStreamDestroy(ctx->scatter_stream);
    ctx->scatter_stream = nullptr;
    for (int j = 0; j < 4; ++j) {
        if (ctx->copy_stream[j]) cudaStreamDestroy(ctx->copy_stream[j]);
        if (ctx->ev_copied[j]) cudaEventDestroy(ctx->ev_copied[j]);
        if (ctx->ev_filled[j]) cudaEventDestroy(ctx->ev_filled[j]);
        ctx->copy_stream[j] = nullptr;
        ctx->ev_copied[j] = ctx->ev_filled[j] = nullptr;
    }
    for (int j = 0; j < 2; ++j) {
        if (ctx->ev_stage_join[j]) cudaEventDestroy(ctx->ev_stage_join[j]);
        if (ctx->ev_packed[j]) cudaEventDestroy(ctx->ev_packed[j]);
        if (ctx->ev_scattered[j]) cudaEventDestroy(ctx->ev_scattered[j]);
        ctx->ev_stage_join[j] = ctx->ev_packed[j] = ctx->ev_scattered[j] = nullptr;
    }
    if (ctx->ev_stage_fork) cudaEventDestroy(ctx->ev_stage_fork);
    ctx->ev_stage_fork = nullptr;
    ctx->stage_ring = nullptr;
    ctx->stage_bytes = 0;
}

static cudaError_t make_event(cudaEvent_t *e) { return cudaEventCreateWithFlags(e, cudaEventDisableTiming); }

extern "C" int cs_set_mover_staging(cs_ctx *ctx, void *dev_ring, size_t bytes)
{
    if (!ctx) return CS_EINVAL;
    if (!dev_ring) { cs_release_staging(ctx); return CS_OK; }
    if ((((uintptr_t)dev_ring) & 255u) || bytes < 4096) return CS_EINVAL;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, dev_ring) != cudaSuccess || at.type != cudaMemoryTypeDevice) {
        (void)cudaGetLastError();
        return CS_EINVAL;                                   // the ring must be device memory
    }
    if (!ctx->copy_stream[0]) {                             // host objects, made once
        cudaError_t e = make_event(&ctx->ev_stage_fork);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->scatter_stream, cudaStreamNonBlocking);
        for (int j = 0; j < 4 && e == cudaSuccess; ++j) {
            e = cudaStreamCreateWithFlags(&ctx->copy_stream[j], cudaStreamNonBlocking);
            if (e == cudaSuccess) e = make_event(&ctx->ev_copied[j]);
            if (e == cudaSuccess) e = make_event(&ctx->ev_filled[j]);
        }
        for (int j = 0; j < 2 && e == cudaSuccess; ++j) {
            e = make_event(&ctx->ev_stage_join[j]);
            if (e == cudaSuccess) e = make_event(&ctx->ev_packed[j]);
            if (e == cudaSuccess) e = make_event(&ctx->ev_scattered[j]);
        }
        if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; cs_release_staging(ctx); return CS_ECUDA; }
    }
    ctx->stage_ring = (unsigned char *)dev_ring;
    ctx->stage_bytes = bytes;
    return CS_OK;
}

struct StagedPlan {
    cs_kv_pool ring[2][2];          // [direction][buffer]: packed, block-major pools over the ring's sub-buffers
    uint32_t cap;                   // blocks per sub-buffer
    size_t block_bytes;
};

static int plan_staging(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, StagedPlan &P)
{
    if (!ctx->stage_ring) return CS_EINVAL;                 // cs_set_mover_staging() first
    if (host->layout != CS_BLOCK_MAJOR) return CS_EINVAL;   // a host block must be one contiguous run of bytes
    const size_t chunk = (size_t)gpu->block_tokens * gpu->n_kv_heads * gpu->head_dim * gpu->elem_bytes;
    P.block_bytes = 2 * (size_t)gpu->n_layers * chunk;
    const size_t sub = (ctx->stage_bytes / 4) & ~(size_t)255;
    if (sub / P.block_bytes < 1) return CS_ECAPACITY;
    P.cap = (uint32_t)(sub / P.block_bytes < 0xFFFFFFFFull ? sub / P.block_bytes : 0xFFFFFFFFull);
    for (int d = 0; d < 2; ++d)
        for (int b = 0; b < 2; ++b) {
            cs_kv_pool &r = P.ring[d][b];
            r = *gpu;
            r.base = ctx->stage_ring + (size_t)(2 * d + b) * sub;
            r.n_slots = P.cap;
            r.layout = CS_BLOCK_MAJOR;
            r.first_id = 0;
        }
    return CS_OK;
}

// Host-side check of a list of host-tier ids (host memory): every id in range.  CS_ID_NONE is not accepted
// here: the device-side pack / scatter launch could not know that the host skipped the entry.
static bool host_ids_ok(const cs_kv_pool *host, const uint32_t *ids, uint32_t n)
{
    for (uint32_t i = 0; i < n; ++i)
        if ((uint32_t)(ids[i] - host->first_id) >= host->n_slots) return false;
    return true;
}

// One cudaMemcpyAsync per run of consecutive host slots within ring positions [lo, hi) of a sub-buffer, the runs
// dealt alternately to two streams so that two copies of a direction are in flight (a copy of a single 2 MiB block
// carries a few microseconds of fixed cost on its engine, which a second engine hides).
static cudaError_t copy_runs(const cs_kv_pool *host, const uint32_t *ids, uint32_t lo, uint32_t hi, unsigned char *ring,
                             size_t bb, bool to_host, cudaStream_t s0, cudaStream_t s1)
{
    cudaError_t e = cudaSuccess;
    uint32_t i = lo, turn = 0;
    while (i < hi && e == cudaSuccess) {
        cudaStream_t s = (turn++ & 1u) ? s1 : s0;
        uint32_t j = i + 1;
        while (j < hi && ids[j] == ids[j - 1] + 1) ++j;
        unsigned char *h = (unsigned char *)host->base + (size_t)(ids[i] - host->first_id) * bb;
        unsigned char *r = ring + (size_t)(i - lo) * bb;
        const size_t len = (size_t)(j - i) * bb;
        e = to_host ? cudaMemcpyAsync(h, r, len, cudaMemcpyDeviceToHost, s) : cudaMemcpyAsync(r, h, len, cudaMemcpyHostToDevice, s);
        i = j;
    }
    return e;
}

#define CK(call) do { if (e == cudaSuccess) e = (call); } while (0)

extern "C" int cs_exchange_blocks_staged(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host,
                                         const uint32_t *off_gpu_slots, const uint32_t *off_host_ids, uint32_t n_off,
                                         const uint32_t *pre_host_ids, const uint32_t *pre_gpu_slots, uint32_t n_pre,
                                         cs_stream_t stream)
{
    CS_RANGE("cs_exchange_blocks_staged");
    if (!ctx || !gpu || !host || !gpu->base || !host->base) return CS_EINVAL;
    if (gpu->n_layers != host->n_layers || gpu->n_kv_heads != host->n_kv_heads || gpu->head_dim != host->head_dim ||
        gpu->block_tokens != host->block_tokens || gpu->elem_bytes != host->elem_bytes || gpu->layout > 1)
        return CS_EINVAL;
    if ((n_off && (!off_gpu_slots || !off_host_ids)) || (n_pre && (!pre_host_ids || !pre_gpu_slots))) return CS_EINVAL;
    if ((((uintptr_t)off_gpu_slots) & 3u) || (((uintptr_t)pre_gpu_slots) & 3u)) return CS_EINVAL;
    if (!cs_device_can_address(gpu->base) || !cs_device_can_address(host->base)) return CS_EINVAL;
    StagedPlan P;
    int rc = plan_staging(ctx, gpu, host, P);
    if (rc != CS_OK) return rc;
    if (!host_ids_ok(host, off_host_ids, n_off) || !host_ids_ok(host, pre_host_ids, n_pre)) return CS_EINVAL;
    if (n_off == 0 && n_pre == 0) return CS_OK;
    // The two directions are independent pipelines: pack launches on the caller's stream feed the device-to-host
    // copies, host-to-device copies feed scatter launches on a stream of the context; neither waits for the other.
    cudaStream_t S = (cudaStream_t)stream, KP = ctx->scatter_stream;
    cudaStream_t *CO = &ctx->copy_stream[0], *CP = &ctx->copy_stream[2];          // two streams per DMA direction
    const uint32_t cap = P.cap;
    const uint32_t nco = (n_off + cap - 1) / cap, ncp = (n_pre + cap - 1) / cap;
    cudaError_t e = cudaSuccess;
    // everything starts after what is already on the caller's stream (the previous user of the ring included)
    CK(cudaEventRecord(ctx->ev_stage_fork, S));
    for (int j = 0; j < 4; ++j) CK(cudaStreamWaitEvent(ctx->copy_stream[j], ctx->ev_stage_fork, 0));
    CK(cudaStreamWaitEvent(KP, ctx->ev_stage_fork, 0));
    for (uint32_t c = 0; c < (nco > ncp ? nco : ncp) && e == cudaSuccess && rc == CS_OK; ++c) {
        const int b = (int)(c & 1u);
        const uint32_t lo = c * cap;
        if (c < ncp) {                                       // prefetch part c: host -> ring on the copy engines, then scatter
            const uint32_t hi = lo + cap < n_pre ? lo + cap : n_pre;
            for (int j = 0; j < 2; ++j) {
                if (c >= 2) CK(cudaStreamWaitEvent(CP[j], ctx->ev_scattered[b], 0));      // the ring buffer is free again
            }
            CK(copy_runs(host, pre_host_ids, lo, hi, (unsigned char *)P.ring[1][b].base, P.block_bytes, false, CP[0], CP[1]));
            for (int j = 0; j < 2; ++j) {
                CK(cudaEventRecord(ctx->ev_filled[2 * b + j], CP[j]));
                CK(cudaStreamWaitEvent(KP, ctx->ev_filled[2 * b + j], 0));
            }
            if (e == cudaSuccess)
                rc = cs_launch_mover_as(ctx, &P.ring[1][b], gpu, nullptr, pre_gpu_slots + lo, hi - lo, nullptr, CS_MOVE_STAGE,
                                        CS_MOVE_PREFETCH, KP);
            CK(cudaEventRecord(ctx->ev_scattered[b], KP));
        }
        if (c < nco && rc == CS_OK) {                        // offload part c: pack on the SMs, ring -> host on the copy engines
            const uint32_t hi = lo + cap < n_off ? lo + cap : n_off;
            if (c >= 2) {
                CK(cudaStreamWaitEvent(S, ctx->ev_copied[2 * b], 0));
                CK(cudaStreamWaitEvent(S, ctx->ev_copied[2 * b + 1], 0));
            }
            if (e == cudaSuccess)
                rc = cs_launch_mover_as(ctx, gpu, &P.ring[0][b], off_gpu_slots + lo, nullptr, hi - lo, nullptr, CS_MOVE_STAGE,
                                        CS_MOVE_OFFLOAD, S);
            CK(cudaEventRecord(ctx->ev_packed[b], S));
            for (int j = 0; j < 2; ++j) CK(cudaStreamWaitEvent(CO[j], ctx->ev_packed[b], 0));
            CK(copy_runs(host, off_host_ids, lo, hi, (unsigned char *)P.ring[0][b].base, P.block_bytes, true, CO[0], CO[1]));
            for (int j = 0; j < 2; ++j) CK(cudaEventRecord(ctx->ev_copied[2 * b + j], CO[j]));
        }
    }
    // the caller's stream ends after the last copies to the host and the last scatter
    if (nco) {
        for (int j = 0; j < 4; ++j) CK(cudaStreamWaitEvent(S, ctx->ev_copied[j], 0));   // (an event never recorded counts as done)
    }
    CK(cudaEventRecord(ctx->ev_stage_join[1], KP));
    CK(cudaStreamWaitEvent(S, ctx->ev_stage_join[1], 0));
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return rc;
}

extern "C" int cs_offload_blocks_staged(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host,
                                        const uint32_t *src_slots, const uint32_t *host_ids, uint32_t n, cs_stream_t stream)
{
    return cs_exchange_blocks_staged(ctx, gpu, host, src_slots, host_ids, n, nullptr, nullptr, 0, stream);
}

extern "C" int cs_prefetch_blocks_staged(cs_ctx *ctx, const cs_kv_pool *host, const cs_kv_pool *gpu,
                                         const uint32_t *host_ids, const uint32_t *dst_slots, uint32_t n, cs_stream_t stream)
{
    return cs_exchange_blocks_staged(ctx, gpu, host, nullptr, nullptr, 0, host_ids, dst_slots, n, stream);
}
