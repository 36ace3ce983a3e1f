// Paged-KV block mover: gathers / scatters whole multi-layer KV blocks between two pools that
// may differ in location (HBM or pinned host memory), slot count and layout.  The paper reuses
// its serving engine's offload path unchanged (Sec. 4); this file is that path for B200.
//
// Unit of work: one "piece" (<= 16 KiB) of one chunk (one layer, one plane, one block).
// Consecutive work items are consecutive pieces of the same chunk, so neighbouring CTAs
// stream neighbouring addresses.  A CTA issues all loads of its piece (4 x 128-bit per thread)
// before the first store, which keeps 16 KiB per CTA in flight; the slot lists and the
// optional device-resident count come straight from the select kernels' output, so no host
// round trip sits between a decision and its transfer.  Pinned host memory is addressed
// directly by the SMs (unified addressing), which lets the destination slots stay scattered.
#include "cs_common.cuh"

#define MV_THREADS 256
#define MV_UNROLL 4
#define MV_PIECE (MV_THREADS * MV_UNROLL * 16)      // bytes per work item

struct MoverArgs {
    const char *src;
    char *dst;
    uint32_t src_total, dst_total, src_layout, dst_layout, L, pieces, src_first, dst_first;
    unsigned long long chunk;
    const uint32_t *src_slots, *dst_slots, *n_dev;
    uint32_t n_max;
    uint32_t *status;
};

__device__ __forceinline__ unsigned long long chunk_offset(uint32_t layout, uint32_t L, uint32_t n_slots, uint32_t l,
                                                           uint32_t p, uint32_t s, unsigned long long chunk)
{
    if (layout == CS_LAYER_MAJOR) return (((unsigned long long)l * 2 + p) * n_slots + s) * chunk;
    return (((unsigned long long)s * L + l) * 2 + p) * chunk;
}

__global__ void __launch_bounds__(MV_THREADS) cs_mover_kernel(MoverArgs a)
{
    uint32_t n = a.n_max;
    if (a.n_dev) { const uint32_t nd = *a.n_dev; n = nd < n ? nd : n; }
    const uint32_t per_block = 2u * a.L * a.pieces;
    const unsigned long long total = (unsigned long long)n * per_block;
    for (unsigned long long w = blockIdx.x; w < total; w += gridDim.x) {
        const uint32_t i = (uint32_t)(w / per_block);
        const uint32_t r = (uint32_t)(w - (unsigned long long)i * per_block);
        const uint32_t lp = r / a.pieces, piece = r - lp * a.pieces;
        uint32_t s = __ldg(a.src_slots + i), d = __ldg(a.dst_slots + i);
        if (s == CS_ID_NONE || d == CS_ID_NONE) continue;
        s -= a.src_first;                                   // ids below first_id wrap and fail the range check
        d -= a.dst_first;
        if (s >= a.src_total || d >= a.dst_total) {
            if (threadIdx.x == 0 && r == 0) atomicOr(a.status, CS_ST_BAD_SLOT);
            continue;
        }
        const unsigned long long in_chunk = (unsigned long long)piece * MV_PIECE;
        const uint4 *sp = (const uint4 *)(a.src + chunk_offset(a.src_layout, a.L, a.src_total, lp >> 1, lp & 1, s, a.chunk) + in_chunk);
        uint4 *dp = (uint4 *)(a.dst + chunk_offset(a.dst_layout, a.L, a.dst_total, lp >> 1, lp & 1, d, a.chunk) + in_chunk);
        const unsigned long long left = a.chunk - in_chunk;
        const uint32_t nvec = (uint32_t)((left < MV_PIECE ? left : MV_PIECE) >> 4);
        uint4 v[MV_UNROLL];
#pragma unroll
        for (int u = 0; u < MV_UNROLL; ++u) {
            const uint32_t x = threadIdx.x + u * MV_THREADS;
            if (x < nvec) v[u] = __ldcs(sp + x);
        }
#pragma unroll
        for (int u = 0; u < MV_UNROLL; ++u) {
            const uint32_t x = threadIdx.x + u * MV_THREADS;
            if (x < nvec) __stcs(dp + x, v[u]);
        }
    }
}

int cs_launch_mover(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                    const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, int crosses_host_link,
                    cudaStream_t s)
{
    MoverArgs a;
    a.src = (const char *)src->base;
    a.dst = (char *)dst->base;
    a.src_total = src->n_slots;
    a.dst_total = dst->n_slots;
    a.src_first = src->first_id;
    a.dst_first = dst->first_id;
    a.src_layout = src->layout;
    a.dst_layout = dst->layout;
    a.L = src->n_layers;
    a.chunk = (unsigned long long)src->block_tokens * src->n_kv_heads * src->head_dim * src->elem_bytes;
    a.pieces = (uint32_t)((a.chunk + MV_PIECE - 1) / MV_PIECE);
    a.src_slots = src_slots;
    a.dst_slots = dst_slots;
    a.n_dev = n_dev;
    a.n_max = n_max;
    a.status = &ctx->ws.sc->status;
    const unsigned long long total = (unsigned long long)n_max * 2ull * a.L * a.pieces;
    unsigned long long cap = crosses_host_link ? (ctx->host_link_ctas ? ctx->host_link_ctas : 64u)
                                               : (ctx->d2d_ctas ? ctx->d2d_ctas : 8u * (uint32_t)ctx->sm_count);
    const uint32_t grid = (uint32_t)(total < cap ? total : cap);
    cs_mover_kernel<<<grid ? grid : 1u, MV_THREADS, 0, s>>>(a);
    return cs_check_launch(ctx);
}
