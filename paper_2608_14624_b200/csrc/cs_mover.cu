// Paged-KV block mover: gathers / scatters whole multi-layer KV blocks between two pools that
// may differ in location (HBM or pinned host memory), slot count and layout.  The paper reuses
// its serving engine's offload path unchanged (Sec. 4); this file is that path for B200.
//
// Unit of work: one "piece" of one chunk (one layer, one plane, one block).  Consecutive work
// items are consecutive pieces, so neighbouring CTAs stream neighbouring addresses.  The slot
// lists and the optional device-resident count come straight from the select kernels' output,
// so no host round trip sits between a decision and its transfer.  Pinned host memory is
// addressed directly by the SMs (unified addressing), which lets both slot lists stay scattered.
//
// Two data paths:
//  * bulk path (default): every warp of a CTA runs its own software pipeline of 1-D bulk
//    asynchronous copies (TMA): global -> shared memory ring (mbarrier completion), shared ->
//    global (bulk groups).  One lane per warp issues; the copy engines of the SM move the
//    bytes, so a handful of CTAs keep hundreds of KiB in flight without occupying the
//    load/store pipelines that co-resident kernels need.
//  * load/store path: 4 x 128-bit loads per thread in flight, streaming cache hints.  Used when
//    asked for (cs_set_mover_path) and as the comparison point in the profiles.
// No copy is multicast and no kernel waits on another CTA; every mbarrier wait is bounded.
#include <mutex>

#include "cs_common.cuh"

#define MV_THREADS 256
#define MV_UNROLL 4
#define MV_PIECE (MV_THREADS * MV_UNROLL * 16)      // bytes per work item of the load/store path

#ifndef TM_WARPS
#define TM_WARPS 4                                   // independent pipelines per CTA
#endif
#ifndef TM_STAGES
#define TM_STAGES 3                                  // ring slots per pipeline
#endif
#ifndef TM_PIECE
#define TM_PIECE 16384u                              // bytes per ring slot
#endif
#define TM_SMEM (TM_WARPS * TM_STAGES * TM_PIECE)    // 192 KiB
#define CS_EXCHANGE_PIPES 32u                         // default width of the two-way transfer, in warp pipelines
#define TM_SPIN_LIMIT (1u << 20)                     // bounded mbarrier wait (polls with back-off: >= 0.1 s)

struct MoverArgs {
    const char *src;
    char *dst;
    uint32_t src_total, dst_total, src_layout, dst_layout, L, pieces, src_first, dst_first, piece_bytes, n_pipes;
    unsigned long long chunk;
    const uint32_t *src_slots, *dst_slots, *n_dev;
    uint32_t n_max;
    uint32_t *status;
    cs_counters *cnt;                 // work counters: blocks and bytes per direction, skipped entries
    uint32_t kind;                    // CS_MOVE_*
    unsigned long long block_bytes;
};

__device__ __forceinline__ unsigned long long chunk_offset(uint32_t layout, uint32_t L, uint32_t n_slots, uint32_t l,
                                                           uint32_t p, uint32_t s, unsigned long long chunk)
{
    if (layout == CS_LAYER_MAJOR) return (((unsigned long long)l * 2 + p) * n_slots + s) * chunk;
    return (((unsigned long long)s * L + l) * 2 + p) * chunk;
}

// Resolves work item w to a source / destination address and a byte count; false = skip.
__device__ __forceinline__ bool resolve_piece(const MoverArgs &a, unsigned long long w, uint32_t per_block,
                                              const char *&sp, char *&dp, uint32_t &bytes, bool report)
{
    const uint32_t i = (uint32_t)(w / per_block);
    const uint32_t r = (uint32_t)(w - (unsigned long long)i * per_block);
    const uint32_t lp = r / a.pieces, piece = r - lp * a.pieces;
    // a missing list means "packed": entry i is slot i (the staging ring of the copy-engine path)
    uint32_t s = a.src_slots ? __ldg(a.src_slots + i) : i, d = a.dst_slots ? __ldg(a.dst_slots + i) : i;
    const bool first = report && r == 0;                // one piece per block does the block's bookkeeping
    if (s == CS_ID_NONE || d == CS_ID_NONE) {
        if (first) atomicAdd((unsigned long long *)&a.cnt->blocks_skipped, 1ull);
        return false;
    }
    s -= a.src_first;                                   // ids below first_id wrap and fail the range check
    d -= a.dst_first;
    if (s >= a.src_total || d >= a.dst_total) {
        if (first) { atomicOr(a.status, CS_ST_BAD_SLOT); atomicAdd((unsigned long long *)&a.cnt->blocks_skipped, 1ull); }
        return false;
    }
    if (first) {
        atomicAdd((unsigned long long *)&a.cnt->blocks_moved[a.kind], 1ull);
        atomicAdd((unsigned long long *)&a.cnt->bytes_moved[a.kind], a.block_bytes);
    }
    const unsigned long long in_chunk = (unsigned long long)piece * a.piece_bytes;
    sp = a.src + chunk_offset(a.src_layout, a.L, a.src_total, lp >> 1, lp & 1, s, a.chunk) + in_chunk;
    dp = a.dst + chunk_offset(a.dst_layout, a.L, a.dst_total, lp >> 1, lp & 1, d, a.chunk) + in_chunk;
    const unsigned long long left = a.chunk - in_chunk;
    bytes = (uint32_t)(left < a.piece_bytes ? left : a.piece_bytes);
    return true;
}

__device__ __forceinline__ uint32_t mover_count(const MoverArgs &a)
{
    uint32_t n = a.n_max;
    if (a.n_dev) { const uint32_t nd = *a.n_dev; n = nd < n ? nd : n; }
    return n;
}

// ---------------------------------------------------------------------------------------------
// load/store path
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(MV_THREADS) cs_mover_kernel(MoverArgs a)
{
    const uint32_t n = mover_count(a);
    const uint32_t per_block = 2u * a.L * a.pieces;
    const unsigned long long total = (unsigned long long)n * per_block;
    for (unsigned long long w = blockIdx.x; w < total; w += gridDim.x) {
        const char *sp0;
        char *dp0;
        uint32_t bytes;
        if (!resolve_piece(a, w, per_block, sp0, dp0, bytes, threadIdx.x == 0)) continue;
        const uint4 *sp = (const uint4 *)sp0;
        uint4 *dp = (uint4 *)dp0;
        const uint32_t nvec = bytes >> 4;
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

// ---------------------------------------------------------------------------------------------
// bulk (TMA) path
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after TM_SPIN_LIMIT polls (each poll may itself block for a short,
// hardware-bounded time) and reports failure instead of spinning forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = TM_SPIN_LIMIT)
{
    for (uint32_t spin = 0; spin < limit; ++spin) {
        if (mbar_test(bar, parity)) return true;
        if (spin > 64) __nanosleep(128);
    }
    return false;
}
// KV blocks stream through once: both directions of every copy carry an evict-first L2 policy, so the
// gigabytes a step moves do not push the (L2-resident) block index and tables of the select kernels out.
#ifndef TM_EVICT_FIRST
#define TM_EVICT_FIRST 1
#endif
__device__ __forceinline__ unsigned long long l2_stream_policy()
{
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar,
                                          unsigned long long pol)
{
#if TM_EVICT_FIRST
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar), "l"(pol)
                 : "memory");
#else
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
#endif
}
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes, unsigned long long pol)
{
#if TM_EVICT_FIRST
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::"l"(dst), "r"(src_smem),
                 "r"(bytes), "l"(pol)
                 : "memory");
#else
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes)
                 : "memory");
#endif
}

// One pipeline per warp, driven by lane 0.  Iteration `it` first stores item it-(STAGES-1)
// (whose load was issued STAGES-1 iterations ago) and then issues the load of item `it` into
// the ring slot whose previous store has finished reading shared memory.  `item(it, sp, dp, bytes)`
// resolves the pipeline's it-th item; false = nothing to copy.
template <class Item>
__device__ __forceinline__ void bulk_pipeline(unsigned char *my_ring, const uint32_t (&bar)[TM_STAGES],
                                              unsigned long long n_items, uint32_t *status, Item item)
{
    constexpr int LAG = TM_STAGES - 1;
    const unsigned long long pol = l2_stream_policy();
    char *dst_of[TM_STAGES];          // destination of the item loaded into each ring slot
    uint32_t bytes_of[TM_STAGES];
    uint32_t phase_bits = 0;          // parity to wait for, one bit per ring slot
    uint32_t pending = 0;             // ring slots with a load in flight that nobody has waited for yet
    bool failed = false;
    for (unsigned long long it = 0; it < n_items + LAG && !failed; ++it) {
        if (it >= LAG) {                                      // store item j = it - LAG
            const int st = (int)((it - LAG) % TM_STAGES);
            if (pending & (1u << st)) {
                if (!mbar_wait_bounded(bar[st], (phase_bits >> st) & 1u)) {
                    failed = true;
                    atomicOr(status, CS_ST_TIMEOUT);
                    break;
                }
                pending &= ~(1u << st);
                phase_bits ^= 1u << st;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                bulk_store(dst_of[st], smem_u32(my_ring + (size_t)st * TM_PIECE), bytes_of[st], pol);
            }
            // one group per item, empty for a skipped item, so that group counts match item counts
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        if (it < n_items) {                                   // load item `it`
            const int st = (int)(it % TM_STAGES);
            const char *sp;
            char *dp;
            uint32_t bytes;
            if (item(it, sp, dp, bytes)) {
                // the slot's previous store (item it-STAGES) was committed one iteration ago, so at
                // most the newest group may still be reading shared memory
                asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                dst_of[st] = dp;
                bytes_of[st] = bytes;
                pending |= 1u << st;
                mbar_expect_tx(bar[st], bytes);
                bulk_load(smem_u32(my_ring + (size_t)st * TM_PIECE), sp, bytes, bar[st], pol);
            }
        }
    }
    if (failed) {
        // give the loads still in flight a bounded chance to land before shared memory is released
        for (int st = 0; st < TM_STAGES; ++st)
            if (pending & (1u << st)) mbar_wait_bounded(bar[st], (phase_bits >> st) & 1u);
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores written
}

// Per-warp set-up shared by the bulk kernels: ring slice and barriers.  Returns false for the
// lanes and warps that have nothing to do.
__device__ __forceinline__ bool bulk_setup(unsigned char *ring, unsigned long long *bars, uint32_t n_pipes,
                                           unsigned char *&my_ring, uint32_t (&bar)[TM_STAGES],
                                           unsigned long long &first)
{
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane != 0) return false;                             // the other lanes have nothing to do
    my_ring = ring + (size_t)warp * TM_STAGES * TM_PIECE;
#pragma unroll
    for (int st = 0; st < TM_STAGES; ++st) {
        bar[st] = smem_u32(&bars[warp * TM_STAGES + st]);
        mbar_init(bar[st], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    first = (unsigned long long)blockIdx.x * (blockDim.x >> 5) + warp;
    return first < n_pipes;
}

__device__ __forceinline__ unsigned long long items_of_pipe(unsigned long long total, unsigned long long first,
                                                            unsigned long long n_pipes)
{
    return first < total ? (total - first + n_pipes - 1) / n_pipes : 0;
}

// One transfer: pipeline `first` of n_pipes takes the pieces first, first + n_pipes, ...
__global__ void __launch_bounds__(TM_WARPS * 32, 1) cs_mover_bulk_kernel(MoverArgs a)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[TM_WARPS * TM_STAGES];
    unsigned char *my_ring;
    uint32_t bar[TM_STAGES];
    unsigned long long first;
    if (!bulk_setup(ring, bars, a.n_pipes, my_ring, bar, first)) return;
    const uint32_t per_block = 2u * a.L * a.pieces;
    const unsigned long long total = (unsigned long long)mover_count(a) * per_block;
    const unsigned long long n_pipes = a.n_pipes;
    bulk_pipeline(my_ring, bar, items_of_pipe(total, first, n_pipes), a.status,
                  [&](unsigned long long it, const char *&sp, char *&dp, uint32_t &bytes) {
                      return resolve_piece(a, first + it * n_pipes, per_block, sp, dp, bytes, true);
                  });
}

// Two transfers in opposite directions over the host link in one launch.  Every pipeline takes its
// share of both piece lists and walks them interleaved in proportion to their lengths, so the two
// directions advance in lock step and finish together whatever the link's arbitration between reads
// and writes would otherwise give each of them.
__global__ void __launch_bounds__(TM_WARPS * 32, 1) cs_exchange_bulk_kernel(MoverArgs off, MoverArgs pre)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ __align__(8) unsigned long long bars[TM_WARPS * TM_STAGES];
    unsigned char *my_ring;
    uint32_t bar[TM_STAGES];
    unsigned long long first;
    if (!bulk_setup(ring, bars, off.n_pipes, my_ring, bar, first)) return;
    const uint32_t per_block = 2u * off.L * off.pieces;
    const unsigned long long n_pipes = off.n_pipes;
    const unsigned long long n_o = items_of_pipe((unsigned long long)mover_count(off) * per_block, first, n_pipes);
    const unsigned long long n_p = items_of_pipe((unsigned long long)mover_count(pre) * per_block, first, n_pipes);
    const unsigned long long n_items = n_o + n_p;
    bulk_pipeline(my_ring, bar, n_items, off.status,
                  [&](unsigned long long it, const char *&sp, char *&dp, uint32_t &bytes) {
                      // offload pieces among the first `it` items: floor(it * n_o / n_items)
                      const unsigned long long before = it * n_o / n_items, after = (it + 1) * n_o / n_items;
                      if (after != before) return resolve_piece(off, first + before * n_pipes, per_block, sp, dp, bytes, true);
                      return resolve_piece(pre, first + (it - before) * n_pipes, per_block, sp, dp, bytes, true);
                  });
}

// ---------------------------------------------------------------------------------------------
static void fill_mover_args(cs_ctx *ctx, MoverArgs &a, const cs_kv_pool *src, const cs_kv_pool *dst,
                            const uint32_t *src_slots, const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev,
                            uint32_t piece_bytes, int kind)
{
    a.cnt = ctx->ws.cnt;
    a.kind = (uint32_t)kind;
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
    a.src_slots = src_slots;
    a.dst_slots = dst_slots;
    a.n_dev = n_dev;
    a.n_max = n_max;
    a.status = &ctx->ws.sc->status;
    a.n_pipes = 0;
    a.piece_bytes = piece_bytes;
    a.pieces = (uint32_t)((a.chunk + piece_bytes - 1) / piece_bytes);
    a.block_bytes = 2ull * a.L * a.chunk;
}

// Shape of a bulk launch.  Narrow transfers (every host-link transfer: at most a few dozen pipelines) run one
// pipeline per CTA with a 48 KiB ring, which fits the SMs' default shared-memory split; only wide device-to-device
// moves pack four pipelines (192 KiB) into a CTA.  A launch that needs the large split costs ~8 us more before
// its first copy is issued, which is most of what a one-block transfer loses against a plain memcpy.
static uint32_t bulk_warps_per_cta(uint32_t n_pipes)
{
    return n_pipes <= 64u ? 1u : TM_WARPS;
}

// Shared-memory opt-in of the bulk kernels: an attribute of the function on a device, so it is set once per
// process and device (always to the same fixed size).
static std::mutex g_bulk_mu;
static bool g_bulk_opted[64];
static int bulk_opt_in(cs_ctx *ctx)
{
    if (ctx->device < 0 || ctx->device >= 64) return CS_EINVAL;
    std::lock_guard<std::mutex> lock(g_bulk_mu);
    if (g_bulk_opted[ctx->device]) return CS_OK;
    cudaError_t e = cudaFuncSetAttribute(cs_mover_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TM_SMEM);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(cs_exchange_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TM_SMEM);
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    g_bulk_opted[ctx->device] = true;
    return CS_OK;
}

int cs_launch_mover(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                    const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, int kind, cudaStream_t s)
{
    return cs_launch_mover_as(ctx, src, dst, src_slots, dst_slots, n_max, n_dev, kind, kind, s);
}

// `kind` decides the width of the launch (which memory the bytes cross), `count_as` the direction the work
// counters book the blocks under (the pack and scatter launches of the copy-engine path move blocks inside the
// device on behalf of an offload or a prefetch).
int cs_launch_mover_as(cs_ctx *ctx, const cs_kv_pool *src, const cs_kv_pool *dst, const uint32_t *src_slots,
                       const uint32_t *dst_slots, uint32_t n_max, const uint32_t *n_dev, int kind, int count_as,
                       cudaStream_t s)
{
    const bool bulk = ctx->mover_path != CS_MOVER_LDST;
    MoverArgs a;
    fill_mover_args(ctx, a, src, dst, src_slots, dst_slots, n_max, n_dev, bulk ? TM_PIECE : MV_PIECE, count_as);
    const unsigned long long total = (unsigned long long)n_max * 2ull * a.L * a.pieces;
    unsigned long long cap;
    if (bulk) {
        // width in warp pipelines (each keeps <= 2 loads and 2 stores of 16 KiB in flight)
        // (a pack / scatter launch of the copy-engine path only has to keep ahead of the host link: 64 pipelines move
        //  about 1.5 TB/s and leave most SMs to the kernels running beside it)
        const uint32_t dflt = kind == CS_MOVE_D2D ? 2u * (uint32_t)ctx->sm_count
                            : (kind == CS_MOVE_STAGE ? 64u : (kind == CS_MOVE_OFFLOAD ? 8u : 24u));
        const uint32_t asked = kind == CS_MOVE_D2D ? ctx->d2d_ctas : (kind == CS_MOVE_STAGE ? 0u : ctx->host_link_ctas);
        cap = asked ? asked : dflt;
        a.n_pipes = (uint32_t)(total < cap ? total : cap);
        if (a.n_pipes == 0) a.n_pipes = 1;
        const uint32_t wpc = bulk_warps_per_cta(a.n_pipes);
        const uint32_t grid = (a.n_pipes + wpc - 1) / wpc;
        const int rc = bulk_opt_in(ctx);
        if (rc != CS_OK) return rc;
        cs_mover_bulk_kernel<<<grid, wpc * 32, (size_t)wpc * TM_STAGES * TM_PIECE, s>>>(a);
    } else {
        const uint32_t dflt = kind == CS_MOVE_D2D ? 8u * (uint32_t)ctx->sm_count
                            : (kind == CS_MOVE_STAGE ? 64u : (kind == CS_MOVE_OFFLOAD ? 8u : 12u));
        const uint32_t asked = kind == CS_MOVE_D2D ? ctx->d2d_ctas : (kind == CS_MOVE_STAGE ? 0u : ctx->host_link_ctas);
        cap = asked ? asked : dflt;
        const uint32_t grid = (uint32_t)(total < cap ? total : cap);
        cs_mover_kernel<<<grid ? grid : 1u, MV_THREADS, 0, s>>>(a);
    }
    return cs_check_launch(ctx);
}

// Offload and prefetch of one step as a single launch (bulk path only).
int cs_launch_exchange(cs_ctx *ctx, const cs_kv_pool *gpu, const cs_kv_pool *host, const uint32_t *off_gpu_slots,
                       const uint32_t *off_host_slots, uint32_t n_off_max, const uint32_t *n_off_dev,
                       const uint32_t *pre_host_slots, const uint32_t *pre_gpu_slots, uint32_t n_pre_max,
                       const uint32_t *n_pre_dev, cudaStream_t s)
{
    MoverArgs off, pre;
    fill_mover_args(ctx, off, gpu, host, off_gpu_slots, off_host_slots, n_off_max, n_off_dev, TM_PIECE, CS_MOVE_OFFLOAD);
    fill_mover_args(ctx, pre, host, gpu, pre_host_slots, pre_gpu_slots, n_pre_max, n_pre_dev, TM_PIECE, CS_MOVE_PREFETCH);
    const unsigned long long total = ((unsigned long long)n_off_max + n_pre_max) * 2ull * off.L * off.pieces;
    const unsigned long long cap = ctx->host_link_ctas ? ctx->host_link_ctas : CS_EXCHANGE_PIPES;
    uint32_t n_pipes = (uint32_t)(total < cap ? total : cap);
    if (n_pipes == 0) n_pipes = 1;
    off.n_pipes = pre.n_pipes = n_pipes;
    const uint32_t wpc = bulk_warps_per_cta(n_pipes);
    const uint32_t grid = (n_pipes + wpc - 1) / wpc;
    const int rc = bulk_opt_in(ctx);
    if (rc != CS_OK) return rc;
    cs_exchange_bulk_kernel<<<grid, wpc * 32, (size_t)wpc * TM_STAGES * TM_PIECE, s>>>(off, pre);
    return cs_check_launch(ctx);
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one warp, one barrier, no copy.  The wait cannot succeed, so it runs out
// after `max_polls` polls and the kernel reports exactly as a stalled transfer would.  Nothing is in flight.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(32) cs_bounded_wait_selftest_kernel(uint32_t max_polls, uint32_t *status)
{
    __shared__ __align__(8) unsigned long long bar_mem;
    if (threadIdx.x != 0) return;
    const uint32_t bar = smem_u32(&bar_mem);
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_bounded(bar, 0, max_polls)) atomicOr(status, CS_ST_TIMEOUT);
}

int cs_launch_bounded_wait_selftest(cs_ctx *ctx, uint32_t max_polls, cudaStream_t s)
{
    cs_bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(max_polls, &ctx->ws.sc->status);
    return cs_check_launch(ctx);
}
