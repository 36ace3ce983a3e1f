// Checker kernels (debugging aids, no counterpart in the paper): they look at the RESULT of a select, or at
// the slot lists of a transfer about to be issued, and report through the device status word.  They share
// the eligibility rules and the key with the select kernels (cs_select_common.cuh) and nothing of the
// selection algorithm itself: a list is accepted when it is the ordered k best, however it was produced.
#include "cs_select_common.cuh"

// Position i of the list: a valid, eligible entry and its key.
template <bool PF>
__device__ __forceinline__ bool list_key(const SelArgs &a, const Tables &T, uint32_t *status, const uint32_t *ids,
                                         uint32_t pos, unsigned long long &km, uint32_t &id)
{
    id = ids[pos];
    if (id >= a.n) return false;
    uint32_t pr, se;
    const uint32_t tok = a.ntok ? a.ntok[id] : a.block_tokens;
    if (!entry_key<PF>(a, T, status, a.agent[id], a.depth[id], a.ref[id], a.flags[id], a.la[id], tok, pr, se)) return false;
    km = ((unsigned long long)pr << 32) | se;
    return true;
}

template <bool PF>
__global__ void __launch_bounds__(SEL_THREADS)
cs_validate_selection_kernel(SelArgs a, cs_workspace ws, const uint32_t *__restrict__ ids, const uint32_t *__restrict__ n_out_dev)
{
    extern __shared__ float smem[];
    __shared__ uint32_t s_le, s_el;
    __shared__ bool s_flag;
    resolve_now(a);
    Tables T;
    load_tables(a, ws, smem, T, PF && a.anchor);
    if (threadIdx.x == 0) { s_le = 0; s_el = 0; }
    __syncthreads();
    uint32_t *status = &ws.sc->status;
    const bool enabled = !PF || prefetch_enabled(ws, a.A);
    const uint32_t gtid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
    uint32_t n = *n_out_dev;
    bool bad = false;
    if (n > a.k) { bad = true; n = a.k; }
    if (!enabled && n != 0) bad = true;
    // the list itself: eligible entries, keys strictly increasing, padded tail
    for (uint32_t i = gtid; i < a.k; i += nth) {
        if (i >= n) { bad |= ids[i] != CS_ID_NONE; continue; }
        unsigned long long k0, k1;
        uint32_t i0, i1;
        if (!list_key<PF>(a, T, status, ids, i, k0, i0)) { bad = true; continue; }
        if (i + 1 < n && list_key<PF>(a, T, status, ids, i + 1, k1, i1)) bad |= !key_less(k0, i0, k1, i1);
    }
    // completeness: exactly n eligible entries lie at or below the last key, and n = min(k, eligible)
    unsigned long long kl = 0;
    uint32_t il = 0;
    const bool have_last = n > 0 && list_key<PF>(a, T, status, ids, n - 1, kl, il);
    uint32_t le = 0, el = 0;
    if (enabled)
        for_each_eligible<PF>(a, T, status, [&](uint32_t id, uint32_t pr, uint32_t se) {
            const unsigned long long km = ((unsigned long long)pr << 32) | se;
            ++el;
            if (have_last && !key_less(kl, il, km, id)) ++le;
        });
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        le += __shfl_xor_sync(0xFFFFFFFFu, le, d);
        el += __shfl_xor_sync(0xFFFFFFFFu, el, d);
    }
    if ((threadIdx.x & 31) == 0) { atomicAdd(&s_le, le); atomicAdd(&s_el, el); }
    if (__syncthreads_or(bad)) { if (threadIdx.x == 0) atomicOr(status, CS_ST_BAD_SELECTION); }
    if (threadIdx.x == 0) { atomicAdd(&ws.sc->val_le, s_le); atomicAdd(&ws.sc->val_elig, s_el); }
    if (!last_cta_done(&ws.sc->val_ticket, &s_flag)) return;
    if (threadIdx.x == 0) {
        const uint32_t tot_le = __ldcg(&ws.sc->val_le), tot_el = __ldcg(&ws.sc->val_elig);
        const uint32_t want = enabled ? (tot_el < a.k ? tot_el : a.k) : 0u;
        if (*n_out_dev != want || (n > 0 && have_last && tot_le != n)) atomicOr(status, CS_ST_BAD_SELECTION);
        ws.sc->val_le = 0;
        ws.sc->val_elig = 0;
        ws.sc->val_ticket = 0;
    }
}

int cs_launch_validate_selection(cs_ctx *ctx, const cs_block_index *idx, uint32_t now, int prefetch, uint32_t tier,
                                 uint32_t k, const uint32_t *ids, const uint32_t *n_out, cudaStream_t s)
{
    SelArgs a;
    cs_fill_sel_args(ctx, idx, now, ctx->fsurv_override ? ctx->fsurv_override : ctx->ws.fsurv, a);
    a.tier = tier;
    a.k = k;
    const uint32_t grid = cs_scan_grid(ctx, idx->n_blocks, SEL_THREADS * GRP);
    const size_t sm = cs_table_smem(ctx);
    if (prefetch) cs_validate_selection_kernel<true><<<grid, SEL_THREADS, sm, s>>>(a, ctx->ws, ids, n_out);
    else cs_validate_selection_kernel<false><<<grid, SEL_THREADS, sm, s>>>(a, ctx->ws, ids, n_out);
    return cs_check_launch(ctx);
}

// ---------------------------------------------------------------------------------------------
// Slot-list conflicts.  Thread i owns entry i of list W and looks for the same slot in list X (entries
// before i only, when both are the same list).  An entry counts only if the mover would copy it: neither
// it nor its partner on the other side of the copy is CS_ID_NONE.  X passes through shared memory in tiles.
// ---------------------------------------------------------------------------------------------
#define VL_THREADS 256
__global__ void __launch_bounds__(VL_THREADS)
cs_validate_lists_kernel(const uint32_t *__restrict__ w, const uint32_t *__restrict__ wp, uint32_t nw_max,
                         const uint32_t *__restrict__ nw_dev, const uint32_t *__restrict__ x,
                         const uint32_t *__restrict__ xp, uint32_t nx_max, const uint32_t *__restrict__ nx_dev, int self,
                         uint32_t *status)
{
    __shared__ uint32_t s_x[VL_THREADS];
    const uint32_t nw = nw_dev ? min(nw_max, *nw_dev) : nw_max, nx = nx_dev ? min(nx_max, *nx_dev) : nx_max;
    const uint32_t i = blockIdx.x * VL_THREADS + threadIdx.x;
    uint32_t mine = CS_ID_NONE;
    if (i < nw && wp[i] != CS_ID_NONE) mine = w[i];
    bool hit = false;
    for (uint32_t base = 0; base < nx; base += VL_THREADS) {
        __syncthreads();
        const uint32_t j = base + threadIdx.x;
        s_x[threadIdx.x] = (j < nx && xp[j] != CS_ID_NONE) ? x[j] : CS_ID_NONE;
        __syncthreads();
        if (mine == CS_ID_NONE) continue;
        uint32_t lim = min((uint32_t)VL_THREADS, nx - base);
        if (self) lim = i > base ? min(lim, i - base) : 0u;           // entries before i only
        for (uint32_t q = 0; q < lim; ++q) hit |= s_x[q] == mine;
    }
    if (hit) atomicOr(status, CS_ST_LIST_CONFLICT);
}

int cs_launch_validate_lists(cs_ctx *ctx, const uint32_t *w_list, const uint32_t *w_partner, uint32_t nw_max,
                             const uint32_t *nw_dev, const uint32_t *x_list, const uint32_t *x_partner, uint32_t nx_max,
                             const uint32_t *nx_dev, int self, cudaStream_t s)
{
    const uint32_t grid = (nw_max + VL_THREADS - 1) / VL_THREADS;
    cs_validate_lists_kernel<<<grid ? grid : 1u, VL_THREADS, 0, s>>>(w_list, w_partner, nw_max, nw_dev, x_list, x_partner,
                                                                    nx_max, nx_dev, self, &ctx->ws.sc->status);
    return cs_check_launch(ctx);
}
