// Single-launch select: the whole top-k (histogram -> threshold -> collect -> order) inside ONE
// thread-block cluster, for index sizes where a handful of SMs can stream the metadata in a few
// microseconds (every configuration of this library's workloads).  Compared with the
// five-launch path (cs_select.cu) it replaces four kernel boundaries by hardware cluster
// barriers, reduces the per-CTA histograms through distributed shared memory instead of global
// atomics, loads the small tables once, and occupies at most 16 SMs, which leaves the rest of
// the GPU to the serving kernels.  Same key, same eligibility rules, same exact ordered output.
//
// Phases (cluster.sync() between them; no spin-waits of our own):
//   1 every CTA scans its slice of the index and builds a 4096-bin histogram of the top 12
//     primary-key bits in its shared memory;
//   2 CTA r sums bins [r*B/CL, (r+1)*B/CL) over all CTAs through DSMEM and writes the sums into
//     every CTA's copy of the total histogram; each CTA then finds the threshold bin b0;
//   3 every CTA re-scans its slice (L2-resident) and appends the entries with bin <= b0 to the
//     candidate buffer (c >= min(k, eligible) keys);
//   4 c <= 4096: CTA 0 sorts the candidates in shared memory (bitonic) and emits the list;
//     otherwise a sample sort across the cluster: CTA 0 sorts a 1024-key sample and publishes
//     <= 255 splitters; all CTAs bucket their candidates; offsets by prefix sum; scatter into
//     bucket order; each needed bucket is sorted in a shared-memory tile.
#include <cooperative_groups.h>

#include "cs_select_common.cuh"

namespace cg = cooperative_groups;

#define CSEL_THREADS 512
#define CSEL_SORT_MAX 4096u       // keys one CTA orders in shared memory
#define CSEL_MAX_CLUSTER 16

struct ClusterSmem {
    float *tables;
    uint32_t *hist;                 // [4096] this CTA's histogram
    uint32_t *tot;                  // [4096] cluster-wide histogram (same in every CTA after phase 2)
    unsigned long long *km;         // [CSEL_SORT_MAX]
    uint32_t *id;                   // [CSEL_SORT_MAX]
    uint32_t *part;                 // [CSEL_THREADS] scan scratch
    uint32_t *misc;                 // [8]
};

__host__ __device__ inline size_t csel_table_bytes(uint32_t A, uint32_t gtab_len)
{
    return (((size_t)(A + gtab_len) * 4 + (size_t)A * 2) + 15) / 16 * 16;
}
static size_t csel_smem_bytes(uint32_t A, uint32_t gtab_len)
{
    return csel_table_bytes(A, gtab_len) + 2 * CS_HIST_BINS * 4 + CSEL_SORT_MAX * 12 + CSEL_THREADS * 4 + 64;
}

__device__ __forceinline__ void csel_carve(unsigned char *base, uint32_t A, uint32_t gtab_len, ClusterSmem &S)
{
    S.tables = (float *)base;
    S.hist = (uint32_t *)(base + csel_table_bytes(A, gtab_len));
    S.tot = S.hist + CS_HIST_BINS;
    S.km = (unsigned long long *)(S.tot + CS_HIST_BINS);
    S.id = (uint32_t *)(S.km + CSEL_SORT_MAX);
    S.part = S.id + CSEL_SORT_MAX;
    S.misc = S.part + CSEL_THREADS;
}

// Exclusive prefix sum of one value per thread over the CTA (CSEL_THREADS threads); also returns the total.
__device__ __forceinline__ uint32_t csel_block_scan(uint32_t v, uint32_t *s_part, uint32_t &total)
{
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += t;
    }
    __syncthreads();
    if (lane == 31) s_part[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < (CSEL_THREADS / 32) ? s_part[lane] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, w, d);
            if (lane >= d) w += t;
        }
        s_part[32 + lane] = w;                         // inclusive warp totals
    }
    __syncthreads();
    total = s_part[32 + CSEL_THREADS / 32 - 1];
    const uint32_t before = warp ? s_part[32 + warp - 1] : 0;
    return before + incl - v;
}

// In-place bitonic sort of P (power of two) keys in shared memory, ascending by (km, id).
__device__ __forceinline__ void csel_bitonic(unsigned long long *km, uint32_t *id, uint32_t P)
{
    if (P >= 64 && P <= 2 * CSEL_THREADS) { bitonic_sort_fast(km, id, P, whole_cta()); return; }
    for (uint32_t size = 2; size <= P; size <<= 1) {
        for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
            for (uint32_t t = threadIdx.x; t < P / 2; t += blockDim.x) {
                const uint32_t lo = 2 * t - (t & (stride - 1));
                const uint32_t hi = lo + stride;
                const bool up = (lo & size) == 0;
                const unsigned long long ka = km[lo], kb = km[hi];
                const uint32_t ia = id[lo], ib = id[hi];
                if (key_less(kb, ib, ka, ia) == up) {
                    km[lo] = kb; id[lo] = ib;
                    km[hi] = ka; id[hi] = ia;
                }
            }
            __syncthreads();
        }
    }
}

// One whole select by the calling cluster.  `ws` carries this select's private candidate / sort regions
// and its row of per-call scalars, so several clusters of one launch can run different selects at once.
template <bool PF>
__device__ __forceinline__ void csel_body(SelArgs a, const cs_workspace &ws, uint32_t *__restrict__ ids_out,
                                          uint32_t *__restrict__ n_out_dev, unsigned char *dsm)
{
    resolve_now(a);
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t CL = cluster.num_blocks(), rank = cluster.block_rank();
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    ClusterSmem S;
    csel_carve(dsm, a.A, a.gtab_len, S);
    Tables T;
    load_tables(a, ws, S.tables, T, PF && a.anchor);
    for (uint32_t i = tid; i < CS_HIST_BINS; i += CSEL_THREADS) S.hist[i] = 0;
    const uint32_t c_slot = *(volatile uint32_t *)&ws.sel->toggle & 1u;   // read here, before any CTA can flip it (first cluster barrier)
    uint32_t *cand_count = &ws.sel->cc[c_slot];                   // zero on entry: the previous call cleared it
    if (rank == 0 && tid == 0) ws.sel->cc[c_slot ^ 1u] = 0;
    if (tid == 0) S.misc[1] = 0;
    __syncthreads();
    const bool enabled = !PF || prefetch_enabled(ws, a.A);
    const uint32_t n_tiles = a.n / TILE;
    const uint32_t cthreads = CL * CSEL_THREADS, ctid = rank * CSEL_THREADS + tid;   // cluster-wide thread id
    const uint32_t t0 = n_tiles * TILE;                                              // start of the ragged tail

    // One routine serves both scans: per warp tile it computes the keys of the eligible entries, feeds
    // the histogram (first scan) and appends the entries whose first digit is <= `limit` to the
    // candidate buffer (warp-aggregated reservation, keys recomputed for the few that are written).
    uint32_t run_bin = 0xFFFFFFFFu, run_cnt = 0;              // adjacent entries often share a bin
    auto hist_add = [&](uint32_t pr) {
        const uint32_t bin = pr >> 20;
        if (bin == run_bin) { ++run_cnt; return; }
        if (run_cnt) atomicAdd(&S.hist[run_bin], run_cnt);
        run_bin = bin;
        run_cnt = 1;
    };
    auto scan = [&](bool do_hist, bool do_collect, uint32_t limit) {
        const uint32_t n_warps = cthreads >> 5;
        const uint32_t n_iter = (n_tiles + n_warps - 1) / n_warps;       // whole warps stay in the ballots
        WarpStage st;
        stage_init(st, S.km, S.id);                                      // the sort tile is free during the scans
        for (uint32_t it = 0; it < n_iter; ++it) {
            const uint32_t t = it * n_warps + (ctid >> 5);
            Group G;
            uint32_t em = 0;
            if (t < n_tiles) {
                load_group<PF>(a, t, lane, G);
                em = group_elig<PF>(a, G);
            }
            if (!__any_sync(0xFFFFFFFFu, em != 0)) continue;
#pragma unroll
            for (int j = 0; j < GRP; ++j) {
                uint32_t pr = 0, se = 0;
                bool cand = false;
                if ((em >> j) & 1u) {
                    const uint32_t tok = a.ntok ? grp_u8(G.tk, j) : a.block_tokens;
                    const uint32_t dp = (PF && a.anchor) ? grp_u16(G.dp0, G.dp1, j) : 0u;
                    if (entry_key_rest<PF>(a, T, &ws.sc->status, grp_u16(G.ag0, G.ag1, j), dp, grp_u8(G.fl, j), grp_u32(G, j), tok, pr, se)) {
                        if (do_hist) hist_add(pr);
                        cand = (pr >> 20) <= limit;
                    }
                }
                if (do_collect) stage_push(st, cand, pr, se, grp_id(t, lane, j), cand_count, ws.cand_km, ws.cand_id);
            }
        }
        stage_flush(st, cand_count, ws.cand_km, ws.cand_id);
        if (ctid < a.n - t0) {                                 // ragged tail, one entry per thread
            const uint32_t i = t0 + ctid;
            uint32_t p, se;
            const uint32_t tok = a.ntok ? a.ntok[i] : a.block_tokens;
            if (entry_key<PF>(a, T, &ws.sc->status, a.agent[i], a.depth[i], a.ref[i], a.flags[i], a.la[i], tok, p, se)) {
                if (do_hist) hist_add(p);
                if (do_collect && (p >> 20) <= limit) {
                    const uint32_t pos = atomicAdd(cand_count, 1u);
                    ws.cand_km[pos] = ((unsigned long long)p << 32) | se;
                    ws.cand_id[pos] = i;
                }
            }
        }
    };

    // ---- phase 1: histogram of this CTA's slice, and candidates up to the remembered threshold bin -----
    const uint32_t hint = ws.sc->sel_hint[a.hint_slot];       // ~0: nothing remembered
    if (enabled) {
        scan(true, hint != 0xFFFFFFFFu, hint);
        if (run_cnt) atomicAdd(&S.hist[run_bin], run_cnt);
    }
    __threadfence();
    cluster.sync();

    // ---- phase 2: reduce the histograms through DSMEM, broadcast, find the threshold bin ---------------
    {
        const uint32_t per = CS_HIST_BINS / CL;                     // CL is a power of two <= 16
        for (uint32_t b = tid; b < per; b += CSEL_THREADS) {
            const uint32_t bin = rank * per + b;
            uint32_t sum = 0;
            for (uint32_t q = 0; q < CL; ++q) sum += cluster.map_shared_rank(S.hist, q)[bin];
            for (uint32_t q = 0; q < CL; ++q) cluster.map_shared_rank(S.tot, q)[bin] = sum;
        }
    }
    cluster.sync();
    if (rank == 0 && tid == 0) ws.sel->toggle = c_slot ^ 1u;       // every CTA has read it: the next call takes the other counter
    constexpr uint32_t PER = CS_HIST_BINS / CSEL_THREADS;
    uint32_t loc[PER], sum = 0;
#pragma unroll
    for (uint32_t q = 0; q < PER; ++q) { loc[q] = S.tot[tid * PER + q]; sum += loc[q]; }
    uint32_t n_elig;
    const uint32_t before = csel_block_scan(sum, S.part, n_elig);
    if (tid == 0) S.misc[0] = (a.k == 0) ? 0xFFFFFFFFu : CS_HIST_BINS - 1;      // k = 0: nothing; k > eligible: everything
    __syncthreads();
    if (a.k && n_elig >= a.k && before < a.k && a.k <= before + sum) {
        uint32_t run = before;
#pragma unroll
        for (uint32_t q = 0; q < PER; ++q) {
            run += loc[q];
            if (run >= a.k) { S.misc[0] = tid * PER + q; break; }
        }
    }
    __syncthreads();
    const uint32_t b0 = S.misc[0];
    const uint32_t n_out = n_elig < a.k ? n_elig : a.k;
    // the tail of the list is known now: pad it while the candidates are being collected
    for (uint32_t i = n_out + ctid; i < a.k; i += cthreads) ids_out[i] = CS_ID_NONE;
    if (ctid == 0) { *n_out_dev = n_out; count_select(ws, a.kind, n_elig, n_out); }

    // ---- phase 3: collect the candidates (bin <= b0), unless the first scan already has them ----------------
    const bool spec_ok = hint != 0xFFFFFFFFu && b0 != 0xFFFFFFFFu && b0 <= hint;     // same verdict in every CTA
    const bool have_b0 = a.k && n_elig >= a.k;
    if (rank == 0) {                                           // whole CTA 0: same histogram in every CTA
        const uint32_t ahead = have_b0 ? collect_ahead_limit<PER>(loc, tid * PER, before, a.k, b0, &S.misc[2], whole_cta()) : 0u;
        if (tid == 0) remember_threshold(ws.sc, a.hint_slot, have_b0, ahead);
    }
    if (!spec_ok) {
        if (hint != 0xFFFFFFFFu) {                            // drop what the first scan appended
            if (rank == 0 && tid == 0) *cand_count = 0;
            __threadfence();
            cluster.sync();
        }
        if (enabled && b0 != 0xFFFFFFFFu) scan(false, true, b0);
        __threadfence();
        cluster.sync();
    }
    const uint32_t c = __ldcg(cand_count);
    if (ctid == 0) count_candidates(ws, a.kind, c, spec_ok);

    // ---- phase 4, small: ordered in shared memory ---------------------------------------------------------------
    if (c <= CSEL_SORT_MAX) {
        if (c == 0) return;
        constexpr uint32_t CH = 2 * CSEL_THREADS;                // keys one CTA orders with the register sort
        const uint32_t n_chunks = (c + CH - 1) / CH;
        if (n_chunks > 1 && n_chunks <= CL && n_chunks * n_out <= CH) {
            // Several CTAs order one chunk each, side by side: the n_out smallest keys of the union lie among the
            // n_out smallest of every chunk, so CTA 0 only has to order n_chunks * n_out survivors afterwards.
            if (rank < n_chunks) {
                const uint32_t beg = rank * CH, m = min(CH, c - beg);
                for (uint32_t i = tid; i < CH; i += CSEL_THREADS) {
                    S.km[i] = i < m ? __ldcg(&ws.cand_km[beg + i]) : ~0ull;
                    S.id[i] = i < m ? __ldcg(&ws.cand_id[beg + i]) : 0xFFFFFFFFu;
                }
                __syncthreads();
                csel_bitonic(S.km, S.id, CH);
                for (uint32_t i = tid; i < n_out; i += CSEL_THREADS) {
                    ws.sort_km[rank * n_out + i] = S.km[i];
                    ws.sort_id[rank * n_out + i] = S.id[i];
                }
            }
            __threadfence();
            cluster.sync();                                     // every CTA of the cluster gets here
            if (rank != 0) return;
            const uint32_t tot = n_chunks * n_out;
            uint32_t P = 64;
            while (P < tot) P <<= 1;
            __syncthreads();
            for (uint32_t i = tid; i < P; i += CSEL_THREADS) {
                S.km[i] = i < tot ? __ldcg(&ws.sort_km[i]) : ~0ull;
                S.id[i] = i < tot ? __ldcg(&ws.sort_id[i]) : 0xFFFFFFFFu;
            }
            __syncthreads();
            csel_bitonic(S.km, S.id, P);
            for (uint32_t i = tid; i < n_out; i += CSEL_THREADS) ids_out[i] = S.id[i];
            return;
        }
        if (rank != 0) return;
        uint32_t P = 64;
        while (P < c) P <<= 1;
        for (uint32_t i = tid; i < P; i += CSEL_THREADS) {
            S.km[i] = i < c ? __ldcg(&ws.cand_km[i]) : ~0ull;
            S.id[i] = i < c ? __ldcg(&ws.cand_id[i]) : 0xFFFFFFFFu;
        }
        __syncthreads();
        csel_bitonic(S.km, S.id, P);
        for (uint32_t i = tid; i < n_out; i += CSEL_THREADS) ids_out[i] = S.id[i];
        return;
    }

    // ---- phase 4, large: sample sort across the cluster ---------------------------------------------------------
    if (rank == 0) {
        for (uint32_t i = tid; i < CS_SAMPLE; i += CSEL_THREADS) {
            const uint32_t pos = (uint32_t)(((unsigned long long)i * c) / CS_SAMPLE);
            S.km[i] = __ldcg(&ws.cand_km[pos]);
            S.id[i] = __ldcg(&ws.cand_id[pos]);
        }
        __syncthreads();
        csel_bitonic(S.km, S.id, CS_SAMPLE);
        for (uint32_t j = tid; j <= CS_MAX_SPLITTERS; j += CSEL_THREADS) {
            if (j < CS_MAX_SPLITTERS) {
                const uint32_t q = (uint32_t)(((unsigned long long)(j + 1) * CS_SAMPLE) / (CS_MAX_SPLITTERS + 1));
                ws.spl_km[j] = S.km[q];
                ws.spl_id[j] = S.id[q];
            }
            CS_BCOUNT(ws, j) = 0;
        }
    }
    __threadfence();
    cluster.sync();
    // bucket: number of splitters <= key; slot by a global counter per bucket
    unsigned long long *spl_km = S.km;               // shared-memory copy of the splitters
    uint32_t *spl_id = S.id;
    __syncthreads();
    for (uint32_t j = tid; j < CS_MAX_SPLITTERS; j += CSEL_THREADS) { spl_km[j] = __ldcg(&ws.spl_km[j]); spl_id[j] = __ldcg(&ws.spl_id[j]); }
    __syncthreads();
    for (uint32_t i = ctid; i < c; i += cthreads) {
        const unsigned long long km = __ldcg(&ws.cand_km[i]);
        const uint32_t id = __ldcg(&ws.cand_id[i]);
        uint32_t lo = 0, hi = CS_MAX_SPLITTERS;
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (key_less(km, id, spl_km[mid], spl_id[mid])) hi = mid;
            else lo = mid + 1;
        }
        ws.cand_bkt[i] = lo;
        ws.cand_slot[i] = atomicAdd(&CS_BCOUNT(ws, lo), 1u);
    }
    __threadfence();
    cluster.sync();
    // offsets (every CTA computes the same prefix sum), then scatter the needed buckets into bucket order
    uint32_t *s_off = S.hist;                        // reuse: [CS_MAX_SPLITTERS + 2]
    {
        const uint32_t mine = tid <= CS_MAX_SPLITTERS ? __ldcg(&CS_BCOUNT(ws, tid)) : 0u;
        uint32_t total;
        const uint32_t excl = csel_block_scan(mine, S.part, total);
        if (tid <= CS_MAX_SPLITTERS) s_off[tid] = excl;
        if (tid == CS_MAX_SPLITTERS) s_off[CS_MAX_SPLITTERS + 1] = excl + mine;
        if (mine && excl <= n_out - 1 && n_out - 1 < excl + mine) S.misc[1] = tid;     // last needed bucket (n_out > 0 here)
        __syncthreads();
    }
    const uint32_t b_last = S.misc[1];
    for (uint32_t i = ctid; i < c; i += cthreads) {
        const uint32_t b = __ldcg(&ws.cand_bkt[i]);
        if (b > b_last) continue;
        const uint32_t pos = s_off[b] + __ldcg(&ws.cand_slot[i]);
        ws.sort_km[pos] = __ldcg(&ws.cand_km[i]);
        ws.sort_id[pos] = __ldcg(&ws.cand_id[i]);
    }
    __threadfence();
    cluster.sync();
    // rank: buckets round-robin over the CTAs; a bucket is ranked from a shared-memory tile
    for (uint32_t b = rank; b <= b_last; b += CL) {
        const uint32_t beg = s_off[b], end = s_off[b + 1], m = end - beg;
        __syncthreads();
        if (m <= CSEL_SORT_MAX) {
            uint32_t P = 64;
            while (P < m) P <<= 1;
            for (uint32_t i = tid; i < P; i += CSEL_THREADS) {
                S.km[i] = i < m ? __ldcg(&ws.sort_km[beg + i]) : ~0ull;
                S.id[i] = i < m ? __ldcg(&ws.sort_id[beg + i]) : 0xFFFFFFFFu;
            }
            __syncthreads();
            csel_bitonic(S.km, S.id, P);
            for (uint32_t i = tid; i < m; i += CSEL_THREADS)
                if (beg + i < n_out) ids_out[beg + i] = S.id[i];
        } else {                                     // a bucket larger than the tile: rank straight from global memory
            for (uint32_t i = tid; i < m; i += CSEL_THREADS) {
                const unsigned long long km = __ldcg(&ws.sort_km[beg + i]);
                const uint32_t id = __ldcg(&ws.sort_id[beg + i]);
                uint32_t r = 0;
                for (uint32_t q = beg; q < end; ++q) r += key_less(__ldcg(&ws.sort_km[q]), __ldcg(&ws.sort_id[q]), km, id) ? 1u : 0u;
                if (beg + r < n_out) ids_out[beg + r] = id;
            }
        }
    }
}

template <bool PF>
__global__ void __launch_bounds__(CSEL_THREADS, 1)
cs_select_cluster_kernel(SelArgs a, cs_workspace ws, uint32_t *__restrict__ ids_out, uint32_t *__restrict__ n_out_dev)
{
    extern __shared__ __align__(16) unsigned char dsm[];
    csel_body<PF>(a, ws, ids_out, n_out_dev, dsm);
}

// The three selects of a step in one launch: cluster q of the grid runs select q (GPU-tier victims,
// host-tier victims, prefetch candidates).  The selects share the index and the tables and nothing else.
struct SelJob {
    SelArgs a;
    cs_workspace ws;
    uint32_t *ids_out, *n_out;
    uint32_t prefetch;
};
struct SelJobs { SelJob j[3]; };     // the grid holds one cluster per job in use

__global__ void __launch_bounds__(CSEL_THREADS, 1) cs_select_step_kernel(const __grid_constant__ SelJobs jobs)
{
    extern __shared__ __align__(16) unsigned char dsm[];
    const uint32_t q = blockIdx.x / cg::this_cluster().num_blocks();
    const SelJob &J = jobs.j[q];
    if (J.prefetch) csel_body<true>(J.a, J.ws, J.ids_out, J.n_out, dsm);
    else csel_body<false>(J.a, J.ws, J.ids_out, J.n_out, dsm);
}

// ---------------------------------------------------------------------------------------------
// Per-device set-up of the three cluster kernels, done once per process and device.  The dynamic shared-memory
// opt-in is an attribute of the FUNCTION (on a device), not of a context, so it is raised once to the fixed
// maximum any parameter set can ask for (CS_MAX_AGENTS agents, the longest recency table) and never lowered:
// contexts of different shape and the static-scratch entry point can then share the kernels.  The largest
// usable cluster is probed with that same maximum, which makes the answer independent of the caller's sizes.
#include <mutex>

#define CSEL_MAX_DEVICES 64
struct CselDevice {
    int ready;                       // 0 = not set up yet
    int max_v, max_pf, max_step;     // largest usable cluster per kernel (-1 = none)
};
static std::mutex g_csel_mu;
static CselDevice g_csel_dev[CSEL_MAX_DEVICES];

template <class Kernel>
static int csel_probe(Kernel kernel, size_t smem, int clusters_needed)
{
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(CSEL_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    for (int cl = CSEL_MAX_CLUSTER; cl >= 1; cl >>= 1) {
        cfg.gridDim = dim3(clusters_needed * cl);
        attr[0].val.clusterDim.x = cl;
        int n_clusters = 0;
        const cudaError_t e = cudaOccupancyMaxActiveClusters(&n_clusters, kernel, &cfg);
        if (e == cudaSuccess && n_clusters >= clusters_needed) return cl;
        (void)cudaGetLastError();
    }
    return -1;
}

// Returns the device's entry (set up on first use, with `device` current), or nullptr for a device index out of range.
static const CselDevice *csel_device(int device)
{
    if (device < 0 || device >= CSEL_MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(g_csel_mu);
    CselDevice &d = g_csel_dev[device];
    if (!d.ready) {
        const size_t smem_max = csel_smem_bytes(CS_MAX_AGENTS, CS_GTAB_MAX);
        d.max_v = csel_probe(cs_select_cluster_kernel<false>, smem_max, 1);
        d.max_pf = csel_probe(cs_select_cluster_kernel<true>, smem_max, 1);
        d.max_step = csel_probe(cs_select_step_kernel, smem_max, 3);
        d.ready = 1;
    }
    return &d;
}

// smallest power-of-two cluster that gives every 16-entry group its own thread, at most max_cl
static int csel_cluster_size(uint32_t n, int max_cl)
{
    const uint32_t n_groups = n / GRP;                   // 16 entries per thread and pass
    int cl = 1;
    while (cl < max_cl && (uint32_t)cl * CSEL_THREADS < n_groups) cl <<= 1;
    return cl;
}

template <bool PF>
static int launch_cluster(cs_ctx *ctx, const SelArgs &a, const cs_workspace &ws, uint32_t *ids_out, uint32_t *n_out,
                          cudaStream_t s)
{
    const CselDevice *d = csel_device(ctx->device);
    const int max_cl = d ? (PF ? d->max_pf : d->max_v) : -1;
    if (max_cl < 1) return CS_ENOTIMPL;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    const int cl = csel_cluster_size(a.n, max_cl);
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(cl);
    cfg.blockDim = dim3(CSEL_THREADS);
    cfg.dynamicSmemBytes = csel_smem_bytes(a.A, a.gtab_len);      // <= the opted-in maximum by construction
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, cs_select_cluster_kernel<PF>, a, ws, ids_out, n_out);
    ctx->n_launches++;
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return CS_OK;
}

int cs_launch_select_clusters(cs_ctx *ctx, int n_jobs, const void *sel_args, const uint32_t *prefetch,
                              uint32_t *const *ids_out, uint32_t *const *n_out, cudaStream_t s)
{
    const SelArgs *aj = (const SelArgs *)sel_args;
    const CselDevice *d = csel_device(ctx->device);
    const int max_cl = d ? d->max_step : -1;
    if (max_cl < 1) return CS_ENOTIMPL;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    const int cl = csel_cluster_size(aj[0].n, max_cl);
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(n_jobs * cl);
    cfg.blockDim = dim3(CSEL_THREADS);
    cfg.dynamicSmemBytes = csel_smem_bytes(aj[0].A, aj[0].gtab_len);
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    SelJobs jobs;
    for (int q = 0; q < n_jobs; ++q) {
        jobs.j[q].a = aj[q];
        jobs.j[q].ws = q == 0 ? ctx->ws : ctx->ws_job[q - 1];
        jobs.j[q].ids_out = ids_out[q];
        jobs.j[q].n_out = n_out[q];
        jobs.j[q].prefetch = prefetch[q];
    }
    for (int q = n_jobs; q < 3; ++q) jobs.j[q] = jobs.j[0];          // unused slots: defined contents
    cudaError_t e = cudaLaunchKernelEx(&cfg, cs_select_step_kernel, jobs);
    ctx->n_launches++;
    if (e != cudaSuccess) { ctx->last_cuda_error = (int)e; return CS_ECUDA; }
    return CS_OK;
}

int cs_launch_select_cluster(cs_ctx *ctx, const void *sel_args, const cs_workspace *ws, int prefetch, uint32_t *ids_out,
                             uint32_t *n_out, cudaStream_t s)
{
    const SelArgs &a = *(const SelArgs *)sel_args;
    return prefetch ? launch_cluster<true>(ctx, a, *ws, ids_out, n_out, s) : launch_cluster<false>(ctx, a, *ws, ids_out, n_out, s);
}
