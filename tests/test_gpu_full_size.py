"""Parity at the sizes and in the launch configuration bench.py times (Llama-3-8B-shaped KV:
20,000-block GPU pool = 39 GiB, 80,000-entry index, 2 MiB blocks), plus a teacher-forced closed
loop at the tiny configuration and the 70B block geometry.

At full size the id lists are compared with the oracle bit for bit; the moved KV bytes are checked
on sampled blocks that the oracle copies one by one between small stand-in pools."""
import argparse

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import cs_oracle as orc
from paper_2608_14624_b200 import binding as cs
from tests import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def block_bytes_from_pool(buf_u8, layout, n_slots, L, chunk, slot):
    """The 2L chunks of one block as a host array [L, 2, chunk] (device gather, then one copy)."""
    if layout == synth.LAYER_MAJOR:
        return buf_u8.view(L, 2, n_slots, chunk)[:, :, slot, :].cpu().numpy()
    return buf_u8.view(n_slots, L, 2, chunk)[slot].cpu().numpy()


@pytest.mark.parametrize("cfg_name,transfers", [("llama8b", "exchange"), ("llama8b", "split"), ("llama70b", "exchange")])
def test_bench_step_at_full_size_matches_oracle(cfg_name, transfers):
    """The step exactly as bench.py times it (full-size GPU pool and index of the 8B- and the 70B-shaped
    configuration, the bench's launch configuration), lists against the oracle and sampled blocks byte for byte."""
    import bench
    free = torch.cuda.mem_get_info()[0]
    if free < 70 * (1 << 30) or bench.mem_available_bytes() < 60 * (1 << 30):
        pytest.skip("needs 70 GiB of free device memory and 60 GiB of host memory")
    args = argparse.Namespace(quick=False, host_slots=8192 if cfg_name == "llama8b" else 4096, host_frac=0.4, offload_width=0,
                              prefetch_width=0, transfers=transfers, exchange_width=0)
    w = bench.StepWorkload(args, torch.device(DEV), 1, cfg_name)
    cfg, G, L, chunk = w.cfg, w.cfg.gpu_blocks, w.cfg.n_layers, w.cfg.chunk_bytes
    o = orc.Oracle(H.oracle_params(w.params))
    o.observe(w.tr.chain[:2000], w.tr.agent[:2000], w.tr.evflags[:2000])
    H.compare_model(w.c, o)
    idx = w.idx_host                                      # the index as uploaded (no step has run yet)
    gpu_u8 = w.gpu_buf.view(torch.uint8)
    for s in range(2):
        now = w.now0 + s
        st = (600 + s) % (w.n_steps - 1)
        lo, hi = int(w.tr.step_off[st]), int(w.tr.step_off[st + 1])
        b, prev = s % w.RING, (s - 1) % w.RING
        dst_prev = w.dst[prev].cpu().numpy().view(np.uint32).copy()
        # source blocks of the transfers, read before the step overwrites anything
        w.step(s)
        w.drain()
        torch.cuda.synchronize()
        o.observe(w.tr.chain[lo:hi], w.tr.agent[lo:hi], w.tr.evflags[lo:hi])
        s64, s32 = o.scores(idx, now)
        ov, ovn = o.select_victims(idx, now, 0, w.k_v, s32)
        oh, ohn = o.select_victims(idx, now, 1, w.k_v, s32)
        op, opn = o.select_prefetch(idx, now, w.k_p, s32)
        gv = w.dst[b][:w.k_v].cpu().numpy().view(np.uint32)
        gh = w.hv[b][:w.k_v].cpu().numpy().view(np.uint32)
        gp = w.pf[b][:w.k_p].cpu().numpy().view(np.uint32)
        assert H.assert_list_matches(gv, int(w.vn[b][0].item()), ov, ovn, s64) == 0
        assert H.assert_list_matches(gh, int(w.hn[b][0].item()), oh, ohn, s64) == 0
        assert H.assert_list_matches(gp, int(w.pn[b][0].item()), op, opn, s64) == 0
        assert ovn == w.k_v and ohn == w.k_v and opn == w.k_p
        # offload: sampled victims, oracle copies the block between one-slot stand-in pools
        rng = np.random.default_rng(s)
        for i in rng.choice(w.k_v, 6, replace=False):
            src_block = block_bytes_from_pool(gpu_u8, synth.LAYER_MAJOR, G, L, chunk, int(ov[i]))
            if int(ov[i]) in set(dst_prev.tolist()):
                continue                                   # overwritten by this step's prefetch afterwards
            stand_src = np.ascontiguousarray(src_block).reshape(-1)      # 1 slot: both layouts coincide
            stand_dst = np.zeros_like(stand_src)
            orc.move_blocks(stand_src, synth.LAYER_MAJOR, 1, stand_dst, synth.BLOCK_MAJOR, 1, L, chunk, [0], [0])
            host_slot = int(oh[i]) - G
            got = w.host_buf[host_slot * cfg.block_bytes:(host_slot + 1) * cfg.block_bytes].numpy()
            assert np.array_equal(got, stand_dst), ("offload", s, i)
        # prefetch: sampled candidates landed in the free GPU slots of the previous step
        for i in rng.choice(w.k_p, 6, replace=False):
            host_slot = int(op[i]) - G
            if host_slot in set((oh[:ohn] - G).tolist()):
                continue                                   # that host slot received an offloaded block in this step
            stand_src = w.host_buf[host_slot * cfg.block_bytes:(host_slot + 1) * cfg.block_bytes].numpy().copy()
            stand_dst = np.zeros_like(stand_src)
            orc.move_blocks(stand_src, synth.BLOCK_MAJOR, 1, stand_dst, synth.LAYER_MAJOR, 1, L, chunk, [0], [0])
            got = block_bytes_from_pool(gpu_u8, synth.LAYER_MAJOR, G, L, chunk, int(dst_prev[i])).reshape(-1)
            assert np.array_equal(got, stand_dst), ("prefetch", s, i)
        # compaction: the staging pool holds the victims packed, block-major
        for i in rng.choice(w.k_v, 4, replace=False):
            if int(ov[i]) in set(dst_prev.tolist()):
                continue
            src_block = block_bytes_from_pool(gpu_u8, synth.LAYER_MAJOR, G, L, chunk, int(ov[i])).reshape(-1)
            got = w.stage_buf[i * cfg.block_bytes:(i + 1) * cfg.block_bytes].cpu().numpy()
            assert np.array_equal(got, src_block), ("compact", s, i)
        # bookkeeping of the harness, mirrored on the host copy of the index
        idx.last_access[ov[:ovn].astype(np.int64)] = now
        idx.flags[op[:opn].astype(np.int64)] |= synth.FLAG_OTHER_COPY
    assert w.c.get_status() == 0
    moved = w.take_moved_bytes()                           # the mover's own counters: every block of both steps
    assert moved == 2 * (w.k_v + w.k_p) * cfg.block_bytes
    w.release()


def test_mover_70b_block_geometry():
    """80 layers x 8 KV heads x 128, bf16: 5 MiB blocks of 160 chunks, both layouts, bulk path."""
    cfg = synth.CONFIGS["llama70b"]
    L, chunk, G, Hs, n = cfg.n_layers, cfg.chunk_bytes, 40, 24, 13
    assert cfg.block_bytes == 5 * (1 << 20)
    rng = synth.rng_for(cfg, 5)
    c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, max_blocks=64), DEV)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    for gpu_layout in (synth.LAYER_MAJOR, synth.BLOCK_MAJOR):
        gpu = cs.KVPool(dev(gpu_np), G, gpu_layout, L)
        host_t = torch.zeros(Hs * L * 2 * chunk, dtype=torch.uint8).pin_memory()
        host = cs.KVPool(host_t, Hs, synth.BLOCK_MAJOR, L, first_id=1000)
        src, dst = synth.mover_batch(n, G, Hs, rng)
        c.offload_blocks(gpu, host, dev(src), dev(dst + 1000))
        back = rng.choice(G, size=n, replace=False).astype(np.uint32)
        c.prefetch_blocks(host, gpu, dev(dst + 1000), dev(back))
        torch.cuda.synchronize()
        want_host = np.zeros(Hs * L * 2 * chunk, np.uint8)
        orc.move_blocks(gpu_np, gpu_layout, G, want_host, synth.BLOCK_MAJOR, Hs, L, chunk, src, dst)
        assert np.array_equal(host_t.numpy(), want_host)
        want_gpu = gpu_np.copy()
        orc.move_blocks(want_host, synth.BLOCK_MAJOR, Hs, want_gpu, gpu_layout, G, L, chunk, dst, back)
        assert np.array_equal(gpu.buf.cpu().numpy(), want_gpu)
        # ids below first_id are out of range for the host pool: skipped and reported
        c.offload_blocks(gpu, host, dev(src[:1]), dev(np.array([5], np.uint32)))
        assert c.get_status() == cs.CS_ST_BAD_SLOT


@pytest.mark.parametrize("chain_mode", ["session", "single", "llama70b-shape"])
def test_closed_loop_teacher_forced_tiny(chain_mode):
    """Tiny configuration end to end: 4 agents, 200 invocations, 512-block GPU pool, 2,048-slot host
    tier, 32 victims / 64 prefetch candidates per step.  Every step both sides get the same state;
    outputs are compared and the oracle's output advances the state, so a mismatch cannot cascade."""
    cfg = synth.CONFIGS["tiny"]
    if chain_mode == "session":
        cfg = synth.shrink(cfg, sessions=4, n_chains=4, events_per_step=(1, 3))
    elif chain_mode == "llama70b-shape":          # 30 agents, sparse workflow matrix, 5 MiB blocks; pools cut to fit the oracle
        cfg = synth.shrink(synth.CONFIGS["llama70b"], gpu_blocks=64, host_blocks=128, invocations=240, sessions=16,
                           n_chains=16, k_victims=8, k_prefetch=12)
    G, Hs, L, chunk = cfg.gpu_blocks, cfg.host_blocks, cfg.n_layers, cfg.chunk_bytes
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=cfg.n_index,
                       block_tokens=cfg.block_tokens, r_min=0.05)
    c, o = cs.CacheScout(p, DEV), orc.Oracle(H.oracle_params(p))
    tr = synth.make_trace(cfg, warmup_frac=0.05)
    idx = synth.make_block_index(cfg, now0=1000)
    rng = synth.rng_for(cfg, 31)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    host_np = synth.kv_pool_u16(Hs, L, chunk, rng).view(np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, synth.LAYER_MAJOR, L)
    host_t = torch.from_numpy(host_np.copy()).pin_memory()
    host = cs.KVPool(host_t, Hs, synth.BLOCK_MAJOR, L, first_id=G)
    side = torch.cuda.Stream(device=DEV)
    n_steps = len(tr.step_off) - 1
    free_gpu = np.arange(G - cfg.k_prefetch, G, dtype=np.uint32)           # slots the first prefetch may fill
    idx.flags[free_gpu.astype(np.int64)] &= np.uint8(~synth.FLAG_VALID & 0xFF)
    compared = 0
    for s in range(n_steps):
        now = 1000 + s
        lo, hi = int(tr.step_off[s]), int(tr.step_off[s + 1])
        c.observe_invocations(dev(tr.chain[lo:hi]), dev(tr.agent[lo:hi]), dev(tr.evflags[lo:hi]))
        o.observe(tr.chain[lo:hi], tr.agent[lo:hi], tr.evflags[lo:hi])
        d = cs.DeviceIndex.from_host(idx, DEV)
        s64, s32 = o.scores(idx, now)
        gv, gvn = c.select_victims(d, now, 0, cfg.k_victims)
        gh, ghn = c.select_victims(d, now, 1, cfg.k_victims)
        gp, gpn = c.select_prefetch(d, now, cfg.k_prefetch)
        ov, ovn = o.select_victims(idx, now, 0, cfg.k_victims, s32)
        oh, ohn = o.select_victims(idx, now, 1, cfg.k_victims, s32)
        op, opn = o.select_prefetch(idx, now, cfg.k_prefetch, s32)
        H.assert_list_matches(gv.cpu().numpy().view(np.uint32)[:cfg.k_victims], int(gvn.item()), ov, ovn, s64)
        H.assert_list_matches(gh.cpu().numpy().view(np.uint32)[:cfg.k_victims], int(ghn.item()), oh, ohn, s64)
        H.assert_list_matches(gp.cpu().numpy().view(np.uint32)[:cfg.k_prefetch], int(gpn.item()), op, opn, s64)
        # carry the decisions out on both sides, driven by the ORACLE's lists (teacher forcing)
        n_off = min(ovn, ohn)
        side.wait_stream(torch.cuda.current_stream())
        c.offload_blocks(gpu, host, dev(ov[:n_off]), dev(oh[:n_off]), stream=side)
        orc.move_blocks(gpu_np, synth.LAYER_MAJOR, G, host_np, synth.BLOCK_MAJOR, Hs, L, chunk, ov[:n_off], oh[:n_off] - G)
        pf_src = op[:opn][~np.isin(op[:opn], oh[:n_off])]                   # a slot just overwritten is not prefetched
        n_pf = min(len(pf_src), len(free_gpu))
        if n_pf:
            c.prefetch_blocks(host, gpu, dev(pf_src[:n_pf]), dev(free_gpu[:n_pf]), stream=side)
            orc.move_blocks(host_np, synth.BLOCK_MAJOR, Hs, gpu_np, synth.LAYER_MAJOR, G, L, chunk, pf_src[:n_pf] - G, free_gpu[:n_pf])
        side.synchronize()
        # engine bookkeeping on the shared host index
        vi, hi_, pi = ov[:n_off].astype(np.int64), oh[:n_off].astype(np.int64), pf_src[:n_pf].astype(np.int64)
        idx.agent[hi_], idx.depth[hi_], idx.last_access[hi_] = idx.agent[vi], idx.depth[vi], idx.last_access[vi]
        idx.flags[hi_] = synth.FLAG_VALID | synth.FLAG_TIER_HOST
        fi = free_gpu[:n_pf].astype(np.int64)
        idx.agent[fi], idx.depth[fi], idx.last_access[fi] = idx.agent[pi], idx.depth[pi], now
        idx.flags[fi] = synth.FLAG_VALID
        idx.flags[pi] |= synth.FLAG_OTHER_COPY
        free_gpu = ov[:ovn].copy()                                           # evicted slots are free for the next step
        idx.flags[free_gpu.astype(np.int64)] &= np.uint8(~synth.FLAG_VALID & 0xFF)
        if s % 20 == 0 or s == n_steps - 1:
            assert np.array_equal(gpu.buf.cpu().numpy(), gpu_np), ("GPU pool differs at step", s)
            assert np.array_equal(host_t.numpy(), host_np), ("host tier differs at step", s)
            H.compare_model(c, o)
            compared += 1
    assert compared >= 3 and c.get_status() == 0
