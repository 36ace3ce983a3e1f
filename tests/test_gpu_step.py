"""cs_step: one whole scheduler step (observe, three selects, compaction, two-way transfer) as one
call, run as a closed loop at the tiny configuration and compared with the oracle every step.

Two ways of issuing it: the call made afresh every step (clock and event count by value), and the
call captured ONCE into a CUDA graph that reads the clock and the event count from device memory
and is replayed for every later step.  The loop is driven by the library's own lists, so every
list must equal the oracle's exactly for the two sides to stay in step."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import cs_oracle as orc
from paper_2608_14624_b200 import binding as cs
from tests import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
EV_CAP = 16


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def i32(n, fill=0):
    return torch.full((max(n, 4),), fill, dtype=torch.int32, device=DEV)


@pytest.mark.parametrize("mode", ["call", "graph"])
def test_step_closed_loop_matches_oracle(mode):
    cfg = synth.CONFIGS["tiny"]
    G, Hs, L, chunk = cfg.gpu_blocks, cfg.host_blocks, cfg.n_layers, cfg.chunk_bytes
    kv, kp = cfg.k_victims, cfg.k_prefetch
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=cfg.n_index,
                       block_tokens=cfg.block_tokens, r_min=0.05)
    c, o = cs.CacheScout(p, DEV), orc.Oracle(H.oracle_params(p))
    tr = synth.make_trace(cfg, warmup_frac=0.05)
    idx = synth.make_block_index(cfg, now0=1000)
    rng = synth.rng_for(cfg, 41)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    host_np = synth.kv_pool_u16(Hs, L, chunk, rng).view(np.uint8)
    stage_np = np.zeros(kv * L * 2 * chunk, np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, synth.LAYER_MAJOR, L)
    host_t = torch.from_numpy(host_np.copy()).pin_memory()
    host = cs.KVPool(host_t, Hs, synth.BLOCK_MAJOR, L, first_id=G)
    stage = cs.KVPool(torch.zeros(kv * L * 2 * chunk, dtype=torch.uint8, device=DEV), kv, synth.BLOCK_MAJOR, L)
    packed = torch.arange(kv, dtype=torch.int32, device=DEV)
    free_np = np.full(kp, orc.ID_NONE, np.uint32)                          # GPU slots the prefetch may fill
    free_np[:kv] = np.arange(G - kv, G, dtype=np.uint32)
    idx.flags[free_np[:kv].astype(np.int64)] &= np.uint8(~synth.FLAG_VALID & 0xFF)

    # persistent device buffers: a captured graph keeps their addresses
    d = cs.DeviceIndex.from_host(idx, DEV)
    gv, gh, gp, free_d = i32(kv), i32(kv), i32(kp), i32(kp)
    gvn, ghn, gpn = i32(1), i32(1), i32(1)
    ev_chain = torch.zeros(EV_CAP, dtype=torch.int32, device=DEV)             # u32 / u16 payloads behind signed views
    ev_agent = torch.zeros(EV_CAP, dtype=torch.int16, device=DEV)
    ev_flags = torch.zeros(EV_CAP, dtype=torch.uint8, device=DEV)
    now_d, nev_d = i32(1), i32(1)
    main, side = torch.cuda.Stream(device=DEV), torch.cuda.Stream(device=DEV)

    def issue(now, n_ev, by_value):
        c.step(d, now if by_value else 0, ev_chain, ev_agent, ev_flags, n_ev if by_value else EV_CAP, kv, kp,
               gv, gvn, gh, ghn, gp, gpn, gpu, host, free_d, stage=stage, stage_slots=packed,
               now_dev=None if by_value else now_d, n_events_dev=None if by_value else nev_d,
               main=main, side=side, join_main=True)

    graph = None
    if mode == "graph":
        # every kind of launch once outside capture, on inputs that change nothing the loop depends on
        scratch, scr_n = i32(4), i32(1)
        none4 = i32(4, -1)
        with torch.cuda.stream(main):
            c.select_victims(d, 1000, 0, 1, scratch, scr_n, stream=main)
            c.select_prefetch(d, 1000, 1, scratch, scr_n, stream=main)
            c.compact_blocks(gpu, stage, none4, none4, n_max=4, stream=main)
            c.exchange_blocks(gpu, host, none4, none4, none4, none4, stream=main)
        main.synchronize()
        assert c.get_status() == 0
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=main, capture_error_mode="relaxed"):
            issue(0, 0, by_value=False)

    n_steps = min(len(tr.step_off) - 1, 60)
    launches0 = c.launch_count()
    for s in range(n_steps):
        now = 1000 + s
        lo, hi = int(tr.step_off[s]), int(tr.step_off[s + 1])
        n_ev = hi - lo
        assert n_ev <= EV_CAP
        with torch.cuda.stream(main):
            for k in ("agent", "depth", "ref_count", "flags", "last_access", "n_tokens"):
                getattr(d, k).copy_(torch.from_numpy(getattr(idx, k)), non_blocking=False)
            ev_chain[:n_ev] = dev(tr.chain[lo:hi].view(np.int32))
            ev_agent[:n_ev] = dev(tr.agent[lo:hi].view(np.int16))
            ev_flags[:n_ev] = dev(tr.evflags[lo:hi].view(np.uint8))
            free_d[:kp] = dev(free_np.view(np.int32))
            now_d.fill_(now)
            nev_d.fill_(n_ev)
            if graph is None:
                issue(now, n_ev, by_value=True)
            else:
                graph.replay()
        main.synchronize()
        side.synchronize()

        o.observe(tr.chain[lo:hi], tr.agent[lo:hi], tr.evflags[lo:hi])
        s64, s32 = o.scores(idx, now)
        ov, ovn = o.select_victims(idx, now, 0, kv, s32)
        oh, ohn = o.select_victims(idx, now, 1, kv, s32)
        op, opn = o.select_prefetch(idx, now, kp, s32)
        as_u32 = lambda t, n: t.cpu().numpy().view(np.uint32)[:n]
        assert H.assert_list_matches(as_u32(gv, kv), int(gvn[0].item()), ov, ovn, s64) == 0, ("GPU victims", s)
        assert H.assert_list_matches(as_u32(gh, kv), int(ghn[0].item()), oh, ohn, s64) == 0, ("host victims", s)
        # a prefetch candidate whose host slot receives an offloaded block in this step is dropped from the list
        n_off = min(ovn, ohn)
        op = op.copy()
        op[:opn][np.isin(op[:opn], oh[:n_off])] = orc.ID_NONE
        got_p = as_u32(gp, kp)
        assert int(gpn[0].item()) == opn and np.array_equal(got_p[:opn], op[:opn]), ("prefetch", s)
        assert np.all(got_p[opn:] == orc.ID_NONE)
        # the oracle carries the same decisions out: compaction, then offload and prefetch on disjoint slots
        orc.move_blocks(gpu_np, synth.LAYER_MAJOR, G, stage_np, synth.BLOCK_MAJOR, kv, L, chunk, ov[:ovn], np.arange(ovn))
        orc.move_blocks(gpu_np, synth.LAYER_MAJOR, G, host_np, synth.BLOCK_MAJOR, Hs, L, chunk, ov[:n_off], oh[:n_off] - G)
        ok = (free_np[:opn] != orc.ID_NONE) & (op[:opn] != orc.ID_NONE)
        pf_src, pf_dst = op[:opn][ok], free_np[:opn][ok]
        orc.move_blocks(host_np, synth.BLOCK_MAJOR, Hs, gpu_np, synth.LAYER_MAJOR, G, L, chunk, pf_src - G, pf_dst)
        # engine bookkeeping on the shared host index
        vi, hi_, pi, fi = (x.astype(np.int64) for x in (ov[:n_off], oh[:n_off], pf_src, pf_dst))
        idx.agent[hi_], idx.depth[hi_], idx.last_access[hi_] = idx.agent[vi], idx.depth[vi], idx.last_access[vi]
        idx.flags[hi_] = synth.FLAG_VALID | synth.FLAG_TIER_HOST
        idx.agent[fi], idx.depth[fi], idx.last_access[fi] = idx.agent[pi], idx.depth[pi], now
        idx.flags[fi] = synth.FLAG_VALID
        idx.flags[pi] |= synth.FLAG_OTHER_COPY
        free_np[:] = orc.ID_NONE
        free_np[:ovn] = ov[:ovn]                                             # evicted slots are free for the next step
        idx.flags[ov[:ovn].astype(np.int64)] &= np.uint8(~synth.FLAG_VALID & 0xFF)
        if s % 15 == 0 or s == n_steps - 1:
            assert np.array_equal(stage.buf.cpu().numpy(), stage_np), ("staging pool differs at step", s)
            assert np.array_equal(gpu.buf.cpu().numpy(), gpu_np), ("GPU pool differs at step", s)
            assert np.array_equal(host_t.numpy(), host_np), ("host tier differs at step", s)
            H.compare_model(c, o)
    assert c.get_status() == 0
    if graph is None:
        assert c.launch_count() - launches0 >= 5 * n_steps           # every step really launched its kernels


def test_step_argument_errors():
    cfg = synth.CONFIGS["tiny"]
    c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, max_blocks=64), DEV)
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_step(c.ctx, cs.cs_step_io())                                   # no index, no pools
    assert e.value.code == cs.CS_EINVAL


@pytest.mark.parametrize("kv,kp,same_stream,with_stage", [(32, 0, True, False), (0, 16, False, True), (8, 8, True, True)])
def test_step_variants_one_step(kv, kp, same_stream, with_stage):
    """One step with an empty list, without a staging pool, and with both transfers on the caller's one stream."""
    cfg = synth.CONFIGS["tiny"]
    G, Hs, L, chunk = cfg.gpu_blocks, cfg.host_blocks, cfg.n_layers, cfg.chunk_bytes
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=cfg.n_index,
                       block_tokens=cfg.block_tokens, r_min=0.02)
    c, o = cs.CacheScout(p, DEV), orc.Oracle(H.oracle_params(p))
    tr = synth.make_trace(cfg)
    n0 = len(tr.agent) - 4
    c.observe_invocations(dev(tr.chain[:n0]), dev(tr.agent[:n0]), dev(tr.evflags[:n0]))
    o.observe(tr.chain[:n0], tr.agent[:n0], tr.evflags[:n0])
    idx = synth.make_block_index(cfg, now0=1000)
    free_np = np.arange(G - max(kp, 1), G, dtype=np.uint32)[:kp]
    idx.flags[free_np.astype(np.int64)] &= np.uint8(~synth.FLAG_VALID & 0xFF)
    d = cs.DeviceIndex.from_host(idx, DEV)
    rng = synth.rng_for(cfg, 43)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    host_np = synth.kv_pool_u16(Hs, L, chunk, rng).view(np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, synth.BLOCK_MAJOR, L)
    host_t = torch.from_numpy(host_np.copy()).pin_memory()
    host = cs.KVPool(host_t, Hs, synth.LAYER_MAJOR, L, first_id=G)
    ks = max(kv, 1)
    stage = cs.KVPool(torch.zeros(ks * L * 2 * chunk, dtype=torch.uint8, device=DEV), ks, synth.LAYER_MAJOR, L) if with_stage else None
    packed = torch.arange(ks, dtype=torch.int32, device=DEV)
    gv, gh, gp, free_d = i32(kv, -1), i32(kv, -1), i32(kp, -1), i32(kp, -1)
    if kp:
        free_d[:kp] = dev(free_np.view(np.int32))
    gvn, ghn, gpn = i32(1), i32(1), i32(1)
    main = torch.cuda.Stream(device=DEV)
    side = main if same_stream else torch.cuda.Stream(device=DEV)
    main.wait_stream(torch.cuda.current_stream())
    now = 1000 + 7
    c.step(d, now, dev(tr.chain[n0:].view(np.int32)), dev(tr.agent[n0:].view(np.int16)), dev(tr.evflags[n0:]), 4, kv, kp,
           gv, gvn, gh, ghn, gp, gpn, gpu, host, free_d, stage=stage, stage_slots=packed if with_stage else None,
           main=main, side=side, join_main=not same_stream)
    main.synchronize()
    o.observe(tr.chain[n0:], tr.agent[n0:], tr.evflags[n0:])
    H.compare_model(c, o)
    s64, s32 = o.scores(idx, now)
    ov, ovn = o.select_victims(idx, now, 0, kv, s32)
    oh, ohn = o.select_victims(idx, now, 1, kv, s32)
    op, opn = o.select_prefetch(idx, now, kp, s32)
    n_off = min(ovn, ohn)
    op = op.copy()
    op[:opn][np.isin(op[:opn], oh[:n_off])] = orc.ID_NONE
    as_u32 = lambda t, n: t.cpu().numpy().view(np.uint32)[:n]
    assert int(gvn[0].item()) == ovn and np.array_equal(as_u32(gv, ovn), ov[:ovn])
    assert int(ghn[0].item()) == ohn and np.array_equal(as_u32(gh, ohn), oh[:ohn])
    assert int(gpn[0].item()) == opn and np.array_equal(as_u32(gp, opn), op[:opn])
    want_g, want_h = gpu_np.copy(), host_np.copy()
    orc.move_blocks(gpu_np, synth.BLOCK_MAJOR, G, want_h, synth.LAYER_MAJOR, Hs, L, chunk, ov[:n_off], oh[:n_off] - G)
    ok = op[:opn] != orc.ID_NONE
    orc.move_blocks(host_np, synth.LAYER_MAJOR, Hs, want_g, synth.BLOCK_MAJOR, G, L, chunk, op[:opn][ok] - G, free_np[:opn][ok])
    assert np.array_equal(host_t.numpy(), want_h) and np.array_equal(gpu.buf.cpu().numpy(), want_g)
    if with_stage and ovn:
        want_s = np.zeros(ks * L * 2 * chunk, np.uint8)
        orc.move_blocks(gpu_np, synth.BLOCK_MAJOR, G, want_s, synth.LAYER_MAJOR, ks, L, chunk, ov[:ovn], np.arange(ovn))
        assert np.array_equal(stage.buf.cpu().numpy(), want_s)
    assert c.get_status() == 0
