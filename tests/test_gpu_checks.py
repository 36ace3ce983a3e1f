"""Failure detection, race detection and metrics of the library, all without faulting a GPU:
the bounded wait is made to run out by a self-test kernel that has nothing in flight, the list
checkers are shown lists that are wrong on purpose (host-made failures), the counters are compared
with what the oracle counts, and contexts of different shape share the kernels' shared-memory opt-in."""
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
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def warm(cfg, n_inv, max_blocks, **kw):
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=max_blocks,
                       block_tokens=cfg.block_tokens, **kw)
    c, o = cs.CacheScout(p, DEV), orc.Oracle(H.oracle_params(p))
    tr = synth.make_trace(cfg, n_invocations=n_inv)
    c.observe_invocations(dev(tr.chain), dev(tr.agent), dev(tr.evflags))
    o.observe(tr.chain, tr.agent, tr.evflags)
    return c, o, tr


def test_bounded_wait_runs_out_and_the_context_stays_usable():
    cfg = synth.CONFIGS["tiny"]
    c, _, _ = warm(cfg, 50, 64)
    assert c.get_status() == 0
    c.selftest_bounded_wait(1000)
    assert c.get_status() == cs.CS_ST_TIMEOUT           # the status path of a stalled transfer
    assert c.get_status() == 0
    # a normal transfer on the same context afterwards, byte for byte
    L, chunk, G = cfg.n_layers, cfg.chunk_bytes, 24
    rng = synth.rng_for(cfg, 41)
    src_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    a = cs.KVPool(dev(src_np), G, 0, L)
    host_t = torch.zeros(G * L * 2 * chunk, dtype=torch.uint8).pin_memory()
    b = cs.KVPool(host_t, G, 1, L)
    s, d = synth.mover_batch(9, G, G, rng)
    c.offload_blocks(a, b, dev(s), dev(d))
    torch.cuda.synchronize()
    want = np.zeros_like(src_np)
    orc.move_blocks(src_np, 0, G, want, 1, G, L, chunk, s, d)
    assert np.array_equal(host_t.numpy(), want)
    assert c.get_status() == 0
    with pytest.raises(cs.CacheScoutError):
        c.selftest_bounded_wait(0)


@pytest.mark.parametrize("path", [cs.CS_SELECT_CLUSTER, cs.CS_SELECT_MULTI])
def test_selection_checker_accepts_the_oracle_list_and_catches_every_kind_of_damage(path):
    cfg = synth.CONFIGS["llama8b"]
    n, k = 30_000 + 11, 500
    c, o, _ = warm(cfg, 1000, n, r_min=0.02)
    c.set_select_path(path)
    idx = synth.make_block_index(cfg, n=n)
    d = cs.DeviceIndex.from_host(idx, DEV)
    now = 100_000
    s64, s32 = o.scores(idx, now)
    for prefetch, tier in ((False, 0), (False, 1), (True, 1)):
        ids_o, n_o = (o.select_prefetch(idx, now, k, s32) if prefetch else o.select_victims(idx, now, tier, k, s32))
        assert n_o == k
        good = dev(ids_o.copy())
        cnt = dev(np.array([n_o, 0, 0, 0], np.uint32))
        c.validate_selection(d, now, prefetch, tier, k, good, cnt)          # the oracle's own list passes
        assert c.get_status() == 0
        damaged = []
        x = ids_o.copy(); x[[10, 11]] = x[[11, 10]]; damaged.append((x, n_o, "order"))
        x = ids_o.copy(); x[7] = x[6]; damaged.append((x, n_o, "duplicate"))
        x = ids_o.copy(); x[3] = n + 5; damaged.append((x, n_o, "id out of range"))
        pinned = np.flatnonzero(idx.flags & synth.FLAG_PINNED)[0]
        x = ids_o.copy(); x[0] = pinned; damaged.append((x, n_o, "ineligible entry"))
        x = ids_o.copy(); x[-1] = orc.ID_NONE; damaged.append((x, n_o - 1, "one entry short"))
        # the (k+1)-th best in place of the k-th: ordered, unique, eligible, but not the k best
        ids_k1, _ = (o.select_prefetch(idx, now, k + 1, s32) if prefetch else o.select_victims(idx, now, tier, k + 1, s32))
        x = ids_o.copy(); x[-1] = ids_k1[-1]; damaged.append((x, n_o, "a better entry left out"))
        x = ids_o.copy(); damaged.append((x, n_o + 1, "count beyond k"))
        for lst, cnt_v, what in damaged:
            c.validate_selection(d, now, prefetch, tier, k, dev(lst), dev(np.array([cnt_v, 0, 0, 0], np.uint32)))
            assert c.get_status() & cs.CS_ST_BAD_SELECTION, what
        c.validate_selection(d, now, prefetch, tier, k, good, cnt)          # and the checker's own state was left clean
        assert c.get_status() == 0
    # fewer eligible entries than k: the list must hold all of them
    small = synth.make_block_index(cfg, n=700)
    ds = cs.DeviceIndex.from_host(small, DEV)
    ids, cnt = c.select_victims(ds, now, 0, 2000)
    c.validate_selection(ds, now, False, 0, 2000, ids, cnt)
    assert c.get_status() == 0
    cnt2 = cnt.clone(); cnt2 -= 1
    ids2 = ids.clone(); ids2[int(cnt.item()) - 1] = -1
    c.validate_selection(ds, now, False, 0, 2000, ids2, cnt2)
    assert c.get_status() & cs.CS_ST_BAD_SELECTION


def test_list_checker_reports_slots_used_twice():
    cfg = synth.CONFIGS["tiny"]
    c, _, _ = warm(cfg, 20, 64)
    L, G, Hs = cfg.n_layers, 64, 64
    gpu = cs.KVPool(torch.zeros(G * cfg.block_bytes, dtype=torch.uint8, device=DEV), G, 0, L)
    gpu2 = cs.KVPool(torch.zeros(G * cfg.block_bytes, dtype=torch.uint8, device=DEV), G, 1, L)
    host = cs.KVPool(torch.zeros(Hs * cfg.block_bytes, dtype=torch.uint8).pin_memory(), Hs, 1, L)
    u = lambda *v: dev(np.array(v, np.uint32))
    NONE = orc.ID_NONE
    ok = lambda: c.get_status() == 0
    bad = lambda: c.get_status() == cs.CS_ST_LIST_CONFLICT
    c.validate_move_lists(gpu, host, u(1, 2, 3), u(5, 6, 7)); assert ok()
    c.validate_move_lists(gpu, host, u(1, 2, 3), u(5, 6, 5)); assert bad()                    # one destination twice
    c.validate_move_lists(gpu, host, u(1, NONE, 3), u(5, 6, 5)); assert bad()
    c.validate_move_lists(gpu, host, u(1, 2, NONE), u(5, 6, 5)); assert ok()                  # the mover skips that entry
    c.validate_move_lists(gpu, host, u(1, 2, 3), u(5, 6, 5), n_dev=u(2, 0, 0, 0)); assert ok()  # beyond the device count
    c.validate_move_lists(gpu, gpu2, u(1, 2, 3), u(3, 4, 5)); assert ok()                     # two pools: no overlap rule
    c.validate_move_lists(gpu, gpu, u(1, 2, 3), u(3, 4, 5)); assert bad()                     # one pool: slot 3 read and written
    c.validate_move_lists(gpu, gpu, u(1, 2, 3), u(7, 8, 9)); assert ok()
    # a list longer than one tile of the checker, conflict between its two ends
    big_dst = np.arange(1000, dtype=np.uint32); big_dst[999] = 0
    c.validate_move_lists(gpu, host, dev(np.arange(1000, dtype=np.uint32)), dev(big_dst)); assert bad()
    # two-way transfer: a host slot written by the offload and read by the prefetch; a GPU slot the other way round
    c.validate_exchange_lists(gpu, host, u(1, 2), u(10, 11), u(20, 21), u(30, 31)); assert ok()
    c.validate_exchange_lists(gpu, host, u(1, 2), u(10, 11), u(20, 11), u(30, 31)); assert bad()
    c.validate_exchange_lists(gpu, host, u(1, 2), u(10, 11), u(20, 21), u(30, 2)); assert bad()
    c.validate_exchange_lists(gpu, host, u(1, 2), u(10, 10), None, None); assert bad()
    c.validate_exchange_lists(gpu, host, None, None, u(20, 21), u(30, 30)); assert bad()
    c.validate_exchange_lists(gpu, host, None, None, u(20, 21), u(30, 31)); assert ok()


def test_counters_agree_with_the_oracle_and_the_lists():
    cfg = synth.CONFIGS["tiny"]
    n = 2560
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=n, block_tokens=cfg.block_tokens, r_min=0.02)
    c, o = cs.CacheScout(p, DEV), orc.Oracle(H.oracle_params(p))
    tr = synth.make_trace(cfg, n_invocations=200, warmup_frac=0.1)
    agent = tr.agent.copy(); agent[17] = cfg.n_agents + 1          # one bad id: skipped
    c.observe_invocations(dev(tr.chain), dev(agent), dev(tr.evflags))
    o.observe(tr.chain, agent, tr.evflags)
    assert c.get_status() == cs.CS_ST_BAD_AGENT
    cn = c.counters()
    assert cn["events_seen"] == 200
    n_warm = int(np.count_nonzero(tr.evflags & synth.EV_WARMUP))
    assert cn["events_skipped"] == n_warm + (0 if tr.evflags[17] & synth.EV_WARMUP else 1)
    assert cn["transitions_counted"] == int(o.C.sum())
    idx = synth.make_block_index(cfg, n=n)
    d = cs.DeviceIndex.from_host(idx, DEV)
    now = 100_000
    elig = lambda tier: int(np.count_nonzero(((idx.flags & 7) == (1 | (tier << 2))) & (idx.ref_count == 0)))
    i32 = lambda m: torch.zeros(max(m, 4), dtype=torch.int32, device=DEV)
    gv, gh, gp, gvn, ghn, gpn = i32(32), i32(32), i32(64), i32(1), i32(1), i32(1)
    c.select_step(d, now, 32, 64, gv, gvn, gh, ghn, gp, gpn)
    c.set_select_path(cs.CS_SELECT_MULTI)
    ids, cnt = c.select_victims(d, now, 0, 2560)                    # more than there are eligible entries
    cn = c.counters()
    assert cn["selects"] == [2, 1, 1]
    assert cn["eligible"][0] == elig(0) and cn["eligible"][1] == elig(1)
    assert cn["selected"] == [32 + int(cnt.item()), 32, int(gpn[0].item())]
    assert int(cnt.item()) == elig(0)
    # mover: blocks and bytes per direction, skipped entries
    L, G = cfg.n_layers, cfg.gpu_blocks
    gpu = cs.KVPool(torch.zeros(G * cfg.block_bytes, dtype=torch.uint8, device=DEV), G, 0, L)
    host = cs.KVPool(torch.zeros(64 * cfg.block_bytes, dtype=torch.uint8).pin_memory(), 64, 1, L)
    lst = gv[:32].clone(); lst[3] = -1                              # a sentinel
    c.offload_blocks(gpu, host, lst, dev(np.arange(32, dtype=np.uint32)), n_max=32, n_dev=gvn)
    c.prefetch_blocks(host, gpu, dev(np.arange(8, dtype=np.uint32)), dev(np.arange(8, dtype=np.uint32)))
    c.compact_blocks(gpu, gpu, dev(np.arange(100, 105, dtype=np.uint32)), dev(np.array([200, 201, 202, 203, G + 9], np.uint32)))
    c.exchange_blocks(gpu, host, dev(np.arange(40, 46, dtype=np.uint32)), dev(np.arange(40, 46, dtype=np.uint32)),
                      dev(np.arange(3, dtype=np.uint32)), dev(np.arange(300, 303, dtype=np.uint32)))
    torch.cuda.synchronize()
    assert c.get_status() == cs.CS_ST_BAD_SLOT
    cn = c.counters(reset=True)
    assert cn["blocks_moved"] == [4, 31 + 6, 8 + 3]
    assert cn["bytes_moved"] == [m * cfg.block_bytes for m in cn["blocks_moved"]]
    assert cn["blocks_skipped"] == 2
    z = c.counters()
    assert z["events_seen"] == 0 and z["blocks_moved"] == [0, 0, 0] and z["selects"] == [0, 0, 0]


def test_contexts_of_different_shape_share_the_select_kernels():
    """The shared-memory opt-in of the cluster select belongs to the kernel, not to a context: a context with
    few agents must not shrink it under a live context with many (and a longer recency table)."""
    now = 100_000
    big_cfg = synth.shrink(synth.CONFIGS["meta1m"], n_chains=4, sessions=4)
    small_cfg = synth.CONFIGS["tiny"]
    c1, o1, _ = warm(big_cfg, 600, 60_000, lam=0.0056)               # 256 agents, table of ~4,040 ages
    idx1 = synth.make_block_index(big_cfg, n=60_000)
    d1 = cs.DeviceIndex.from_host(idx1, DEV)

    def check(c, o, idx, d, k):
        s64, s32 = o.scores(idx, now)
        for tier in (0, 1):
            ids, cnt = c.select_victims(d, now, tier, k)
            oi, on = o.select_victims(idx, now, tier, k, s32)
            assert H.assert_list_matches(ids.cpu().numpy().view(np.uint32)[:k], int(cnt.item()), oi, on, s64) == 0
        i32 = lambda m: torch.zeros(max(m, 4), dtype=torch.int32, device=DEV)
        gv, gh, gp, gvn, ghn, gpn = i32(k), i32(k), i32(k), i32(1), i32(1), i32(1)
        c.select_step(d, now, k, k, gv, gvn, gh, ghn, gp, gpn)
        oi, on = o.select_prefetch(idx, now, k, s32)
        assert H.assert_list_matches(gp.cpu().numpy().view(np.uint32)[:k], int(gpn[0].item()), oi, on, s64) == 0
        assert c.get_status() == 0

    check(c1, o1, idx1, d1, 300)
    c2, o2, _ = warm(small_cfg, 100, 3000, lam=0.1)                   # 4 agents, short table
    idx2 = synth.make_block_index(small_cfg, n=3000)
    d2 = cs.DeviceIndex.from_host(idx2, DEV)
    check(c2, o2, idx2, d2, 64)
    check(c1, o1, idx1, d1, 300)                                      # the first context again
    c3, o3, _ = warm(synth.shrink(synth.CONFIGS["llama70b"], n_agents=1024, transitions=("sparse", 4)), 300, 20_000, lam=0.0056)
    idx3 = synth.make_block_index(synth.shrink(synth.CONFIGS["llama70b"], n_agents=1024), n=20_000)
    check(c3, o3, idx3, cs.DeviceIndex.from_host(idx3, DEV), 100)     # the largest shape there is
    check(c2, o2, idx2, d2, 64)
    check(c1, o1, idx1, d1, 300)


def test_status_bits_set_between_two_reads_are_not_lost():
    cfg = synth.CONFIGS["tiny"]
    c, _, _ = warm(cfg, 20, 64)
    side = torch.cuda.Stream(device=DEV)
    for _ in range(20):
        c.selftest_bounded_wait(50, stream=side)                     # sets the bit on the side stream ...
        a = c.get_status()                                            # ... while the main stream reads and clears
        side.synchronize()
        b = c.get_status()
        assert (a | b) == cs.CS_ST_TIMEOUT                            # seen exactly once or twice, never dropped


def test_clock_read_from_device_memory_when_the_kernels_run():
    """cs_set_device_clock: the select takes `now` from a device word at execution time (what a captured
    CUDA graph needs), on both select paths, and goes back to its argument afterwards."""
    cfg = synth.CONFIGS["llama8b"]
    n, k = 40_000 + 3, 300
    c, o, _ = warm(cfg, 800, n, r_min=0.02)
    idx = synth.make_block_index(cfg, n=n)
    d = cs.DeviceIndex.from_host(idx, DEV)
    clock = torch.zeros(4, dtype=torch.int32, device=DEV)
    c.set_device_clock(clock)
    for path in (cs.CS_SELECT_CLUSTER, cs.CS_SELECT_MULTI):
        c.set_select_path(path)
        for now in (100_000, 100_777):
            clock.fill_(now)
            s64, s32 = o.scores(idx, now)
            ids, cnt = c.select_victims(d, 5, 0, k)                       # the argument (5) is ignored
            oi, on = o.select_victims(idx, now, 0, k, s32)
            assert H.assert_list_matches(ids.cpu().numpy().view(np.uint32)[:k], int(cnt.item()), oi, on, s64) == 0
            assert np.array_equal(c.score_blocks(d, 5).cpu().numpy(), s32)
    c.set_device_clock(None)
    s64, s32 = o.scores(idx, 100_100)
    ids, cnt = c.select_victims(d, 100_100, 0, k)
    oi, on = o.select_victims(idx, 100_100, 0, k, s32)
    assert H.assert_list_matches(ids.cpu().numpy().view(np.uint32)[:k], int(cnt.item()), oi, on, s64) == 0
    with pytest.raises(cs.CacheScoutError):
        c.set_device_clock(torch.zeros(4, dtype=torch.int32))                # pageable host memory: refused
    assert c.get_status() == 0


def test_phase_stamps_need_the_profiling_build():
    """cs_debug_phase_stamps() belongs to builds with -DCS_PHASE_STAMPS; the ordinary library says so and stores nothing."""
    cfg = synth.CONFIGS["tiny"]
    c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=64, block_tokens=cfg.block_tokens), DEV)
    with pytest.raises(cs.CacheScoutError) as e:
        c.phase_stamps()
    assert e.value.code == cs.CS_ENOTIMPL
