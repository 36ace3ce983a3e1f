"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Counts, tables, lists and copied bytes are compared bit-exactly;
fp32 scores within 1e-6 relative of the fp64 oracle."""
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


def make_ctx(cfg, max_blocks, **kw):
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=max_blocks,
                       block_tokens=cfg.block_tokens, **kw)
    return cs.CacheScout(p, DEV), orc.Oracle(H.oracle_params(p))


def feed_trace(c, o, tr, steps=None, check_every=0):
    n_steps = len(tr.step_off) - 1 if steps is None else steps
    for s in range(n_steps):
        lo, hi = int(tr.step_off[s]), int(tr.step_off[s + 1])
        c.observe_invocations(dev(tr.chain[lo:hi]), dev(tr.agent[lo:hi]), dev(tr.evflags[lo:hi]))
        o.observe(tr.chain[lo:hi], tr.agent[lo:hi], tr.evflags[lo:hi])
        if check_every and s % check_every == 0:
            H.compare_model(c, o)


# ---- learner + scorer state ---------------------------------------------------------------------------
@pytest.mark.parametrize("name,n_inv,chain_mode", [
    ("tiny", 200, "session"), ("llama8b", 3000, "session"), ("llama8b", 3000, "single"),
    ("llama70b", 4000, "session"), ("meta1m", 6400, "session")])
def test_model_parity_stepwise(name, n_inv, chain_mode):
    cfg = synth.CONFIGS[name]
    if chain_mode == "single":                      # the paper's single current-agent register
        cfg = synth.shrink(cfg, n_chains=1)
    tr = synth.make_trace(cfg, n_invocations=n_inv, warmup_frac=0.05)
    c, o = make_ctx(cfg, 64)
    H.compare_model(c, o)                           # initial state: uniform matrix, no current agent
    n_steps = len(tr.step_off) - 1
    feed_trace(c, o, tr, check_every=max(1, n_steps // 25))
    H.compare_model(c, o)
    assert c.get_status() == 0


def test_model_big_batches_and_bad_ids():
    cfg = synth.shrink(synth.CONFIGS["llama70b"], n_chains=7)
    tr = synth.make_trace(cfg, n_invocations=5000, warmup_frac=0.1)
    c, o = make_ctx(cfg, 64)
    agent = tr.agent.copy()
    chain = tr.chain.copy()
    agent[100] = cfg.n_agents + 3                   # skipped, status bit set
    chain[2500] = 7
    for lo, hi in ((0, 1), (1, 2400), (2400, 5000)):   # batches above the 1024-event shared-memory tile
        c.observe_invocations(dev(chain[lo:hi]), dev(agent[lo:hi]), dev(tr.evflags[lo:hi]))
        o.observe(chain[lo:hi], agent[lo:hi], tr.evflags[lo:hi])
    H.compare_model(c, o)
    assert c.get_status() == (cs.CS_ST_BAD_AGENT | cs.CS_ST_BAD_CHAIN)
    assert c.get_status() == 0                      # cleared by the read
    c.observe_invocations(None, None, None, n_events=0)     # refresh only
    H.compare_model(c, o)


def test_worked_examples_on_gpu(golden):
    for fixture, A in (("worked_example_a.txt", 3), ("worked_example_b.txt", 4)):
        g = golden(fixture)
        trace = np.array(g["trace"][0], np.uint16)
        p = cs.make_params(n_agents=A, max_blocks=16)
        c = cs.CacheScout(p, DEV)
        c.observe_invocations(dev(np.zeros(len(trace), np.uint32)), dev(trace), None)
        m = c.get_model()
        assert abs(m["R"] - g["R"][0][0]) < 1e-5
        assert m["hops"].tolist() == [int(x) for x in g["E"][0]]
        assert np.allclose(m["fsurv"], np.array(g["ptilde"][0]) + 0.01, rtol=1e-6)


# ---- scores ----------------------------------------------------------------------------------------------
def warm_state(cfg, n_inv, max_blocks, **kw):
    tr = synth.make_trace(cfg, n_invocations=n_inv)
    c, o = make_ctx(cfg, max_blocks, **kw)
    c.observe_invocations(dev(tr.chain), dev(tr.agent), dev(tr.evflags))
    o.observe(tr.chain, tr.agent, tr.evflags)
    return c, o


@pytest.mark.parametrize("name,n", [("tiny", 2560), ("tiny", 37), ("llama8b", 80000), ("llama70b", 52000 + 5)])
@pytest.mark.parametrize("with_tokens", [True, False])
def test_score_parity(name, n, with_tokens):
    cfg = synth.CONFIGS[name]
    c, o = warm_state(cfg, 500, n)
    idx = synth.make_block_index(cfg, n=n, with_tokens=with_tokens)
    idx.last_access[::97] = 100_000 + 5             # in the future: age clamps to 0
    idx.last_access[1::89] = 3                      # far beyond saturation
    d = cs.DeviceIndex.from_host(idx, DEV)
    s = c.score_blocks(d, 100_000).cpu().numpy()
    s64, s32 = o.scores(idx, 100_000)
    assert np.all(np.abs(s - s64) <= H.REL_TOL * s64)
    assert np.array_equal(s, s32)
    # explicit sources (multi-source BFS), used for that call only
    src = np.array([0, cfg.n_agents - 1], np.uint16)
    s_b = c.score_blocks(d, 100_000, sources=dev(src)).cpu().numpy()
    o.survival(src)
    s64b, s32b = o.scores(idx, 100_000)
    o.survival()
    assert np.array_equal(s_b, s32b) and np.all(np.abs(s_b - s64b) <= H.REL_TOL * s64b)
    assert np.array_equal(c.score_blocks(d, 100_000).cpu().numpy(), s32)    # cached table untouched
    assert c.get_status() == 0


def test_score_slow_decay_uses_direct_path():
    """A decay rate so small that the recency table does not cover all unsaturated ages."""
    cfg = synth.CONFIGS["tiny"]
    c, o = warm_state(cfg, 200, 4096, lam=0.0007)
    idx = synth.make_block_index(cfg, n=4096)
    d = cs.DeviceIndex.from_host(idx, DEV)
    s = c.score_blocks(d, 100_000).cpu().numpy()
    s64, s32 = o.scores(idx, 100_000)
    assert np.all(np.abs(s - s64) <= H.REL_TOL * s64)
    assert np.mean(s == s32) > 0.999                # device exp vs libm exp may differ in the last fp64 bit


# ---- selections ---------------------------------------------------------------------------------------------
def run_selects(c, o, idx, now, ks, tiers=(0, 1)):
    d = cs.DeviceIndex.from_host(idx, DEV)
    s64, s32 = o.scores(idx, now)
    tolerated = 0
    for path, k in [(p_, k_) for p_ in (cs.CS_SELECT_CLUSTER, cs.CS_SELECT_MULTI, -1) for k_ in ks]:
        c.set_select_path(cs.CS_SELECT_MULTI if path == -1 else path)
        c.set_select_speculation(path != -1)          # -1: multi-launch path without the remembered threshold
        for tier in tiers:
            ids, n_out = c.select_victims(d, now, tier, k)
            ids2, n_out2 = c.select_victims(d, now, tier, k)           # determinism: identical on a second run
            g_ids, g_n = ids.cpu().numpy().view(np.uint32)[:k], int(n_out.item())
            assert np.array_equal(g_ids, ids2.cpu().numpy().view(np.uint32)[:k]) and g_n == int(n_out2.item())
            o_ids, o_n = o.select_victims(idx, now, tier, k, s32)
            tolerated += H.assert_list_matches(g_ids, g_n, o_ids, o_n, s64)
            c.validate_selection(d, now, False, tier, k, ids, n_out)        # the device-side checker agrees (status stays 0)
            sel = g_ids[:g_n].astype(np.int64)
            assert not np.any(idx.flags[sel] & synth.FLAG_PINNED) and np.all(idx.ref_count[sel] == 0)
        ids, n_out = c.select_prefetch(d, now, k)
        g_ids, g_n = ids.cpu().numpy().view(np.uint32)[:k], int(n_out.item())
        o_ids, o_n = o.select_prefetch(idx, now, k, s32)
        tolerated += H.assert_list_matches(g_ids, g_n, o_ids, o_n, s64)
        c.validate_selection(d, now, True, 1, k, ids, n_out)
    assert c.get_status() == 0
    return tolerated


@pytest.mark.parametrize("name,n,ks", [
    ("tiny", 2560, (1, 32, 64, 700, 2560)),
    ("tiny", 0, (4,)), ("tiny", 5, (1, 8)), ("tiny", 16, (3,)), ("tiny", 1029, (32, 1029)),
    ("llama8b", 80000, (256, 384, 5000)),
    ("llama70b", 52000, (256, 384)),
])
def test_select_parity(name, n, ks):
    cfg = synth.CONFIGS[name]
    c, o = warm_state(cfg, 1000, max(n, max(ks)), r_min=0.02)
    H.reject_fragile(o)
    assert o.gate
    idx = synth.make_block_index(cfg, n=n)
    assert run_selects(c, o, idx, 100_000, ks) == 0


def test_select_massive_ties_and_lru_case():
    """tau > 1 removes every edge: survival is flat and eviction must be exact LRU (Sec. 3.3),
    with most keys tied in score so that last_access and id decide."""
    cfg = synth.CONFIGS["llama8b"]
    c, o = warm_state(cfg, 1000, 40000, tau=1.5)
    idx = synth.make_block_index(cfg, n=40000, with_tokens=False)
    idx.last_access[:] = 100_000 - 3000 - (np.arange(40000) % 211) * 5        # all ages saturated
    assert run_selects(c, o, idx, 100_000, (1, 300, 4000, 40000)) == 0
    ids, n_out = c.select_victims(cs.DeviceIndex.from_host(idx, DEV), 100_000, 0, 300)
    sel = ids.cpu().numpy().view(np.uint32)[:int(n_out.item())].astype(np.int64)
    la = int(o.last_agent[0])
    rest = sel[idx.agent[sel] != la]                 # the current agent keeps its survival bonus
    assert np.all(np.diff(idx.last_access[rest].astype(np.int64)) >= 0)


def test_select_gate_closed_and_cold_start():
    cfg = synth.CONFIGS["tiny"]
    idx = synth.make_block_index(cfg, n=2560)
    c, o = warm_state(cfg, 200, 2560, r_min=5.0)     # gate can never open
    assert run_selects(c, o, idx, 100_000, (64,)) == 0
    c2, o2 = make_ctx(cfg, 2560, r_min=-1.0)          # gate open but no current agent yet
    assert run_selects(c2, o2, idx, 100_000, (64,)) == 0


def test_select_without_optional_tables_and_capacity_errors():
    cfg = synth.CONFIGS["llama70b"]
    c, o = warm_state(cfg, 2000, 9000, r_min=0.02)
    idx = synth.make_block_index(cfg, n=9000, with_tokens=False, with_anchor=False)
    assert run_selects(c, o, idx, 100_000, (100,)) == 0
    d = cs.DeviceIndex.from_host(idx, DEV)
    with pytest.raises(cs.CacheScoutError) as e:
        c.select_victims(d, 1, 0, 9001)
    assert e.value.code == cs.CS_ECAPACITY
    big = cs.DeviceIndex.from_host(synth.make_block_index(cfg, n=9016), DEV)
    with pytest.raises(cs.CacheScoutError) as e:
        c.select_victims(big, 1, 0, 4)
    assert e.value.code == cs.CS_ECAPACITY
    off = cs.DeviceIndex(d.agent[1:], d.depth, d.ref_count, d.flags, d.last_access)      # misaligned pointer
    with pytest.raises(cs.CacheScoutError) as e:
        c.select_victims(off, 1, 0, 4)
    assert e.value.code == cs.CS_EINVAL


def test_metadata_scale_first_calls():
    """1,000,000-entry index, 256 agents, k = 10,000 victims / 2,000 prefetch candidates, state evolving between
    calls (the launch configuration the benchmark times): every one of the first 100 calls against the oracle, then
    every 50th up to call 600 (between those the library's own lists advance the state, so a checked call also
    vouches for the calls before it), issued alternately as two calls and as one cs_select_step call."""
    cfg = synth.CONFIGS["meta1m"]
    N = 1_000_000
    n_calls = 601
    tr = synth.make_trace(cfg, n_invocations=64 * (n_calls + 8))
    c, o = make_ctx(cfg, N, r_min=0.02)
    idx = synth.make_block_index(cfg, n=N, tier="random")
    rng = synth.rng_for(cfg, 9)
    now0 = 100_000
    checked = 0
    v_ids = torch.empty(cfg.k_victims, dtype=torch.int32, device=DEV)
    p_ids = torch.empty(cfg.k_prefetch, dtype=torch.int32, device=DEV)
    v_n, p_n = torch.zeros(4, dtype=torch.int32, device=DEV), torch.zeros(4, dtype=torch.int32, device=DEV)
    d = cs.DeviceIndex.from_host(idx, DEV)
    for call in range(n_calls):
        lo, hi = int(tr.step_off[call * 4]), int(tr.step_off[call * 4 + 4])
        c.observe_invocations(dev(tr.chain[lo:hi]), dev(tr.agent[lo:hi]), None)
        o.observe(tr.chain[lo:hi], tr.agent[lo:hi])
        now = now0 + call
        for name in ("agent", "depth", "ref_count", "flags", "last_access"):       # the evolved index, same device arrays
            getattr(d, name).copy_(torch.from_numpy(getattr(idx, name)))
        if call % 2:
            c.select_step(d, now, cfg.k_victims, cfg.k_prefetch, v_ids, v_n, None, None, p_ids, p_n)
        else:
            c.select_victims(d, now, 0, cfg.k_victims, v_ids, v_n)
            c.select_prefetch(d, now, cfg.k_prefetch, p_ids, p_n)
        gv, gp = v_ids.cpu().numpy().view(np.uint32)[:cfg.k_victims], p_ids.cpu().numpy().view(np.uint32)[:cfg.k_prefetch]
        if call < 100 or call % 50 == 0:
            s64, s32 = o.scores(idx, now)
            ov, ovn = o.select_victims(idx, now, 0, cfg.k_victims, s32)
            op, opn = o.select_prefetch(idx, now, cfg.k_prefetch, s32)
            assert H.assert_list_matches(gv, int(v_n[0].item()), ov, ovn, s64) == 0, call
            assert H.assert_list_matches(gp, int(p_n[0].item()), op, opn, s64) == 0, call
            checked += 1
        synth.mutate_index(idx, rng, now, gv, gp, int(o.last_agent[0]), cfg.n_agents)
    assert checked == 100 + 11
    H.compare_model(c, o)
    cn = c.counters()
    assert cn["selects"][0] == n_calls and cn["selects"][2] == n_calls
    assert cn["fast_hits"][0] > n_calls // 2                  # the remembered threshold holds in most calls
    assert c.get_status() == 0


# ---- mover -----------------------------------------------------------------------------------------------------
def pinned_zeros(nbytes):
    return torch.zeros(nbytes, dtype=torch.uint8).pin_memory()


PATHS = [cs.CS_MOVER_BULK, cs.CS_MOVER_LDST]


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("gpu_layout", [synth.LAYER_MAJOR, synth.BLOCK_MAJOR])
@pytest.mark.parametrize("host_layout", [synth.BLOCK_MAJOR, synth.LAYER_MAJOR])
def test_mover_offload_prefetch_compact(gpu_layout, host_layout, path):
    cfg = synth.CONFIGS["tiny"]
    L, chunk, G, Hs = cfg.n_layers, cfg.chunk_bytes, 96, 160
    rng = synth.rng_for(cfg, 5)
    c, _ = make_ctx(cfg, 64)
    c.set_mover_path(path)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, gpu_layout, L)
    host_t = pinned_zeros(Hs * L * 2 * chunk)
    host = cs.KVPool(host_t, Hs, host_layout, L)
    host_np = np.zeros(Hs * L * 2 * chunk, np.uint8)

    n = 41
    src, dst = synth.mover_batch(n, G, Hs, rng)
    src[5] = orc.ID_NONE                                       # sentinel: skipped
    side = torch.cuda.Stream(device=DEV)
    n_dev = dev(np.array([37, 0, 0, 0], np.uint32))            # device-resident count below n_max
    side.wait_stream(torch.cuda.current_stream())
    c.offload_blocks(gpu, host, dev(src), dev(dst), n_dev=n_dev, stream=side)
    side.synchronize()
    orc.move_blocks(gpu_np, gpu_layout, G, host_np, host_layout, Hs, L, chunk, src[:37], dst[:37])
    assert np.array_equal(host_t.numpy(), host_np)

    # prefetch the same blocks back into other GPU slots, byte-for-byte
    back = rng.choice(G, size=37, replace=False).astype(np.uint32)
    c.prefetch_blocks(host, gpu, dev(dst[:37]), dev(back), stream=side)
    side.synchronize()
    want = gpu_np.copy()
    orc.move_blocks(host_np, host_layout, Hs, want, gpu_layout, G, L, chunk, dst[:37], back)
    got = gpu.buf.cpu().numpy()
    assert np.array_equal(got, want)
    ok = src[:37] != orc.ID_NONE
    assert np.array_equal(H.pool_view(got, gpu_layout, G, L, chunk)[back[ok]],
                          H.pool_view(gpu_np, gpu_layout, G, L, chunk)[src[:37][ok]])

    # device-to-device compaction into a packed staging pool of the other layout
    stage = cs.KVPool(torch.zeros(n * L * 2 * chunk, dtype=torch.uint8, device=DEV), n, 1 - gpu_layout, L)
    s2, d2 = synth.mover_batch(n, G, n, rng, packed_dst=True)
    c.compact_blocks(gpu, stage, dev(s2), dev(d2))
    torch.cuda.synchronize()
    want_s = np.zeros(n * L * 2 * chunk, np.uint8)
    orc.move_blocks(got, gpu_layout, G, want_s, 1 - gpu_layout, n, L, chunk, s2, d2)
    assert np.array_equal(stage.buf.cpu().numpy(), want_s)
    assert c.get_status() == 0

    # an out-of-range slot is skipped and reported, nothing else is touched
    bad_src = src.copy()
    bad_src[0] = G
    before = host_t.numpy().copy()
    c.offload_blocks(gpu, host, dev(bad_src[:1]), dev(dst[:1]), stream=side)
    side.synchronize()
    assert c.get_status() == cs.CS_ST_BAD_SLOT
    assert np.array_equal(host_t.numpy(), before)


@pytest.mark.parametrize("path", PATHS)
def test_mover_small_chunks_and_geometry_errors(path):
    """Chunks that are not a whole number of 16 KiB pieces, and a one-block batch."""
    cfg = synth.CONFIGS["tiny"]
    c, _ = make_ctx(cfg, 64)
    c.set_mover_path(path)
    rng = synth.rng_for(cfg, 6)
    for heads, hd, tok in ((3, 40, 16), (8, 128, 16), (1, 8, 1), (5, 128, 9)):
        chunk = tok * heads * hd * 2
        L, G = 3, 17
        src_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
        a = cs.KVPool(dev(src_np), G, 0, L, heads, hd, tok)
        b = cs.KVPool(torch.zeros(G * L * 2 * chunk, dtype=torch.uint8, device=DEV), G, 1, L, heads, hd, tok)
        s, d = synth.mover_batch(1 if heads == 1 else 9, G, G, rng)
        c.compact_blocks(a, b, dev(s), dev(d))
        want = np.zeros_like(src_np)
        orc.move_blocks(src_np, 0, G, want, 1, G, L, chunk, s, d)
        assert np.array_equal(b.buf.cpu().numpy(), want)
    bad = cs.KVPool(b.buf, G, 1, L + 1, heads, hd, tok)
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_compact_blocks(c.ctx, a.struct(), cs.cs_kv_pool(bad.buf.data_ptr(), G, 1, L + 1, heads, hd, tok, 2, 0),
                             dev(s), dev(d), 1)
    assert e.value.code == cs.CS_EINVAL
    # a pool in pageable host memory is refused on the host: nothing is launched, the device never sees the address
    pageable = torch.zeros(G * L * 2 * chunk + 64, dtype=torch.uint8)
    ptr = (pageable.data_ptr() + 15) & ~15
    l_before = c.launch_count()
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_offload_blocks(c.ctx, a.struct(), cs.cs_kv_pool(ptr, G, 1, L, heads, hd, tok, 2, 0), dev(s), dev(d), 1)
    assert e.value.code == cs.CS_EINVAL and c.launch_count() == l_before
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_exchange_blocks(c.ctx, a.struct(), cs.cs_kv_pool(ptr, G, 1, L, heads, hd, tok, 2, 0), dev(s), dev(d), 1, None,
                              dev(d), dev(s), 1, None)
    assert e.value.code == cs.CS_EINVAL and c.launch_count() == l_before
    odd = cs.cs_kv_pool(a.buf.data_ptr(), G, 0, L, 1, 3, 1, 2, 0)          # 6-byte chunks: not 16-byte multiples
    with pytest.raises(cs.CacheScoutError):
        cs.cs_compact_blocks(c.ctx, odd, odd, dev(s), dev(d), 1)


@pytest.mark.parametrize("gpu_layout,host_layout", [(0, 1), (1, 0)])
@pytest.mark.parametrize("n_off,n_pre,width", [(41, 67, 0), (50, 0, 3), (0, 33, 0), (1, 1, 64), (37, 5, 7)])
def test_exchange_matches_offload_then_prefetch(gpu_layout, host_layout, n_off, n_pre, width):
    """Both directions in one launch: byte-exact against the oracle's two transfers on disjoint slots,
    for uneven list lengths, empty lists, device-resident counts and sentinels."""
    cfg = synth.CONFIGS["tiny"]
    L, chunk, G, Hs = cfg.n_layers, cfg.chunk_bytes, 160, 200
    rng = synth.rng_for(cfg, 15)
    c, _ = make_ctx(cfg, 64)
    c.set_mover_ctas(width, 0)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    host_np = synth.kv_pool_u16(Hs, L, chunk, rng).view(np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, gpu_layout, L)
    host_t = pinned_zeros(Hs * L * 2 * chunk)
    host_t.numpy()[:] = host_np
    host = cs.KVPool(host_t, Hs, host_layout, L)
    g_perm = rng.permutation(G).astype(np.uint32)              # disjoint GPU slots: sources then destinations
    h_perm = rng.permutation(Hs).astype(np.uint32)
    off_src, pre_dst = g_perm[:n_off].copy(), g_perm[n_off:n_off + n_pre].copy()
    off_dst, pre_src = h_perm[:n_off].copy(), h_perm[n_off:n_off + n_pre].copy()
    m_off, m_pre = n_off, n_pre
    if n_off > 8:
        off_src[3] = orc.ID_NONE                                # skipped
        m_off = n_off - 4                                       # device-resident count below n_max
    if n_pre > 8:
        pre_dst[2] = orc.ID_NONE
        m_pre = n_pre - 1
    side = torch.cuda.Stream(device=DEV)
    side.wait_stream(torch.cuda.current_stream())
    c.exchange_blocks(gpu, host, dev(off_src) if n_off else None, dev(off_dst) if n_off else None,
                      dev(pre_src) if n_pre else None, dev(pre_dst) if n_pre else None,
                      n_off_dev=dev(np.array([m_off], np.uint32)) if n_off else None,
                      n_pre_dev=dev(np.array([m_pre], np.uint32)) if n_pre else None, stream=side)
    side.synchronize()
    want_h, want_g = host_np.copy(), gpu_np.copy()
    orc.move_blocks(gpu_np, gpu_layout, G, want_h, host_layout, Hs, L, chunk, off_src[:m_off], off_dst[:m_off])
    orc.move_blocks(host_np, host_layout, Hs, want_g, gpu_layout, G, L, chunk, pre_src[:m_pre], pre_dst[:m_pre])
    assert np.array_equal(host_t.numpy(), want_h)
    assert np.array_equal(gpu.buf.cpu().numpy(), want_g)
    assert c.get_status() == 0


@pytest.mark.parametrize("gpu_layout", [0, 1])
@pytest.mark.parametrize("n_off,n_pre,ring_blocks", [(41, 67, 3), (50, 0, 1), (0, 33, 2), (1, 1, 64), (37, 5, 7), (64, 64, 16)])
def test_staged_exchange_matches_the_oracle(gpu_layout, n_off, n_pre, ring_blocks):
    """The copy-engine path (pack -> cudaMemcpyAsync -> host, host -> cudaMemcpyAsync -> scatter) against the
    oracle's two transfers: rings of 1 to 64 blocks per sub-buffer (many parts, double buffering, a ragged last
    part), runs of consecutive host ids (merged copies) next to scattered ones, sentinels on either side."""
    cfg = synth.CONFIGS["tiny"]
    L, chunk, G, Hs, first_h = cfg.n_layers, cfg.chunk_bytes, 160, 200, 1000
    bb = cfg.block_bytes
    rng = synth.rng_for(cfg, 15 + ring_blocks)
    c, _ = make_ctx(cfg, 64)
    ring = torch.empty(4 * ring_blocks * bb + 256, dtype=torch.uint8, device=DEV)
    c.set_mover_staging(ring)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    host_np = synth.kv_pool_u16(Hs, L, chunk, rng).view(np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, gpu_layout, L)
    host_t = pinned_zeros(Hs * bb)
    host_t.numpy()[:] = host_np
    host = cs.KVPool(host_t, Hs, synth.BLOCK_MAJOR, L, first_id=first_h)
    g_perm = rng.permutation(G).astype(np.uint32)
    off_src, pre_dst = g_perm[:n_off].copy(), g_perm[n_off:n_off + n_pre].copy()
    # host slots: the first half of each list is one run of consecutive slots, the rest scattered
    h_free = rng.permutation(np.arange(Hs // 2, Hs)).astype(np.uint32)
    run_o, run_p = n_off // 2, n_pre // 2
    off_dst = np.concatenate([np.arange(run_o, dtype=np.uint32), h_free[:n_off - run_o]])
    pre_src = np.concatenate([np.arange(run_o, run_o + run_p, dtype=np.uint32), h_free[n_off - run_o:n_off - run_o + n_pre - run_p]])
    unspecified = []
    if n_off > 8:
        unspecified.append(int(off_dst[6]))
        off_src[6] = orc.ID_NONE                                # skipped on the device: that host slot gets unspecified bytes
    if n_pre > 8:
        pre_dst[2] = orc.ID_NONE                                # skipped on the device
    side = torch.cuda.Stream(device=DEV)
    side.wait_stream(torch.cuda.current_stream())
    ids = lambda a: np.where(a == orc.ID_NONE, a, a + np.uint32(first_h))
    c.exchange_blocks_staged(gpu, host, dev(off_src) if n_off else None, ids(off_dst) if n_off else None,
                             ids(pre_src) if n_pre else None, dev(pre_dst) if n_pre else None, stream=side)
    side.synchronize()
    want_h, want_g = host_np.copy(), gpu_np.copy()
    orc.move_blocks(gpu_np, gpu_layout, G, want_h, synth.BLOCK_MAJOR, Hs, L, chunk, off_src, off_dst)
    orc.move_blocks(host_np, synth.BLOCK_MAJOR, Hs, want_g, gpu_layout, G, L, chunk, pre_src, pre_dst)
    got_h = host_t.numpy().copy()
    for slot in unspecified:
        got_h[slot * bb:(slot + 1) * bb] = want_h[slot * bb:(slot + 1) * bb]
    assert np.array_equal(got_h, want_h)
    assert np.array_equal(gpu.buf.cpu().numpy(), want_g)
    cn = c.counters()
    assert cn["blocks_moved"][1] == np.count_nonzero(off_src != orc.ID_NONE)
    assert cn["blocks_moved"][2] == np.count_nonzero(pre_dst != orc.ID_NONE)
    assert c.get_status() == 0
    # a second transfer right behind the first on the same stream reuses the ring safely: move everything back
    if n_off and n_pre == 0:
        keep = np.ones(n_off, bool)
        back = off_src
        cs.cs_prefetch_blocks_staged(c.ctx, host.struct(), gpu.struct(), ids(off_dst[keep]), dev(back[keep]),
                                     int(keep.sum()), stream=side)
        side.synchronize()
        ok = keep & (off_src != orc.ID_NONE)
        assert np.array_equal(H.pool_view(gpu.buf.cpu().numpy(), gpu_layout, G, L, chunk)[off_src[ok]],
                              H.pool_view(gpu_np, gpu_layout, G, L, chunk)[off_src[ok]])
    # errors: no ring, host ids out of range, a layer-major host pool
    with pytest.raises(cs.CacheScoutError) as e:
        c.exchange_blocks_staged(gpu, host, dev(g_perm[:1]), np.array([first_h + Hs], np.uint32), None, None)
    assert e.value.code == cs.CS_EINVAL
    with pytest.raises(cs.CacheScoutError) as e:             # a sentinel in a host list: the device could not know of the skip
        c.exchange_blocks_staged(gpu, host, dev(g_perm[:1]), np.array([orc.ID_NONE], np.uint32), None, None)
    assert e.value.code == cs.CS_EINVAL
    bad_host = cs.KVPool(host_t, Hs, synth.LAYER_MAJOR, L, first_id=first_h)
    with pytest.raises(cs.CacheScoutError) as e:
        c.exchange_blocks_staged(gpu, bad_host, dev(g_perm[:1]), np.array([first_h], np.uint32), None, None)
    assert e.value.code == cs.CS_EINVAL
    c.set_mover_staging(None)
    with pytest.raises(cs.CacheScoutError) as e:
        c.exchange_blocks_staged(gpu, host, dev(g_perm[:1]), np.array([first_h], np.uint32), None, None)
    assert e.value.code == cs.CS_EINVAL
    tiny_ring = torch.empty(2 * bb, dtype=torch.uint8, device=DEV)          # less than four blocks
    c.set_mover_staging(tiny_ring)
    with pytest.raises(cs.CacheScoutError) as e:
        c.exchange_blocks_staged(gpu, host, dev(g_perm[:1]), np.array([first_h], np.uint32), None, None)
    assert e.value.code == cs.CS_ECAPACITY


def test_offload_straight_from_select_output():
    """The victim list and its device-resident count drive the mover without a host round trip."""
    cfg = synth.CONFIGS["tiny"]
    L, chunk, G, Hs = cfg.n_layers, cfg.chunk_bytes, cfg.gpu_blocks, 64
    c, o = warm_state(cfg, 200, cfg.n_index)
    idx = synth.make_block_index(cfg)                            # ids [0,512) GPU tier, rest host tier
    d = cs.DeviceIndex.from_host(idx, DEV)
    rng = synth.rng_for(cfg, 7)
    gpu_np = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, synth.LAYER_MAJOR, L)
    host_t = pinned_zeros(Hs * L * 2 * chunk)
    host = cs.KVPool(host_t, Hs, synth.BLOCK_MAJOR, L)
    k = cfg.k_victims
    ids, n_out = c.select_victims(d, 100_000, 0, k)
    dst = dev(np.arange(k, dtype=np.uint32))
    c.offload_blocks(gpu, host, ids, dst, n_max=k, n_dev=n_out)
    torch.cuda.synchronize()
    o_ids, o_n = o.select_victims(idx, 100_000, 0, k)
    want = np.zeros(Hs * L * 2 * chunk, np.uint8)
    orc.move_blocks(gpu_np, synth.LAYER_MAJOR, G, want, synth.BLOCK_MAJOR, Hs, L, chunk, o_ids[:o_n], np.arange(o_n))
    assert np.array_equal(host_t.numpy(), want)
    assert c.get_status() == 0
    assert c.launch_count() > 0


# ---- exact survival probability (Eq. 6) as an alternative scorer -----------------------------------------
@pytest.mark.parametrize("name,K", [("tiny", 4), ("llama8b", 3), ("llama70b", 5), ("meta1m", 4)])
def test_exact_survival_parity_and_select(name, K):
    cfg = synth.CONFIGS[name]
    n = 20000
    c, o = warm_state(cfg, 3000, n, r_min=0.02)
    ps, fs = c.exact_survival(K)
    want = o.exact_survival(K)
    got = ps.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want) <= H.REL_TOL * np.maximum(want, 1e-3)), np.abs(got - want).max()
    assert np.all(np.abs(fs.cpu().numpy() - (want + float(np.float32(0.01)))) <= 2e-7 * (want + 0.01) + 1e-9)
    assert abs(float(want.sum()) - float(got.sum())) < 1e-4 and np.all(got >= 0) and np.all(got <= 1 + 1e-6)
    # explicit start agent, K = 1 is the row of the transition matrix
    ps1, _ = c.exact_survival(1, a0=2)
    assert np.allclose(ps1.cpu().numpy(), o.P64[2], rtol=1e-6, atol=1e-9)
    # selections driven by the exact table: same kernels, other first factor of Eq. 9
    idx = synth.make_block_index(cfg, n=n)
    d = cs.DeviceIndex.from_host(idx, DEV)
    c.use_survival_table(fs)
    o.ptilde = want.copy()
    o.fsurv32 = (want + float(np.float32(o.p.delta))).astype(np.float32)
    s64, s32 = o.scores(idx, 100_000)
    s = c.score_blocks(d, 100_000).cpu().numpy()
    assert np.all(np.abs(s - s64) <= H.REL_TOL * s64)
    for k in (64, 2000):
        ids, n_out = c.select_victims(d, 100_000, 0, k)
        o_ids, o_n = o.select_victims(idx, 100_000, 0, k, s32)
        H.assert_list_matches(ids.cpu().numpy().view(np.uint32)[:k], int(n_out.item()), o_ids, o_n, s64)
    c.use_survival_table(None)                           # back to the hop-distance table of Eq. 8
    o.survival()
    _, s32b = o.scores(idx, 100_000)
    assert np.array_equal(c.score_blocks(d, 100_000).cpu().numpy(), s32b)
    assert c.get_status() == 0


def test_select_with_other_tier_copy_preference():
    """cs_params.prefer_other_copy = 1: (score, has no copy, last_access, id), both select paths."""
    cfg = synth.CONFIGS["llama8b"]
    c, o = warm_state(cfg, 1000, 40000, r_min=0.02, prefer_other_copy=1)
    idx = synth.make_block_index(cfg, n=40000, with_tokens=False)
    idx.last_access[:] = 100_000 - (np.arange(40000) % 37)                 # many equal scores
    assert run_selects(c, o, idx, 100_000, (64, 3000)) == 0
    c2, o2 = warm_state(synth.CONFIGS["meta1m"], 2000, 300_000, r_min=0.02, prefer_other_copy=1)
    idx2 = synth.make_block_index(synth.CONFIGS["meta1m"], n=300_000, tier="random")     # above the cluster limit
    assert run_selects(c2, o2, idx2, 100_000, (10_000,), tiers=(0,)) == 0


# ---- corners of the parameter space -----------------------------------------------------------------------
@pytest.mark.parametrize("kw", [
    dict(lam=0.0), dict(e_max=1), dict(tau=0.0), dict(tau=1.5), dict(delta=0.5, eps=1.0),
    dict(lam=3.0, delta=1e-4), dict(e_max=37, tau=0.2), dict(block_tokens=255), dict(lam=1e-5)])
def test_parameter_corners(kw):
    cfg = synth.shrink(synth.CONFIGS["llama70b"], block_tokens=kw.pop("block_tokens", 16))
    c, o = warm_state(cfg, 2000, 5000, r_min=0.02, **kw)
    H.compare_model(c, o)
    idx = synth.make_block_index(cfg, n=5000)
    idx.last_access[::3] = 100_000 - np.arange(len(idx.last_access[::3])) % 9000    # ages across the whole table range
    d = cs.DeviceIndex.from_host(idx, DEV)
    s = c.score_blocks(d, 100_000).cpu().numpy()
    s64, s32 = o.scores(idx, 100_000)
    assert np.all(np.abs(s - s64) <= H.REL_TOL * s64)
    run_selects(c, o, idx, 100_000, (100,))


def test_maximum_agent_count():
    """1,024 agents: 32-word adjacency rows, 4 MiB transition matrix, rows that span several warps."""
    cfg = synth.shrink(synth.CONFIGS["meta1m"], n_agents=1024, sessions=64, n_chains=64, events_per_step=(8, 8))
    tr = synth.make_trace(cfg, n_invocations=30000)
    c, o = make_ctx(cfg, 20000, r_min=0.02, tau=0.1)
    for lo in range(0, 30000, 7000):
        c.observe_invocations(dev(tr.chain[lo:lo + 7000]), dev(tr.agent[lo:lo + 7000]), None)
        o.observe(tr.chain[lo:lo + 7000], tr.agent[lo:lo + 7000])
        H.compare_model(c, o)
    idx = synth.make_block_index(cfg, n=20000)
    assert run_selects(c, o, idx, 100_000, (500,)) == 0
    ps, _ = c.exact_survival(3)
    want = o.exact_survival(3)
    assert np.all(np.abs(ps.cpu().numpy() - want) <= H.REL_TOL * np.maximum(want, 1e-3))


@pytest.mark.parametrize("A,chains,all_sources", [(4, 3, False), (256, 40, False), (256, 40, True), (1024, 9, False), (70, 1, True)])
def test_small_batches_ride_with_the_refresh(A, chains, all_sources):
    """Batches of up to 256 events are applied inside the refresh launch (every row CTA adds the batch's transitions
    to its own rows, the last CTA writes the shared state); larger ones take the launch of their own.  Sizes on both
    sides of that limit, chains that repeat inside a batch, warm-up events, bad agent and chain ids, one and all
    chains as BFS sources: the learner state after every batch, the status bits and the event counters."""
    base = synth.CONFIGS["tiny"] if A <= 5 else synth.CONFIGS["meta1m"]
    cfg = synth.shrink(base, n_agents=A, sessions=chains, n_chains=chains, events_per_step=(4, 4))
    tr = synth.make_trace(cfg, n_invocations=3000, warmup_frac=0.15)
    agent, chain, evflags = tr.agent.copy(), tr.chain.copy(), tr.evflags.copy()
    bad_at = [70, 700, 1400, 1500]                   # 70, 1400, 1500 fall into batches of <= 256 events, 700 into one of 257
    evflags[bad_at] = 0
    agent[70] = A + 1
    chain[700] = chains
    chain[1400] = chains + 5
    agent[1500] = 0xFFFE
    c, o = make_ctx(cfg, 64, r_min=0.0)
    if all_sources:
        c.set_survival_sources(cs.CS_SOURCES_ALL_CHAINS)
    l0 = c.launch_count()
    lo = 0
    for size in (1, 2, 64, 255, 256, 257, 256, 300, 5, 256, 1024, 130):
        hi = lo + size
        c.observe_invocations(dev(chain[lo:hi]), dev(agent[lo:hi]), dev(evflags[lo:hi]))
        o.observe(chain[lo:hi], agent[lo:hi], evflags[lo:hi])
        if all_sources:
            o.survival(sources=np.unique(o.cur[o.cur != orc.AGENT_NONE]))
        H.compare_model(c, o)
        lo = hi
    assert c.launch_count() - l0 == 12 + 3           # one launch per batch, one more for the three batches above 256 events
    assert c.get_status() == (cs.CS_ST_BAD_AGENT | cs.CS_ST_BAD_CHAIN)
    cn = c.counters()
    live = (evflags[:lo] & cs.CS_EV_WARMUP) == 0
    bad = np.zeros(lo, bool); bad[bad_at] = True
    assert cn["events_seen"] == lo and cn["events_skipped"] == int(np.sum(~live | bad))
    assert cn["transitions_counted"] == int(o.C.sum())


@pytest.mark.parametrize("A,stride", [(40, 1), (300, 1), (300, 7), (512, 1), (512, 33), (544, 1), (96, 5)])
def test_bfs_on_deep_path_graphs(A, stride):
    """A workflow that is one long path (agent i is followed by agent i + stride mod A, over and over): the BFS from
    the current agent is as deep as the graph allows, the adjacency rows have 2 .. 17 words, and every hop count up
    to the depth appears once in the exported table."""
    cfg = synth.shrink(synth.CONFIGS["meta1m"], n_agents=A, sessions=2, n_chains=2, events_per_step=(8, 8))
    order = (np.arange(3 * A + 11, dtype=np.int64) * stride) % A
    chain = np.zeros(len(order), dtype=np.uint32)
    agent = order.astype(np.uint16)
    c, o = make_ctx(cfg, 64, tau=0.3, e_max=50, r_min=0.0)
    for lo in range(0, len(order), 97):                     # ragged batches, so predecessors are carried between calls
        c.observe_invocations(dev(chain[lo:lo + 97]), dev(agent[lo:lo + 97]), None)
        o.observe(chain[lo:lo + 97], agent[lo:lo + 97])
    m = H.compare_model(c, o)
    reach = m["hops"][m["hops"] != 0xFFFF]
    assert int(reach.max()) == A // int(np.gcd(A, stride)) - 1      # the path was walked to its end


def test_checkpoint_and_resume_of_the_learner():
    cfg = synth.CONFIGS["llama70b"]
    tr = synth.make_trace(cfg, n_invocations=4000, warmup_frac=0.05)
    c1, o = make_ctx(cfg, 64)
    c1.observe_invocations(dev(tr.chain[:2500]), dev(tr.agent[:2500]), dev(tr.evflags[:2500]))
    o.observe(tr.chain[:2500], tr.agent[:2500], tr.evflags[:2500])
    m = c1.get_model()
    c2, _ = make_ctx(cfg, 64)
    c2.import_state(dev(m["C"].astype(np.uint32).ravel()), dev(m["cur"]), m["last_agent"])
    H.compare_model(c2, o)                                     # restored state = the oracle's after the same events
    for c in (c1, c2):
        c.observe_invocations(dev(tr.chain[2500:]), dev(tr.agent[2500:]), dev(tr.evflags[2500:]))
    o.observe(tr.chain[2500:], tr.agent[2500:], tr.evflags[2500:])
    H.compare_model(c1, o)
    H.compare_model(c2, o)
    c3, o3 = make_ctx(cfg, 64)
    c3.import_state(dev(np.zeros(cfg.n_agents ** 2, np.uint32)), None, cs.CS_AGENT_NONE)
    H.compare_model(c3, o3)                                    # importing nothing is the initial state


@pytest.mark.parametrize("with_tokens,prefer", [(True, 0), (False, 0), (True, 1)])
def test_select_large_index_uses_age_limits(with_tokens, prefer):
    """Above 2^21 entries the collect pass decides by per-(agent, size) age limits; the lists must
    still equal the full sort, including sizes outside the table (0 and > block_tokens)."""
    cfg = synth.CONFIGS["meta1m"]
    n = (1 << 21) + 100_037
    c, o = warm_state(cfg, 3000, n, r_min=0.02, prefer_other_copy=prefer)
    idx = synth.make_block_index(cfg, n=n, tier="random", with_tokens=with_tokens)
    if with_tokens:
        idx.n_tokens[::1001] = 0
        idx.n_tokens[7::1003] = 200
    d = cs.DeviceIndex.from_host(idx, DEV)
    s64, s32 = o.scores(idx, 100_000)
    for k, tier in ((10_000, 0), (333, 1)):
        ids, n_out = c.select_victims(d, 100_000, tier, k)
        o_ids, o_n = o.select_victims(idx, 100_000, tier, k, s32)
        assert H.assert_list_matches(ids.cpu().numpy().view(np.uint32)[:k], int(n_out.item()), o_ids, o_n, s64) == 0
    ids, n_out = c.select_prefetch(d, 100_000, 2000)
    o_ids, o_n = o.select_prefetch(idx, 100_000, 2000, s32)
    assert o_n == 2000
    assert H.assert_list_matches(ids.cpu().numpy().view(np.uint32)[:2000], int(n_out.item()), o_ids, o_n, s64) == 0
    assert c.get_status() == 0


@pytest.mark.parametrize("max_keys", [0, 1, 40, 100_000])
def test_bucket_regions_and_their_fallback(max_keys):
    """With few candidates the sample sort's buckets live in fixed regions of the sort arrays that the bucket launch
    fills directly; a bucket that outgrows its region sends the call down the general route (buckets grouped by a
    launch of its own).  Capping the region (1 and 40 keys against buckets of ~64) forces that route on every call;
    the lists must not change.  Three clocks in a row, so that both the first call (full histogram and collect passes)
    and the calls that reuse the remembered threshold are covered; the cluster path is unaffected by the setting."""
    cfg = synth.CONFIGS["meta1m"]
    n = 400_000
    c, o = warm_state(cfg, 3000, n, r_min=0.02)
    c.set_select_bucket_regions(max_keys)
    idx = synth.make_block_index(cfg, n=n, tier="random")
    for now in (100_000, 100_001, 100_007):
        assert run_selects(c, o, idx, now, (9_000, 700)) == 0
    cn = c.counters()
    assert all(x > 0 for x in cn["region_selects"])          # 8 c <= 400,000 for k = 700, and mostly for k = 9,000
    if max_keys in (1, 40):
        assert all(x > 0 for x in cn["region_overflows"])
    else:
        assert cn["region_overflows"] == [0, 0, 0]


# ---- hop table from every live session's current agent ----------------------------------------------------
@pytest.mark.parametrize("name,n_inv", [("tiny", 60), ("llama8b", 400), ("meta1m", 3000)])
def test_survival_from_all_chains(name, n_inv):
    """CS_SOURCES_ALL_CHAINS: the cached BFS starts at the current agent of every chain; the oracle runs its
    multi-source BFS (pinned by brute force) from the same set, and the selects follow the new table."""
    cfg = synth.CONFIGS[name]
    if name == "tiny":
        cfg = synth.shrink(cfg, sessions=4, n_chains=4)
    n = 20000
    c, o = warm_state(cfg, n_inv, n, r_min=0.02)
    c.set_survival_sources(cs.CS_SOURCES_ALL_CHAINS)
    srcs = np.unique(o.cur[o.cur != orc.AGENT_NONE])
    assert len(srcs) >= 2, "needs several live chains"
    o.survival(sources=srcs)
    H.compare_model(c, o)
    assert np.all(o.E[srcs] == 0)
    # the mode persists across observe calls
    tr = synth.make_trace(cfg, n_invocations=n_inv + 40)
    lo = len(tr.agent) - 40
    c.observe_invocations(dev(tr.chain[lo:]), dev(tr.agent[lo:]), dev(tr.evflags[lo:]))
    o.observe(tr.chain[lo:], tr.agent[lo:], tr.evflags[lo:])
    o.survival(sources=np.unique(o.cur[o.cur != orc.AGENT_NONE]))
    H.compare_model(c, o)
    idx = synth.make_block_index(cfg, n=n, tier="random")
    d = cs.DeviceIndex.from_host(idx, DEV)
    s64, s32 = o.scores(idx, 100_000)
    assert np.array_equal(c.score_blocks(d, 100_000).cpu().numpy(), s32)
    k = 300
    ids, n_out = c.select_victims(d, 100_000, 0, k)
    o_ids, o_n = o.select_victims(idx, 100_000, 0, k, s32)
    assert H.assert_list_matches(ids.cpu().numpy().view(np.uint32)[:k], int(n_out[0].item()), o_ids, o_n, s64) == 0
    # back to the single source
    c.set_survival_sources(cs.CS_SOURCES_LAST_AGENT)
    o.survival()
    H.compare_model(c, o)
    assert c.get_status() == 0


# ---- the three selects of a step in one launch --------------------------------------------------------------
@pytest.mark.parametrize("name,n,kv,kp", [
    ("tiny", 2560, 32, 64), ("tiny", 0, 4, 4), ("tiny", 5, 8, 1), ("tiny", 1029, 1029, 700),
    ("llama8b", 80000, 256, 384), ("llama8b", 80000, 9000, 6000), ("llama70b", 52000 + 5, 128, 192),
    ("meta1m", 262144, 10000, 2000), ("meta1m", 300000, 500, 500), ("meta1m", 1_000_000, 10000, 2000)])
@pytest.mark.parametrize("path", [cs.CS_SELECT_AUTO, cs.CS_SELECT_MULTI])
def test_select_step_matches_three_calls_and_oracle(name, n, kv, kp, path):
    """cs_select_step: one launch of three clusters where the single-launch select applies, three kernel chains
    side by side elsewhere (300,000 entries, or the multi-launch path forced); lists bit-exact against the oracle,
    and again on a second and third call with a later clock (remembered thresholds in play)."""
    cfg = synth.CONFIGS[name]
    c, o = warm_state(cfg, 800, max(n, 16), r_min=0.02)
    c.set_select_path(path)
    idx = synth.make_block_index(cfg, n=n, tier="random" if name == "meta1m" else "range")
    d = cs.DeviceIndex.from_host(idx, DEV)
    i32 = lambda m: torch.full((max(m, 4),), 7, dtype=torch.int32, device=DEV)
    gv, gh, gp, gvn, ghn, gpn = i32(kv), i32(kv), i32(kp), i32(1), i32(1), i32(1)
    l0 = c.launch_count()
    for rep, now in enumerate((100_000, 100_001, 100_009)):
        c.select_step(d, now, kv, kp, gv, gvn, gh, ghn, gp, gpn)
        s64, s32 = o.scores(idx, now)
        for got, got_n, k, (o_ids, o_n) in ((gv, gvn, kv, o.select_victims(idx, now, 0, kv, s32)),
                                            (gh, ghn, kv, o.select_victims(idx, now, 1, kv, s32)),
                                            (gp, gpn, kp, o.select_prefetch(idx, now, kp, s32))):
            g = got.cpu().numpy().view(np.uint32)[:k]
            assert H.assert_list_matches(g, int(got_n[0].item()), o_ids, o_n, s64) == 0, (rep, k)
    fused = path == cs.CS_SELECT_AUTO and n <= 262144
    assert c.launch_count() - l0 == (3 if fused else 3 * 3 * 6)
    # a select whose count pointer is NULL is left out
    gh.fill_(7)
    ghn.fill_(7)
    now = 100_020
    c.select_step(d, now, kv, kp, gv, gvn, None, None, gp, gpn)
    s64, s32 = o.scores(idx, now)
    for got, got_n, k, (o_ids, o_n) in ((gv, gvn, kv, o.select_victims(idx, now, 0, kv, s32)),
                                        (gp, gpn, kp, o.select_prefetch(idx, now, kp, s32))):
        assert H.assert_list_matches(got.cpu().numpy().view(np.uint32)[:k], int(got_n[0].item()), o_ids, o_n, s64) == 0
    assert bool((gh == 7).all()) and int(ghn[0].item()) == 7
    assert c.get_status() == 0


def test_select_step_side_by_side_is_stable_over_many_calls():
    """The three kernel chains of a step run side by side on three streams with private scratch: over many
    consecutive calls with a moving clock and a changing index every list must equal the one the same select
    produces alone (bitwise), and the last call is checked against the oracle."""
    cfg = synth.CONFIGS["meta1m"]
    n, kv, kp = 300_000, 3000, 1500
    c, o = warm_state(cfg, 800, n, r_min=0.02)
    idx = synth.make_block_index(cfg, n=n, tier="random")
    d = cs.DeviceIndex.from_host(idx, DEV)
    i32 = lambda m: torch.full((max(m, 4),), 7, dtype=torch.int32, device=DEV)
    gv, gh, gp, gvn, ghn, gpn = i32(kv), i32(kv), i32(kp), i32(1), i32(1), i32(1)
    sv, sh, sp, svn, shn, spn = i32(kv), i32(kv), i32(kp), i32(1), i32(1), i32(1)
    la = d.last_access.view(torch.int32)
    bad = torch.zeros(1, dtype=torch.int64, device=DEV)
    for it in range(120):
        now = 100_000 + 3 * it
        if it:
            la[gv[:kv].long().clamp_(min=0)] = now - 3          # the index changes between calls
        c.select_step(d, now, kv, kp, gv, gvn, gh, ghn, gp, gpn)
        c.select_victims(d, now, 0, kv, sv, svn)
        c.select_victims(d, now, 1, kv, sh, shn)
        c.select_prefetch(d, now, kp, sp, spn)
        bad += (gv != sv).sum() + (gh != sh).sum() + (gp != sp).sum() + (gvn != svn).sum() + (ghn != shn).sum() + (gpn != spn).sum()
    assert int(bad.item()) == 0
    idx.last_access[:] = d.last_access.cpu().numpy()
    s64, s32 = o.scores(idx, now)
    for got, got_n, k, (o_ids, o_n) in ((gv, gvn, kv, o.select_victims(idx, now, 0, kv, s32)),
                                        (gh, ghn, kv, o.select_victims(idx, now, 1, kv, s32)),
                                        (gp, gpn, kp, o.select_prefetch(idx, now, kp, s32))):
        assert H.assert_list_matches(got.cpu().numpy().view(np.uint32)[:k], int(got_n[0].item()), o_ids, o_n, s64) == 0
    assert c.get_status() == 0


# ---- randomised small configurations ------------------------------------------------------------------------
@pytest.mark.parametrize("case", range(48))
def test_random_small_configurations(case):
    """Seeded random draws of everything the paper leaves open (agent count, chains, E_max, tau, lambda, delta,
    eps, block size, index size, k, with / without token counts and anchors, the copy preference, both BFS source
    modes): learner state, scores and all three lists on both select paths against the oracle."""
    rng = np.random.default_rng(7000 + case)
    A = int(rng.choice([1, 2, 3, 5, 12, 31, 32, 33, 70, 129]))
    chains = int(rng.choice([1, 3, 17]))
    base = synth.CONFIGS["tiny"] if A <= 5 else synth.CONFIGS["llama70b"]
    cfg = synth.shrink(base, n_agents=A, sessions=chains, n_chains=chains, seed=base.seed + 100 + case,
                       transitions=("dirichlet", float(rng.choice([0.3, 1.0]))) if A < 9 else ("sparse", int(min(4, A - 1))),
                       block_tokens=int(rng.choice([2, 7, 16, 32])), events_per_step=(1, int(rng.integers(1, 6))))
    n = int(rng.choice([1, 15, 16, 511, 512, 513, 3000, 9001]))
    kw = dict(e_max=int(rng.choice([1, 3, 4, 7])), tau=float(rng.choice([0.0, 0.02, 0.2, 1.5])),
              lam=float(rng.choice([0.0, 0.003, 0.05, 1.0])), delta=float(rng.choice([1e-3, 0.01, 0.5])),
              eps=float(rng.choice([1e-3, 0.01, 1.0])), r_min=float(rng.choice([0.0, 0.02])),
              prefer_other_copy=int(rng.integers(0, 2)))
    tr = synth.make_trace(cfg, n_invocations=int(rng.integers(1, 400)), warmup_frac=float(rng.choice([0.0, 0.2])))
    c, o = make_ctx(cfg, max(n, 16), **kw)
    all_chains = bool(rng.integers(0, 2))
    if all_chains:
        c.set_survival_sources(cs.CS_SOURCES_ALL_CHAINS)
    c.observe_invocations(dev(tr.chain), dev(tr.agent), dev(tr.evflags))
    o.observe(tr.chain, tr.agent, tr.evflags)
    if all_chains:
        o.survival(sources=np.unique(o.cur[o.cur != orc.AGENT_NONE]))
    if abs(o.R - o.p.r_min) < H.R_FRAGILE:
        pytest.skip("R within the fragile band of r_min for this draw")
    H.compare_model(c, o)
    idx = synth.make_block_index(cfg, n=n, tier="random", with_tokens=bool(rng.integers(0, 2)),
                                 with_anchor=bool(rng.integers(0, 2)))
    now = 100_000 + int(rng.integers(0, 5000))
    d = cs.DeviceIndex.from_host(idx, DEV)
    if n:
        s64, s32 = o.scores(idx, now)
        got = c.score_blocks(d, now).cpu().numpy()
        assert np.all(np.abs(got - s64) <= H.REL_TOL * s64)
        if kw["lam"] not in (0.003,):                  # (a table that does not cover every age may differ in the last bit)
            assert np.mean(got == s32) > 0.999
    ks = sorted({1, int(rng.integers(1, n + 1)), n})
    assert run_selects(c, o, idx, now, ks) == 0


@pytest.mark.parametrize("case", range(16))
def test_random_mover_geometries(case):
    """Seeded random block geometries (layers, heads, head size, tokens, element size), layouts, id offsets, list
    lengths and sentinels: offload, prefetch, compaction (bulk and load/store paths) and the two-way transfer."""
    rng = np.random.default_rng(9000 + case)
    L, heads = int(rng.integers(1, 7)), int(rng.choice([1, 2, 3, 8]))
    hd, tok, eb = int(rng.choice([8, 40, 64, 128])), int(rng.choice([1, 4, 9, 16])), int(rng.choice([1, 2, 4]))
    chunk = tok * heads * hd * eb
    if chunk % 16:
        hd, chunk = 128, tok * heads * 128 * eb
    G, Hs = int(rng.integers(20, 60)), int(rng.integers(20, 60))
    lay_g, lay_h = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    first_h = int(rng.choice([0, G, 1000]))
    c = cs.CacheScout(cs.make_params(n_agents=4, max_blocks=64), DEV)
    c.set_mover_path(cs.CS_MOVER_LDST if case % 4 == 3 else cs.CS_MOVER_BULK)
    c.set_mover_ctas(int(rng.choice([0, 1, 5, 40])), int(rng.choice([0, 3, 64])))
    gpu_np = rng.integers(0, 256, G * L * 2 * chunk, dtype=np.uint8)
    host_np = rng.integers(0, 256, Hs * L * 2 * chunk, dtype=np.uint8)
    gpu = cs.KVPool(dev(gpu_np), G, lay_g, L, heads, hd, tok, eb)
    host_t = torch.from_numpy(host_np.copy()).pin_memory()
    host = cs.KVPool(host_t, Hs, lay_h, L, heads, hd, tok, eb, first_id=first_h)
    n_off, n_pre = int(rng.integers(0, 12)), int(rng.integers(0, 12))
    g_perm, h_perm = rng.permutation(G).astype(np.uint32), rng.permutation(Hs).astype(np.uint32)
    off_src, pre_dst = g_perm[:n_off].copy(), g_perm[n_off:n_off + n_pre].copy()
    off_dst, pre_src = h_perm[:n_off] + np.uint32(first_h), h_perm[n_off:n_off + n_pre] + np.uint32(first_h)
    if n_off > 2:
        off_src[1] = orc.ID_NONE
    if n_pre > 2:
        pre_src[0] = orc.ID_NONE
    opt = lambda a: dev(a) if len(a) else None
    c.validate_exchange_lists(gpu, host, opt(off_src), opt(off_dst), opt(pre_src), opt(pre_dst))     # no slot used twice
    c.exchange_blocks(gpu, host, opt(off_src), opt(off_dst), opt(pre_src), opt(pre_dst))
    torch.cuda.synchronize()
    want_h, want_g = host_np.copy(), gpu_np.copy()
    unoff = lambda a: np.where(a == orc.ID_NONE, a, a - np.uint32(first_h))
    orc.move_blocks(gpu_np, lay_g, G, want_h, lay_h, Hs, L, chunk, off_src, unoff(off_dst))
    orc.move_blocks(host_np, lay_h, Hs, want_g, lay_g, G, L, chunk, unoff(pre_src), pre_dst)
    assert np.array_equal(host_t.numpy(), want_h) and np.array_equal(gpu.buf.cpu().numpy(), want_g)
    # the single calls, starting from the state just reached
    n = int(rng.integers(1, 15))
    s_g, d_h = rng.permutation(G).astype(np.uint32)[:n], rng.permutation(Hs).astype(np.uint32)[:n] + np.uint32(first_h)
    c.validate_move_lists(gpu, host, dev(s_g), dev(d_h))
    c.offload_blocks(gpu, host, dev(s_g), dev(d_h))
    torch.cuda.synchronize()
    orc.move_blocks(want_g, lay_g, G, want_h, lay_h, Hs, L, chunk, s_g, unoff(d_h))
    assert np.array_equal(host_t.numpy(), want_h)
    back = rng.permutation(G).astype(np.uint32)[:n]
    c.validate_move_lists(host, gpu, dev(d_h), dev(back))
    c.prefetch_blocks(host, gpu, dev(d_h), dev(back))
    torch.cuda.synchronize()
    src_h = want_h.copy()
    orc.move_blocks(src_h, lay_h, Hs, want_g, lay_g, G, L, chunk, unoff(d_h), back)
    assert np.array_equal(gpu.buf.cpu().numpy(), want_g)
    stage = cs.KVPool(torch.zeros(n * L * 2 * chunk, dtype=torch.uint8, device=DEV), n, 1 - lay_g, L, heads, hd, tok, eb)
    c.compact_blocks(gpu, stage, dev(back), dev(np.arange(n, dtype=np.uint32)))
    torch.cuda.synchronize()
    want_s = np.zeros(n * L * 2 * chunk, np.uint8)
    orc.move_blocks(want_g, lay_g, G, want_s, 1 - lay_g, n, L, chunk, back, np.arange(n))
    assert np.array_equal(stage.buf.cpu().numpy(), want_s)
    assert c.get_status() == 0
    if lay_h == synth.BLOCK_MAJOR:          # the copy-engine path needs contiguous host blocks
        bb = L * 2 * chunk
        c.set_mover_staging(torch.empty(4 * int(rng.integers(1, 6)) * bb + 512, dtype=torch.uint8, device=DEV))
        m = int(rng.integers(1, 12))
        gp2, hp2 = rng.permutation(G).astype(np.uint32), rng.permutation(Hs).astype(np.uint32)
        o_src, p_dst = gp2[:m], gp2[m:2 * m]
        o_dst, p_src = hp2[:m] + np.uint32(first_h), hp2[m:2 * m] + np.uint32(first_h)
        host_before = host_t.numpy().copy()
        c.exchange_blocks_staged(gpu, host, dev(o_src), o_dst, p_src, dev(p_dst))
        torch.cuda.synchronize()
        orc.move_blocks(want_g, lay_g, G, want_h, lay_h, Hs, L, chunk, o_src, unoff(o_dst))
        want_g2 = want_g.copy()
        orc.move_blocks(host_before, lay_h, Hs, want_g2, lay_g, G, L, chunk, unoff(p_src), p_dst)
        assert np.array_equal(host_t.numpy(), want_h) and np.array_equal(gpu.buf.cpu().numpy(), want_g2)
        assert c.get_status() == 0
