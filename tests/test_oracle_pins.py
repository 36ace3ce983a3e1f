"""Pins of the CPU oracle against things other than itself: brute force on tiny inputs,
closed forms, invariants, hand-derived worked examples (tests/golden) and special cases.

All of this runs without a GPU.  Each test is chosen so that a plausible slip in the oracle
(a dropped term, a wrong sign or index, a transposed operand, a wrong tie order) fails it.
"""
import itertools
import math

import numpy as np
import pytest

from oracle import cs_oracle as orc
from tests import synth
from tests.conftest import read_golden

P = orc.Params


def run_trace(agents, A, chains=None, flags=None, n_chains=1, **kw):
    o = orc.Oracle(P(n_agents=A, n_chains=n_chains, **kw))
    chains = np.zeros(len(agents), np.uint32) if chains is None else chains
    o.observe(chains, np.asarray(agents, np.uint16), flags)
    return o


# ---- transition counts: brute force by direct counting of the trace ---------------------
def brute_counts(chain, agent, flags, A, n_chains):
    """Dictionary count of consecutive distinct pairs per chain (Sec. 3.2, Algorithm 1)."""
    C = np.zeros((A, A), np.int64)
    prev = {}
    last = None
    for c, a, f in zip(chain.tolist(), agent.tolist(), flags.tolist()):
        if f & 1 or a >= A or c >= n_chains:
            continue
        if c in prev and prev[c] != a:
            C[prev[c], a] += 1
        prev[c] = a
        last = a
    return C, prev, last


@pytest.mark.parametrize("seed", range(6))
def test_counts_vs_direct_counting(seed):
    rng = np.random.default_rng(seed)
    A, n_chains, E = 5, 3, 60
    chain = rng.integers(0, n_chains, E).astype(np.uint32)
    agent = rng.integers(0, A, E).astype(np.uint16)
    flags = (rng.random(E) < 0.15).astype(np.uint8)
    if seed == 5:                       # invalid ids are skipped, not counted
        agent[7] = A + 2
        chain[11] = n_chains
    o = orc.Oracle(P(n_agents=A, n_chains=n_chains))
    # feed in three batches: state must carry over batch boundaries
    for lo, hi in ((0, 13), (13, 14), (14, E)):
        o.observe(chain[lo:hi], agent[lo:hi], flags[lo:hi])
    Cb, prev, last = brute_counts(chain, agent, flags, A, n_chains)
    assert np.array_equal(o.C.astype(np.int64), Cb)
    assert np.all(np.diag(o.C) == 0)
    for c in range(n_chains):
        assert int(o.cur[c]) == prev.get(c, orc.AGENT_NONE)
    assert int(o.last_agent[0]) == last
    if seed == 5:
        assert o.n_bad_events == 2


def test_counts_single_chain_is_algorithm_1():
    # with one chain the number of counted transitions = number of agent changes
    agents = [2, 2, 0, 0, 0, 1, 2, 2, 1]
    o = run_trace(agents, 3)
    changes = sum(1 for x, y in zip(agents, agents[1:]) if x != y)
    assert int(o.C.sum()) == changes
    assert o.C[2, 0] == 1 and o.C[0, 1] == 1 and o.C[1, 2] == 1 and o.C[2, 1] == 1


def test_counts_direction_not_transposed():
    o = run_trace([0, 1], 2)
    assert o.C[0, 1] == 1 and o.C[1, 0] == 0


# ---- Eq. 3: normalisation -----------------------------------------------------------------
@pytest.mark.parametrize("A", [2, 3, 7, 24])
def test_rows_sum_to_one_and_match_definition(A):
    rng = np.random.default_rng(A)
    o = orc.Oracle(P(n_agents=A))
    o.C[:] = rng.integers(0, 50, (A, A))
    np.fill_diagonal(o.C, 0)
    o.C[A - 1, :] = 0                        # a cold row must come out uniform
    o.refresh()
    assert np.allclose(o.P64.sum(1), 1.0, atol=1e-14)
    assert np.all(np.abs(o.P32.astype(np.float64).sum(1) - 1.0) <= A * 2.0 ** -23)
    assert np.allclose(o.P64[A - 1], 1.0 / A, rtol=0, atol=1e-15)
    eps = float(np.float32(0.01))
    want = (o.C + eps) / (o.C.sum(1, keepdims=True) + A * eps)      # NumPy restatement
    assert np.allclose(o.P64, want, rtol=1e-13)
    assert np.all(np.abs(o.P32 - o.P64) <= 1e-6 * o.P64)
    assert np.array_equal(o.amax, np.argmax(o.P32, axis=1))          # first max wins


def test_worked_example_a():
    g = read_golden("worked_example_a.txt")
    trace = [int(x) for x in g["trace"][0]]
    o = run_trace(trace, 3)
    assert o.C.tolist() == [[0, 2, 0], [0, 0, 2], [2, 0, 0]]
    p_hi, p_lo = g["p_hi"][0][0], g["p_lo"][0][0]
    # tolerance: eps is the fp32 value nearest 0.01, the fixture uses the decimal 0.01
    want = np.array([[p_lo, p_hi, p_lo], [p_lo, p_lo, p_hi], [p_hi, p_lo, p_lo]])
    assert np.allclose(o.P64, want, rtol=1e-7)
    assert math.isclose(o.R, g["R"][0][0], rel_tol=1e-6)
    assert o.E.tolist() == [int(x) for x in g["E"][0]]
    assert np.allclose(o.ptilde, g["ptilde"][0], atol=0)
    assert int(o.amax[0]) == int(g["a_star_of_0"][0][0])
    assert o.gate
    for a, age, tok, want_s in g["score"]:
        idx = synth.BlockIndex(np.array([a], np.uint16), np.zeros(1, np.uint16), np.zeros(1, np.uint8),
                               np.ones(1, np.uint8), np.array([1000], np.uint32),
                               np.array([tok], np.uint8), None)
        s64, s32 = o.scores(idx, 1000 + int(age))
        assert math.isclose(s64[0], want_s, rel_tol=2e-7), (a, age, tok)
        assert math.isclose(float(s32[0]), want_s, rel_tol=1e-6)


def test_worked_example_b_ties_and_hub():
    g = read_golden("worked_example_b.txt")
    trace = [int(x) for x in g["trace"][0]]
    o = run_trace(trace, 4)
    assert o.C.ravel().tolist() == [int(x) for x in g["C"][0]]
    assert np.allclose(o.P64[0], g["row0"][0], rtol=1e-7)
    assert np.allclose(o.P64[1], g["row1"][0], rtol=1e-7)
    assert np.allclose(o.P64[2], g["row2"][0], rtol=1e-7)
    assert np.allclose(o.P64[3], g["row2"][0], rtol=1e-7)
    assert o.amax.tolist() == [int(x) for x in g["amax"][0]]       # row 1: tie -> lowest index
    assert math.isclose(o.R, g["R"][0][0], rel_tol=1e-6)
    assert int(o.last_agent[0]) == 1
    assert o.E.tolist() == [int(x) for x in g["E"][0]]
    assert np.array_equal(o.ptilde, np.array(g["ptilde"][0]))


# ---- Eq. 2: predictability --------------------------------------------------------------------
def test_R_deterministic_cycle_tends_to_one():
    agents = list(range(6)) * 40
    r_prev = 0.0
    for eps in (1e-1, 1e-2, 1e-4, 1e-7):
        o = run_trace(agents, 6, eps=eps)
        assert o.R > r_prev
        r_prev = o.R
    assert r_prev > 1 - 1e-4                   # Pipeline topology: R = 1.0 (Sec. 2.2)


def test_R_zero_when_next_agent_independent():
    # every row the same distribution => next agent independent of the current one
    A = 4
    o = orc.Oracle(P(n_agents=A))
    o.C[:] = np.array([5, 1, 3, 7], np.uint32)[None, :] * 2   # includes the diagonal on purpose
    o.refresh()
    assert abs(o.R) < 1e-12
    o2 = orc.Oracle(P(n_agents=A))
    assert o2.R == 0.0 and not o2.gate          # nothing counted yet


@pytest.mark.parametrize("seed", range(4))
def test_R_equals_mutual_information_ratio(seed):
    """R * H(next) = I(cur; next) = sum pi_i P_ij ln(P_ij / q_j): an independent formula."""
    rng = np.random.default_rng(seed)
    A = 6
    o = orc.Oracle(P(n_agents=A))
    o.C[:] = rng.integers(0, 30, (A, A))
    np.fill_diagonal(o.C, 0)
    o.refresh()
    pi = o.C.sum(1) / o.C.sum()
    J = pi[:, None] * o.P64
    q = J.sum(0)
    I = float((J * np.log(o.P64 / q[None, :])).sum())
    Hm = float(-(q * np.log(q)).sum())
    assert math.isclose(o.R, I / Hm, rel_tol=1e-10)
    assert 0.0 <= o.R <= 1.0


def test_recoverability_of_generating_matrix():
    """With chain = session the learner recovers the jump chain of the generating matrix."""
    cfg = synth.shrink(synth.CONFIGS["llama8b"], n_agents=5, sessions=8, n_chains=8,
                       session_len=(2000, 2000), events_per_step=(1, 4))
    tr = synth.make_trace(cfg, n_invocations=16000)
    o = orc.Oracle(P(n_agents=5, n_chains=8, eps=1e-6))
    o.observe(tr.chain, tr.agent, tr.evflags)
    J = tr.M.copy()
    np.fill_diagonal(J, 0.0)
    J /= J.sum(1, keepdims=True)
    n_i = o.C.sum(1, keepdims=True).astype(np.float64)
    assert n_i.min() > 30 and n_i.max() > 1000
    bound = 4.5 * np.sqrt(J * (1 - J) / n_i) + 2.0 / n_i     # binomial error of each row estimate
    assert np.all(np.abs(o.P64 - J) <= bound)
    assert np.max(np.abs(o.P64 - J)) < 0.1


# ---- Eq. 7 + BFS + Eq. 8 --------------------------------------------------------------------
def brute_hops(adj, sources):
    """min t with (adj^t)[s][a] > 0 by boolean matrix powers."""
    A = adj.shape[0]
    E = np.full(A, orc.INF, np.uint64)
    reach = np.zeros(A, bool)
    reach[list(sources)] = True
    E[list(sources)] = 0
    front = reach.copy()
    for t in range(1, A + 1):
        front = (front.astype(np.int64) @ adj.astype(np.int64)) > 0
        new = front & ~reach
        E[new] = t
        reach |= new
    return E


@pytest.mark.parametrize("seed", range(8))
def test_graph_and_bfs_vs_matrix_powers(seed):
    rng = np.random.default_rng(100 + seed)
    A = int(rng.integers(2, 12))
    o = orc.Oracle(P(n_agents=A, tau=0.12, e_max=3))
    o.C[:] = rng.integers(0, 4, (A, A)) * (rng.random((A, A)) < 0.35)
    np.fill_diagonal(o.C, 0)
    srcs = [int(rng.integers(0, A))] if seed % 2 == 0 else rng.choice(A, 2, replace=False).tolist()
    o.refresh(sources=srcs)
    adj = (o.P32 >= np.float32(0.12))
    assert np.array_equal(o.adj.astype(bool), adj)
    assert np.array_equal(o.E.astype(np.uint64), brute_hops(adj, srcs))
    m = np.minimum(o.E.astype(np.float64), 3)
    assert np.array_equal(o.ptilde, 1 - m / 3)
    assert all(o.ptilde[s] == 1.0 for s in srcs)              # the current agent is fully protected
    assert np.all(o.ptilde[o.E == orc.INF] == 0.0)            # unreachable -> floor only


def test_threshold_is_inclusive_and_no_source_means_no_protection():
    o = orc.Oracle(P(n_agents=2, tau=0.5, eps=0.25))           # cold rows: P = 0.5 exactly
    assert o.adj.tolist() == [[1, 1], [1, 1]]
    assert np.all(o.E == orc.INF) and np.all(o.ptilde == 0.0)  # no current agent yet
    assert np.allclose(o.fsurv32, 0.01)


# ---- Eq. 9: block score ----------------------------------------------------------------------
def make_idx(agent, last_access, n_tokens=None, flags=None, ref=None, depth=None, anchor=None):
    n = len(agent)
    return synth.BlockIndex(
        np.asarray(agent, np.uint16),
        np.zeros(n, np.uint16) if depth is None else np.asarray(depth, np.uint16),
        np.zeros(n, np.uint8) if ref is None else np.asarray(ref, np.uint8),
        np.full(n, synth.FLAG_VALID, np.uint8) if flags is None else np.asarray(flags, np.uint8),
        np.asarray(last_access, np.uint32),
        None if n_tokens is None else np.asarray(n_tokens, np.uint8),
        None if anchor is None else np.asarray(anchor, np.uint16))


def test_score_closed_forms_and_monotonicity():
    lam = math.log(2.0) / 8                              # recency halves every 8 steps
    o = run_trace([0, 1, 2, 0], 3, lam=lam, delta=0.01)
    # E = [0,1,2] from agent 0
    ages = np.arange(0, 64)
    for a, pt in ((0, 1.0), (1, 0.75), (2, 0.5)):
        idx = make_idx([a] * 64, 500 - ages, n_tokens=[16] * 64)
        s64, s32 = o.scores(idx, 500)
        d = float(np.float32(0.01))
        lam32 = float(np.float32(lam))
        for age in (0, 8, 16, 24):                       # exp(-lam*age) = 2^-(age/8)
            want = (pt + d) * (2.0 ** (-age / 8) * math.exp(-(lam32 - lam) * age) + d) * 16
            assert math.isclose(s64[age], want, rel_tol=1e-12)
        assert np.all(np.diff(s64) < 0)                  # strictly decreasing in age
        assert np.all(np.abs(s32 - s64) <= 1e-6 * s64)
        assert np.all(s32 > 0)
    # decreasing in hop distance, proportional to |b|
    idx = make_idx([0, 1, 2, 2], [490] * 4, n_tokens=[16, 16, 16, 8])
    s64, _ = o.scores(idx, 500)
    assert s64[0] > s64[1] > s64[2] and math.isclose(s64[3] * 2, s64[2], rel_tol=1e-15)
    # future last_access clamps age to 0; default |b| = block_tokens
    s_f, _ = o.scores(make_idx([1], [777]), 500)
    s_0, _ = o.scores(make_idx([1], [500], n_tokens=[16]), 500)
    assert s_f[0] == s_0[0]


def test_score_saturates_at_delta_floor():
    o = run_trace([0, 1], 2)
    idx = make_idx([1, 1, 1], [10 ** 6 - 2194, 0, 10 ** 6 - 2000])
    _, s32 = o.scores(idx, 10 ** 6)
    assert s32[0] == s32[1]                              # both recency factors round to delta
    assert s32[2] > s32[1]
    assert s32[1] == np.float32(np.float32(1.01) * np.float32(0.01)) * np.float32(16)


# ---- selections: brute force by a full Python sort -------------------------------------------
def brute_victims(idx, s32, tier, k, A):
    rows = []
    for b in range(idx.n):
        f = int(idx.flags[b])
        if not f & 1 or f & 2 or idx.ref_count[b] != 0 or ((f >> 2) & 1) != tier or idx.agent[b] >= A:
            continue
        rows.append((float(s32[b]), int(idx.last_access[b]), b))
    rows.sort()
    ids = [r[2] for r in rows[:k]]
    return ids + [orc.ID_NONE] * (k - len(ids)), len(ids), len(rows)


def brute_prefetch(idx, s32, k, A, gate, last_agent, amax):
    if not gate or last_agent == orc.AGENT_NONE:
        return [orc.ID_NONE] * k, 0
    a_star = int(amax[last_agent])
    rows = []
    for b in range(idx.n):
        f = int(idx.flags[b])
        if not f & 1 or f & 2 or idx.ref_count[b] != 0 or not f & 4 or f & 8 or idx.agent[b] >= A:
            continue
        if idx.anchor_blocks is not None and not idx.depth[b] < idx.anchor_blocks[idx.agent[b]]:
            continue
        rows.append((0 if idx.agent[b] == a_star else 1, -float(s32[b]), -int(idx.last_access[b]), b))
    rows.sort()
    ids = [r[3] for r in rows[:k]]
    return ids + [orc.ID_NONE] * (k - len(ids)), len(ids)


def small_state(seed, A=6, N=64, n_chains=2):
    cfg = synth.shrink(synth.CONFIGS["tiny"], n_agents=A, sessions=n_chains, n_chains=n_chains,
                       gpu_blocks=N // 2, host_blocks=N - N // 2, seed=synth.BASE_SEED + 100 + seed)
    tr = synth.make_trace(cfg, n_invocations=50)
    o = orc.Oracle(P(n_agents=A, n_chains=n_chains, r_min=0.05))
    o.observe(tr.chain, tr.agent, tr.evflags)
    idx = synth.make_block_index(cfg, n=N, now0=3000)
    idx.anchor_blocks[:] = np.random.default_rng(seed).integers(100, 400, A)
    # force ties: quantise ages so many blocks share (score, last_access)
    idx.last_access[:] = 3000 - (3000 - idx.last_access.astype(np.int64)) // 700 * 700
    return cfg, o, idx


@pytest.mark.parametrize("seed", range(10))
def test_victims_vs_full_sort(seed):
    cfg, o, idx = small_state(seed)
    _, s32 = o.scores(idx, 3000)
    for tier in (0, 1):
        for k in (1, 5, 32, 100):
            ids, n_out = o.select_victims(idx, 3000, tier, k)
            want, wn, n_elig = brute_victims(idx, s32, tier, k, cfg.n_agents)
            assert n_out == wn == min(k, n_elig)
            assert ids.tolist() == want
            sel = ids[:n_out].astype(np.int64)
            assert len(set(sel.tolist())) == n_out
            assert not np.any(idx.flags[sel] & synth.FLAG_PINNED)
            assert np.all(idx.ref_count[sel] == 0) and np.all(idx.flags[sel] & synth.FLAG_VALID)


@pytest.mark.parametrize("seed", range(10))
def test_prefetch_vs_full_sort(seed):
    cfg, o, idx = small_state(seed)
    _, s32 = o.scores(idx, 3000)
    assert o.gate
    for k in (1, 7, 64):
        ids, n_out = o.select_prefetch(idx, 3000, k)
        want, wn = brute_prefetch(idx, s32, k, cfg.n_agents, o.gate, int(o.last_agent[0]), o.amax)
        assert (ids.tolist(), n_out) == (want, wn)
        sel = ids[:n_out].astype(np.int64)
        assert np.all(idx.flags[sel] & synth.FLAG_TIER_HOST)
        assert not np.any(idx.flags[sel] & (synth.FLAG_OTHER_COPY | synth.FLAG_PINNED))
    # a* blocks come first
    ids, n_out = o.select_prefetch(idx, 3000, 64)
    a_star = int(o.amax[int(o.last_agent[0])])
    is_star = idx.agent[ids[:n_out].astype(np.int64)] == a_star
    assert np.all(np.diff(is_star.astype(int)) <= 0)


def test_prefetch_gate_closed_or_no_agent_gives_empty_list():
    cfg, o, idx = small_state(0)
    o.p.r_min = 2.0
    ids, n_out = o.select_prefetch(idx, 3000, 8)
    assert n_out == 0 and np.all(ids == orc.ID_NONE)
    o2 = orc.Oracle(P(n_agents=cfg.n_agents, r_min=-1.0))       # gate open, but no current agent
    ids, n_out = o2.select_prefetch(idx, 3000, 8)
    assert n_out == 0


def test_lru_special_case():
    """No graph edges (tau > 1) and constant |b|: eviction order is exactly LRU (Sec. 3.3)."""
    cfg, o, idx = small_state(3)
    o.p.tau = 1.5
    o.refresh()
    assert o.adj.sum() == 0
    idx.n_tokens = None
    la = int(o.last_agent[0])
    keep = idx.agent != la                                  # the current agent itself stays protected
    idx.flags[~keep] &= np.uint8(~synth.FLAG_VALID & 0xFF)
    idx.last_access[::5] = 10                                # far past the recency saturation point
    ids, n_out = o.select_victims(idx, 3000, 0, 40)
    sel = ids[:n_out].astype(np.int64)
    order = sorted(sel.tolist(), key=lambda b: (int(idx.last_access[b]), b))
    assert sel.tolist() == order
    elig = [b for b in range(idx.n) if idx.flags[b] & 1 and not idx.flags[b] & 2
            and idx.ref_count[b] == 0 and not idx.flags[b] & 4]
    assert sel.tolist() == sorted(elig, key=lambda b: (int(idx.last_access[b]), b))[:40]


def test_equal_reuse_probability_evicts_cheaper_block_first():
    o = run_trace([0, 1], 2)
    idx = make_idx([0, 0], [90, 90], n_tokens=[16, 5])
    ids, n = o.select_victims(idx, 100, 0, 2)
    assert ids.tolist() == [1, 0]


# ---- mover: NumPy fancy indexing on a reshaped pool ---------------------------------------------
@pytest.mark.parametrize("src_layout,dst_layout", list(itertools.product((0, 1), (0, 1))))
def test_mover_vs_fancy_indexing(src_layout, dst_layout):
    rng = np.random.default_rng(7)
    L, chunk, ns, nd, n = 3, 64, 11, 9, 6
    src = rng.integers(0, 256, ns * L * 2 * chunk, dtype=np.uint8)
    dst = rng.integers(0, 256, nd * L * 2 * chunk, dtype=np.uint8)
    dst0 = dst.copy()
    s_ids, d_ids = synth.mover_batch(n, ns, nd, rng)
    s_ids[2] = orc.ID_NONE                                   # sentinel entries are skipped
    bad = orc.move_blocks(src, src_layout, ns, dst, dst_layout, nd, L, chunk, s_ids, d_ids)
    assert bad == 0

    def view(buf, layout, slots):                            # -> [slot, layer, plane, byte]
        if layout == 0:
            return buf.reshape(L, 2, slots, chunk).transpose(2, 0, 1, 3)
        return buf.reshape(slots, L, 2, chunk)
    want = view(dst0.copy(), dst_layout, nd).copy()
    ok = s_ids != orc.ID_NONE
    want[d_ids[ok]] = view(src, src_layout, ns)[s_ids[ok]]
    assert np.array_equal(view(dst, dst_layout, nd), want)
    untouched = np.setdiff1d(np.arange(nd), d_ids[ok])
    assert np.array_equal(view(dst, dst_layout, nd)[untouched], view(dst0, dst_layout, nd)[untouched])


def test_offload_then_prefetch_roundtrip_is_bytewise_identity():
    rng = np.random.default_rng(11)
    L, chunk, G, H, n = 4, 128, 16, 32, 10
    gpu = synth.kv_pool_u16(G, L, chunk, rng).view(np.uint8)
    host = np.zeros(H * L * 2 * chunk, np.uint8)
    back = np.zeros_like(gpu)
    g_ids, h_ids = synth.mover_batch(n, G, H, rng)
    for lay in (0, 1):
        orc.move_blocks(gpu, lay, G, host, 1, H, L, chunk, g_ids, h_ids)
        orc.move_blocks(host, 1, H, back, lay, G, L, chunk, h_ids, g_ids)
        v = (lambda b: b.reshape(L, 2, G, chunk).transpose(2, 0, 1, 3)) if lay == 0 else \
            (lambda b: b.reshape(G, L, 2, chunk))
        assert np.array_equal(v(back)[g_ids], v(gpu)[g_ids])
    bad = orc.move_blocks(gpu, 0, G, host, 1, H, L, chunk, np.array([G], np.uint32), np.array([0], np.uint32))
    assert bad == 1


# ---- Eq. 6: exact survival probability --------------------------------------------------------------
def brute_survival(Pm, a0, K):
    """Enumerate every path of K steps from a0 and add up the probability of those that visit a."""
    A = Pm.shape[0]
    out = np.zeros(A)
    for path in itertools.product(range(A), repeat=K):
        pr, cur = 1.0, a0
        for nxt in path:
            pr *= Pm[cur, nxt]
            cur = nxt
        for a in set(path):
            out[a] += pr
    return out


@pytest.mark.parametrize("seed", range(4))
def test_exact_survival_vs_path_enumeration(seed):
    rng = np.random.default_rng(40 + seed)
    A, K = 4, 4
    o = orc.Oracle(P(n_agents=A))
    o.C[:] = rng.integers(0, 9, (A, A))
    np.fill_diagonal(o.C, 0)
    o.refresh()
    for a0 in range(A):
        got = o.exact_survival(K, a0)
        assert np.allclose(got, brute_survival(o.P64, a0, K), rtol=1e-12, atol=1e-15)
        assert np.allclose(o.exact_survival(1, a0), o.P64[a0], rtol=1e-13)         # one step: the row itself
        assert np.all(np.diff([o.exact_survival(k, a0) for k in range(0, 6)], axis=0) >= -1e-15)   # grows with K
    assert np.all(o.exact_survival(0, 0) == 0.0)
    assert np.all(o.exact_survival(3, orc.AGENT_NONE) == 0.0)                      # no current agent yet


def test_exact_survival_on_a_deterministic_cycle():
    """Pipeline topology: agent at distance d is reached within K steps iff d <= K (Sec. 2.2)."""
    o = run_trace(list(range(5)) * 30, 5, eps=1e-9)
    for K in (1, 2, 4, 5):
        got = o.exact_survival(K)                       # current agent is 4; distances: 0->1, 1->2, ... 4->5
        want = np.array([1.0 if ((a - 4) % 5 or 5) <= K else 0.0 for a in range(5)])
        assert np.allclose(got, want, atol=1e-6)
    # the hop-distance proxy of Eq. 8 orders the agents the same way on this chain
    assert np.array_equal(np.argsort(-o.exact_survival(3), kind="stable")[:3], np.argsort(o.E, kind="stable")[1:4])


def test_preference_for_blocks_with_a_copy_on_the_other_tier():
    """Sec. 4: among equally scored victims, those whose contents already exist on the other tier
    go first (they need no offload); the score still dominates."""
    for seed in range(4):
        cfg, o, idx = small_state(seed)
        o.p.prefer_other_copy = 1
        _, s32 = o.scores(idx, 3000)
        for tier in (0, 1):
            ids, n_out = o.select_victims(idx, 3000, tier, 40)
            rows = []
            for b in range(idx.n):
                f = int(idx.flags[b])
                if not f & 1 or f & 2 or idx.ref_count[b] != 0 or ((f >> 2) & 1) != tier:
                    continue
                rows.append((float(s32[b]), 0 if f & 8 else 1, int(idx.last_access[b]), b))
            rows.sort()
            assert ids[:n_out].tolist() == [r[3] for r in rows[:40]]
    o = run_trace([0, 1], 2, prefer_other_copy=1)
    # equal scores need equal ages: blocks 0 and 1 tie, block 1 has a copy and goes first
    idx = make_idx([0, 0], [90, 90], flags=[1, 1 | 8])
    assert o.select_victims(idx, 100, 0, 2)[0].tolist() == [1, 0]
    o.p.prefer_other_copy = 0
    assert o.select_victims(idx, 100, 0, 2)[0].tolist() == [0, 1]
