"""Shared helpers of the GPU parity tests: build both sides from one seeded input and compare."""
import numpy as np

from oracle import cs_oracle as orc
from tests import synth

REL_TOL = 1e-6          # fp32 reuse scores vs the fp64 oracle (relative)
R_ABS_TOL = 1e-5        # predictability: sum of A^2 entropy terms
R_FRAGILE = 1e-4        # inputs whose R lies this close to r_min are rejected as threshold-fragile


def oracle_params(p) -> orc.Params:
    """cs_params (ctypes) -> oracle Params."""
    return orc.Params(n_agents=p.n_agents, n_chains=p.n_chains, block_tokens=p.block_tokens, e_max=p.e_max,
                      eps=p.eps, tau=p.tau, lam=p.lambda_, delta=p.delta, r_min=p.r_min,
                      prefer_other_copy=p.prefer_other_copy)


def compare_model(cs, o: orc.Oracle):
    """Learner / scorer state of the CUDA context against the oracle's."""
    m = cs.get_model()
    assert np.array_equal(m["C"], o.C), "transition counts differ"
    assert np.array_equal(m["cur"], o.cur), "per-chain current agents differ"
    assert m["last_agent"] == int(o.last_agent[0])
    assert np.all(np.abs(m["P"].astype(np.float64) - o.P64) <= REL_TOL * o.P64), "Eq. 3 beyond 1e-6"
    assert np.array_equal(m["P"], o.P32), "Eq. 3 canonical fp32 differs"
    assert np.array_equal(m["amax"], o.amax), "row arg-max differs"
    assert abs(m["R"] - o.R) <= R_ABS_TOL, ("R", m["R"], o.R)
    hops = np.where(o.E == orc.INF, 0xFFFF, np.minimum(o.E, 0xFFFE)).astype(np.uint16)
    assert np.array_equal(m["hops"], hops), "BFS hop table differs"
    assert np.array_equal(m["fsurv"], o.fsurv32), "survival factor differs"
    return m


def assert_list_matches(ids_gpu, n_gpu, ids_orc, n_orc, score64):
    """Bit-exact lists; a differing position is tolerated only between entries whose oracle
    scores agree within REL_TOL (several correct answers), and then the id sets must agree
    up to such entries.  Returns the number of tolerated positions (0 expected)."""
    ids_gpu = np.asarray(ids_gpu, np.uint32)
    assert n_gpu == n_orc, ("n_out", n_gpu, n_orc)
    assert np.all(ids_gpu[n_gpu:] == orc.ID_NONE), "tail not padded with the sentinel"
    diff = np.flatnonzero(ids_gpu[:n_orc] != ids_orc[:n_orc])
    for pos in diff:
        a, b = float(score64[ids_gpu[pos]]), float(score64[ids_orc[pos]])
        assert abs(a - b) <= REL_TOL * max(abs(a), abs(b)), ("list differs beyond score tolerance", pos)
    assert len(np.unique(ids_gpu[:n_gpu])) == n_gpu, "duplicate ids"
    return len(diff)


def reject_fragile(o: orc.Oracle):
    assert abs(o.R - o.p.r_min) >= R_FRAGILE, "threshold-fragile input: choose another seed"


def pool_view(buf_u8: np.ndarray, layout: int, n_slots: int, n_layers: int, chunk: int):
    """[slot, layer, plane, byte] view of a flat pool."""
    if layout == synth.LAYER_MAJOR:
        return buf_u8.reshape(n_layers, 2, n_slots, chunk).transpose(2, 0, 1, 3)
    return buf_u8.reshape(n_slots, n_layers, 2, chunk)
