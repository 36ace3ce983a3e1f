"""The closed-loop harness itself, with the oracle alone (no GPU): the simulated cache stays consistent,
the loop is deterministic, evicted blocks come back from the host tier byte for byte, and the two
workload shapes have the reuse structure they are meant to have."""
import numpy as np

from tests import closed_loop as CL

GEO = CL.KVGeometry(n_layers=2, n_kv_heads=1, head_dim=8)


def test_simulated_cache_stays_consistent_and_deterministic():
    runs = []
    for _ in range(2):
        loop = CL.make_loop("tiny", GEO, workload="anchor")
        for s in range(199):
            loop.step(s)
            if s % 10 == 0:
                loop.check_invariants()
        loop.check_invariants()
        runs.append((loop.stats.gpu_hit_tokens, loop.stats.evicted, loop.stats.offloaded, loop.stats.prefetched,
                     loop.oe.gpu.copy(), loop.oe.host.copy()))
    assert runs[0][:4] == runs[1][:4]
    assert np.array_equal(runs[0][4], runs[1][4]) and np.array_equal(runs[0][5], runs[1][5])
    st = loop.stats
    assert st.evicted > 0 and st.offloaded > 0 and st.prefetched > 0 and st.host_dropped > 0      # every path of the loop ran
    assert 0.0 < st.gpu_hit_rate <= st.hit_rate < 1.0


def test_blocks_in_the_pools_are_the_blocks_the_maps_say():
    """After evictions, offloads, reloads and prefetches every cached block still holds the bytes written for its key."""
    loop = CL.make_loop("tiny", GEO, workload="anchor")
    loop.run(150)
    g = loop.geo
    from tests import helpers as H
    gv = H.pool_view(loop.oe.gpu, g.gpu_layout, loop.G, g.n_layers, g.chunk)
    hv = H.pool_view(loop.oe.host, g.host_layout, loop.Hs, g.n_layers, g.chunk)
    for key, slot in loop.gpu_of.items():
        assert np.array_equal(gv[slot].reshape(-1), CL.block_content(key, g.block_bytes)), key
    for key, slot in loop.host_of.items():
        assert np.array_equal(hv[slot].reshape(-1), CL.block_content(key, g.block_bytes)), key


def test_history_workload_reuses_history_blocks_and_fixed_contexts():
    """Fixed contexts are shared by every invocation of an agent, history blocks by the later turns of a session
    (the paper reports 49-173 uses against 12-15, Sec. 2.2); fresh suffixes are used once."""
    loop = CL.make_loop("llama8b", GEO, workload="history", with_pools=False, gpu_blocks=4000, host_blocks=8000,
                        n_invocations=1500)
    loop.run(10 ** 9)
    a, h = CL.history_kinds(loop)
    assert a > 40 and 6.0 < h < 20.0 and h < a          # history blocks: about a dozen uses; fixed contexts: many more
    assert loop.stats.hit_rate > 0.5
    anchor = CL.make_loop("llama8b", GEO, workload="anchor", with_pools=False, gpu_blocks=4000, host_blocks=8000, n_invocations=300)
    anchor.run(10 ** 9)
    assert max(n for k, n in anchor.uses.items() if k[0] == "S") == 1
