"""The configurations run as traces through the closed-loop harness, CUDA library teacher-forced against the
oracle at every call: victim lists (both tiers) and prefetch lists bit for bit (and re-checked on the device by
cs_validate_selection), slot lists checked by cs_validate_move_lists, learner state and both KV pools byte for
byte at checkpoints.  Tiny in full (its real 512 KiB blocks and pool sizes); the 8B- and 70B-shaped configurations
with their full index (80,000 / 52,000 entries) and agent structure and the KV geometry cut to what the oracle can
copy in seconds; session = chain and the paper's single current-agent register; both workload shapes."""
import pytest

torch = pytest.importorskip("torch")

from tests import closed_loop as CL

pytestmark = pytest.mark.gpu
SMALL = CL.KVGeometry(n_layers=2, n_kv_heads=1, head_dim=8)            # 1 KiB blocks


@pytest.mark.parametrize("workload,chain_mode", [("anchor", "session"), ("anchor", "single"), ("history", "session")])
def test_tiny_config_in_full(workload, chain_mode):
    geo = CL.KVGeometry(n_layers=8)                                     # the configuration's own 512 KiB blocks
    loop = CL.make_loop("tiny", geo, workload=workload, chain_mode=chain_mode, gpu=True)
    st = loop.run(10 ** 9, check_every=50)                              # all 200 invocations
    loop.check_invariants()
    assert st.evicted > 0 and st.offloaded > 0 and st.prefetched > 0 and st.select_calls > 100


@pytest.mark.parametrize("name,workload,chain_mode", [
    ("llama8b", "anchor", "session"), ("llama8b", "history", "single"),
    ("llama70b", "anchor", "session"), ("llama70b", "history", "single")])
def test_full_index_configs_as_traces(name, workload, chain_mode):
    loop = CL.make_loop(name, SMALL, workload=workload, chain_mode=chain_mode, gpu=True, n_invocations=2600)
    n_steps = len(loop.tr.step_off) - 1
    assert n_steps >= 500
    st = loop.run(520, check_every=130)
    loop.check_invariants()
    assert st.evicted > 0 and st.offloaded > 0 and st.select_calls >= 500
