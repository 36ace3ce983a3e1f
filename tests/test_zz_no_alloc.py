"""cs_select_victims_static: victim selection for callers that cannot allocate device memory
(an engine that owns the whole GPU, a hook that runs while allocation is forbidden).  Its
scratch is a static array inside the library, so the call takes no context and no workspace.

Checked through the C ABI against cs_select_victims() on the same index, twice in a row (the
array keeps the first call's contents, which must not leak into the second), bit for bit: both
entry points run the same kernels, so the lists must be identical.  This file sorts last on
purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2608_14624_b200 import binding as cs
from paper_2608_14624_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def up(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def test_static_scratch_select_matches_workspace_select_twice():
    cfg = synth.CONFIGS["tiny"]
    n = 50_000 + 7                                    # several tiles and a ragged tail, below the limit
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=n, block_tokens=cfg.block_tokens)
    c = cs.CacheScout(p, DEV)
    tr = synth.make_trace(cfg)
    c.observe_invocations(up(tr.chain), up(tr.agent), up(tr.evflags))
    fsurv = up(c.get_model()["fsurv"])                # an input the caller already owns
    idx = synth.make_block_index(cfg, n=n)
    d = cs.DeviceIndex.from_host(idx, DEV)
    ids_s = torch.empty(4096, dtype=torch.int32, device=DEV)
    n_s = torch.zeros(4, dtype=torch.int32, device=DEV)
    # two calls in a row, the second with another time, tier and k: stale scratch must not matter
    for now, tier, k in ((100_000, 0, 4096), (100_321, 1, 333), (100_321, 0, 1)):
        ids_w, n_w = c.select_victims(d, now, tier, k)
        ids_s.fill_(7)
        cs.cs_select_victims_static(p, fsurv, d.struct(), now, tier, k, ids_s, n_s)
        torch.cuda.synchronize()
        assert int(n_s[0].item()) == int(n_w.item()) > 0
        assert torch.equal(ids_s[:k], ids_w[:k])
    assert c.get_status() == 0


def test_static_scratch_select_rejects_sizes_beyond_its_array():
    cfg = synth.CONFIGS["tiny"]
    p = cs.make_params(n_agents=cfg.n_agents)
    fsurv = torch.ones(cfg.n_agents, dtype=torch.float32, device=DEV)
    big = cs.DeviceIndex.from_host(synth.make_block_index(cfg, n=cs.CS_STATIC_MAX_BLOCKS + 16), DEV)
    out, cnt = torch.empty(16, dtype=torch.int32, device=DEV), torch.zeros(4, dtype=torch.int32, device=DEV)
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_select_victims_static(p, fsurv, big.struct(), 1, 0, 8, out, cnt)
    assert e.value.code == cs.CS_ECAPACITY
    ok = cs.DeviceIndex.from_host(synth.make_block_index(cfg, n=1024), DEV)
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_select_victims_static(p, fsurv, ok.struct(), 1, 0, cs.CS_STATIC_MAX_BLOCKS + 1, out, cnt)
    assert e.value.code == cs.CS_ECAPACITY
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_select_victims_static(p, None, ok.struct(), 1, 0, 8, out, cnt)
    assert e.value.code == cs.CS_EINVAL
