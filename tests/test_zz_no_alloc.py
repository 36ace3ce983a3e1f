"""cs_select_victims_static: victim selection for callers that cannot allocate device memory
(an engine that owns the whole GPU, a hook that runs while allocation is forbidden).  Its
scratch is a static array inside the library, so the call takes no context and no workspace.

Checked through the C ABI against cs_select_victims() on the same index and against the CPU
oracle, on calls in a row whose parameters differ (the array keeps the previous call's contents,
which must not leak into the next; the agent count and the recency table change size between
calls).  This file sorts last on purpose: a run that stops at the first failure has then already
run every other test."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import cs_oracle as orc
from paper_2608_14624_b200 import binding as cs
from tests import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def up(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def test_static_scratch_select_matches_workspace_select_twice():
    cfg = synth.CONFIGS["tiny"]
    n = 50_000 + 7                                    # several tiles and a ragged tail, below the limit
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=n, block_tokens=cfg.block_tokens)
    c = cs.CacheScout(p, DEV)
    o = orc.Oracle(H.oracle_params(p))
    tr = synth.make_trace(cfg)
    c.observe_invocations(up(tr.chain), up(tr.agent), up(tr.evflags))
    o.observe(tr.chain, tr.agent, tr.evflags)
    fsurv = up(c.get_model()["fsurv"])                # an input the caller already owns
    idx = synth.make_block_index(cfg, n=n)
    d = cs.DeviceIndex.from_host(idx, DEV)
    ids_s = torch.empty(4096, dtype=torch.int32, device=DEV)
    n_s = torch.zeros(4, dtype=torch.int32, device=DEV)
    # calls in a row, with another time, tier and k each: stale scratch must not matter
    for now, tier, k in ((100_000, 0, 4096), (100_321, 1, 333), (100_321, 0, 1)):
        ids_w, n_w = c.select_victims(d, now, tier, k)
        ids_s.fill_(7)
        cs.cs_select_victims_static(p, fsurv, d.struct(), now, tier, k, ids_s, n_s)
        torch.cuda.synchronize()
        assert int(n_s[0].item()) == int(n_w.item()) > 0
        assert torch.equal(ids_s[:k], ids_w[:k])
        s64, s32 = o.scores(idx, now)
        o_ids, o_n = o.select_victims(idx, now, tier, k, s32)
        assert H.assert_list_matches(ids_s[:k].cpu().numpy().view(np.uint32), int(n_s[0].item()), o_ids, o_n, s64) == 0
    assert c.get_status() == 0


def test_static_scratch_select_with_changing_parameters_against_the_oracle():
    """(4 agents, lambda 0.1) -> (256 agents, lambda 0.0056, a recency table of ~3,900 ages, copy preference) -> 1,024 agents -> the first
    again: every list equals the oracle's, and no call allocates device memory."""
    now = 100_000
    cases = []
    for cfg, kw, n, k in ((synth.CONFIGS["tiny"], dict(lam=0.1), 20_000 + 3, 500),
                          (synth.shrink(synth.CONFIGS["meta1m"], n_chains=4, sessions=4),
                           dict(lam=0.0056, delta=0.02, prefer_other_copy=1), 65_536, 3000),
                          (synth.shrink(synth.CONFIGS["llama70b"], n_agents=1024, n_chains=2, sessions=2),
                           dict(lam=0.0056), 9_000, 64)):
        p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=64, block_tokens=cfg.block_tokens, **kw)
        o = orc.Oracle(H.oracle_params(p))
        tr = synth.make_trace(cfg, n_invocations=400)
        o.observe(tr.chain, tr.agent, tr.evflags)
        idx = synth.make_block_index(cfg, n=n)
        cases.append((p, o, idx, cs.DeviceIndex.from_host(idx, DEV), up(o.fsurv32), k))
    ids_s = torch.empty(4096, dtype=torch.int32, device=DEV)
    n_s = torch.zeros(4, dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()
    before = None
    for rep, which in enumerate((0, 1, 0, 2, 1, 0)):
        p, o, idx, d, fsurv, k = cases[which]
        tier = rep & 1
        s64, s32 = o.scores(idx, now + rep)
        o_ids, o_n = o.select_victims(idx, now + rep, tier, k, s32)
        ids_s.fill_(7)
        cs.cs_select_victims_static(p, fsurv, d.struct(), now + rep, tier, k, ids_s, n_s)
        torch.cuda.synchronize()
        assert H.assert_list_matches(ids_s[:k].cpu().numpy().view(np.uint32), int(n_s[0].item()), o_ids, o_n, s64) == 0
        mem = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated())
        if rep >= 1:                                   # (the first call may load the kernels' code)
            assert before is None or mem == before, "a static-scratch call changed the device's free memory"
            before = mem


def test_static_scratch_select_rejects_sizes_beyond_its_array_and_memory_the_gpu_cannot_address():
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
    # a pageable host array in place of a device array is refused on the host: the GPU never sees the pointer
    host_idx = synth.make_block_index(cfg, n=1024)
    pageable = torch.from_numpy(host_idx.last_access.copy())
    assert not pageable.is_pinned()
    bad = cs.DeviceIndex(ok.agent, ok.depth, ok.ref_count, ok.flags, pageable, ok.n_tokens)
    cnt.fill_(77)
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_select_victims_static(p, fsurv, bad.struct(), 1, 0, 8, out, cnt)
    assert e.value.code == cs.CS_EINVAL
    with pytest.raises(cs.CacheScoutError) as e:
        cs.cs_select_victims_static(p, torch.ones(cfg.n_agents, dtype=torch.float32), ok.struct(), 1, 0, 8, out, cnt)
    assert e.value.code == cs.CS_EINVAL
    torch.cuda.synchronize()
    assert int(cnt[0].item()) == 77                    # nothing ran
