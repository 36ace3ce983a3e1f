"""Closed-loop cache harness (test infrastructure): runs a configuration AS A TRACE.

It stands in for the agent framework and the serving engine around the library (Algorithm 1's main
loop): every scheduler step takes the step's invocations from a seeded trace, builds each prompt as
a list of blocks, looks the blocks up, allocates GPU slots for what is missing, evicts under memory
pressure through the victim selection, offloads evicted blocks to the host tier, reloads host hits,
and between steps prefetches the candidates the prefetch selection ranks first.

Two engines can sit behind the loop: the CPU oracle (`OracleEngine`) and the CUDA library through
its C ABI (`GpuEngine`).  With both (`teacher-forced`), every call's output is compared (lists bit
for bit, pools byte for byte at checkpoints) and the ORACLE's output advances the state, so one
mismatch cannot cascade.  With the oracle alone the loop yields the hit rate of a policy, which is
reported as context (cached prompt tokens / prompt tokens, the paper's definition in Sec. 5.1).

Simplifications, stated once: a block's identity is a key (anchor block j of agent a; history block
j of session s; suffix block j of invocation i) standing in for the engine's chained prefix hash;
blocks are looked up independently; transfers complete within the step that issues them.

Workloads: "anchor" -- prompt = the agent's fixed context + a fresh suffix (the paper's Sec. 2.2
structure); "history" -- prompt = fixed context + the session's accumulated history + a fresh
suffix, the suffix joining the history afterwards (history blocks are reused on every later turn
of their session, fixed contexts by every invocation of their agent).
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

from oracle import cs_oracle as orc
from tests import synth

from . import helpers as H

NONE = orc.ID_NONE


@dataclass
class KVGeometry:
    n_layers: int
    n_kv_heads: int = 8
    head_dim: int = 128
    block_tokens: int = 16
    elem_bytes: int = 2
    gpu_layout: int = synth.LAYER_MAJOR
    host_layout: int = synth.BLOCK_MAJOR

    @property
    def chunk(self) -> int:
        return self.block_tokens * self.n_kv_heads * self.head_dim * self.elem_bytes

    @property
    def block_bytes(self) -> int:
        return self.n_layers * 2 * self.chunk


def block_content(key: Tuple, nbytes: int) -> np.ndarray:
    """Deterministic stand-in for the KV values a prefill would write for this block."""
    seed = zlib.crc32(repr(key).encode())
    return np.random.Generator(np.random.PCG64(seed)).integers(0, 256, nbytes, dtype=np.uint8)


# ---- engines ---------------------------------------------------------------------------------------------
class OracleEngine:
    def __init__(self, params: orc.Params, geo: KVGeometry, G: int, Hs: int, with_pools: bool = True):
        self.o = orc.Oracle(params)
        self.geo, self.G, self.Hs = geo, G, Hs
        self.gpu = np.zeros(G * geo.block_bytes, np.uint8) if with_pools else None
        self.host = np.zeros(Hs * geo.block_bytes, np.uint8) if with_pools else None
        self._s32 = None

    def observe(self, chain, agent, evflags):
        self.o.observe(chain, agent, evflags)

    def begin_selects(self, idx, now):
        self.s64, self._s32 = self.o.scores(idx, now)

    def select_victims(self, idx, now, tier, k):
        return self.o.select_victims(idx, now, tier, k, self._s32)

    def select_prefetch(self, idx, now, k):
        return self.o.select_prefetch(idx, now, k, self._s32)

    def write_block(self, slot, data):
        if self.gpu is not None:
            g = self.geo
            H.pool_view(self.gpu, g.gpu_layout, self.G, g.n_layers, g.chunk)[slot] = data.reshape(g.n_layers, 2, g.chunk)

    def offload(self, src, dst):
        if self.gpu is not None:
            g = self.geo
            orc.move_blocks(self.gpu, g.gpu_layout, self.G, self.host, g.host_layout, self.Hs, g.n_layers, g.chunk, src, dst)

    def prefetch(self, src, dst):
        if self.gpu is not None:
            g = self.geo
            orc.move_blocks(self.host, g.host_layout, self.Hs, self.gpu, g.gpu_layout, self.G, g.n_layers, g.chunk, src, dst)


class GpuEngine:
    """The CUDA library behind the same calls (device pools, pinned host tier, ids offset by G on the host tier)."""

    def __init__(self, params, geo: KVGeometry, G: int, Hs: int, device="cuda:0", validate=True):
        import torch

        from paper_2608_14624_b200 import binding as cs
        self.torch, self.cs, self.dev = torch, cs, device
        self.geo, self.G, self.Hs, self.validate = geo, G, Hs, validate
        self.c = cs.CacheScout(params, device)
        self.gpu_buf = torch.zeros(G * geo.block_bytes, dtype=torch.uint8, device=device)
        self.host_buf = torch.zeros(Hs * geo.block_bytes, dtype=torch.uint8).pin_memory()
        kw = dict(n_kv_heads=geo.n_kv_heads, head_dim=geo.head_dim, block_tokens=geo.block_tokens, elem_bytes=geo.elem_bytes)
        self.gpu_pool = cs.KVPool(self.gpu_buf, G, geo.gpu_layout, geo.n_layers, **kw)
        self.host_pool = cs.KVPool(self.host_buf, Hs, geo.host_layout, geo.n_layers, first_id=G, **kw)
        self.d = None

    def up(self, a):
        return self.torch.from_numpy(np.ascontiguousarray(a)).to(self.dev)

    def observe(self, chain, agent, evflags):
        self.c.observe_invocations(self.up(chain), self.up(agent), self.up(evflags))

    def begin_selects(self, idx, now):
        self.d = self.cs.DeviceIndex.from_host(idx, self.dev)

    def select_victims(self, idx, now, tier, k):
        ids, n = self.c.select_victims(self.d, now, tier, k)
        if self.validate:
            self.c.validate_selection(self.d, now, False, tier, k, ids, n)
        return ids.cpu().numpy().view(np.uint32)[:k], int(n.item())

    def select_prefetch(self, idx, now, k):
        ids, n = self.c.select_prefetch(self.d, now, k)
        if self.validate:
            self.c.validate_selection(self.d, now, True, 1, k, ids, n)
        return ids.cpu().numpy().view(np.uint32)[:k], int(n.item())

    def write_block(self, slot, data):
        g = self.geo
        t = self.up(data.reshape(g.n_layers, 2, g.chunk))
        if g.gpu_layout == synth.LAYER_MAJOR:
            self.gpu_buf.view(g.n_layers, 2, self.G, g.chunk)[:, :, slot, :] = t
        else:
            self.gpu_buf.view(self.G, g.n_layers, 2, g.chunk)[slot] = t

    def offload(self, src, dst):
        if len(src):
            s, d = self.up(np.asarray(src, np.uint32)), self.up(np.asarray(dst, np.uint32) + np.uint32(self.G))
            if self.validate:
                self.c.validate_move_lists(self.gpu_pool, self.host_pool, s, d)
            self.c.offload_blocks(self.gpu_pool, self.host_pool, s, d)

    def prefetch(self, src, dst):
        if len(src):
            s, d = self.up(np.asarray(src, np.uint32) + np.uint32(self.G)), self.up(np.asarray(dst, np.uint32))
            if self.validate:
                self.c.validate_move_lists(self.host_pool, self.gpu_pool, s, d)
            self.c.prefetch_blocks(self.host_pool, self.gpu_pool, s, d)

    def pools(self):
        self.torch.cuda.synchronize()
        return self.gpu_buf.cpu().numpy(), self.host_buf.numpy()


# ---- the loop ----------------------------------------------------------------------------------------------
@dataclass
class LoopStats:
    prompt_tokens: int = 0
    gpu_hit_tokens: int = 0
    host_hit_tokens: int = 0
    evicted: int = 0
    offloaded: int = 0
    prefetched: int = 0
    prefetch_used: int = 0
    host_dropped: int = 0
    select_calls: int = 0
    uncached_blocks: int = 0
    reuse: Dict[str, List[int]] = field(default_factory=dict)

    @property
    def hit_rate(self) -> float:
        return (self.gpu_hit_tokens + self.host_hit_tokens) / max(1, self.prompt_tokens)

    @property
    def gpu_hit_rate(self) -> float:
        return self.gpu_hit_tokens / max(1, self.prompt_tokens)


class ClosedLoop:
    def __init__(self, cfg: synth.Config, geo: KVGeometry, params: orc.Params, oracle: OracleEngine,
                 gpu: Optional[GpuEngine] = None, workload: str = "anchor", n_invocations: Optional[int] = None,
                 reserve: int = 0, pin_prob: float = 0.01, max_history_blocks: int = 1024, seed_stream: int = 31):
        self.cfg, self.geo, self.p = cfg, geo, params
        self.oe, self.ge = oracle, gpu
        self.workload = workload
        self.G, self.Hs = cfg.gpu_blocks, cfg.host_blocks
        self.N = self.G + self.Hs
        self.tr = synth.make_trace(cfg, n_invocations=n_invocations)
        self.rng = synth.rng_for(cfg, seed_stream)
        A, T = cfg.n_agents, cfg.block_tokens
        lo, hi = cfg.anchor_tokens
        self.anchor_tokens = self.rng.integers(lo, hi + 1, size=A)
        self.idx = synth.BlockIndex(
            agent=np.zeros(self.N, np.uint16), depth=np.zeros(self.N, np.uint16), ref_count=np.zeros(self.N, np.uint8),
            flags=np.zeros(self.N, np.uint8), last_access=np.zeros(self.N, np.uint32),
            n_tokens=np.full(self.N, T, np.uint8), anchor_blocks=(self.anchor_tokens // T).astype(np.uint16))
        self.idx.flags[self.G:] = synth.FLAG_TIER_HOST
        self.free_gpu = list(range(self.G - 1, -1, -1))
        self.free_host = list(range(self.Hs - 1, -1, -1))
        self.gpu_of: Dict[Tuple, int] = {}
        self.host_of: Dict[Tuple, int] = {}
        self.key_of_gpu: Dict[int, Tuple] = {}
        self.key_of_host: Dict[int, Tuple] = {}
        self.refs: List[int] = []
        self.pins: List[Tuple[int, int]] = []           # (expiry step, gpu slot)
        self.history: Dict[int, List[Tuple]] = {}       # session -> keys of its history blocks
        self.max_history_blocks = max_history_blocks
        self.reserve = reserve
        self.pin_prob = pin_prob
        self.stats = LoopStats()
        self.uses: Dict[Tuple, int] = {}
        self.now0 = 1000
        self.inv_counter = 0

    # -- prompts ---------------------------------------------------------------------------------------------
    def prompt_blocks(self, agent: int, session: int) -> List[Tuple[Tuple, int]]:
        T = self.cfg.block_tokens
        out = []
        n_anchor = int(self.anchor_tokens[agent])
        for j in range(n_anchor // T):
            out.append((("A", agent, j), T))
        if n_anchor % T:
            out.append((("A", agent, n_anchor // T), n_anchor % T))
        if self.workload == "history":
            for key in self.history.get(session, []):
                out.append((key, T))
        lo, hi = self.cfg.suffix_tokens
        n_suf = int(self.rng.integers(lo, hi + 1))
        self.inv_counter += 1
        suffix = [(("S", self.inv_counter, j), T) for j in range(n_suf // T)]
        if n_suf % T:
            suffix.append((("S", self.inv_counter, n_suf // T), n_suf % T))
        out.extend(suffix)
        if self.workload == "history":                   # the turn's full blocks join the session's history afterwards
            h = self.history.setdefault(session, [])
            h.extend(k for k, nt in suffix if nt == T)
            del h[:-self.max_history_blocks]
        return out

    # -- both engines, compared -------------------------------------------------------------------------------
    def _both(self, name, *args):
        want = getattr(self.oe, name)(*args)
        if self.ge is not None:
            got = getattr(self.ge, name)(*args)
            if name.startswith("select"):
                assert H.assert_list_matches(got[0], got[1], want[0], want[1], self.oe.s64) == 0, (name, args[1:])
        return want

    def _set_gpu_entry(self, slot, agent, depth, ntok, now, ref, flags):
        i = self.idx
        i.agent[slot], i.depth[slot], i.n_tokens[slot] = agent, min(depth, 0xFFFF), ntok
        i.last_access[slot], i.ref_count[slot], i.flags[slot] = now, ref, flags

    def _evict(self, need: int, now: int):
        """Frees at least `need` GPU slots (if that many entries are evictable): victims by Algorithm 1's Evict,
        offloaded to the host tier unless a host copy exists; a full host tier is thinned by the same selector."""
        k = max(self.cfg.k_victims, need)
        self._both("begin_selects", self.idx, now)
        ids, n = self._both("select_victims", self.idx, now, 0, k)
        self.stats.select_calls += 1
        victims = [int(v) for v in ids[:n]]
        to_host = [v for v in victims if not (self.idx.flags[v] & synth.FLAG_OTHER_COPY)]
        short = len(to_host) - len(self.free_host)
        if short > 0:                                     # host tier full: drop its lowest-scored entries
            hk = max(self.cfg.k_victims, short)
            hids, hn = self._both("select_victims", self.idx, now, 1, hk)
            self.stats.select_calls += 1
            for h in hids[:hn]:
                self._drop_host_entry(int(h) - self.G)
            self.stats.host_dropped += int(hn)
        src, dst = [], []
        for v in victims:
            key = self.key_of_gpu.pop(v)
            del self.gpu_of[key]
            if self.idx.flags[v] & synth.FLAG_OTHER_COPY:
                h = self.host_of[key]                     # the host copy stays; it no longer has a GPU twin
                self.idx.flags[self.G + h] &= np.uint8(~synth.FLAG_OTHER_COPY & 0xFF)
                self.idx.last_access[self.G + h] = self.idx.last_access[v]
            elif self.free_host:
                h = self.free_host.pop()
                src.append(v)
                dst.append(h)
                self.host_of[key] = h
                self.key_of_host[h] = key
                e = self.G + h
                self.idx.agent[e], self.idx.depth[e], self.idx.n_tokens[e] = self.idx.agent[v], self.idx.depth[v], self.idx.n_tokens[v]
                self.idx.last_access[e], self.idx.ref_count[e] = self.idx.last_access[v], 0
                self.idx.flags[e] = synth.FLAG_VALID | synth.FLAG_TIER_HOST
            self.idx.flags[v] = 0
            self.free_gpu.append(v)
        self._both("offload", src, dst)
        self.stats.evicted += len(victims)
        self.stats.offloaded += len(src)

    def _drop_host_entry(self, h: int):
        key = self.key_of_host.pop(h)
        del self.host_of[key]
        e = self.G + h
        if self.idx.flags[e] & synth.FLAG_OTHER_COPY:
            g = self.gpu_of[key]
            self.idx.flags[g] &= np.uint8(~synth.FLAG_OTHER_COPY & 0xFF)
        self.idx.flags[e] = synth.FLAG_TIER_HOST
        self.free_host.append(h)

    # -- one scheduler step ------------------------------------------------------------------------------------
    def step(self, s: int):
        tr, st = self.tr, self.stats
        now = self.now0 + s
        lo, hi = int(tr.step_off[s]), int(tr.step_off[s + 1])
        for slot in self.refs:                            # requests of the previous step are done
            self.idx.ref_count[slot] -= 1
        self.refs = []
        keep = []
        for expiry, slot in self.pins:
            if expiry <= s:
                self.idx.flags[slot] &= np.uint8(~synth.FLAG_PINNED & 0xFF)
            else:
                keep.append((expiry, slot))
        self.pins = keep
        self._both("observe", tr.chain[lo:hi], tr.agent[lo:hi], tr.evflags[lo:hi])
        # look-ups
        alloc = []                                        # (key, agent, depth, ntok, host slot or None)
        seen = set()
        for e in range(lo, hi):
            a, sess = int(tr.agent[e]), int(tr.session[e])
            for depth, (key, ntok) in enumerate(self.prompt_blocks(a, sess)):
                st.prompt_tokens += ntok
                self.uses[key] = self.uses.get(key, 0) + 1
                g = self.gpu_of.get(key)
                if g is not None:
                    st.gpu_hit_tokens += ntok
                    self.idx.last_access[g], self.idx.agent[g] = now, a
                    if self.idx.ref_count[g] < 255:
                        self.idx.ref_count[g] += 1
                        self.refs.append(g)
                    continue
                if key in seen:                           # a second request of this step for a block being brought in
                    continue
                seen.add(key)
                h = self.host_of.get(key)
                if h is not None:
                    st.host_hit_tokens += ntok
                alloc.append((key, a, depth, ntok, h))
        # allocation under pressure
        if len(alloc) > len(self.free_gpu):
            self._evict(len(alloc) - len(self.free_gpu), now)
        pre_src, pre_dst = [], []
        for key, a, depth, ntok, h in alloc:
            if not self.free_gpu:
                st.uncached_blocks += 1                   # nothing evictable: served without being cached
                continue
            g = self.free_gpu.pop()
            self.gpu_of[key] = g
            self.key_of_gpu[g] = key
            flags = synth.FLAG_VALID
            h = self.host_of.get(key)                     # (the eviction above may have dropped the host copy)
            if h is not None:
                pre_src.append(h)
                pre_dst.append(g)
                flags |= synth.FLAG_OTHER_COPY
                self.idx.flags[self.G + h] |= synth.FLAG_OTHER_COPY
            else:
                if self.oe.gpu is not None or self.ge is not None:
                    data = block_content(key, self.geo.block_bytes)
                    self.oe.write_block(g, data)
                    if self.ge is not None:
                        self.ge.write_block(g, data)
                if self.rng.random() < self.pin_prob:
                    flags |= synth.FLAG_PINNED
                    self.pins.append((s + int(self.rng.integers(1, 21)), g))
            self._set_gpu_entry(g, a, depth, ntok, now, 1, flags)
            self.refs.append(g)
        self._both("prefetch", pre_src, pre_dst)
        # between steps: warm what the predicted next agent needs (BetweenStep), into free slots above the reserve
        room = len(self.free_gpu) - self.reserve
        if room > 0 and self.cfg.k_prefetch:
            self._both("begin_selects", self.idx, now)
            ids, n = self._both("select_prefetch", self.idx, now, self.cfg.k_prefetch)
            st.select_calls += 1
            src, dst = [], []
            for e in ids[:min(n, room)]:
                h = int(e) - self.G
                key = self.key_of_host[h]
                g = self.free_gpu.pop()
                self.gpu_of[key] = g
                self.key_of_gpu[g] = key
                self._set_gpu_entry(g, int(self.idx.agent[e]), int(self.idx.depth[e]), int(self.idx.n_tokens[e]), now, 0,
                                    synth.FLAG_VALID | synth.FLAG_OTHER_COPY)
                self.idx.flags[e] |= synth.FLAG_OTHER_COPY
                src.append(h)
                dst.append(g)
            self._both("prefetch", src, dst)
            st.prefetched += len(src)

    def check_state(self):
        """Teacher-forced checkpoint: learner state and both pools, GPU against oracle."""
        if self.ge is None:
            return
        H.compare_model(self.ge.c, self.oe.o)
        gpu, host = self.ge.pools()
        assert np.array_equal(gpu, self.oe.gpu), "GPU pool differs from the oracle's"
        assert np.array_equal(host, self.oe.host), "host tier differs from the oracle's"
        assert self.ge.c.get_status() == 0

    def check_invariants(self):
        """Host-side consistency of the simulated cache (no engine involved)."""
        i = self.idx
        valid_gpu = np.flatnonzero(i.flags[:self.G] & synth.FLAG_VALID)
        assert set(valid_gpu.tolist()) == set(self.key_of_gpu) == set(self.gpu_of.values())
        valid_host = np.flatnonzero(i.flags[self.G:] & synth.FLAG_VALID)
        assert set(valid_host.tolist()) == set(self.key_of_host) == set(self.host_of.values())
        assert len(self.free_gpu) + len(valid_gpu) == self.G and len(self.free_host) + len(valid_host) == self.Hs
        assert not (set(self.free_gpu) & set(valid_gpu.tolist()))
        for key, g in self.gpu_of.items():
            both = key in self.host_of
            assert bool(i.flags[g] & synth.FLAG_OTHER_COPY) == both, key
            if both:
                assert i.flags[self.G + self.host_of[key]] & synth.FLAG_OTHER_COPY
        for key, h in self.host_of.items():
            assert bool(i.flags[self.G + h] & synth.FLAG_OTHER_COPY) == (key in self.gpu_of), key
        assert np.all(i.flags[self.G:] & synth.FLAG_TIER_HOST) and not np.any(i.flags[:self.G] & synth.FLAG_TIER_HOST)

    def reuse_counts(self) -> Dict[str, float]:
        """Mean number of uses per block, by kind (A fixed context, H session history, S fresh suffix)."""
        out = {}
        for kind in ("A", "H", "S"):
            v = [n for k, n in self.uses.items() if k[0] == kind]
            if v:
                out[kind] = float(np.mean(v))
        return out

    def run(self, n_steps: int, check_every: int = 0):
        n_steps = min(n_steps, len(self.tr.step_off) - 1)
        for s in range(n_steps):
            self.step(s)
            if check_every and (s + 1) % check_every == 0:
                self.check_state()
        self.check_state()
        return self.stats


def history_kinds(loop: ClosedLoop):
    """In the history workload, blocks that joined a session's history keep their suffix key; count them apart."""
    hist = {k for h in loop.history.values() for k in h}
    a = [n for k, n in loop.uses.items() if k[0] == "A"]
    hh = [n for k, n in loop.uses.items() if k in hist]
    return (float(np.mean(a)) if a else 0.0), (float(np.mean(hh)) if hh else 0.0)


def make_loop(name: str, geo: KVGeometry, workload="anchor", chain_mode="session", policy="cachescout", gpu=False,
              n_invocations=None, device="cuda:0", with_pools=True, gpu_blocks=None, host_blocks=None, **param_kw):
    """A configuration as a closed loop.  policy "lru": tau > 1 removes every edge, survival is flat and the
    selection is exact LRU (Sec. 3.3's fallback), the comparison point for the hit rate."""
    cfg = synth.CONFIGS[name]
    kw = {}
    if chain_mode == "single":
        kw["n_chains"] = 1
    if gpu_blocks is not None:
        kw["gpu_blocks"] = gpu_blocks
    if host_blocks is not None:
        kw["host_blocks"] = host_blocks
    if workload == "history":
        # long sessions with short turns, so that a history block is read again by a dozen later turns of its session
        # (the paper reports 12-15 uses per history block against 49-173 per fixed-context block, Sec. 2.2)
        kw.setdefault("session_len", (20, 32))
        kw.setdefault("suffix_tokens", (64, 512))
    if kw:
        cfg = synth.shrink(cfg, **kw)
    pk = dict(n_agents=cfg.n_agents, n_chains=cfg.n_chains, block_tokens=cfg.block_tokens, r_min=0.02)
    if policy == "lru":
        pk["tau"] = 1.5
    pk.update(param_kw)
    params = orc.Params(**pk)
    oe = OracleEngine(params, geo, cfg.gpu_blocks, cfg.host_blocks, with_pools=with_pools)
    ge = None
    if gpu:
        from paper_2608_14624_b200 import binding as cs
        p = cs.make_params(n_agents=params.n_agents, n_chains=params.n_chains, max_blocks=cfg.gpu_blocks + cfg.host_blocks,
                           block_tokens=params.block_tokens, e_max=params.e_max, eps=params.eps, tau=params.tau,
                           lam=params.lam, delta=params.delta, r_min=params.r_min)
        ge = GpuEngine(p, geo, cfg.gpu_blocks, cfg.host_blocks, device)
    return ClosedLoop(cfg, geo, params, oe, ge, workload=workload, n_invocations=n_invocations)
