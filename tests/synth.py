"""Seeded synthetic inputs: agent traces, block-index metadata, KV pools, mover batches.

This module serves BOTH the CPU oracle's tests and the CUDA path's tests / bench (it is
test infrastructure and lives outside the product package), so it
holds none of the method's arithmetic (no counting, normalising, scoring, selecting or
copying of KV bytes): it only draws shapes and values.  Everything is NumPy on the host,
driven by ``numpy.random.Generator(PCG64(seed))``; callers move arrays to the device.

The workloads stand in for the agentic serving traces the paper evaluates on (shared
per-agent fixed contexts at the head of every prompt, fresh per-invocation suffixes,
Sec. 2.2); no item of any public benchmark is reproduced.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np

# ---- flag bits of the block index (same values as include/cachescout.h) -------------
FLAG_VALID = 1
FLAG_PINNED = 2
FLAG_TIER_HOST = 4
FLAG_OTHER_COPY = 8

EV_WARMUP = 1  # event flag: warmup request, excluded from transition learning (Sec. 4)

LAYER_MAJOR = 0
BLOCK_MAJOR = 1

AGENT_NONE = 0xFFFF
ID_NONE = 0xFFFFFFFF

BASE_SEED = 2608146240


@dataclass(frozen=True)
class Config:
    name: str
    seed: int
    n_agents: int
    transitions: Tuple[str, float]        # ("dirichlet", alpha) | ("sparse", nnz per row)
    n_layers: int
    n_kv_heads: int
    head_dim: int
    block_tokens: int
    elem_bytes: int
    gpu_blocks: int
    host_blocks: int
    sessions: int                         # concurrent live sessions
    invocations: int                      # length of the trace
    session_len: Tuple[int, int]          # invocations per session, inclusive range
    anchor_tokens: Tuple[int, int]        # fixed per-agent context, inclusive range
    suffix_tokens: Tuple[int, int]        # per-invocation user suffix, inclusive range
    events_per_step: Tuple[int, int]      # invocations handled by one scheduler step
    k_victims: int
    k_prefetch: int
    n_chains: int                         # chains tracked by the learner (sessions hashed)

    @property
    def chunk_bytes(self) -> int:
        """One layer, one of K/V, one block: tokens x heads x head_dim x element size."""
        return self.block_tokens * self.n_kv_heads * self.head_dim * self.elem_bytes

    @property
    def block_bytes(self) -> int:
        return self.n_layers * 2 * self.chunk_bytes

    @property
    def n_index(self) -> int:
        return self.gpu_blocks + self.host_blocks


CONFIGS: Dict[str, Config] = {
    # config 0: the small case the oracle finishes in seconds
    "tiny": Config("tiny", BASE_SEED + 1, 4, ("dirichlet", 1.0), 8, 8, 128, 16, 2,
                   512, 2048, 1, 200, (3, 8), (1024, 1024), (64, 512), (1, 1), 32, 64, 1),
    # config 1: Llama-3-8B-shaped KV, the configuration the metric is quoted on
    "llama8b": Config("llama8b", BASE_SEED + 2, 12, ("dirichlet", 0.5), 32, 8, 128, 16, 2,
                      20000, 60000, 64, 20000, (4, 16), (2048, 6144), (128, 2048), (1, 8),
                      256, 384, 64),
    # config 3: 70B-shaped KV
    "llama70b": Config("llama70b", BASE_SEED + 4, 30, ("sparse", 4), 80, 8, 128, 16, 2,
                       12000, 40000, 128, 50000, (3, 6), (2048, 6144), (128, 2048), (1, 8),
                       256, 384, 128),
    # config 4: metadata-scale scoring (no KV bytes)
    "meta1m": Config("meta1m", BASE_SEED + 5, 256, ("sparse", 8), 0, 8, 128, 16, 2,
                     500000, 500000, 16, 640000, (4, 4), (2048, 6144), (128, 2048), (16, 16),
                     10000, 2000, 16),
}


def rng_for(cfg_or_seed, stream: int = 0) -> np.random.Generator:
    seed = cfg_or_seed.seed if isinstance(cfg_or_seed, Config) else int(cfg_or_seed)
    return np.random.Generator(np.random.PCG64([seed, stream]))


# ---- generating transition matrix ---------------------------------------------------
def transition_matrix(cfg: Config, rng: np.random.Generator) -> np.ndarray:
    """Row-stochastic generating matrix M[A, A] (float64) of the agent workflow."""
    A = cfg.n_agents
    kind, par = cfg.transitions
    if kind == "dirichlet":
        return rng.dirichlet(np.full(A, float(par)), size=A)
    if kind == "sparse":
        nnz = int(par)
        M = np.zeros((A, A))
        for i in range(A):
            others = np.delete(np.arange(A), i)
            cols = rng.choice(others, size=min(nnz, A - 1), replace=False)
            M[i, cols] = rng.dirichlet(np.ones(len(cols)))
        return M
    raise ValueError(kind)


@dataclass
class Trace:
    chain: np.ndarray      # u32 [E] chain (session slot) of each invocation
    agent: np.ndarray      # u16 [E]
    evflags: np.ndarray    # u8  [E]
    session: np.ndarray    # u32 [E] global session id (fresh id per new session)
    step_off: np.ndarray   # i64 [S+1] events of scheduler step s are [step_off[s], step_off[s+1])
    M: np.ndarray          # generating matrix


def make_trace(cfg: Config, n_invocations: Optional[int] = None, warmup_frac: float = 0.0,
               stream: int = 1) -> Trace:
    """Sessions of agent invocations drawn from M; ``sessions`` of them are live at a time.

    The first agent of a session is uniform, later ones follow the row of M (self loops
    in M are allowed and produce repeated agents).  A finished session is replaced by a
    new one in the same chain slot.  Events are grouped into scheduler steps of
    U[events_per_step] invocations of distinct live sessions.
    """
    rng = rng_for(cfg, stream)
    M = transition_matrix(cfg, rng)
    A, S = cfg.n_agents, cfg.sessions
    E = int(n_invocations if n_invocations is not None else cfg.invocations)
    cum = np.cumsum(M, axis=1)
    cur = np.full(S, -1, dtype=np.int64)
    left = np.zeros(S, dtype=np.int64)
    sess_id = np.arange(S, dtype=np.int64)
    next_sess = S
    chain = np.empty(E, np.uint32)
    agent = np.empty(E, np.uint16)
    session = np.empty(E, np.uint32)
    step_off = [0]
    e = 0
    lo, hi = cfg.events_per_step
    while e < E:
        m = int(min(rng.integers(lo, hi + 1), S, E - e))
        slots = rng.choice(S, size=m, replace=False) if S > 1 else np.zeros(1, np.int64)
        for s in slots:
            if left[s] == 0:                       # start a fresh session in this slot
                left[s] = rng.integers(cfg.session_len[0], cfg.session_len[1] + 1)
                cur[s] = -1
                sess_id[s] = next_sess
                next_sess += 1
            if cur[s] < 0:
                a = int(rng.integers(0, A))
            else:
                a = int(min(np.searchsorted(cum[cur[s]], rng.random(), side="right"), A - 1))
            cur[s] = a
            left[s] -= 1
            chain[e] = s % cfg.n_chains
            agent[e] = a
            session[e] = sess_id[s]
            e += 1
        step_off.append(e)
    evflags = (rng.random(E) < warmup_frac).astype(np.uint8) * EV_WARMUP
    return Trace(chain, agent, evflags, session, np.asarray(step_off, np.int64), M)


# ---- block index (SoA metadata) --------------------------------------------------------
@dataclass
class BlockIndex:
    agent: np.ndarray          # u16 [N] owning agent
    depth: np.ndarray          # u16 [N] position of the block in its prompt
    ref_count: np.ndarray      # u8  [N]
    flags: np.ndarray          # u8  [N]
    last_access: np.ndarray    # u32 [N] scheduler step of the last touch
    n_tokens: Optional[np.ndarray]       # u8 [N] or None (= block_tokens everywhere)
    anchor_blocks: Optional[np.ndarray]  # u16 [A] or None

    @property
    def n(self) -> int:
        return int(self.agent.shape[0])

    def copy(self) -> "BlockIndex":
        c = lambda x: None if x is None else x.copy()
        return BlockIndex(c(self.agent), c(self.depth), c(self.ref_count), c(self.flags),
                          c(self.last_access), c(self.n_tokens), c(self.anchor_blocks))


def make_block_index(cfg: Config, n: Optional[int] = None, now0: int = 100_000,
                     tier: str = "range", with_tokens: bool = True, with_anchor: bool = True,
                     stream: int = 2, agent_bias: Optional[np.ndarray] = None) -> BlockIndex:
    """Metadata of ``n`` cached blocks with the metadata-scale recipe's distributions.

    ref_count is 0 w.p. 0.90 else U[1,4]; VALID 0.98, PINNED 0.02, HAS_OTHER_TIER_COPY 0.3;
    age = now0 - last_access is 50 % U[0,64), 30 % U[64,1024), 20 % U[1024,65536).
    ``tier="range"`` puts ids [0, gpu_blocks) on the GPU tier and the rest on the host tier
    (scaled when n differs from the config's index size); ``tier="random"`` flips a fair coin.
    """
    rng = rng_for(cfg, stream)
    N = int(n if n is not None else cfg.n_index)
    A = cfg.n_agents
    if agent_bias is None:
        agent = rng.integers(0, A, size=N, dtype=np.uint16)
    else:
        agent = rng.choice(A, size=N, p=agent_bias).astype(np.uint16)
    depth = rng.integers(0, 512, size=N, dtype=np.uint16)
    ref = np.where(rng.random(N) < 0.90, 0, rng.integers(1, 5, size=N)).astype(np.uint8)
    flags = np.zeros(N, np.uint8)
    flags |= (rng.random(N) < 0.98).astype(np.uint8) * FLAG_VALID
    flags |= (rng.random(N) < 0.02).astype(np.uint8) * FLAG_PINNED
    flags |= (rng.random(N) < 0.30).astype(np.uint8) * FLAG_OTHER_COPY
    if tier == "random":
        flags |= (rng.random(N) < 0.5).astype(np.uint8) * FLAG_TIER_HOST
    else:
        n_gpu = int(round(N * cfg.gpu_blocks / max(cfg.n_index, 1)))
        flags[n_gpu:] |= FLAG_TIER_HOST
    u = rng.random(N)
    age = np.where(u < 0.5, rng.integers(0, 64, size=N),
                   np.where(u < 0.8, rng.integers(64, 1024, size=N),
                            rng.integers(1024, 65536, size=N)))
    last_access = (now0 - age).astype(np.uint32)
    n_tokens = None
    if with_tokens:
        n_tokens = np.where(rng.random(N) < 0.95, cfg.block_tokens,
                            rng.integers(1, cfg.block_tokens, size=N)).astype(np.uint8)
    anchor = None
    if with_anchor:
        lo, hi = cfg.anchor_tokens
        anchor = (rng.integers(lo, hi + 1, size=A) // cfg.block_tokens).astype(np.uint16)
    return BlockIndex(agent, depth, ref, flags, last_access, n_tokens, anchor)


def mutate_index(idx: BlockIndex, rng: np.random.Generator, now: int, victims: np.ndarray,
                 prefetched: np.ndarray, last_agent: int, n_agents: int, n_touch: int = 2000):
    """Untimed state evolution between two score+select calls (host copy of the index).

    Victim slots are refilled (agent = last_agent w.p. 0.5 else uniform, fresh depth,
    last_access = now, ref 0); prefetch picks lose TIER_HOST and are touched; ``n_touch``
    random entries of ``last_agent`` are touched.
    """
    v = victims[victims != ID_NONE].astype(np.int64)
    if len(v):
        la = last_agent if last_agent != AGENT_NONE else 0
        idx.agent[v] = np.where(rng.random(len(v)) < 0.5, la,
                                rng.integers(0, n_agents, size=len(v))).astype(np.uint16)
        idx.depth[v] = rng.integers(0, 512, size=len(v), dtype=np.uint16)
        idx.last_access[v] = now
        idx.ref_count[v] = 0
    p = prefetched[prefetched != ID_NONE].astype(np.int64)
    if len(p):
        idx.flags[p] &= np.uint8(~FLAG_TIER_HOST & 0xFF)
        idx.last_access[p] = now
    if last_agent != AGENT_NONE and n_touch:
        mine = np.flatnonzero(idx.agent == last_agent)
        if len(mine):
            t = rng.choice(mine, size=min(n_touch, len(mine)), replace=False)
            idx.last_access[t] = now


# ---- KV pools and mover batches ----------------------------------------------------------
def kv_pool_u16(n_slots: int, n_layers: int, chunk_bytes: int, rng: np.random.Generator) -> np.ndarray:
    """A pool of ``n_slots`` blocks as raw 16-bit words: bf16 bit patterns of N(0,1) draws.

    Returned flat; which (layer, plane, slot) a word belongs to is decided by the layout
    formula of whoever reads it, so the same array serves both layouts.
    """
    n_words = n_slots * n_layers * 2 * chunk_bytes // 2
    x = rng.standard_normal(n_words, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16)


def mover_batch(n: int, src_slots_total: int, dst_slots_total: int, rng: np.random.Generator,
                packed_dst: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """``n`` distinct uniformly random source slots and destination slots (u32, unsorted)."""
    src = rng.choice(src_slots_total, size=n, replace=False).astype(np.uint32)
    if packed_dst:
        dst = np.arange(n, dtype=np.uint32)
    else:
        dst = rng.choice(dst_slots_total, size=n, replace=False).astype(np.uint32)
    return src, dst


def shrink(cfg: Config, **kw) -> Config:
    """A copy of a config with some sizes replaced (parity cases smaller than the named one)."""
    return replace(cfg, **kw)
