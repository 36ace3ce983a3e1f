"""ctypes wrapper of the CPU oracle (cs_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg.  The CUDA path never imports this module and this module never imports
the CUDA path.  Arrays are NumPy; every call goes straight to the C function of the same
name, which cites the passage of the paper it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cs_oracle.c")
_LIB = os.path.join(_HERE, "libcs_oracle.so")

AGENT_NONE = 0xFFFF
ID_NONE = 0xFFFFFFFF
INF = 0xFFFFFFFF


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-shared",
                               "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_predictability.restype = C.c_double
        for name in ("orc_observe", "orc_select_victims", "orc_select_prefetch", "orc_move_blocks"):
            getattr(_lib, name).restype = C.c_uint32
    return _lib


def _p(a: Optional[np.ndarray]):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.c_void_p)


@dataclass
class Params:
    n_agents: int
    n_chains: int = 1
    block_tokens: int = 16
    e_max: int = 4
    eps: float = 0.01
    tau: float = 0.05
    lam: float = 0.01
    delta: float = 0.01
    r_min: float = 0.3
    prefer_other_copy: int = 0


class Oracle:
    """State of Algorithm 1 plus the derived tables, refreshed after every observe()."""

    def __init__(self, p: Params):
        self.p = p
        A = p.n_agents
        self.C = np.zeros((A, A), np.uint32)
        self.cur = np.full(p.n_chains, AGENT_NONE, np.uint16)
        self.last_agent = np.array([AGENT_NONE], np.uint16)
        self.P64 = np.zeros((A, A), np.float64)
        self.P32 = np.zeros((A, A), np.float32)
        self.amax = np.zeros(A, np.uint16)
        self.R = 0.0
        self.adj = np.zeros((A, A), np.uint8)
        self.E = np.full(A, INF, np.uint32)
        self.ptilde = np.zeros(A, np.float64)
        self.fsurv32 = np.zeros(A, np.float32)
        self.n_bad_events = 0
        self.refresh()

    # -- learner -----------------------------------------------------------------------
    def observe(self, chain, agent, evflags=None):
        chain = np.ascontiguousarray(chain, np.uint32)
        agent = np.ascontiguousarray(agent, np.uint16)
        ev = None if evflags is None else np.ascontiguousarray(evflags, np.uint8)
        self.n_bad_events += lib().orc_observe(
            C.c_uint32(self.p.n_agents), C.c_uint32(self.p.n_chains), _p(self.C), _p(self.cur),
            _p(self.last_agent), _p(chain), _p(agent), _p(ev), C.c_uint32(len(agent)))
        self.refresh()

    def refresh(self, sources: Optional[Sequence[int]] = None):
        """Eq. 3 matrix, arg-max rows, Eq. 2, Eq. 7 graph, BFS from the current agent, Eq. 8."""
        A = self.p.n_agents
        L = lib()
        L.orc_normalise(C.c_uint32(A), _p(self.C), C.c_float(self.p.eps), _p(self.P64),
                        _p(self.P32), _p(self.amax))
        self.R = float(L.orc_predictability(C.c_uint32(A), _p(self.C), _p(self.P64)))
        L.orc_threshold_graph(C.c_uint32(A), _p(self.P32), C.c_float(self.p.tau), _p(self.adj))
        self.survival(sources)

    def survival(self, sources: Optional[Sequence[int]] = None):
        A = self.p.n_agents
        if sources is None:
            la = int(self.last_agent[0])
            src = np.array([la] if la != AGENT_NONE else [], np.uint16)
        else:
            src = np.ascontiguousarray(sources, np.uint16)
        L = lib()
        L.orc_bfs(C.c_uint32(A), _p(self.adj), _p(src) if len(src) else None,
                  C.c_uint32(len(src)), _p(self.E))
        L.orc_survival(C.c_uint32(A), _p(self.E), C.c_uint32(self.p.e_max),
                       C.c_float(self.p.delta), _p(self.ptilde), _p(self.fsurv32))

    def exact_survival(self, K: int, a0: Optional[int] = None) -> np.ndarray:
        """Eq. 6 for every agent, from the current agent (or `a0`) over K steps; fp64."""
        A = self.p.n_agents
        a0 = int(self.last_agent[0]) if a0 is None else int(a0)
        out = np.zeros(A, np.float64)
        lib().orc_exact_survival(C.c_uint32(A), _p(self.P64), C.c_uint32(a0), C.c_uint32(K), _p(out))
        return out

    @property
    def gate(self) -> bool:
        """Eq. 11, decided on the fp32 value of R like the kernels do."""
        return bool(np.float32(self.R) >= np.float32(self.p.r_min))

    # -- scorer ------------------------------------------------------------------------
    def scores(self, idx, now: int):
        n = idx.n
        s64 = np.zeros(n, np.float64)
        s32 = np.zeros(n, np.float32)
        lib().orc_scores(C.c_uint32(n), C.c_uint32(self.p.n_agents), _p(idx.agent),
                         _p(idx.last_access), _p(idx.n_tokens), C.c_uint32(self.p.block_tokens),
                         C.c_uint32(now), C.c_float(self.p.lam), C.c_float(self.p.delta),
                         _p(self.ptilde), _p(self.fsurv32), _p(s64), _p(s32))
        return s64, s32

    def select_victims(self, idx, now: int, tier: int, k: int, score32=None):
        if score32 is None:
            score32 = self.scores(idx, now)[1]
        ids = np.empty(k, np.uint32)
        n_out = lib().orc_select_victims(
            C.c_uint32(idx.n), C.c_uint32(self.p.n_agents), _p(idx.agent), _p(idx.ref_count),
            _p(idx.flags), _p(idx.last_access), _p(score32), C.c_uint32(tier), C.c_uint32(k),
            C.c_int(int(self.p.prefer_other_copy)), _p(ids))
        return ids, int(n_out)

    def select_prefetch(self, idx, now: int, k: int, score32=None):
        if score32 is None:
            score32 = self.scores(idx, now)[1]
        ids = np.empty(k, np.uint32)
        n_out = lib().orc_select_prefetch(
            C.c_uint32(idx.n), C.c_uint32(self.p.n_agents), _p(idx.agent), _p(idx.depth),
            _p(idx.ref_count), _p(idx.flags), _p(idx.last_access), _p(idx.anchor_blocks),
            _p(score32), C.c_int(int(self.gate)), C.c_uint16(int(self.last_agent[0])),
            _p(self.amax), C.c_uint32(k), _p(ids))
        return ids, int(n_out)


def move_blocks(src: np.ndarray, src_layout: int, src_slots_total: int, dst: np.ndarray,
                dst_layout: int, dst_slots_total: int, n_layers: int, chunk_bytes: int,
                src_slots, dst_slots) -> int:
    """Chunk-by-chunk memcpy of the listed blocks between two pools (flat byte views)."""
    s = np.ascontiguousarray(src_slots, np.uint32)
    d = np.ascontiguousarray(dst_slots, np.uint32)
    assert src.nbytes == src_slots_total * n_layers * 2 * chunk_bytes
    assert dst.nbytes == dst_slots_total * n_layers * 2 * chunk_bytes
    return int(lib().orc_move_blocks(
        _p(src), C.c_uint32(src_layout), C.c_uint32(src_slots_total), _p(dst),
        C.c_uint32(dst_layout), C.c_uint32(dst_slots_total), C.c_uint32(n_layers),
        C.c_size_t(chunk_bytes), _p(s), _p(d), C.c_uint32(len(s))))
