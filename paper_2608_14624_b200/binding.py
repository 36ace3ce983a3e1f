"""Thin Python binding of libcachescout (argument marshalling only).

Every ``cs_*`` function below calls the C function of the same name declared in
``include/cachescout.h``; all arithmetic runs in the CUDA kernels.  PyTorch is used for
device memory, pinned memory and streams only.  There is no CPU fallback: if the shared
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("CACHESCOUT_LIB") or os.path.join(HERE, "libcachescout.so")   # override: another build of the same ABI

CS_OK = 0
CS_EINVAL, CS_ECAPACITY, CS_ENOTIMPL, CS_ECUDA, CS_EDEVICE_STATUS, CS_ENOMEM = -1, -2, -3, -4, -5, -6
CS_ST_BAD_AGENT, CS_ST_BAD_CHAIN, CS_ST_BAD_SLOT, CS_ST_BAD_SOURCE = 1, 2, 4, 8
CS_AGENT_NONE, CS_ID_NONE, CS_HOP_NONE = 0xFFFF, 0xFFFFFFFF, 0xFFFF
CS_FLAG_VALID, CS_FLAG_PINNED, CS_FLAG_TIER_HOST, CS_FLAG_OTHER_COPY = 1, 2, 4, 8
CS_EV_WARMUP = 1
CS_LAYER_MAJOR, CS_BLOCK_MAJOR = 0, 1
CS_STATIC_MAX_BLOCKS = 65536
CS_MOVER_AUTO, CS_MOVER_LDST, CS_MOVER_BULK = 0, 1, 2
CS_ST_TIMEOUT, CS_ST_LIST_CONFLICT, CS_ST_BAD_SELECTION = 16, 32, 64
CS_SELECT_AUTO, CS_SELECT_CLUSTER, CS_SELECT_MULTI = 0, 1, 2

# every symbol include/cachescout.h declares
EXPORTS = ("cs_workspace_bytes", "cs_create", "cs_destroy", "cs_observe_invocations", "cs_score_blocks",
           "cs_select_victims", "cs_select_prefetch", "cs_offload_blocks", "cs_prefetch_blocks",
           "cs_compact_blocks", "cs_get_model", "cs_get_status", "cs_launch_count", "cs_set_mover_ctas",
           "cs_last_cuda_error", "cs_strerror", "cs_version", "cs_select_victims_static", "cs_set_mover_path", "cs_set_select_path",
           "cs_exact_survival", "cs_use_survival_table", "cs_import_state", "cs_set_select_speculation", "cs_exchange_blocks", "cs_step", "cs_set_survival_sources", "cs_select_step",
           "cs_get_counters", "cs_validate_selection", "cs_validate_move_lists", "cs_validate_exchange_lists",
           "cs_selftest_bounded_wait", "cs_set_device_clock", "cs_set_mover_staging", "cs_exchange_blocks_staged",
           "cs_offload_blocks_staged", "cs_prefetch_blocks_staged", "cs_set_select_bucket_regions", "cs_debug_phase_stamps")


class cs_params(C.Structure):
    _fields_ = [("n_agents", C.c_uint32), ("n_chains", C.c_uint32), ("max_blocks", C.c_uint32),
                ("block_tokens", C.c_uint32), ("e_max", C.c_uint32), ("eps", C.c_float), ("tau", C.c_float),
                ("lambda_", C.c_float), ("delta", C.c_float), ("r_min", C.c_float),
                ("prefer_other_copy", C.c_uint32)]


class cs_block_index(C.Structure):
    _fields_ = [("n_blocks", C.c_uint32), ("agent", C.c_void_p), ("depth", C.c_void_p), ("ref_count", C.c_void_p),
                ("flags", C.c_void_p), ("last_access", C.c_void_p), ("n_tokens", C.c_void_p),
                ("anchor_blocks", C.c_void_p)]


class cs_kv_pool(C.Structure):
    _fields_ = [("base", C.c_void_p), ("n_slots", C.c_uint32), ("layout", C.c_uint32), ("n_layers", C.c_uint32),
                ("n_kv_heads", C.c_uint32), ("head_dim", C.c_uint32), ("block_tokens", C.c_uint32),
                ("elem_bytes", C.c_uint32), ("first_id", C.c_uint32)]


class cs_step_io(C.Structure):
    _fields_ = [("chain", C.c_void_p), ("agent", C.c_void_p), ("evflags", C.c_void_p), ("n_events", C.c_uint32),
                ("n_events_dev", C.c_void_p), ("idx", C.POINTER(cs_block_index)), ("now", C.c_uint32),
                ("now_dev", C.c_void_p), ("k_victims", C.c_uint32), ("k_prefetch", C.c_uint32),
                ("gpu_victims", C.c_void_p), ("n_gpu_victims", C.c_void_p), ("host_victims", C.c_void_p),
                ("n_host_victims", C.c_void_p), ("prefetch_ids", C.c_void_p), ("n_prefetch", C.c_void_p),
                ("gpu", C.POINTER(cs_kv_pool)), ("host", C.POINTER(cs_kv_pool)), ("stage", C.POINTER(cs_kv_pool)),
                ("stage_slots", C.c_void_p), ("free_gpu_slots", C.c_void_p), ("join_main", C.c_uint32)]


class cs_counters(C.Structure):
    _fields_ = [("events_seen", C.c_uint64), ("events_skipped", C.c_uint64), ("transitions_counted", C.c_uint64),
                ("selects", C.c_uint64 * 3), ("eligible", C.c_uint64 * 3), ("selected", C.c_uint64 * 3),
                ("candidates", C.c_uint64 * 3), ("fast_hits", C.c_uint64 * 3),
                ("blocks_moved", C.c_uint64 * 3), ("bytes_moved", C.c_uint64 * 3), ("blocks_skipped", C.c_uint64),
                ("region_selects", C.c_uint64 * 3), ("region_overflows", C.c_uint64 * 3)]


class CacheScoutError(RuntimeError):
    def __init__(self, code: int, where: str, extra: str = ""):
        self.code = code
        msg = "%s: %s (%d)%s" % (where, lib().cs_strerror(code).decode(), code, extra)
        super().__init__(msg)


_lib = None


def lib():
    """Loads libcachescout.so (building is the job of ``build.build_library``); never falls back."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libcachescout.so is missing: build it with "
                               "`python -m paper_2608_14624_b200.build` (there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.cs_strerror.restype = C.c_char_p
        L.cs_strerror.argtypes = [C.c_int]
        vp, u32 = C.c_void_p, C.c_uint32
        L.cs_workspace_bytes.argtypes = [C.POINTER(cs_params), C.POINTER(C.c_size_t)]
        L.cs_create.argtypes = [C.POINTER(cs_params), vp, C.c_size_t, vp, C.POINTER(vp)]
        L.cs_destroy.argtypes = [vp]
        L.cs_observe_invocations.argtypes = [vp, vp, vp, vp, u32, vp]
        L.cs_score_blocks.argtypes = [vp, C.POINTER(cs_block_index), u32, vp, u32, vp, vp]
        L.cs_select_victims.argtypes = [vp, C.POINTER(cs_block_index), u32, u32, u32, vp, vp, vp]
        L.cs_select_prefetch.argtypes = [vp, C.POINTER(cs_block_index), u32, u32, vp, vp, vp]
        L.cs_select_victims_static.argtypes = [C.POINTER(cs_params), vp, C.POINTER(cs_block_index), u32, u32, u32,
                                               vp, vp, vp]
        for name in ("cs_offload_blocks", "cs_prefetch_blocks", "cs_compact_blocks"):
            getattr(L, name).argtypes = [vp, C.POINTER(cs_kv_pool), C.POINTER(cs_kv_pool), vp, vp, u32, vp, vp]
        L.cs_exchange_blocks.argtypes = [vp, C.POINTER(cs_kv_pool), C.POINTER(cs_kv_pool), vp, vp, u32, vp, vp, vp, u32,
                                         vp, vp]
        L.cs_set_survival_sources.argtypes = [vp, u32, vp]
        L.cs_select_step.argtypes = [vp, C.POINTER(cs_block_index), u32, u32, u32, vp, vp, vp, vp, vp, vp, vp]
        L.cs_step.argtypes = [vp, C.POINTER(cs_step_io), vp, vp]
        L.cs_get_model.argtypes = [vp] * 10
        L.cs_get_status.argtypes = [vp, C.POINTER(u32), vp]
        L.cs_launch_count.argtypes = [vp, C.POINTER(C.c_uint64)]
        L.cs_set_mover_ctas.argtypes = [vp, u32, u32]
        L.cs_last_cuda_error.argtypes = [vp]
        L.cs_set_mover_path.argtypes = [vp, u32]
        L.cs_set_select_path.argtypes = [vp, u32]
        L.cs_set_select_speculation.argtypes = [vp, u32]
        L.cs_set_select_bucket_regions.argtypes = [vp, u32]
        L.cs_debug_phase_stamps.argtypes = [vp, vp]
        L.cs_exact_survival.argtypes = [vp, u32, u32, vp, vp, vp]
        L.cs_use_survival_table.argtypes = [vp, vp]
        L.cs_import_state.argtypes = [vp, vp, vp, u32, vp]
        L.cs_get_counters.argtypes = [vp, C.POINTER(cs_counters), u32, vp]
        L.cs_validate_selection.argtypes = [vp, C.POINTER(cs_block_index), u32, u32, u32, u32, vp, vp, vp]
        L.cs_validate_move_lists.argtypes = [vp, C.POINTER(cs_kv_pool), C.POINTER(cs_kv_pool), vp, vp, u32, vp, vp]
        L.cs_validate_exchange_lists.argtypes = [vp, C.POINTER(cs_kv_pool), C.POINTER(cs_kv_pool), vp, vp, u32, vp, vp, vp,
                                                 u32, vp, vp]
        L.cs_selftest_bounded_wait.argtypes = [vp, u32, vp]
        L.cs_set_device_clock.argtypes = [vp, vp]
        L.cs_set_mover_staging.argtypes = [vp, vp, C.c_size_t]
        L.cs_exchange_blocks_staged.argtypes = [vp, C.POINTER(cs_kv_pool), C.POINTER(cs_kv_pool), vp, vp, u32, vp, vp, u32, vp]
        L.cs_offload_blocks_staged.argtypes = [vp, C.POINTER(cs_kv_pool), C.POINTER(cs_kv_pool), vp, vp, u32, vp]
        L.cs_prefetch_blocks_staged.argtypes = [vp, C.POINTER(cs_kv_pool), C.POINTER(cs_kv_pool), vp, vp, u32, vp]
        _lib = L
    return _lib


def _ptr(t) -> Optional[int]:
    """Device (or pinned host) address of a tensor, None for None, ints pass through."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(s) -> Optional[int]:
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _chk(code: int, where: str, ctx=None):
    if code != CS_OK:
        extra = ""
        if code == CS_ECUDA and ctx:
            extra = " [cudaError %d]" % lib().cs_last_cuda_error(ctx)
        raise CacheScoutError(code, where, extra)


# ---- the C-ABI, one Python function per exported call -----------------------------------------------
def cs_workspace_bytes(params: cs_params) -> int:
    n = C.c_size_t(0)
    _chk(lib().cs_workspace_bytes(C.byref(params), C.byref(n)), "cs_workspace_bytes")
    return int(n.value)


def cs_create(params: cs_params, workspace, stream=None) -> int:
    ctx = C.c_void_p()
    _chk(lib().cs_create(C.byref(params), _ptr(workspace), workspace.numel() * workspace.element_size(),
                         _stream(stream), C.byref(ctx)), "cs_create")
    return ctx.value


def cs_destroy(ctx: int):
    _chk(lib().cs_destroy(ctx), "cs_destroy")


def cs_observe_invocations(ctx, chain, agent, evflags, n_events: int, stream=None):
    _chk(lib().cs_observe_invocations(ctx, _ptr(chain), _ptr(agent), _ptr(evflags), n_events, _stream(stream)),
         "cs_observe_invocations", ctx)


def cs_score_blocks(ctx, idx: cs_block_index, now: int, sources, n_sources: int, scores_out, stream=None):
    _chk(lib().cs_score_blocks(ctx, C.byref(idx), now, _ptr(sources), n_sources, _ptr(scores_out), _stream(stream)),
         "cs_score_blocks", ctx)


def cs_select_victims(ctx, idx: cs_block_index, now: int, tier: int, k: int, ids_out, n_out, stream=None):
    _chk(lib().cs_select_victims(ctx, C.byref(idx), now, tier, k, _ptr(ids_out), _ptr(n_out), _stream(stream)),
         "cs_select_victims", ctx)


def cs_select_prefetch(ctx, idx: cs_block_index, now: int, k: int, ids_out, n_out, stream=None):
    _chk(lib().cs_select_prefetch(ctx, C.byref(idx), now, k, _ptr(ids_out), _ptr(n_out), _stream(stream)),
         "cs_select_prefetch", ctx)


def cs_select_victims_static(params: cs_params, fsurv, idx: cs_block_index, now: int, tier: int, k: int, ids_out,
                             n_out, stream=None):
    """Victim selection without a context or workspace, for callers that cannot allocate device
    memory: the kernels' scratch is a static array inside the library.  `fsurv` is the device
    table of survival factors (one fp32 per agent); at most CS_STATIC_MAX_BLOCKS entries / k."""
    _chk(lib().cs_select_victims_static(C.byref(params), _ptr(fsurv), C.byref(idx), now, tier, k, _ptr(ids_out),
                                        _ptr(n_out), _stream(stream)), "cs_select_victims_static")


def cs_offload_blocks(ctx, gpu: cs_kv_pool, host: cs_kv_pool, src_slots, dst_slots, n_max: int, n_dev=None, stream=None):
    _chk(lib().cs_offload_blocks(ctx, C.byref(gpu), C.byref(host), _ptr(src_slots), _ptr(dst_slots), n_max,
                                 _ptr(n_dev), _stream(stream)), "cs_offload_blocks", ctx)


def cs_prefetch_blocks(ctx, host: cs_kv_pool, gpu: cs_kv_pool, src_slots, dst_slots, n_max: int, n_dev=None, stream=None):
    _chk(lib().cs_prefetch_blocks(ctx, C.byref(host), C.byref(gpu), _ptr(src_slots), _ptr(dst_slots), n_max,
                                  _ptr(n_dev), _stream(stream)), "cs_prefetch_blocks", ctx)


def cs_exchange_blocks(ctx, gpu: cs_kv_pool, host: cs_kv_pool, off_gpu_slots, off_host_slots, n_off_max: int, n_off_dev,
                       pre_host_slots, pre_gpu_slots, n_pre_max: int, n_pre_dev, stream=None):
    _chk(lib().cs_exchange_blocks(ctx, C.byref(gpu), C.byref(host), _ptr(off_gpu_slots), _ptr(off_host_slots), n_off_max,
                                  _ptr(n_off_dev), _ptr(pre_host_slots), _ptr(pre_gpu_slots), n_pre_max,
                                  _ptr(n_pre_dev), _stream(stream)), "cs_exchange_blocks", ctx)


CS_SOURCES_LAST_AGENT, CS_SOURCES_ALL_CHAINS = 0, 1


def cs_set_survival_sources(ctx, mode: int, stream=None):
    _chk(lib().cs_set_survival_sources(ctx, mode, _stream(stream)), "cs_set_survival_sources", ctx)


def cs_select_step(ctx, idx: cs_block_index, now: int, k_victims: int, k_prefetch: int, gpu_victims, n_gpu_victims,
                   host_victims, n_host_victims, prefetch_ids, n_prefetch, stream=None):
    _chk(lib().cs_select_step(ctx, C.byref(idx), now, k_victims, k_prefetch, _ptr(gpu_victims), _ptr(n_gpu_victims),
                              _ptr(host_victims), _ptr(n_host_victims), _ptr(prefetch_ids), _ptr(n_prefetch),
                              _stream(stream)), "cs_select_step", ctx)


def cs_step(ctx, io: cs_step_io, main=None, side=None):
    _chk(lib().cs_step(ctx, C.byref(io), _stream(main), _stream(side)), "cs_step", ctx)


def cs_compact_blocks(ctx, src: cs_kv_pool, dst: cs_kv_pool, src_slots, dst_slots, n_max: int, n_dev=None, stream=None):
    _chk(lib().cs_compact_blocks(ctx, C.byref(src), C.byref(dst), _ptr(src_slots), _ptr(dst_slots), n_max,
                                 _ptr(n_dev), _stream(stream)), "cs_compact_blocks", ctx)


def cs_get_model(ctx, C_out=None, P_out=None, amax_out=None, hops_out=None, fsurv_out=None, R_out=None,
                 cur_out=None, last_agent_out=None, stream=None):
    _chk(lib().cs_get_model(ctx, _ptr(C_out), _ptr(P_out), _ptr(amax_out), _ptr(hops_out), _ptr(fsurv_out),
                            _ptr(R_out), _ptr(cur_out), _ptr(last_agent_out), _stream(stream)), "cs_get_model", ctx)


def cs_get_status(ctx, stream=None, raise_on_set: bool = False) -> int:
    st = C.c_uint32(0)
    code = lib().cs_get_status(ctx, C.byref(st), _stream(stream))
    if code not in (CS_OK, CS_EDEVICE_STATUS) or (raise_on_set and code != CS_OK):
        _chk(code, "cs_get_status", ctx)
    return int(st.value)


def cs_get_counters(ctx, reset: bool = False, stream=None) -> dict:
    """Work counters kept by the kernels (synchronises the stream); plain ints and lists of three."""
    out = cs_counters()
    _chk(lib().cs_get_counters(ctx, C.byref(out), 1 if reset else 0, _stream(stream)), "cs_get_counters", ctx)
    return {name: (list(getattr(out, name)) if hasattr(getattr(out, name), "__len__") else int(getattr(out, name)))
            for name, _ in cs_counters._fields_}


def cs_validate_selection(ctx, idx: cs_block_index, now: int, prefetch: bool, tier: int, k: int, ids_out, n_out, stream=None):
    _chk(lib().cs_validate_selection(ctx, C.byref(idx), now, 1 if prefetch else 0, tier, k, _ptr(ids_out), _ptr(n_out),
                                     _stream(stream)), "cs_validate_selection", ctx)


def cs_validate_move_lists(ctx, src: cs_kv_pool, dst: cs_kv_pool, src_slots, dst_slots, n_max: int, n_dev=None, stream=None):
    _chk(lib().cs_validate_move_lists(ctx, C.byref(src), C.byref(dst), _ptr(src_slots), _ptr(dst_slots), n_max,
                                      _ptr(n_dev), _stream(stream)), "cs_validate_move_lists", ctx)


def cs_validate_exchange_lists(ctx, gpu: cs_kv_pool, host: cs_kv_pool, off_gpu_slots, off_host_slots, n_off_max: int,
                               n_off_dev, pre_host_slots, pre_gpu_slots, n_pre_max: int, n_pre_dev, stream=None):
    _chk(lib().cs_validate_exchange_lists(ctx, C.byref(gpu), C.byref(host), _ptr(off_gpu_slots), _ptr(off_host_slots),
                                          n_off_max, _ptr(n_off_dev), _ptr(pre_host_slots), _ptr(pre_gpu_slots),
                                          n_pre_max, _ptr(n_pre_dev), _stream(stream)), "cs_validate_exchange_lists", ctx)


def cs_selftest_bounded_wait(ctx, max_polls: int, stream=None):
    _chk(lib().cs_selftest_bounded_wait(ctx, max_polls, _stream(stream)), "cs_selftest_bounded_wait", ctx)


def _host_ids(a):
    """Host-memory id list for the staged calls: a NumPy uint32 array (or None); returns (keep-alive, address)."""
    if a is None:
        return None, None
    import numpy as np
    arr = np.ascontiguousarray(a, dtype=np.uint32)
    return arr, arr.ctypes.data


def cs_set_mover_staging(ctx, ring):
    if ring is None:
        _chk(lib().cs_set_mover_staging(ctx, None, 0), "cs_set_mover_staging", ctx)
    else:
        _chk(lib().cs_set_mover_staging(ctx, _ptr(ring), ring.numel() * ring.element_size()), "cs_set_mover_staging", ctx)


def cs_exchange_blocks_staged(ctx, gpu: cs_kv_pool, host: cs_kv_pool, off_gpu_slots, off_host_ids, n_off: int,
                              pre_host_ids, pre_gpu_slots, n_pre: int, stream=None):
    ko, po = _host_ids(off_host_ids)
    kp, pp = _host_ids(pre_host_ids)
    _chk(lib().cs_exchange_blocks_staged(ctx, C.byref(gpu), C.byref(host), _ptr(off_gpu_slots), po, n_off, pp,
                                         _ptr(pre_gpu_slots), n_pre, _stream(stream)), "cs_exchange_blocks_staged", ctx)


def cs_offload_blocks_staged(ctx, gpu: cs_kv_pool, host: cs_kv_pool, src_slots, host_ids, n: int, stream=None):
    k, p = _host_ids(host_ids)
    _chk(lib().cs_offload_blocks_staged(ctx, C.byref(gpu), C.byref(host), _ptr(src_slots), p, n, _stream(stream)),
         "cs_offload_blocks_staged", ctx)


def cs_prefetch_blocks_staged(ctx, host: cs_kv_pool, gpu: cs_kv_pool, host_ids, dst_slots, n: int, stream=None):
    k, p = _host_ids(host_ids)
    _chk(lib().cs_prefetch_blocks_staged(ctx, C.byref(host), C.byref(gpu), p, _ptr(dst_slots), n, _stream(stream)),
         "cs_prefetch_blocks_staged", ctx)


def cs_set_device_clock(ctx, now_dev):
    _chk(lib().cs_set_device_clock(ctx, _ptr(now_dev)), "cs_set_device_clock", ctx)


def cs_launch_count(ctx) -> int:
    n = C.c_uint64(0)
    _chk(lib().cs_launch_count(ctx, C.byref(n)), "cs_launch_count")
    return int(n.value)


def cs_set_mover_ctas(ctx, host_link_ctas: int, d2d_ctas: int):
    _chk(lib().cs_set_mover_ctas(ctx, host_link_ctas, d2d_ctas), "cs_set_mover_ctas")


def cs_set_mover_path(ctx, path: int):
    _chk(lib().cs_set_mover_path(ctx, path), "cs_set_mover_path")


def cs_exact_survival(ctx, a0: int, n_steps: int, psurv_out, fsurv_out, stream=None):
    _chk(lib().cs_exact_survival(ctx, a0, n_steps, _ptr(psurv_out), _ptr(fsurv_out), _stream(stream)),
         "cs_exact_survival", ctx)


def cs_import_state(ctx, C_in, cur_in, last_agent: int, stream=None):
    _chk(lib().cs_import_state(ctx, _ptr(C_in), _ptr(cur_in), last_agent, _stream(stream)), "cs_import_state", ctx)


def cs_use_survival_table(ctx, fsurv):
    _chk(lib().cs_use_survival_table(ctx, _ptr(fsurv)), "cs_use_survival_table", ctx)


def cs_set_select_speculation(ctx, enabled: bool):
    _chk(lib().cs_set_select_speculation(ctx, 1 if enabled else 0), "cs_set_select_speculation")


def cs_debug_phase_stamps(ctx):
    """Phase stamps (ns of the GPU's global timer) of the latest calls as a list; a library built without
    -DCS_PHASE_STAMPS raises CS_ENOTIMPL."""
    out = (C.c_uint64 * 64)()
    _chk(lib().cs_debug_phase_stamps(ctx, C.cast(out, C.c_void_p)), "cs_debug_phase_stamps")
    return list(out)


def cs_set_select_bucket_regions(ctx, max_keys: int):
    _chk(lib().cs_set_select_bucket_regions(ctx, int(max_keys)), "cs_set_select_bucket_regions", "cs_debug_phase_stamps")


def cs_set_select_path(ctx, path: int):
    _chk(lib().cs_set_select_path(ctx, path), "cs_set_select_path")


def cs_version() -> int:
    return int(lib().cs_version())


# ---- small holders that keep tensors alive next to the structs that point into them ---------------------
def make_params(n_agents: int, n_chains: int = 1, max_blocks: int = 1, block_tokens: int = 16, e_max: int = 4,
                eps: float = 0.01, tau: float = 0.05, lam: float = 0.01, delta: float = 0.01,
                r_min: float = 0.3, prefer_other_copy: int = 0) -> cs_params:
    return cs_params(n_agents, n_chains, max_blocks, block_tokens, e_max, eps, tau, lam, delta, r_min,
                     prefer_other_copy)


@dataclass
class DeviceIndex:
    """SoA block metadata on the device (torch tensors) plus the struct the C calls take."""
    agent: object
    depth: object
    ref_count: object
    flags: object
    last_access: object
    n_tokens: object = None
    anchor_blocks: object = None

    @classmethod
    def from_host(cls, idx, device="cuda:0"):
        import torch
        up = lambda a: None if a is None else torch.from_numpy(a).to(device)
        return cls(up(idx.agent), up(idx.depth), up(idx.ref_count), up(idx.flags), up(idx.last_access),
                   up(idx.n_tokens), up(idx.anchor_blocks))

    @property
    def n(self) -> int:
        return int(self.agent.numel())

    def struct(self) -> cs_block_index:
        return cs_block_index(self.n, _ptr(self.agent), _ptr(self.depth), _ptr(self.ref_count), _ptr(self.flags),
                              _ptr(self.last_access), _ptr(self.n_tokens), _ptr(self.anchor_blocks))


@dataclass
class KVPool:
    """A paged KV pool: flat tensor (device, or pinned host) + geometry."""
    buf: object
    n_slots: int
    layout: int
    n_layers: int
    n_kv_heads: int = 8
    head_dim: int = 128
    block_tokens: int = 16
    elem_bytes: int = 2
    first_id: int = 0

    @property
    def chunk_bytes(self) -> int:
        return self.block_tokens * self.n_kv_heads * self.head_dim * self.elem_bytes

    @property
    def block_bytes(self) -> int:
        return self.n_layers * 2 * self.chunk_bytes

    def struct(self) -> cs_kv_pool:
        """The C struct (built once: the fields of a pool are not meant to change after construction)."""
        s = self.__dict__.get("_struct")
        if s is None:
            assert self.buf.numel() * self.buf.element_size() >= self.n_slots * self.block_bytes
            s = cs_kv_pool(_ptr(self.buf), self.n_slots, self.layout, self.n_layers, self.n_kv_heads, self.head_dim,
                           self.block_tokens, self.elem_bytes, self.first_id)
            self.__dict__["_struct"] = s
        return s


class CacheScout:
    """One context: owns the torch workspace tensor and forwards to the cs_* calls."""

    def __init__(self, params: cs_params, device="cuda:0", stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("CacheScout needs a CUDA device (sm_100a); there is no CPU fallback")
        self.params = params
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(cs_workspace_bytes(params) + 256, dtype=torch.uint8, device=self.device)
            self.ctx = cs_create(params, self.workspace, stream)

    def close(self):
        if getattr(self, "ctx", None):
            cs_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- calls ---------------------------------------------------------------------------------------
    def observe_invocations(self, chain, agent, evflags=None, n_events=None, stream=None):
        n = int(agent.numel()) if n_events is None and agent is not None else int(n_events or 0)
        cs_observe_invocations(self.ctx, chain, agent, evflags, n, stream)

    def score_blocks(self, idx: DeviceIndex, now: int, sources=None, out=None, stream=None):
        import torch
        if out is None:
            out = torch.empty(idx.n, dtype=torch.float32, device=self.device)
        cs_score_blocks(self.ctx, idx.struct(), now, sources, 0 if sources is None else int(sources.numel()), out, stream)
        return out

    def select_victims(self, idx: DeviceIndex, now: int, tier: int, k: int, ids_out=None, n_out=None, stream=None):
        import torch
        if ids_out is None:
            ids_out = torch.empty(max(k, 4), dtype=torch.int32, device=self.device)
        if n_out is None:
            n_out = torch.empty(1, dtype=torch.int32, device=self.device)
        cs_select_victims(self.ctx, idx.struct(), now, tier, k, ids_out, n_out, stream)
        return ids_out, n_out

    def select_prefetch(self, idx: DeviceIndex, now: int, k: int, ids_out=None, n_out=None, stream=None):
        import torch
        if ids_out is None:
            ids_out = torch.empty(max(k, 4), dtype=torch.int32, device=self.device)
        if n_out is None:
            n_out = torch.empty(1, dtype=torch.int32, device=self.device)
        cs_select_prefetch(self.ctx, idx.struct(), now, k, ids_out, n_out, stream)
        return ids_out, n_out

    def select_step(self, idx: DeviceIndex, now: int, k_victims: int, k_prefetch: int, gpu_victims, n_gpu_victims,
                    host_victims, n_host_victims, prefetch_ids, n_prefetch, stream=None):
        """GPU-tier victims, host-tier victims and prefetch candidates of one step at once."""
        cs_select_step(self.ctx, idx.struct(), now, k_victims, k_prefetch, gpu_victims, n_gpu_victims, host_victims,
                       n_host_victims, prefetch_ids, n_prefetch, stream)

    def offload_blocks(self, gpu: KVPool, host: KVPool, src_slots, dst_slots, n_max=None, n_dev=None, stream=None):
        cs_offload_blocks(self.ctx, gpu.struct(), host.struct(), src_slots, dst_slots,
                          int(src_slots.numel()) if n_max is None else n_max, n_dev, stream)

    def prefetch_blocks(self, host: KVPool, gpu: KVPool, src_slots, dst_slots, n_max=None, n_dev=None, stream=None):
        cs_prefetch_blocks(self.ctx, host.struct(), gpu.struct(), src_slots, dst_slots,
                           int(src_slots.numel()) if n_max is None else n_max, n_dev, stream)

    def exchange_blocks(self, gpu: KVPool, host: KVPool, off_gpu_slots, off_host_slots, pre_host_slots, pre_gpu_slots,
                        n_off_max=None, n_off_dev=None, n_pre_max=None, n_pre_dev=None, stream=None):
        """Offload and prefetch of one step in a single launch; either pair of lists may be None."""
        if n_off_max is None:
            n_off_max = 0 if off_gpu_slots is None else int(off_gpu_slots.numel())
        if n_pre_max is None:
            n_pre_max = 0 if pre_host_slots is None else int(pre_host_slots.numel())
        cs_exchange_blocks(self.ctx, gpu.struct(), host.struct(), off_gpu_slots, off_host_slots, n_off_max, n_off_dev,
                           pre_host_slots, pre_gpu_slots, n_pre_max, n_pre_dev, stream)

    def step(self, idx: "DeviceIndex", now: int, chain, agent, evflags, n_events: int, k_victims: int, k_prefetch: int,
             gpu_victims, n_gpu_victims, host_victims, n_host_victims, prefetch_ids, n_prefetch,
             gpu: KVPool, host: KVPool, free_gpu_slots, stage: Optional[KVPool] = None, stage_slots=None,
             now_dev=None, n_events_dev=None, main=None, side=None, join_main: bool = False):
        """One whole step (observe, three selects, compaction, two-way transfer) as one call."""
        i_s, g_s, h_s = idx.struct(), gpu.struct(), host.struct()
        st_s = stage.struct() if stage is not None else None
        io = cs_step_io(_ptr(chain), _ptr(agent), _ptr(evflags), n_events, _ptr(n_events_dev), C.pointer(i_s), now,
                        _ptr(now_dev), k_victims, k_prefetch, _ptr(gpu_victims), _ptr(n_gpu_victims),
                        _ptr(host_victims), _ptr(n_host_victims), _ptr(prefetch_ids), _ptr(n_prefetch),
                        C.pointer(g_s), C.pointer(h_s), C.pointer(st_s) if st_s is not None else None,
                        _ptr(stage_slots), _ptr(free_gpu_slots), 1 if join_main else 0)
        cs_step(self.ctx, io, main, side)

    def compact_blocks(self, src: KVPool, dst: KVPool, src_slots, dst_slots, n_max=None, n_dev=None, stream=None):
        cs_compact_blocks(self.ctx, src.struct(), dst.struct(), src_slots, dst_slots,
                          int(src_slots.numel()) if n_max is None else n_max, n_dev, stream)

    def get_model(self, stream=None) -> dict:
        """Copies of the learner / scorer state as host NumPy arrays (synchronises)."""
        import torch
        A, nc = self.params.n_agents, self.params.n_chains
        dev = self.device
        out = dict(C=torch.empty(A * A, dtype=torch.int32, device=dev), P=torch.empty(A * A, dtype=torch.float32, device=dev),
                   amax=torch.empty(A + 8, dtype=torch.int16, device=dev), hops=torch.empty(A + 8, dtype=torch.int16, device=dev),
                   fsurv=torch.empty(A, dtype=torch.float32, device=dev), R=torch.empty(1, dtype=torch.float32, device=dev),
                   cur=torch.empty(nc + 8, dtype=torch.int16, device=dev), last_agent=torch.empty(8, dtype=torch.int16, device=dev))
        cs_get_model(self.ctx, out["C"], out["P"], out["amax"], out["hops"], out["fsurv"], out["R"], out["cur"],
                     out["last_agent"], stream)
        torch.cuda.synchronize(dev)
        import numpy as np
        res = {}
        res["C"] = out["C"].cpu().numpy().view(np.uint32).reshape(A, A)
        res["P"] = out["P"].cpu().numpy().reshape(A, A)
        res["amax"] = out["amax"].cpu().numpy().view(np.uint16)[:A]
        res["hops"] = out["hops"].cpu().numpy().view(np.uint16)[:A]
        res["fsurv"] = out["fsurv"].cpu().numpy()
        res["R"] = float(out["R"].item())
        res["cur"] = out["cur"].cpu().numpy().view(np.uint16)[:nc]
        res["last_agent"] = int(out["last_agent"].cpu().numpy().view(np.uint16)[0])
        return res

    def get_status(self, stream=None) -> int:
        return cs_get_status(self.ctx, stream)

    def launch_count(self) -> int:
        return cs_launch_count(self.ctx)

    def counters(self, reset: bool = False, stream=None) -> dict:
        return cs_get_counters(self.ctx, reset, stream)

    def validate_selection(self, idx: DeviceIndex, now: int, prefetch: bool, tier: int, k: int, ids_out, n_out, stream=None):
        cs_validate_selection(self.ctx, idx.struct(), now, prefetch, tier, k, ids_out, n_out, stream)

    def validate_move_lists(self, src: KVPool, dst: KVPool, src_slots, dst_slots, n_max=None, n_dev=None, stream=None):
        cs_validate_move_lists(self.ctx, src.struct(), dst.struct(), src_slots, dst_slots,
                               int(src_slots.numel()) if n_max is None else n_max, n_dev, stream)

    def validate_exchange_lists(self, gpu: KVPool, host: KVPool, off_gpu_slots, off_host_slots, pre_host_slots,
                                pre_gpu_slots, n_off_max=None, n_off_dev=None, n_pre_max=None, n_pre_dev=None, stream=None):
        if n_off_max is None:
            n_off_max = 0 if off_gpu_slots is None else int(off_gpu_slots.numel())
        if n_pre_max is None:
            n_pre_max = 0 if pre_host_slots is None else int(pre_host_slots.numel())
        cs_validate_exchange_lists(self.ctx, gpu.struct(), host.struct(), off_gpu_slots, off_host_slots, n_off_max,
                                   n_off_dev, pre_host_slots, pre_gpu_slots, n_pre_max, n_pre_dev, stream)

    def set_mover_staging(self, ring):
        """Device ring (a torch uint8 tensor, kept alive here) for the copy-engine transfers; None takes it away."""
        cs_set_mover_staging(self.ctx, ring)
        self._ring_keepalive = ring

    def exchange_blocks_staged(self, gpu: KVPool, host: KVPool, off_gpu_slots, off_host_ids, pre_host_ids, pre_gpu_slots,
                               stream=None):
        """Offload + prefetch on the copy engines; the host-side id lists are NumPy arrays (host memory)."""
        n_off = 0 if off_host_ids is None else len(off_host_ids)
        n_pre = 0 if pre_host_ids is None else len(pre_host_ids)
        cs_exchange_blocks_staged(self.ctx, gpu.struct(), host.struct(), off_gpu_slots, off_host_ids, n_off, pre_host_ids,
                                  pre_gpu_slots, n_pre, stream)

    def set_device_clock(self, now_dev):
        """Selects and scores read the clock from this device word when they run (CUDA-graph replay); None = the argument."""
        self._clock_keepalive = now_dev
        cs_set_device_clock(self.ctx, now_dev)

    def selftest_bounded_wait(self, max_polls: int = 1000, stream=None):
        cs_selftest_bounded_wait(self.ctx, max_polls, stream)

    def exact_survival(self, n_steps: int, a0: int = CS_AGENT_NONE, stream=None):
        """Eq. 6 for every agent: returns (p_surv, p_surv + delta) as device tensors."""
        import torch
        A = self.params.n_agents
        ps = torch.empty(A, dtype=torch.float32, device=self.device)
        fs = torch.empty(A, dtype=torch.float32, device=self.device)
        cs_exact_survival(self.ctx, a0, n_steps, ps, fs, stream)
        return ps, fs

    def import_state(self, C, cur, last_agent: int, stream=None):
        """Restores the learner state exported by get_model() (device tensors: counts [A*A] u32, cur [n_chains] u16)."""
        cs_import_state(self.ctx, C, cur, int(last_agent), stream)

    def use_survival_table(self, fsurv):
        self._fsurv_keepalive = fsurv
        cs_use_survival_table(self.ctx, fsurv)

    def set_survival_sources(self, mode: int, stream=None):
        cs_set_survival_sources(self.ctx, mode, stream)

    def set_select_speculation(self, enabled: bool):
        cs_set_select_speculation(self.ctx, enabled)

    def set_select_bucket_regions(self, max_keys: int):
        cs_set_select_bucket_regions(self.ctx, max_keys)

    def phase_stamps(self):
        return cs_debug_phase_stamps(self.ctx)

    def set_select_path(self, path: int):
        cs_set_select_path(self.ctx, path)

    def set_mover_path(self, path: int):
        cs_set_mover_path(self.ctx, path)

    def set_mover_ctas(self, host_link_ctas: int = 0, d2d_ctas: int = 0):
        cs_set_mover_ctas(self.ctx, host_link_ctas, d2d_ctas)
