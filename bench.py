#!/usr/bin/env python
"""Benchmark of the agent-aware KV-cache hot path on B200.

One "step" is one scheduler step of the Llama-3-8B-shaped configuration (32 layers x 8 KV
heads x 128, bf16, 16-token blocks of 2 MiB; GPU pool 20,000 blocks, host tier 60,000, 12
agents): observe the step's agent invocations, select 256 GPU-tier victims, 256 host-tier
victims (their slots receive the offloaded blocks) and 384 prefetch candidates, compact the
victims into a packed device staging pool, offload them to the pinned host tier and prefetch
the candidates into free GPU slots.  The two transfers run as one fused launch on a side
stream (or, with --transfers split, as two launches on two side streams) and overlap the next
step's selection.  value = KV bytes moved across the host link per second over the K steps.

    python bench.py --gpus 1 --steps 20 --warmup 3
    python bench.py --config llama70b         # the 70B-shaped configuration as the timed workload
    python bench.py --impl reference          # the CPU oracle on the host cores, same metric

The default run times the Llama-3-8B-shaped step (the headline line) and then, as extra keys of the same
JSON line, the 70B-shaped step, the mover sweep, the metadata-scale calls and the large-index regime.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "KV block offload/prefetch GB/s vs host-link peak; blocks scored+selected/sec"
GIB = 1 << 30


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llama8b", choices=["llama8b", "llama70b"], help="KV shape of the timed step")
    ap.add_argument("--host-slots", type=int, default=0,
                    help="host-tier slots backed by pinned memory (0 = as many of the configuration's as --host-frac of the free memory holds)")
    ap.add_argument("--host-frac", type=float, default=0.40, help="share of the box's available memory the pinned host tier may take")
    ap.add_argument("--meta-calls", type=int, default=10000, help="score+select calls of the metadata-scale section")
    ap.add_argument("--no-extras", action="store_true", help="skip the mover sweep and the metadata-scale section")
    ap.add_argument("--offload-width", type=int, default=0, help="warp pipelines of the offload mover (0 = library default)")
    ap.add_argument("--prefetch-width", type=int, default=0, help="warp pipelines of the prefetch mover (0 = library default)")
    ap.add_argument("--transfers", default="exchange", choices=["exchange", "split", "staged"],
                    help="offload and prefetch of a step as one fused SM-issued launch (exchange), as two launches on two streams "
                         "(split), or on the copy engines through a device ring after reading the id lists back (staged)")
    ap.add_argument("--ring-mib", type=int, default=256, help="device ring of the staged transfers, MiB")
    ap.add_argument("--selects", default="fused", choices=["fused", "separate"],
                    help="the three selects of a step as one launch (cs_select_step) or as three calls")
    ap.add_argument("--exchange-width", type=int, default=0, help="warp pipelines of the fused transfer (0 = library default)")
    ap.add_argument("--quick", action="store_true", help="small pools (debugging only; not a valid bench line)")
    ap.add_argument("--workload", default="step", choices=["step", "mover", "select", "select80k", "select16m", "select64m"],
                    help="'mover'/'select' run one small case of that kernel family only (profiler captures)")
    ap.add_argument("--kineto", action="store_true",
                    help="with --workload select / select80k: warm per-kernel device times from the CUDA profiler API (torch.profiler)")
    ap.add_argument("--phase-stamps", action="store_true",
                    help="with --workload select: build the profiling variant of the library (kernels store the GPU's global "
                         "timer at phase boundaries) and print where the time of a graph-replayed metadata-scale call goes")
    ap.add_argument("--skip-aux", action="store_true",
                    help="timed steps only: no link-peak probe, end-to-end pass, extras or CPU baseline (profiler launch lists)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def mem_available_bytes():
    """Memory this process may still take: MemAvailable, or what its cgroup leaves, whichever is less."""
    avail = 0
    with open("/proc/meminfo") as f:
        for line in f:
            if line.startswith("MemAvailable:"):
                avail = int(line.split()[1]) * 1024
    try:
        with open("/sys/fs/cgroup/memory.max") as f:
            lim = f.read().strip()
        with open("/sys/fs/cgroup/memory.current") as f:
            cur = int(f.read().strip())
        if lim != "max":
            avail = min(avail, max(0, int(lim) - cur))
    except (OSError, ValueError):
        pass
    return avail


def clear_cuda_last_error(torch):
    """A runtime call that fails (here: cudaHostRegister refused for lack of lockable memory) leaves its code behind as the
    thread's "last error", and torch reads that after its next kernel launch.  cudaGetLastError() of the runtime torch
    uses returns and clears it; where that library cannot be reached by name, one throw-away launch takes the blame."""
    try:
        import ctypes
        ctypes.CDLL("libcudart.so.12").cudaGetLastError()
    except OSError:
        pass
    try:
        torch.empty(1, device="cuda").fill_(0)
        torch.cuda.synchronize()
    except RuntimeError:
        pass


class PinnedBuffer:
    """Page-locked host memory.  First choice: a pageable tensor of the exact size registered with cudaHostRegister
    (torch's own pinned allocator rounds every request up to a power of two, which would double a 117 GiB tier).
    Where registration is refused (a locked-memory limit of the environment), the largest power of two of bytes that
    fits the request comes from torch's pinned allocator (cudaHostAlloc) instead; `nbytes` says what was obtained."""

    def __init__(self, torch, nbytes):
        self.torch, self.registered = torch, False
        t0 = time.time()
        self.t = torch.empty(nbytes, dtype=torch.uint8)
        rc = torch.cuda.cudart().cudaHostRegister(self.t.data_ptr(), nbytes, 0)
        if int(rc) == 0:
            self.registered, self.how, self.nbytes = True, "cudaHostRegister", nbytes
        else:
            self.t = None
            clear_cuda_last_error(torch)             # or the next kernel launch reports the refused registration as its own
            pow2 = 1 << (int(nbytes).bit_length() - 1)
            try:
                self.t = torch.empty(pow2, dtype=torch.uint8, pin_memory=True)
            except RuntimeError as e:
                raise RuntimeError("no page-locked memory: cudaHostRegister of %d bytes failed (%s) and cudaHostAlloc of %d "
                                   "bytes failed (%s)" % (nbytes, rc, pow2, e))
            self.how, self.nbytes = "cudaHostAlloc", pow2
        self.seconds = time.time() - t0

    def free(self):
        if self.registered:
            self.torch.cuda.cudart().cudaHostUnregister(self.t.data_ptr())
            self.registered = False
        self.t = None


def host_tier_slots(named, block_bytes, asked, frac, n_replicas):
    """Slots of the host tier that get pinned memory behind them: all the configuration names, unless the box's
    free memory (times frac, shared by the replicas) is short; then as many as fit (the reduction is reported)."""
    if asked:
        return max(1, min(asked, named))
    budget = int(frac * mem_available_bytes() / max(1, n_replicas))
    return max(1, min(named, budget // block_bytes))


# ---- clocks sampled during the timed region -----------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


# ---- the workload ---------------------------------------------------------------------------------------
class StepWorkload:
    """State of one configuration's scheduler step on one GPU: pools, index, trace, context, ring of id buffers."""
    RING = 3

    def __init__(self, args, device, n_replicas, cfg_name="llama8b"):
        import torch
        from paper_2608_14624_b200 import binding as cs
        from paper_2608_14624_b200 import build
        from tests import synth
        build.build_library()
        self.torch, self.cs, self.synth = torch, cs, synth
        self.dev = device
        cfg = synth.CONFIGS[cfg_name]
        self.cfg_name = cfg_name
        if args.quick:
            cfg = synth.shrink(cfg, gpu_blocks=2048, host_blocks=6144)
        self.cfg = cfg
        G, Hs, L = cfg.gpu_blocks, cfg.host_blocks, cfg.n_layers
        bb = cfg.block_bytes
        # host tier: every slot the configuration names gets pinned memory behind it, unless the box is short of memory
        self.host_backed = host_tier_slots(Hs, bb, args.host_slots, args.host_frac, n_replicas)
        if args.quick:
            self.host_backed = min(self.host_backed, 1024)
        # Page-locking tens of GiB can fail although MemAvailable said otherwise (memory of a process that has just exited
        # is still being returned, a locked-memory limit): wait, ask for less, try again -- the reduction is reported.
        self.pin_attempts = 0
        while True:
            self.pin_attempts += 1
            try:
                self.pinned = PinnedBuffer(torch, self.host_backed * bb)
                self.host_backed = self.pinned.nbytes // bb          # (fewer when the fallback allocator was used)
                break
            except RuntimeError:
                if self.pin_attempts >= 6 or self.host_backed <= 1024:
                    raise
                time.sleep(3.0)
                again = host_tier_slots(Hs, bb, args.host_slots, args.host_frac, n_replicas)
                self.host_backed = max(1024, min(again, int(self.host_backed * 0.75)))
        self.host_buf = self.pinned.t
        self.t_pin = self.pinned.seconds
        self.gpu_buf = torch.empty(G * bb // 2, dtype=torch.bfloat16, device=device)
        step_elems = 1 << 28
        for lo in range(0, self.gpu_buf.numel(), step_elems):           # N(0,1) bf16 KV values, seeded
            g = torch.Generator(device=device)
            g.manual_seed(cfg.seed + lo // step_elems)
            self.gpu_buf[lo:lo + step_elems].normal_(generator=g)
        self.k_v, self.k_p = cfg.k_victims, cfg.k_prefetch
        self.stage_buf = torch.empty(self.k_v * bb, dtype=torch.uint8, device=device)
        self.gpu_pool = cs.KVPool(self.gpu_buf, G, cs.CS_LAYER_MAJOR, L)
        self.host_pool = cs.KVPool(self.host_buf, self.host_backed, cs.CS_BLOCK_MAJOR, L, first_id=G)
        self.stage_pool = cs.KVPool(self.stage_buf, self.k_v, cs.CS_BLOCK_MAJOR, L)

        # index: ids [0, G) GPU tier, [G, G+Hs) host tier; host entries without backing are not VALID
        idx = synth.make_block_index(cfg)
        if self.host_backed < Hs:
            idx.flags[G + self.host_backed:] &= np.uint8(~synth.FLAG_VALID & 0xFF)
        idx.flags[G - cfg.k_prefetch:G] &= np.uint8(~synth.FLAG_VALID & 0xFF)      # initially free GPU slots
        self.idx_host = idx
        self.N = idx.n
        self.didx = cs.DeviceIndex.from_host(idx, device)
        self.la_i32 = self.didx.last_access.view(torch.int32)
        self.pin_idx = {k: torch.from_numpy(getattr(idx, k)).pin_memory()
                        for k in ("agent", "depth", "ref_count", "flags", "last_access", "n_tokens")}
        self.meta_bytes = sum(int(t.numel() * t.element_size()) for t in self.pin_idx.values())

        # trace, events of step s padded to 16 per step so slices are cheap
        self.tr = synth.make_trace(cfg)
        self.n_steps = len(self.tr.step_off) - 1
        self.ev_chain = torch.from_numpy(self.tr.chain).pin_memory()
        self.ev_agent = torch.from_numpy(self.tr.agent).pin_memory()
        self.ev_flags = torch.from_numpy(self.tr.evflags).pin_memory()
        self.d_chain, self.d_agent, self.d_flags = (t.to(device) for t in (self.ev_chain, self.ev_agent, self.ev_flags))
        self.e2e_chain = torch.empty(64, dtype=self.ev_chain.dtype, device=device)
        self.e2e_agent = torch.empty(64, dtype=self.ev_agent.dtype, device=device)
        self.e2e_flags = torch.empty(64, dtype=self.ev_flags.dtype, device=device)

        p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=self.N,
                           block_tokens=cfg.block_tokens, r_min=0.02)
        self.params = p
        self.c = cs.CacheScout(p, device)
        # ring of list buffers: dst[b][:k_v] receives the GPU victims of step s (b = s % RING) and, one
        # step later, serves with the reserve tail as the free GPU slots the prefetch fills
        # (the last k_p GPU slots start out free -- not VALID in the index -- so the first prefetch has a target)
        free0 = torch.arange(G - self.k_p, G, dtype=torch.int32, device=device)
        self.dst = [free0.clone() for _ in range(self.RING)]
        mk = lambda n: [torch.zeros(max(n, 4), dtype=torch.int32, device=device) for _ in range(self.RING)]
        self.hv, self.pf = mk(self.k_v), mk(self.k_p)
        self.vn, self.hn, self.pn = mk(1), mk(1), mk(1)
        self.packed = torch.arange(self.k_v, dtype=torch.int32, device=device)
        self.res_pin = torch.zeros(self.k_v * 2 + self.k_p + 16, dtype=torch.int32).pin_memory()
        self.main = torch.cuda.current_stream(device)
        self.side_o = torch.cuda.Stream(device=device)
        self.side_p = torch.cuda.Stream(device=device)
        self.done_o = [None] * self.RING
        self.done_p = [None] * self.RING
        self.now0 = 100_000
        self.w_off, self.w_pre = args.offload_width, args.prefetch_width
        self.fused, self.w_ex = args.transfers in ("exchange", "staged"), args.exchange_width
        self.staged = args.transfers == "staged"
        if self.staged:
            self.ring = torch.empty(max(getattr(args, "ring_mib", 256), 4 * bb >> 20) << 20, dtype=torch.uint8, device=device)
            self.c.set_mover_staging(self.ring)
            self.dst_host = [free0.cpu().numpy().view(np.uint32).copy() for _ in range(self.RING)]
        self.fused_selects = getattr(args, "selects", "fused") == "fused"
        self.fifo = [torch.zeros(self.k_p, dtype=torch.int64, device=device) for _ in range(8)]
        self.fifo_used = 0
        self.bytes_per_step = (self.k_v + self.k_p) * bb
        self.timers = {"select": [], "compact": [], "offload": [], "prefetch": [], "observe": []}
        # warm the learner so that the prefetch gate has something to work with
        self.c.observe_invocations(self.d_chain[:2000], self.d_agent[:2000], self.d_flags[:2000])
        torch.cuda.synchronize(device)

    def step(self, s, e2e=False, timed=False):
        torch, c = self.torch, self.c
        b, prev = s % self.RING, (s - 1) % self.RING
        self.last_s = s
        main = self.main
        # ring slot b is rewritten now: the transfers that read it (step s - RING) must be over
        if self.done_o[b] is not None:
            main.wait_event(self.done_o[b])
            main.wait_event(self.done_p[b])
        nxt = (s + 1) % self.RING                 # prefetch of step s-2 reads dst[b] as its destination list
        if self.done_p[nxt] is not None:
            main.wait_event(self.done_p[nxt])
        now = self.now0 + s
        st = (600 + s) % (self.n_steps - 1)
        lo, hi = int(self.tr.step_off[st]), int(self.tr.step_off[st + 1])
        n_ev = hi - lo
        ev = (lambda: torch.cuda.Event(enable_timing=True)) if timed else (lambda: None)
        t = [ev() for _ in range(10)]
        rec = lambda e, stream: e.record(stream) if e is not None else None
        if e2e:      # this step's inputs come from pinned host memory
            self.e2e_chain[:n_ev].copy_(self.ev_chain[lo:hi], non_blocking=True)
            self.e2e_agent[:n_ev].copy_(self.ev_agent[lo:hi], non_blocking=True)
            self.e2e_flags[:n_ev].copy_(self.ev_flags[lo:hi], non_blocking=True)
            for k, src in self.pin_idx.items():
                getattr(self.didx, k).copy_(src, non_blocking=True)
            chain, agent, flags = self.e2e_chain, self.e2e_agent, self.e2e_flags
        else:
            chain, agent, flags = self.d_chain[lo:hi], self.d_agent[lo:hi], self.d_flags[lo:hi]
        rec(t[0], main)
        c.observe_invocations(chain, agent, flags, n_events=n_ev)
        rec(t[1], main)
        vict = self.dst[b][:self.k_v]
        if self.fused_selects:         # one launch: three thread-block clusters side by side
            c.select_step(self.didx, now, self.k_v, self.k_p, vict, self.vn[b], self.hv[b], self.hn[b], self.pf[b], self.pn[b])
        else:
            c.select_victims(self.didx, now, 0, self.k_v, vict, self.vn[b])
            c.select_victims(self.didx, now, 1, self.k_v, self.hv[b], self.hn[b])
            c.select_prefetch(self.didx, now, self.k_p, self.pf[b], self.pn[b])
        rec(t[2], main)
        c.compact_blocks(self.gpu_pool, self.stage_pool, vict, self.packed, n_max=self.k_v, n_dev=self.vn[b])
        rec(t[3], main)
        ready = torch.cuda.Event()
        ready.record(main)
        if self.staged:
            # copy-engine path: the host must know the host-tier slots, so the three lists and counts are read back
            # (a few KB and one host synchronisation per step), conflicts are dropped on the host (a candidate whose
            # host slot receives an offloaded block in this step), and the transfers are issued with host id lists
            r, kv, kp = self.res_pin, self.k_v, self.k_p
            r[:kv].copy_(vict, non_blocking=True)
            r[kv:2 * kv].copy_(self.hv[b][:kv], non_blocking=True)
            r[2 * kv:2 * kv + kp].copy_(self.pf[b][:kp], non_blocking=True)
            r[-16:-15].copy_(self.vn[b][:1], non_blocking=True)
            r[-15:-14].copy_(self.hn[b][:1], non_blocking=True)
            r[-14:-13].copy_(self.pn[b][:1], non_blocking=True)
            main.synchronize()
            rv = r.numpy().view(np.uint32)
            n_off, n_pre = int(min(rv[-16], rv[-15])), int(rv[-14])
            off_host, pre_host = rv[kv:kv + n_off].copy(), rv[2 * kv:2 * kv + n_pre].copy()
            keep = ~np.isin(pre_host, off_host)
            pre_gpu = self.dst[prev]
            if not keep.all():
                pre_host = pre_host[keep]
                pre_gpu = torch.from_numpy(self.dst_host[prev][:n_pre][keep].view(np.int32)).to(self.dev)
            self.dst_host[b][:kv] = rv[:kv]
            self.side_o.wait_event(ready)
            rec(t[4], self.side_o)
            c.exchange_blocks_staged(self.gpu_pool, self.host_pool, vict[:n_off], off_host, pre_host, pre_gpu, stream=self.side_o)
            rec(t[5], self.side_o)
            self.done_o[b] = torch.cuda.Event()
            self.done_o[b].record(self.side_o)
            self.done_p[b] = self.done_o[b]
            t[6], t[7] = t[4], t[5]
        elif self.fused:
            # one launch on side stream 1: GPU victims -> the slots of the host-tier victims, and the prefetch
            # candidates -> the slots freed one step earlier (their offload ran in the previous launch of this stream)
            self.side_o.wait_event(ready)
            rec(t[4], self.side_o)
            if self.w_ex:
                c.set_mover_ctas(self.w_ex, 0)
            c.exchange_blocks(self.gpu_pool, self.host_pool, vict, self.hv[b], self.pf[b], self.dst[prev],
                              n_off_max=self.k_v, n_off_dev=self.vn[b], n_pre_max=self.k_p, n_pre_dev=self.pn[b],
                              stream=self.side_o)
            if self.w_ex:
                c.set_mover_ctas(0, 0)
            rec(t[5], self.side_o)
            self.done_o[b] = torch.cuda.Event()
            self.done_o[b].record(self.side_o)
            self.done_p[b] = self.done_o[b]
            t[6], t[7] = t[4], t[5]
        else:
            # offload on side stream 1: GPU victims -> the slots of the host-tier victims
            self.side_o.wait_event(ready)
            rec(t[4], self.side_o)
            if self.w_off:
                c.set_mover_ctas(self.w_off, 0)
            c.offload_blocks(self.gpu_pool, self.host_pool, vict, self.hv[b], n_max=self.k_v, n_dev=self.vn[b],
                             stream=self.side_o)
            rec(t[5], self.side_o)
            self.done_o[b] = torch.cuda.Event()
            self.done_o[b].record(self.side_o)
            # prefetch on side stream 2 into the slots freed one step earlier (their offload must be over)
            self.side_p.wait_event(ready)
            if self.done_o[prev] is not None:
                self.side_p.wait_event(self.done_o[prev])
            rec(t[6], self.side_p)
            if self.w_pre:
                c.set_mover_ctas(self.w_pre, 0)
            c.prefetch_blocks(self.host_pool, self.gpu_pool, self.pf[b], self.dst[prev], n_max=self.k_p, n_dev=self.pn[b],
                              stream=self.side_p)
            if self.w_off or self.w_pre:
                c.set_mover_ctas(0, 0)
            rec(t[7], self.side_p)
            self.done_p[b] = torch.cuda.Event()
            self.done_p[b].record(self.side_p)
        # engine bookkeeping (plumbing, not the method): refilled victim slots are touched now, prefetched
        # host entries now have a GPU copy
        vi = vict.long().clamp_(min=0)
        self.la_i32[vi] = now
        pi = self.pf[b][:self.k_p].long().clamp_(min=0)
        self.didx.flags[pi] |= self.cs.CS_FLAG_OTHER_COPY
        # ... and the GPU copies made 8 steps ago count as evicted again, so the candidate set is stationary
        slot = self.fifo[s % 8]
        if self.fifo_used >= 8:
            self.didx.flags[slot] &= 0xF7
        slot.copy_(pi)
        self.fifo_used += 1
        if e2e:      # the step's result goes back to the host
            r = self.res_pin
            r[:self.k_v].copy_(vict, non_blocking=True)
            r[self.k_v:2 * self.k_v].copy_(self.hv[b][:self.k_v], non_blocking=True)
            r[2 * self.k_v:2 * self.k_v + self.k_p].copy_(self.pf[b][:self.k_p], non_blocking=True)
            r[-16:-15].copy_(self.vn[b][:1], non_blocking=True)
            r[-15:-14].copy_(self.hn[b][:1], non_blocking=True)
            r[-14:-13].copy_(self.pn[b][:1], non_blocking=True)
            main.synchronize()
        if timed:
            self._pending = getattr(self, "_pending", [])
            self._pending.append(t)

    def drain(self):
        self.main.wait_stream(self.side_o)
        self.main.wait_stream(self.side_p)

    def collect_timers(self):
        for t in getattr(self, "_pending", []):
            self.timers["observe"].append(t[0].elapsed_time(t[1]))
            self.timers["select"].append(t[1].elapsed_time(t[2]))
            self.timers["compact"].append(t[2].elapsed_time(t[3]))
            self.timers["offload"].append(t[4].elapsed_time(t[5]))
            self.timers["prefetch"].append(t[6].elapsed_time(t[7]))
        self._pending = []

    def take_moved_bytes(self):
        """KV bytes the transfers since the last call really moved over the link: the library's own work counters
        (kept by the mover kernels, one increment per block copied), read and reset."""
        self.torch.cuda.synchronize(self.dev)
        cn = self.c.counters(reset=True)
        self.last_counters = cn
        return cn["bytes_moved"][1] + cn["bytes_moved"][2]

    def release(self):
        """Gives the pools back (the next workload needs the memory)."""
        self.drain()
        self.torch.cuda.synchronize(self.dev)
        self.c.close()
        self.gpu_buf = self.stage_buf = self.host_buf = None
        self.gpu_pool = self.host_pool = self.stage_pool = None
        self.pinned.free()
        self.torch.cuda.empty_cache()

    def e2e_bytes(self):
        ev = 8 * 7          # <= 8 events x (4 + 2 + 1) bytes
        h2d = self.meta_bytes + ev + self.k_p * self.cfg.block_bytes
        d2h = (2 * self.k_v + self.k_p + 3) * 4 + self.k_v * self.cfg.block_bytes
        return h2d, d2h


def in_flight_factor(alone_ms, both_ms, transfer_ms):
    """Slowdown of the serving loop during the part of it that overlaps the transfer, when the loop outlasts the
    transfer: it does transfer_ms / f of its work while the transfer runs and the rest at full speed."""
    if both_ms <= transfer_ms:
        return both_ms / alone_ms
    done_during = alone_ms - (both_ms - transfer_ms)
    return transfer_ms / done_during if done_during > 0 else float("inf")


def fused_step_section(w, steps=10):
    """The whole step as ONE library call (cs_step): issued afresh every step, and captured once into a CUDA
    graph that reads the clock and the event count from device memory and is replayed; then the interference
    between the two-way transfer on the side stream and synthetic serving kernels on the main stream (a
    bandwidth-bound copy standing in for decode, a bf16 GEMM standing in for prefill; both are torch's
    kernels, they are the disturbed party, not the product).  Steps run back to back without overlap
    (the side stream rejoins the main stream every step, as a graph capture requires)."""
    torch, c, dev = w.torch, w.c, w.dev
    main, side = torch.cuda.Stream(device=dev), w.side_o          # a graph cannot be captured on the default stream
    kv, kp, bb = w.k_v, w.k_p, w.cfg.block_bytes
    i32 = lambda n, fill=0: torch.full((max(n, 4),), fill, dtype=torch.int32, device=dev)
    gv, gh, gp = i32(kv), i32(kv), i32(kp)
    gvn, ghn, gpn, now_d, nev_d = i32(1), i32(1), i32(1), i32(1), i32(1)
    free_d = w.dst[w.last_s % w.RING].clone()                  # slots freed by the last step of the main run + reserve tail
    free_last = free_d.clone()                                 # the destination list the latest step used
    cap = 16
    ev_c = torch.zeros(cap, dtype=w.d_chain.dtype, device=dev)
    ev_a = torch.zeros(cap, dtype=w.d_agent.dtype, device=dev)
    ev_f = torch.zeros(cap, dtype=w.d_flags.dtype, device=dev)
    fifo = [torch.zeros(kp, dtype=torch.int64, device=dev) for _ in range(8)]
    state = {"s": w.last_s + 1, "n": 0}

    def issue(by_value, now=0, n_ev=cap):
        c.step(w.didx, now, ev_c, ev_a, ev_f, n_ev, kv, kp, gv, gvn, gh, ghn, gp, gpn, w.gpu_pool, w.host_pool, free_d,
               stage=w.stage_pool, stage_slots=w.packed, now_dev=None if by_value else now_d,
               n_events_dev=None if by_value else nev_d, main=main, side=side, join_main=True)

    def one_step(graph):
        s = state["s"]
        now = w.now0 + s
        st = (600 + s) % (w.n_steps - 1)
        lo, hi = int(w.tr.step_off[st]), int(w.tr.step_off[st + 1])
        n_ev = hi - lo
        ev_c[:n_ev].copy_(w.d_chain[lo:hi]); ev_a[:n_ev].copy_(w.d_agent[lo:hi]); ev_f[:n_ev].copy_(w.d_flags[lo:hi])
        now_d.fill_(now); nev_d.fill_(n_ev)
        if graph is None:
            issue(True, now, n_ev)
        else:
            graph.replay()
        # engine bookkeeping, as in the main run
        vi = gv[:kv].long().clamp_(min=0)
        w.la_i32[vi] = now
        pi = gp[:kp].long().clamp_(min=0)
        w.didx.flags[pi] |= w.cs.CS_FLAG_OTHER_COPY
        if state["n"] >= 8:
            w.didx.flags[fifo[state["n"] % 8]] &= 0xF7
        fifo[state["n"] % 8].copy_(pi)
        free_last.copy_(free_d)
        free_d[:kv].copy_(gv[:kv])
        state["s"] += 1
        state["n"] += 1

    def timed(graph, k):
        with torch.cuda.stream(main):
            for _ in range(3):
                one_step(graph)
            main.synchronize()
            l0 = c.launch_count()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c.counters(reset=True)
            e0.record(main)
            for _ in range(k):
                one_step(graph)
            e1.record(main)
            main.synchronize()
            cn = c.counters()          # blocks the steps really moved (dropped prefetch candidates are not copied)
        ms = e0.elapsed_time(e1) / k
        return ms, (c.launch_count() - l0) / k, (cn["bytes_moved"][1] + cn["bytes_moved"][2]) / k / ms / 1e6

    w.drain()
    torch.cuda.synchronize(dev)
    with torch.cuda.stream(main):                               # buffers made above belong to this stream from here on
        pass
    ms_call, launches_call, gbps_call = timed(None, steps)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=main, capture_error_mode="relaxed"):
        issue(False)
    ms_graph, _, gbps_graph = timed(g, steps)
    out = {"what": "cs_step: observe + 3 selects + conflict filter + compaction + two-way transfer as one call; steps back to back, no overlap between steps",
           "ms_per_step_call": ms_call, "GBps_call": gbps_call, "kernel_launches_per_step": launches_call,
           "ms_per_step_graph_replay": ms_graph, "GBps_graph_replay": gbps_graph,
           "n_out_last_step": [int(gvn[0].item()), int(ghn[0].item()), int(gpn[0].item())], "device_status": c.get_status()}

    # ---- interference with synthetic serving kernels ------------------------------------------------------
    x = torch.empty(1 << 30, dtype=torch.float32, device=dev).normal_()
    y = torch.empty_like(x)
    a = torch.randn(8192, 8192, dtype=torch.bfloat16, device=dev)
    b = torch.randn(8192, 8192, dtype=torch.bfloat16, device=dev)
    o = torch.empty(8192, 8192, dtype=torch.bfloat16, device=dev)
    small = torch.zeros(1 << 18, dtype=torch.float32, device=dev)          # 1 MiB: a latency-bound kernel per call
    loads = {"hbm_copy_8GiB_x16": (lambda: y.copy_(x), 16), "bf16_gemm_8192_x24": (lambda: torch.matmul(a, b, out=o), 24),
             "small_kernel_chain_x4000": (lambda: small.add_(1.0), 4000)}

    def transfer():
        c.exchange_blocks(w.gpu_pool, w.host_pool, gv, gh, gp, free_last, n_off_max=kv, n_off_dev=gvn, n_pre_max=kp,
                          n_pre_dev=gpn, stream=side)

    def run(load, with_transfer, with_load=True):
        fn, reps = load
        ts = []
        for _ in range(3):
            torch.cuda.synchronize(dev)
            m0, m1, s0, s1 = (torch.cuda.Event(enable_timing=True) for _ in range(4))
            m0.record(main)
            side.wait_event(m0)
            if with_transfer:
                s0.record(side)
                transfer()
                s1.record(side)
            with torch.cuda.stream(main):
                if with_load:
                    for _ in range(reps):
                        fn()
            m1.record(main)
            torch.cuda.synchronize(dev)
            ts.append((m0.elapsed_time(m1), s0.elapsed_time(s1) if with_transfer else 0.0))
        return min(t[0] for t in ts), min(t[1] for t in ts)

    _, x_alone = run(loads["hbm_copy_8GiB_x16"], True, with_load=False)
    inter = {"transfer_alone_ms": x_alone}
    for name, load in loads.items():
        run(load, False)
        alone, _ = run(load, False)
        both, x_both = run(load, True)
        inter[name] = {"serving_alone_ms": alone, "serving_with_transfer_ms": both, "serving_slowdown": both / alone,
                       "serving_slowdown_while_transfer_in_flight": in_flight_factor(alone, both, x_both),
                       "transfer_with_serving_ms": x_both, "transfer_slowdown": x_both / x_alone}
    # the same chain as a CUDA graph (no per-kernel host traffic), disturbed by this library's transfer and by the
    # same bytes moved by the copy engines (two pinned cudaMemcpyAsync copies, 512 MiB out while 768 MiB come in)
    cg = torch.cuda.CUDAGraph()
    with torch.cuda.graph(cg, stream=main, capture_error_mode="relaxed"):
        for _ in range(1000):
            small.add_(1.0)
    side2 = torch.cuda.Stream(device=dev)
    ce_out_h, ce_in_h = w.host_buf[:512 << 20], w.host_buf[(1 << 30):(1 << 30) + (768 << 20)]
    ce_out_d = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    ce_in_d = torch.empty(768 << 20, dtype=torch.uint8, device=dev)

    def copy_engines():
        with torch.cuda.stream(side):
            ce_out_h.copy_(ce_out_d, non_blocking=True)
        with torch.cuda.stream(side2):
            ce_in_d.copy_(ce_in_h, non_blocking=True)
        side.wait_stream(side2)

    def run_graph(disturber):
        best = None
        for _ in range(3):
            torch.cuda.synchronize(dev)
            m0, m1, s0, s1 = (torch.cuda.Event(enable_timing=True) for _ in range(4))
            m0.record(main)
            side.wait_event(m0)
            side2.wait_event(m0)
            s0.record(side)
            if disturber is not None:
                disturber()
            s1.record(side)
            with torch.cuda.stream(main):
                for _ in range(4):
                    cg.replay()
            m1.record(main)
            torch.cuda.synchronize(dev)
            t = (m0.elapsed_time(m1), s0.elapsed_time(s1))
            best = t if best is None or t[0] < best[0] else best
        return best

    g_alone, _ = run_graph(None)
    g_ours, g_ours_x = run_graph(transfer)
    g_ce, g_ce_x = run_graph(copy_engines)
    inter["graph_chain_4x1000_small_kernels"] = {
        "alone_ms": g_alone,
        "with_this_library_transfer_ms": g_ours, "slowdown_while_in_flight": in_flight_factor(g_alone, g_ours, g_ours_x),
        "with_copy_engine_transfer_ms": g_ce, "copy_engine_transfer_ms": g_ce_x,
        "slowdown_while_copy_engines_in_flight": in_flight_factor(g_alone, g_ce, g_ce_x)}
    del ce_out_d, ce_in_d
    # the knob: a narrower transfer disturbs latency-bound kernels less and moves fewer bytes per second
    c.set_mover_ctas(8, 0)
    _, x8 = run(loads["small_kernel_chain_x4000"], True, with_load=False)
    both8, x8_both = run(loads["small_kernel_chain_x4000"], True)
    c.set_mover_ctas(0, 0)
    alone_small = inter["small_kernel_chain_x4000"]["serving_alone_ms"]
    inter["small_kernel_chain_x4000_transfer_width_8"] = {
        "transfer_alone_ms": x8, "serving_with_transfer_ms": both8, "serving_slowdown": both8 / alone_small,
        "serving_slowdown_while_transfer_in_flight": in_flight_factor(alone_small, both8, x8_both),
        "transfer_with_serving_ms": x8_both, "transfer_slowdown": x8_both / x8}
    # ---- the same 256 out + 384 in through three forms of transfer: what each gives the link and what it costs the
    #      kernels running beside it (a graph-replayed chain of small kernels, this library's own fused select, and the
    #      in-step compaction) ------------------------------------------------------------------------------------
    r_np = lambda t, n: t[:n].cpu().numpy().view(np.uint32).copy()
    n_off, n_pre = int(min(gvn[0].item(), ghn[0].item())), int(gpn[0].item())
    off_host, pre_host = r_np(gh, n_off), r_np(gp, n_pre)
    keep = (pre_host != 0xFFFFFFFF) & ~np.isin(pre_host, off_host)
    pre_host_k = pre_host[keep]
    pre_gpu_k = torch.from_numpy(r_np(free_last, n_pre)[keep].view(np.int32)).to(dev)
    ring = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    c.set_mover_staging(ring)
    sv, sh, sp, svn, shn, spn = i32(kv), i32(kv), i32(kp), i32(1), i32(1), i32(1)
    now_sel = w.now0 + state["s"]

    def staged():
        c.exchange_blocks_staged(w.gpu_pool, w.host_pool, gv[:n_off], off_host, pre_host_k, pre_gpu_k, stream=side)

    # the same transfer when the engine numbers the host tier itself, as consecutive runs (a log-structured host tier:
    # the i-th offloaded block of a step goes to slot first + i): a step's transfer is a handful of large copies
    G0 = w.cfg.gpu_blocks
    run_off = (G0 + np.arange(n_off)).astype(np.uint32)
    run_pre = (G0 + n_off + np.arange(len(pre_host_k))).astype(np.uint32)

    def staged_runs():
        c.exchange_blocks_staged(w.gpu_pool, w.host_pool, gv[:n_off], run_off, run_pre, pre_gpu_k, stream=side)

    def beside(op, reps, disturber):
        """Per-call time of `reps` back-to-back calls of op on the main stream while the disturber runs on the side stream."""
        best, x_ms = None, 0.0
        for _ in range(3):
            torch.cuda.synchronize(dev)
            m0, e0, e1, s0, s1 = (torch.cuda.Event(enable_timing=True) for _ in range(5))
            m0.record(main)
            side.wait_event(m0)
            s0.record(side)
            if disturber is not None:
                disturber()
            s1.record(side)
            with torch.cuda.stream(main):
                e0.record(main)
                for _ in range(reps):
                    op()
                e1.record(main)
            torch.cuda.synchronize(dev)
            t = e0.elapsed_time(e1) / reps
            if best is None or t < best:
                best, x_ms = t, s0.elapsed_time(s1)
        return best, x_ms

    sel_op = lambda: c.select_step(w.didx, now_sel, kv, kp, sv, svn, sh, shn, sp, spn, stream=main)
    cmp_op = lambda: c.compact_blocks(w.gpu_pool, w.stage_pool, gv, w.packed, n_max=kv, n_dev=gvn, stream=main)
    sel_alone, _ = beside(sel_op, 20, None)
    cmp_alone, _ = beside(cmp_op, 10, None)
    variants = []
    for name, width, fn in (("sm_direct_width_32", 0, transfer), ("sm_direct_width_8", 8, transfer),
                            ("staged_copy_engines_scattered_host_slots", 0, staged),
                            ("staged_copy_engines_consecutive_host_slots", 0, staged_runs)):
        c.set_mover_ctas(width, 0)
        _, x_alone_ms = beside(lambda: None, 1, fn)
        g_ms, g_x = run_graph(fn)
        sel_ms, _ = beside(sel_op, 20, fn)
        cmp_ms, _ = beside(cmp_op, 10, fn)
        moved = (n_off + (n_pre if fn is transfer else len(pre_host_k))) * bb
        variants.append({"transfer": name, "transfer_alone_ms": x_alone_ms, "link_GBps": moved / x_alone_ms / 1e6,
                         "graph_chain_slowdown_while_in_flight": in_flight_factor(g_alone, g_ms, g_x),
                         "fused_select_ms_alone": sel_alone, "fused_select_ms_beside": sel_ms, "fused_select_slowdown": sel_ms / sel_alone,
                         "compaction_ms_alone": cmp_alone, "compaction_ms_beside": cmp_ms,
                         "compaction_GBps_beside": 2 * kv * bb / cmp_ms / 1e6, "compaction_slowdown": cmp_ms / cmp_alone})
    c.set_mover_ctas(0, 0)
    c.set_mover_staging(None)
    inter["transfer_variants"] = variants
    out["interference"] = inter
    del x, y, a, b, o, small, ring
    return out


def host_link_peak(torch, device, n_bytes=GIB, reps=10):
    """Pinned cudaMemcpyAsync of one contiguous buffer, each direction alone, both at once, and both at once in
    the step's proportions (2 bytes out for every 3 bytes in: 256 blocks offloaded, 384 prefetched)."""
    h = torch.empty(n_bytes, dtype=torch.uint8, pin_memory=True)
    h2 = torch.empty(n_bytes, dtype=torch.uint8, pin_memory=True)
    d = torch.empty(n_bytes, dtype=torch.uint8, device=device)
    d2 = torch.empty(n_bytes, dtype=torch.uint8, device=device)
    s1, s2 = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
    out = {}
    n_out = (n_bytes * 2 // 3) & ~4095
    for name in ("d2h", "h2d", "bidir", "bidir_step_mix"):
        best = 0.0
        for _ in range(reps):
            torch.cuda.synchronize(device)
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record(s1)
            s2.wait_event(e0)
            if name in ("d2h", "bidir"):
                with torch.cuda.stream(s1):
                    h.copy_(d, non_blocking=True)
            if name == "bidir_step_mix":
                with torch.cuda.stream(s1):
                    h[:n_out].copy_(d[:n_out], non_blocking=True)
            if name in ("h2d", "bidir", "bidir_step_mix"):
                with torch.cuda.stream(s2):
                    d2.copy_(h2, non_blocking=True)
            e2.record(s2)
            s1.wait_event(e2)
            e1.record(s1)
            torch.cuda.synchronize(device)
            ms = e0.elapsed_time(e1)
            moved = {"bidir": 2 * n_bytes, "bidir_step_mix": n_bytes + n_out}.get(name, n_bytes)
            best = max(best, moved / ms / 1e6)
        out[name] = best
    del h, h2, d, d2
    return out


def time_call(torch, stream, fn, reps, warm=1, hide_host=True):
    """Median and best device time of fn's work on `stream` (CUDA events).  With hide_host the stream is first given
    ~150 us of busy-waiting, during which the host enqueues the first event, fn's launches and the second event:
    the measured span is then the device's time for the work itself, not the host's time to issue it (what a
    pipelined caller sees; it matters for transfers of a few tens of microseconds)."""
    for _ in range(warm):
        fn()
    stream.synchronize()
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if hide_host:
            with torch.cuda.stream(stream):
                torch.cuda._sleep(300_000)
        e0.record(stream)
        fn()
        e1.record(stream)
        stream.synchronize()
        ts.append(e0.elapsed_time(e1))
    return float(np.median(ts)), float(min(ts))


def _block_from_pool(buf_u8, layout, n_slots, L, chunk, slot):
    """The 2L chunks of one block of a device pool as a flat host array in [layer][plane][byte] order (plain indexing)."""
    if layout == 0:
        return buf_u8.view(L, 2, n_slots, chunk)[:, :, slot, :].contiguous().cpu().numpy().reshape(-1)
    return buf_u8.view(n_slots, L, 2, chunk)[slot].cpu().numpy().reshape(-1)


def _check_moved_blocks(orc, get_src, get_dst, src_layout, dst_layout, L, chunk, n, rng, n_samples=32):
    """After a timed transfer: sampled blocks (every one of their 2L chunks) against the oracle's chunk-by-chunk copy
    between one-slot stand-in pools.  Returns the number of blocks compared; raises on any differing byte."""
    picks = rng.choice(n, size=min(n_samples, n), replace=False)
    for i in picks:
        stand_src = np.ascontiguousarray(get_src(int(i)))
        stand_dst = np.zeros_like(stand_src)
        orc.move_blocks(stand_src, src_layout, 1, stand_dst, dst_layout, 1, L, chunk, [0], [0])
        if not np.array_equal(get_dst(int(i)), stand_dst):
            raise RuntimeError("mover sweep: block %d of a %d-block batch differs from the oracle's copy" % (i, n))
    return len(picks)


def mover_sweep(w, hbm_peak, link):
    """Batches of 1..4096 uniformly random scattered blocks: offload, prefetch, device-to-device,
    GPU pool addressed layer-major and block-major (same memory, two address formulas).  After the last
    repetition of every transfer 32 sampled blocks are compared byte for byte with the oracle's copy."""
    from oracle import cs_oracle as orc
    torch, cs, synth, c = w.torch, w.cs, w.synth, w.c
    cfg, dev = w.cfg, w.dev
    rng = synth.rng_for(cfg, 11)
    G, L, bb, chunk = cfg.gpu_blocks, cfg.n_layers, cfg.block_bytes, cfg.chunk_bytes
    rows = []
    side = w.side_o
    gpu_u8 = w.gpu_buf.view(torch.uint8)
    up = lambda a: torch.from_numpy(a.view(np.int32)).to(dev)
    host_block = lambda slot: w.host_buf[slot * bb:(slot + 1) * bb].numpy()
    for n in (1, 8, 64, 512, 4096):
        if n > w.host_backed or 2 * n > G:
            continue
        src, dst_h = synth.mover_batch(n, G - n, w.host_backed, rng)
        back = (G - n + np.arange(n)).astype(np.uint32)                     # disjoint from every src
        src_rot = np.roll(src, 1)                                           # the compaction moves other blocks than the prefetch did
        d_src, d_dst_h = up(src.astype(np.uint32)), up((dst_h + G).astype(np.uint32))   # host pool ids start at G
        d_back, d_src_rot = up(back), up(src_rot.astype(np.uint32))
        reps = 20 if n <= 512 else 8                                        # after 3 warm-up repetitions
        # fair comparator for the latency-bound small batches: one contiguous pinned copy of the same size
        tmp = torch.empty(n * bb, dtype=torch.uint8, device=dev)
        hview = w.host_buf[:n * bb]
        with torch.cuda.stream(side):
            _, cp_o = time_call(torch, side, lambda: hview.copy_(tmp, non_blocking=True), reps)
            _, cp_p = time_call(torch, side, lambda: tmp.copy_(hview, non_blocking=True), reps)
        del tmp
        for lay_name, lay in (("layer_major", cs.CS_LAYER_MAJOR), ("block_major", cs.CS_BLOCK_MAJOR)):
            gp = cs.KVPool(w.gpu_buf, G, lay, L)
            pool_block = lambda slot: _block_from_pool(gpu_u8, lay, G, L, chunk, slot)
            checked = 0
            med_o, best_o = time_call(torch, side, lambda: c.offload_blocks(gp, w.host_pool, d_src, d_dst_h, stream=side), reps, warm=3)
            checked += _check_moved_blocks(orc, lambda i: pool_block(int(src[i])), lambda i: host_block(int(dst_h[i])),
                                           lay, cs.CS_BLOCK_MAJOR, L, chunk, n, rng)
            med_p, best_p = time_call(torch, side, lambda: c.prefetch_blocks(w.host_pool, gp, d_dst_h, d_back, stream=side), reps, warm=3)
            checked += _check_moved_blocks(orc, lambda i: host_block(int(dst_h[i])), lambda i: pool_block(int(back[i])),
                                           cs.CS_BLOCK_MAJOR, lay, L, chunk, n, rng)
            med_c, best_c = time_call(torch, side, lambda: c.compact_blocks(gp, gp, d_src_rot, d_back, stream=side), reps, warm=3)
            checked += _check_moved_blocks(orc, lambda i: pool_block(int(src_rot[i])), lambda i: pool_block(int(back[i])),
                                           lay, lay, L, chunk, n, rng)
            gb = n * bb / 1e9
            rows.append({"blocks": n, "gpu_layout": lay_name,
                         "offload_GBps": gb / (med_o / 1e3), "offload_frac_of_link": gb / (med_o / 1e3) / link["d2h"],
                         "prefetch_GBps": gb / (med_p / 1e3), "prefetch_frac_of_link": gb / (med_p / 1e3) / link["h2d"],
                         "memcpy_same_size_d2h_GBps": gb / (cp_o / 1e3), "memcpy_same_size_h2d_GBps": gb / (cp_p / 1e3),
                         "offload_frac_of_memcpy_same_size": cp_o / med_o, "prefetch_frac_of_memcpy_same_size": cp_p / med_p,
                         "d2d_GBps_rw": 2 * gb / (med_c / 1e3), "d2d_frac_of_hbm": 2 * gb / (med_c / 1e3) / hbm_peak,
                         "offload_ms": med_o, "prefetch_ms": med_p, "d2d_ms": med_c,
                         "offload_ms_best": best_o, "prefetch_ms_best": best_p, "d2d_ms_best": best_c, "repetitions": reps,
                         "blocks_byte_checked_against_oracle": checked})
    return rows


def metadata_scale(torch, cs, synth, dev, hbm_peak, calls=10000):
    """1,000,000-entry index, 256 agents: observe 64 events + select 10,000 victims + 2,000 prefetch
    candidates per call, `calls` calls in a row with the index evolving between them; every call is timed
    with CUDA events on the stream (median and 99th percentile).  Three ways of issuing the same call:
    the two selects as separate calls, both in one cs_select_step call, and that call replayed from a CUDA graph."""
    cfg = synth.CONFIGS["meta1m"]
    N = 1_000_000
    idx = synth.make_block_index(cfg, n=N, tier="random")
    d = cs.DeviceIndex.from_host(idx, dev)
    n_tr = min(calls, 2000)                                    # the event trace is cycled beyond 2,000 calls
    tr = synth.make_trace(cfg, n_invocations=64 * (n_tr + 40))
    p = cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=N, block_tokens=cfg.block_tokens, r_min=0.02)
    c = cs.CacheScout(p, dev)
    ch, ag = torch.from_numpy(tr.chain).to(dev), torch.from_numpy(tr.agent).to(dev)
    c.observe_invocations(ch[:64 * 30], ag[:64 * 30], None)
    v = torch.empty(cfg.k_victims, dtype=torch.int32, device=dev)
    pf = torch.empty(cfg.k_prefetch, dtype=torch.int32, device=dev)
    vn, pn = torch.zeros(4, dtype=torch.int32, device=dev), torch.zeros(4, dtype=torch.int32, device=dev)
    la = d.last_access.view(torch.int32)
    stream = torch.cuda.current_stream(dev)
    fifo = [torch.zeros(cfg.k_prefetch, dtype=torch.int64, device=dev) for _ in range(8)]
    state = {"call": 0}

    def bookkeeping(now):                                      # untimed: victims refilled, prefetched entries leave the
        la[v.long().clamp_(min=0)] = now                       # host tier and return to it 8 calls later (stationary state)
        pi = pf.long().clamp_(min=0)
        d.flags[pi] &= 0xFB
        if state["call"] >= 8:
            d.flags[fifo[state["call"] % 8]] |= 4
        fifo[state["call"] % 8].copy_(pi)
        state["call"] += 1

    def run(issue, n_calls, warm=5):
        evs = []
        l0 = c.launch_count()
        for k in range(n_calls + warm):
            call = state["call"]
            now = 100_000 + call
            lo = 64 * (30 + call % n_tr)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            issue(now, lo)
            e1.record(stream)
            bookkeeping(now)
            if k >= warm:
                evs.append((e0, e1))
        torch.cuda.synchronize(dev)
        us = np.array([a.elapsed_time(b) for a, b in evs]) * 1e3
        return {"us_median": float(np.median(us)), "us_p99": float(np.percentile(us, 99)), "us_min": float(us.min()),
                "us_mean": float(us.mean()), "launches_per_call": (c.launch_count() - l0) / (n_calls + warm)}

    def separate(now, lo):
        c.observe_invocations(ch[lo:lo + 64], ag[lo:lo + 64], None)
        c.select_victims(d, now, 0, cfg.k_victims, v, vn)
        c.select_prefetch(d, now, cfg.k_prefetch, pf, pn)

    def together(now, lo):
        c.observe_invocations(ch[lo:lo + 64], ag[lo:lo + 64], None)
        c.select_step(d, now, cfg.k_victims, cfg.k_prefetch, v, vn, None, None, pf, pn)

    t_wall = time.perf_counter()
    r_sep = run(separate, calls)
    r_tog = run(together, calls)
    # the same call captured once into a CUDA graph that reads the clock from device memory, replayed with fresh events
    now_d = torch.zeros(4, dtype=torch.int32, device=dev)
    ev_c, ev_a = torch.zeros(64, dtype=ch.dtype, device=dev), torch.zeros(64, dtype=ag.dtype, device=dev)
    cap = torch.cuda.Stream(device=dev)
    cap.wait_stream(stream)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=cap, capture_error_mode="relaxed"):
        c.observe_invocations(ev_c, ev_a, None, stream=cap)
        c.set_device_clock(now_d)                  # the captured selects read the clock when they run, not when captured
        c.select_step(d, 0, cfg.k_victims, cfg.k_prefetch, v, vn, None, None, pf, pn, stream=cap)
        c.set_device_clock(None)
    cap.synchronize()

    def replay_timed(n_calls, warm=5):
        evs = []
        with torch.cuda.stream(cap):
            for k in range(n_calls + warm):
                call = state["call"]
                now = 100_000 + call
                lo = 64 * (30 + call % n_tr)
                ev_c.copy_(ch[lo:lo + 64]); ev_a.copy_(ag[lo:lo + 64]); now_d.fill_(now)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(cap)
                g.replay()
                e1.record(cap)
                bookkeeping(now)
                if k >= warm:
                    evs.append((e0, e1))
        cap.synchronize()
        us = np.array([a.elapsed_time(b) for a, b in evs]) * 1e3
        return {"us_median": float(np.median(us)), "us_p99": float(np.percentile(us, 99)), "us_min": float(us.min()),
                "us_mean": float(us.mean())}

    stream.wait_stream(cap)
    r_graph = replay_timed(calls)
    wall = time.perf_counter() - t_wall
    best = min(r_sep["us_median"], r_tog["us_median"], r_graph["us_median"]) * 1e-6
    algo_bytes = N * (9 + 11) + (cfg.k_victims + cfg.k_prefetch) * 4        # one scan per select when the remembered
    #                                                                        threshold holds: 9 B (victims) + 11 B (prefetch) per entry
    cn = c.counters()
    return {"workload": "metadata-scale (BASELINE.json configs[4]): 1,000,000-entry index, 256 agents, observe 64 events + k=10000 victims + 2000 prefetch candidates per call",
            "calls_timed_per_form": calls, "wall_seconds_all_forms": wall,
            "separate_calls": r_sep, "one_select_step_call": r_tog, "graph_replay": r_graph,
            "us_per_call_median": best * 1e6, "blocks_scored_selected_per_s": 2 * N / best,
            "algorithmic_GBps": algo_bytes / best / 1e9, "frac_of_hbm_peak": algo_bytes / best / 1e9 / hbm_peak,
            "target_frac_of_hbm_peak": 0.60, "target_met": bool(algo_bytes / best / 1e9 / hbm_peak >= 0.60),
            "note": "11 MB of metadata per call: at 0.60 of the HBM peak a call would last 2.6 us, less than one kernel launch; "
                    "the call is latency-bound and the fraction is reported as measured",
            "selects_counted_by_the_kernels": cn["selects"], "selects_whose_threshold_held": cn["fast_hits"],
            "selects_with_buckets_filled_in_place": cn["region_selects"], "of_those_regrouped": cn["region_overflows"],
            "n_out": [int(vn[0].item()), int(pn[0].item())],
            "device_status": c.get_status()}


def hbm_regime_section(torch, cs, synth, dev, hbm_peak, n_entries=64_000_000):
    """Score and select over an index far larger than L2 (64,000,000 entries = 704 MB of metadata), where
    the scans are bound by memory or instruction issue instead of launch latency: the regime in which a
    fraction of the HBM roofline is meaningful for these kernels."""
    cfg = synth.CONFIGS["meta1m"]
    idx = synth.make_block_index(cfg, n=n_entries, tier="random")
    d = cs.DeviceIndex.from_host(idx, dev)
    del idx
    tr = synth.make_trace(cfg, n_invocations=4000)
    c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=n_entries,
                                     block_tokens=cfg.block_tokens, r_min=0.02), dev)
    c.observe_invocations(torch.from_numpy(tr.chain).to(dev), torch.from_numpy(tr.agent).to(dev), None)
    k = cfg.k_victims
    v = torch.empty(k, dtype=torch.int32, device=dev)
    vn = torch.zeros(4, dtype=torch.int32, device=dev)
    sc = torch.empty(n_entries, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev)
    t_score, _ = time_call(torch, stream, lambda: c.score_blocks(d, 100_000, out=sc), 5, warm=2)
    t_sel, _ = time_call(torch, stream, lambda: c.select_victims(d, 100_000, 0, k, v, vn), 5, warm=2)
    score_bytes = n_entries * (2 + 4 + 1 + 4)             # agent, last_access, n_tokens in; fp32 score out
    sel_bytes = n_entries * 9 + 4 * k                     # one scan of agent, ref_count, flags, last_access, n_tokens:
    #                                                     the threshold bin remembered from the previous call holds,
    #                                                     so the histogram pass also collects the candidates
    cn = c.counters()
    return {"entries": n_entries, "k": k, "candidates_ordered_per_select": cn["candidates"][0],
            "selects": cn["selects"][0], "selects_that_read_the_index_once": cn["fast_hits"][0],
            "score_ms": t_score, "score_GBps": score_bytes / t_score / 1e6, "score_frac_of_hbm_peak": score_bytes / t_score / 1e6 / hbm_peak,
            "select_ms": t_sel, "select_GBps": sel_bytes / t_sel / 1e6, "select_frac_of_hbm_peak": sel_bytes / t_sel / 1e6 / hbm_peak,
            "blocks_scored_selected_per_s": n_entries / (t_sel / 1e3), "n_out": int(vn[0].item())}


def exact_survival_section(torch, cs, synth, dev):
    """Eq. 6 as an alternative scorer: time of one table (CUDA events) and how far the victim list it
    gives is from the list of the hop-distance proxy of Eq. 8 (context for the approximation)."""
    rows = []
    for name, n_idx, k, K in (("llama8b", 80_000, 256, 4), ("llama70b", 52_000, 256, 4), ("meta1m", 1_000_000, 10_000, 4)):
        cfg = synth.CONFIGS[name]
        tr = synth.make_trace(cfg, n_invocations=6000)
        c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=n_idx,
                                         block_tokens=cfg.block_tokens, r_min=0.02), dev)
        c.observe_invocations(torch.from_numpy(tr.chain).to(dev), torch.from_numpy(tr.agent).to(dev), None)
        stream = torch.cuda.current_stream(dev)
        A = cfg.n_agents
        ps = torch.empty(A, dtype=torch.float32, device=dev)
        fs = torch.empty(A, dtype=torch.float32, device=dev)
        med, best = time_call(torch, stream, lambda: cs.cs_exact_survival(c.ctx, cs.CS_AGENT_NONE, K, ps, fs), 20, warm=3)
        d = cs.DeviceIndex.from_host(synth.make_block_index(cfg, n=n_idx, tier="random" if name == "meta1m" else "range"), dev)
        v_proxy, _ = c.select_victims(d, 100_000, 0, k)
        c.use_survival_table(fs)
        v_exact, _ = c.select_victims(d, 100_000, 0, k)
        c.use_survival_table(None)
        common = len(set(v_proxy[:k].tolist()) & set(v_exact[:k].tolist()))
        rows.append({"config": name, "agents": A, "steps_K": K, "us_per_table_median": med * 1e3, "us_min": best * 1e3,
                     "fp64_GFLOPs": 2.0 * A ** 3 * K / (med / 1e3) / 1e9,
                     "victims_shared_with_hop_proxy": common / k})
    return rows


# ---- the oracle on the host cores (cpu_baseline and --impl reference) ----------------------------------------
class OracleStep:
    """The same scheduler step computed by the CPU oracle.  Bounded sample: the selections run over
    the configuration's full index, the mover copies the step's 256 + 384 blocks at their real size but
    between two stand-in pools of 4 GiB in host memory (ids taken modulo their slot count), single thread."""

    def __init__(self, cfg_name="llama8b"):
        from oracle import cs_oracle as orc
        from tests import synth
        self.orc, self.synth = orc, synth
        cfg = synth.CONFIGS[cfg_name]
        self.cfg = cfg
        self.o = orc.Oracle(orc.Params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, block_tokens=cfg.block_tokens, r_min=0.02))
        self.tr = synth.make_trace(cfg)
        self.o.observe(self.tr.chain[:2000], self.tr.agent[:2000], self.tr.evflags[:2000])
        self.idx = synth.make_block_index(cfg)
        self.S = (4 * GIB) // cfg.block_bytes            # 2,048 slots of 2 MiB, 819 of 5 MiB
        self.sample = ("selections over the full %d-entry index; mover copies the step's %d+%d blocks of %.0f MiB between two "
                       "%d-slot host stand-in pools (ids modulo %d)" % (cfg.n_index, cfg.k_victims, cfg.k_prefetch,
                                                                        cfg.block_bytes / 2**20, self.S, self.S))
        rng = synth.rng_for(cfg, 21)
        self.a = synth.kv_pool_u16(self.S, cfg.n_layers, cfg.chunk_bytes, rng).view(np.uint8)
        self.b = np.zeros_like(self.a)
        self.bytes_per_step = (cfg.k_victims + cfg.k_prefetch) * cfg.block_bytes

    def step(self, s):
        cfg, o, idx = self.cfg, self.o, self.idx
        now = 100_000 + s
        st = (250 + s) % (len(self.tr.step_off) - 2)
        lo, hi = int(self.tr.step_off[st]), int(self.tr.step_off[st + 1])
        o.observe(self.tr.chain[lo:hi], self.tr.agent[lo:hi], self.tr.evflags[lo:hi])
        _, s32 = o.scores(idx, now)
        v, vn = o.select_victims(idx, now, 0, cfg.k_victims, s32)
        h, hn = o.select_victims(idx, now, 1, cfg.k_victims, s32)
        p, pn = o.select_prefetch(idx, now, cfg.k_prefetch, s32)
        L, ch, S = cfg.n_layers, cfg.chunk_bytes, self.S
        m = lambda x, n: (x[:n] % S).astype(np.uint32)
        self.orc.move_blocks(self.a, 0, S, self.b, 1, S, L, ch, m(v, vn), m(h, vn))                       # offload
        self.orc.move_blocks(self.b, 1, S, self.a, 0, S, L, ch, m(p, pn), np.arange(pn, dtype=np.uint32) % S)  # prefetch
        idx.last_access[v[:vn].astype(np.int64)] = now
        return vn + pn


def run_reference(args):
    """--impl reference: the oracle, as it stands, timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    ow = OracleStep(args.config)
    for s in range(args.warmup):
        ow.step(s)
    t0 = time.perf_counter()
    for s in range(args.steps):
        ow.step(args.warmup + s)
    dt = time.perf_counter() - t0
    gbps = ow.bytes_per_step * args.steps / dt / 1e9
    sample = ow.sample
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbps, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.config] + ": observe + 3 selects over the full index + offload 256 / prefetch 384 blocks",
                   "sample": sample},
        "cpu_baseline": {"value": gbps, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample,
                         "blocks_scored_selected_per_s": 3 * ow.idx.n * args.steps / dt},
        "e2e": {"value": gbps, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


PHASE_NAMES = {0: "refresh: entry", 1: "refresh: dependency wait over", 2: "refresh: rows of CTA 0 done (events applied, Eq. 3, arg-max, adjacency)",
               3: "refresh: last CTA starts", 4: "refresh: cur[] / last agent written, Eq. 2 done", 5: "refresh: BFS and Eq. 8 done",
               8: "scan: entry", 9: "scan: tables, thresholds, histogram set up", 10: "scan: dependency wait over",
               11: "scan: index read, queues worked off (CTA 0)", 12: "scan: candidates and histogram flushed (CTA 0)",
               13: "scan: last CTA starts", 14: "scan: threshold found, splitters published",
               24: "bucket: dependency wait over (histogram and collect launches returned)", 25: "bucket: CTA 0 done",
               26: "scatter: dependency wait over", 27: "rank: dependency wait over", 28: "rank: CTA 0 done",
               29: "bucket: state, splitters and keys arrived (CTA 0)", 30: "bucket: buckets found (CTA 0)",
               31: "bucket: slots taken (CTA 0)",
               40: "rank: bucket offsets known (CTA 0)", 41: "rank: bucket 0 in the tile", 42: "rank: bucket 0 sorted",
               56: "scan: per-call tables loaded [victims]", 57: "scan: age cuts built [victims]",
               58: "scan: index tiles walked, whole rounds of the queue worked off (CTA 0) [victims]",
               60: "scan: per-call tables loaded [prefetch]", 61: "scan: age cuts built [prefetch]",
               62: "scan: index tiles walked, whole rounds of the queue worked off (CTA 0) [prefetch]"}


def phase_timeline(args, torch, device):
    """Where the time of one metadata-scale call goes (1,000,000 entries, 256 agents: observe 64 events, 10,000 victims,
    2,000 prefetch candidates as one cs_select_step, replayed from a CUDA graph).  Needs the profiling build of the
    library: every kernel stores the GPU's global nanosecond timer at its phase boundaries, read back after each call.
    Prints medians over the calls after a warm-up, in microseconds from the first stamp of the call."""
    from paper_2608_14624_b200 import binding as cs
    from paper_2608_14624_b200 import build
    from tests import synth
    assert cs._lib is None, "the library is loaded already"
    cs.LIB_PATH = build.build_stamped_library()                           # the binding loads it on first use
    cfg = synth.CONFIGS["meta1m"]
    N, calls, warm = 1_000_000, max(20, args.steps), 20
    d = cs.DeviceIndex.from_host(synth.make_block_index(cfg, n=N, tier="random"), device)
    tr = synth.make_trace(cfg, n_invocations=64 * (calls + warm + 40))
    c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=N, block_tokens=cfg.block_tokens,
                                     r_min=0.02), device)
    ch, ag = torch.from_numpy(tr.chain).to(device), torch.from_numpy(tr.agent).to(device)
    c.observe_invocations(ch[:64 * 30], ag[:64 * 30], None)
    v = torch.empty(cfg.k_victims, dtype=torch.int32, device=device)
    pf = torch.empty(cfg.k_prefetch, dtype=torch.int32, device=device)
    vn, pn = torch.zeros(4, dtype=torch.int32, device=device), torch.zeros(4, dtype=torch.int32, device=device)
    la = d.last_access.view(torch.int32)
    fifo = [torch.zeros(cfg.k_prefetch, dtype=torch.int64, device=device) for _ in range(8)]
    now_d = torch.zeros(4, dtype=torch.int32, device=device)
    ev_c, ev_a = torch.zeros(64, dtype=ch.dtype, device=device), torch.zeros(64, dtype=ag.dtype, device=device)
    cap = torch.cuda.Stream(device=device)
    cap.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=cap, capture_error_mode="relaxed"):
        c.observe_invocations(ev_c, ev_a, None, stream=cap)
        c.set_device_clock(now_d)
        c.select_step(d, 0, cfg.k_victims, cfg.k_prefetch, v, vn, None, None, pf, pn, stream=cap)
        c.set_device_clock(None)
    cap.synchronize()
    rows, timed = [], []
    with torch.cuda.stream(cap):
        for i in range(calls + warm):
            now, lo = 100_000 + i, 64 * (30 + i)
            ev_c.copy_(ch[lo:lo + 64]); ev_a.copy_(ag[lo:lo + 64]); now_d.fill_(now)
            torch.cuda._sleep(400_000)                                     # the host gets ahead: nothing below waits for it
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(cap); g.replay(); e1.record(cap)
            cap.synchronize()
            if i >= warm:
                timed.append(e0.elapsed_time(e1) * 1e3)
                rows.append(np.array(c.phase_stamps(), dtype=np.int64))
            la[v.long().clamp_(min=0)] = now                              # the index evolves as in metadata_scale
            pi = pf.long().clamp_(min=0); d.flags[pi] &= 0xFB
            if i >= 8:
                d.flags[fifo[i % 8]] |= 4
            fifo[i % 8].copy_(pi)
            cap.synchronize()
    R = np.stack(rows)
    rel = (R - R[:, 0:1]) / 1000.0
    line = {"workload": "phase stamps: metadata-scale call replayed from a CUDA graph", "calls": calls,
            "event_timed_us_median": float(np.median(timed)), "fast_hits": c.counters()["fast_hits"], "phases_us_median": []}
    for base, who in ((0, ""), (8, " [victims]"), (16, " [prefetch]"), (24, " [victims]"), (32, " [prefetch]"), (40, " [victims]"),
                      (48, " [prefetch]"), (56, "")):
        for k in range(8):
            name = PHASE_NAMES.get((base - 8 if base in (16, 32, 48) else base) + k)
            if name is None or R[0, base + k] == 0:
                continue
            line["phases_us_median"].append([round(float(np.median(rel[:, base + k])), 2), name + who])
    line["phases_us_median"].sort()
    print(json.dumps(line))


def profile_case(args, torch, device):
    """Small cases for profiler captures (a few GB on the device, inputs larger than L2).
    mover : 2,048-block GPU pool (4 GiB), 512-slot pinned host tier (1 GiB); per step one
            device-to-device move of 512 scattered blocks, one offload and one prefetch of 256, and
            one fused two-way transfer of 170 blocks out and 256 in.
    select: metadata-scale index (1,000,000 entries, 256 agents); per step observe 64 events,
            select 10,000 victims and 2,000 prefetch candidates (multi-launch select path).
    select80k: the 80,000-entry index of the Llama-8B configuration, 256 victims / 384 prefetch
            candidates (single-launch cluster select path), then the step's three selects as one launch."""
    from paper_2608_14624_b200 import binding as cs
    from paper_2608_14624_b200 import build
    from tests import synth
    if args.phase_stamps:
        return phase_timeline(args, torch, device)
    build.build_library()
    if args.workload in ("select16m", "select64m"):
        # one kind of select over an index far larger than L2 (176 MB / 704 MB of metadata): the regime in which the
        # scans are bound by memory or instruction issue; the first call has no remembered threshold, the rest do
        cfg = synth.CONFIGS["meta1m"]
        N = 16_000_000 if args.workload == "select16m" else 64_000_000
        d = cs.DeviceIndex.from_host(synth.make_block_index(cfg, n=N, tier="random"), device)
        tr = synth.make_trace(cfg, n_invocations=4000)
        c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=N,
                                         block_tokens=cfg.block_tokens, r_min=0.02), device)
        c.observe_invocations(torch.from_numpy(tr.chain).to(device), torch.from_numpy(tr.agent).to(device), None)
        v = torch.empty(cfg.k_victims, dtype=torch.int32, device=device)
        vn = torch.zeros(4, dtype=torch.int32, device=device)
        for s in range(max(1, args.steps)):
            c.select_victims(d, 100_000, 0, cfg.k_victims, v, vn)
        torch.cuda.synchronize(device)
        print(json.dumps({"workload": args.workload, "launches": c.launch_count(), "counters": c.counters(),
                          "device_status": c.get_status()}))
        return
    if args.workload == "mover":
        cfg = synth.CONFIGS["llama8b"]
        G, Hs, L, bb = 2048, 512, cfg.n_layers, cfg.block_bytes
        c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, max_blocks=64), device)
        gpu = cs.KVPool(torch.randint(0, 255, (G * bb,), dtype=torch.uint8, device=device), G, cs.CS_LAYER_MAJOR, L)
        host = cs.KVPool(torch.empty(Hs * bb, dtype=torch.uint8, pin_memory=True), Hs, cs.CS_BLOCK_MAJOR, L)
        rng = synth.rng_for(cfg, 11)
        up = lambda a: torch.from_numpy(a.view(np.int32)).to(device)
        src, _ = synth.mover_batch(512, G - 512, 512, rng)
        d_src, d_back = up(src), torch.arange(G - 512, G, dtype=torch.int32, device=device)
        hs, hd = synth.mover_batch(256, G, Hs, rng)
        d_hs, d_hd = up(hs), up(hd)
        h_perm = rng.permutation(Hs).astype(np.uint32)
        x_off_src, x_off_dst = up(src[:170].copy()), up(h_perm[:170].copy())
        x_pre_src, x_pre_dst = up(h_perm[170:426].copy()), torch.arange(G - 512, G - 256, dtype=torch.int32, device=device)
        if args.offload_width or args.prefetch_width:
            c.set_mover_ctas(max(args.offload_width, args.prefetch_width), 0)
        for _ in range(max(1, args.steps)):
            c.compact_blocks(gpu, gpu, d_src, d_back)
            c.offload_blocks(gpu, host, d_hs, d_hd)
            c.prefetch_blocks(host, gpu, d_hd, d_hs)
            c.exchange_blocks(gpu, host, x_off_src, x_off_dst, x_pre_src, x_pre_dst)
    else:
        big = args.workload == "select"
        cfg = synth.CONFIGS["meta1m" if big else "llama8b"]
        N = 1_000_000 if big else cfg.n_index
        d = cs.DeviceIndex.from_host(synth.make_block_index(cfg, n=N, tier="random" if big else "range"), device)
        tr = synth.make_trace(cfg, n_invocations=64 * (args.steps + 40))
        c = cs.CacheScout(cs.make_params(n_agents=cfg.n_agents, n_chains=cfg.n_chains, max_blocks=N,
                                         block_tokens=cfg.block_tokens, r_min=0.02), device)
        ch, ag = torch.from_numpy(tr.chain).to(device), torch.from_numpy(tr.agent).to(device)
        c.observe_invocations(ch[:64 * 30], ag[:64 * 30], None)
        v = torch.empty(cfg.k_victims, dtype=torch.int32, device=device)
        pf = torch.empty(cfg.k_prefetch, dtype=torch.int32, device=device)
        vn, pn = torch.zeros(4, dtype=torch.int32, device=device), torch.zeros(4, dtype=torch.int32, device=device)
        hv = torch.empty(cfg.k_victims, dtype=torch.int32, device=device)
        hn = torch.zeros(4, dtype=torch.int32, device=device)
        def one(s):
            lo = 64 * (30 + s)
            c.observe_invocations(ch[lo:lo + 64], ag[lo:lo + 64], None)
            c.select_victims(d, 100_000 + s, 0, cfg.k_victims, v, vn)
            c.select_prefetch(d, 100_000 + s, cfg.k_prefetch, pf, pn)
            if not big:        # the step's three selects as one launch
                c.select_step(d, 100_000 + s, cfg.k_victims, cfg.k_prefetch, v, vn, hv, hn, pf, pn)

        n_steps = max(1, args.steps)
        if args.kineto:        # warm device times per kernel (L2-resident index, no serialisation), first 5 steps untimed
            from torch.profiler import ProfilerActivity, profile
            for s in range(min(5, n_steps)):
                one(s)
            torch.cuda.synchronize(device)
            with profile(activities=[ProfilerActivity.CUDA]) as prof:
                for s in range(min(5, n_steps), n_steps):
                    one(s)
                torch.cuda.synchronize(device)
            # All launches of this workload are on one stream.  A kernel launched with programmatic dependent launch starts
            # early and waits for its predecessor, so its own time is taken from the end of the kernel before it.
            evs = sorted((e for e in prof.events() if e.device_type == torch.autograd.DeviceType.CUDA and "cs_" in e.name),
                         key=lambda e: e.time_range.start)
            per, prev_end = {}, 0
            for e in evs:
                own = e.time_range.end - max(e.time_range.start, prev_end)
                prev_end = max(prev_end, e.time_range.end)
                per.setdefault(e.name.split("(")[0], []).append(own)
            calls = n_steps - min(5, n_steps)
            print(json.dumps({"kernel_us_median_warm": {k: round(float(np.median(x)), 2) for k, x in per.items()},
                              "launches_per_call": {k: len(x) / calls for k, x in per.items()},
                              "us_of_kernel_time_per_call": round(sum(float(np.sum(x)) for x in per.values()) / calls, 1),
                              "note": "own time of each kernel: from the end of the kernel before it on the stream (or its own start) to its end"}))
        else:
            for s in range(n_steps):
                one(s)
    torch.cuda.synchronize(device)
    print(json.dumps({"workload": args.workload, "launches": c.launch_count(), "device_status": c.get_status()}))


WORKLOAD_TEXT = {
    "tiny": "tiny step (BASELINE.json configs[0]): 8 layers x 8 KV heads x 128 bf16, 512 KiB blocks",
    "llama8b": "llama8b-kv step (BASELINE.json configs[1]): 32 layers x 8 KV heads x 128 bf16, 2 MiB blocks",
    "llama70b": "llama70b-kv step (BASELINE.json configs[3]): 80 layers x 8 KV heads x 128 bf16, 5 MiB blocks",
}


def oracle_baseline(cfg_name, budget_s):
    """The oracle as it stands, timed on this machine's host cores for about budget_s seconds of steps."""
    ow = OracleStep(cfg_name)
    ow.step(0)
    t0 = time.perf_counter()
    n_or = 0
    while time.perf_counter() - t0 < budget_s and n_or < 40:
        ow.step(1 + n_or)
        n_or += 1
    dt = time.perf_counter() - t0
    return {"value": ow.bytes_per_step * n_or / dt / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": "%d oracle steps: %s" % (n_or, ow.sample),
            "blocks_scored_selected_per_s": 3 * ow.idx.n * n_or / dt, "ms_per_step": dt / n_or * 1e3}


def measure_step_workload(args, w, ctx):
    """Warm-up, K timed steps with device-resident inputs (the headline value), K steps end to end, and the
    per-kernel figures of the step; returns the JSON object of this workload (rank 0's view)."""
    torch, world, rank, device = ctx["torch"], ctx["world"], ctx["rank"], ctx["device"]
    barrier, link, hbm_peak, peak_kind = ctx["barrier"], ctx["link"], ctx["hbm_peak"], ctx["peak_kind"]
    for s in range(args.warmup):
        w.step(s)
    w.drain()
    barrier()
    sampler = ClockSampler(ctx["local"])
    if rank == 0:
        sampler.start()
    l0 = w.c.launch_count()
    w.take_moved_bytes()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(w.main)
    for s in range(args.steps):
        w.step(args.warmup + s, timed=True)
    w.drain()
    e1.record(w.main)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    launches = w.c.launch_count() - l0
    moved_bytes = w.take_moved_bytes()                 # what the timed steps really moved (this rank)
    counters = w.last_counters
    total_ms = reduce_max_ms(e0.elapsed_time(e1), world, device)
    w.collect_timers()
    status = w.c.get_status()
    last = (args.warmup + args.steps - 1) % w.RING
    n_out = [int(w.vn[last][0].item()), int(w.hn[last][0].item()), int(w.pn[last][0].item())]
    if args.skip_aux:
        return {"workload": "step", "config": w.cfg_name, "ms_per_step": total_ms / args.steps, "gpu_launches": int(launches),
                "value": job_value(world, moved_bytes / args.steps, args.steps, total_ms), "n_out": n_out}

    # ---- end to end: inputs from pinned host memory, results read back, every step ---------------------------
    base = args.warmup + args.steps
    for s in range(2):
        w.step(base + s, e2e=True)
    w.drain()
    barrier()
    w.take_moved_bytes()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(w.main)
    for s in range(args.steps):
        w.step(base + 2 + s, e2e=True)
    w.drain()
    f1.record(w.main)
    barrier()
    e2e_ms = reduce_max_ms(f0.elapsed_time(f1), world, device)
    e2e_moved = w.take_moved_bytes()
    w._pending = []
    if rank != 0:
        return {}

    cfg = w.cfg
    value = job_value(world, moved_bytes / args.steps, args.steps, total_ms)
    e2e_value = job_value(world, e2e_moved / args.steps, args.steps, e2e_ms)
    bb = cfg.block_bytes
    med = lambda k: float(np.median(w.timers[k])) if w.timers[k] else None
    t_c, t_o, t_p, t_s, t_ob = med("compact"), med("offload"), med("prefetch"), med("select"), med("observe")
    d2d_gbps = 2 * w.k_v * bb / (t_c / 1e3) / 1e9
    off_gbps = w.k_v * bb / (t_o / 1e3) / 1e9
    pre_gbps = w.k_p * bb / (t_p / 1e3) / 1e9
    sel_bytes = 3 * w.N * 11 + (2 * w.k_v + w.k_p) * 4
    h2d, d2h = w.e2e_bytes()
    traffic, traffic_x = None, None
    tpath = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if os.path.exists(tpath) and w.cfg_name == "llama8b":
        with open(tpath) as f:
            tj = json.load(f)
        traffic = tj.get("cs_mover_kernel_d2d_256_blocks_bytes")
        traffic_x = tj.get("cs_exchange_bulk_kernel_256_out_384_in_dram_bytes")
    # the two-way transfer: bytes of one launch over its duration on the side stream, against what the link gives two
    # concurrent pinned cudaMemcpyAsync copies in the same out:in proportion, measured in this run
    x_ms = t_o if w.fused else max(t_o, t_p)
    x_bytes = moved_bytes / args.steps                   # what a launch really moved (the nominal 256 + 384 blocks at full size)
    x_gbps = x_bytes / (x_ms / 1e3) / 1e9
    # time a perfect duplex link would need for the step's bytes, from the one-direction peaks of this run
    ideal_ms = max(w.k_v * bb / link["d2h"], w.k_p * bb / link["h2d"]) / 1e6
    ideal_ms *= x_bytes / float((w.k_v + w.k_p) * bb)    # a launch that found fewer eligible blocks moved fewer bytes
    named, backed = cfg.host_blocks, w.host_backed
    return {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u8", "data": "synthetic",
        "config": {"workload": "%s; GPU pool %d blocks layer-major, host tier %d blocks; %d agents; per step: observe <= 8 invocations, "
                               "select %d GPU victims + %d host victims + %d prefetch candidates over %d entries, compact %d, "
                               "offload %d, prefetch %d blocks" % (WORKLOAD_TEXT[w.cfg_name], cfg.gpu_blocks, named, cfg.n_agents,
                                                                  w.k_v, w.k_v, w.k_p, w.N, w.k_v, w.k_v, w.k_p),
                   "host_tier": {"named_slots": named, "backed_slots": backed, "reduction": round(1.0 - backed / named, 4),
                                 "why": "all named slots are pinned" if backed == named else
                                        "pinned memory limited to %.2f of the box's available memory" % args.host_frac,
                                 "pin_attempts": w.pin_attempts, "pinned_by": w.pinned.how,
                                 "pinned_GiB": round(backed * bb / GIB, 1), "pin_seconds": round(w.t_pin, 2)},
                   "l2_policy": "inputs larger than L2: every step moves %.2f GiB of scattered blocks; the %.1f MB index is L2-resident by design"
                                % ((2 * w.k_v + w.k_p) * bb / GIB, w.N * 11 / 1e6),
                   "replicas": "replicas only (no data-path collective)", "quick": bool(args.quick)},
        "blocks_moved_in_timed_steps": {"counted_by_the_mover_kernels": [counters["blocks_moved"][1], counters["blocks_moved"][2]],
                                        "skipped_list_entries": counters["blocks_skipped"],
                                        "nominal": args.steps * (w.k_v + w.k_p)},
        "blocks_scored_selected_per_s": world * 3 * w.N / (t_s / 1e3),
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"kernel": ("cs_exchange_bulk_kernel: offload %d + prefetch %d blocks as one launch on the side stream (98 %% of the step's device time)"
                                % (w.k_v, w.k_p)) if w.fused else "cs_mover_bulk_kernel: offload and prefetch launches on two side streams",
                     "bound": "host_link", "achieved": x_gbps, "peak": link["bidir_step_mix"], "unit": "GB/s",
                     "frac": x_gbps / link["bidir_step_mix"], "traffic": traffic_x,
                     "peak_kind": "measured in this run: two concurrent pinned cudaMemcpyAsync copies of contiguous buffers in the step's "
                                  "2:3 out:in proportion (PCIe Gen5 x16 is neither HBM nor a tensor pipe)",
                     "peak_per_direction": {"d2h": link["d2h"], "h2d": link["h2d"], "both_1to1": link["bidir"]},
                     "ideal_duplex_ms": ideal_ms, "frac_of_ideal_duplex": ideal_ms / x_ms,
                     "algorithmic_bytes_per_launch": x_bytes, "ms_per_launch": x_ms,
                     "traffic_note": "DRAM bytes of one launch (ncu, profiles/): each block crosses HBM once"},
        "roofline_hbm": {"kernel": "cs_mover_bulk_kernel (device-to-device compaction of the %d victims, inside the step, while the host-link "
                                   "transfer of the previous step runs beside it)" % w.k_v, "bound": "hbm",
                         "achieved": d2d_gbps, "peak": hbm_peak, "unit": "GB/s", "frac": d2d_gbps / hbm_peak, "traffic": traffic,
                         "peak_kind": "of %s" % peak_kind, "algorithmic_bytes_per_launch": 2 * w.k_v * bb, "ms_per_launch": t_c},
        "host_link": {"peak_d2h_GBps": link["d2h"], "peak_h2d_GBps": link["h2d"], "peak_bidir_GBps": link["bidir"],
                      "peak_bidir_step_mix_GBps": link["bidir_step_mix"],
                      "how": "pinned cudaMemcpyAsync of 1 GiB, best of 10, same run; step_mix = 2/3 GiB out while 1 GiB comes in, "
                             "the proportions of a step, whose inbound direction is the longer one",
                      "offload_GBps": off_gbps, "offload_frac": off_gbps / link["d2h"], "offload_ms": t_o,
                      "prefetch_GBps": pre_gbps, "prefetch_frac": pre_gbps / link["h2d"], "prefetch_ms": t_p,
                      "step_frac_of_bidir": value / world / link["bidir"],
                      "step_frac_of_bidir_step_mix": value / world / link["bidir_step_mix"],
                      "transfers": args.transfers,
                      "note": ("offload and prefetch of a step run as one fused launch (cs_exchange_blocks): both per-direction times "
                               "are that launch's duration" if w.fused else
                               "offload and prefetch of a step overlap (full duplex); per-direction times are measured while the other direction is busy")},
        "select": {"how": "cs_select_step: one launch of three 16-CTA clusters" if w.fused_selects else "three calls", "ms_three_selects": t_s, "ms_observe": t_ob, "algorithmic_bytes": sel_bytes,
                   "achieved_GBps": sel_bytes / (t_s / 1e3) / 1e9, "frac_of_hbm_peak": sel_bytes / (t_s / 1e3) / 1e9 / hbm_peak,
                   "n_out_last_step": n_out, "device_status": status},
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / args.steps,
                "includes": "per step: H2D of the step's events and of the whole index from pinned memory, D2H of the three id lists and counts, host sync on the result"},
    }


def reduce_max_ms(local_ms: float, world: int, device) -> float:
    """Job time = the slowest rank's device time (all-reduce MAX; identity for one rank)."""
    if world <= 1:
        return float(local_ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world: int, bytes_per_step_per_rank: int, steps: int, job_ms: float) -> float:
    """Whole-job GB/s of independent replicas: every rank moves the same bytes per step."""
    return world * bytes_per_step_per_rank * steps / (job_ms / 1e3) / 1e9


# ---- main ------------------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    hbm_peak, peak_kind = measured_peaks()
    if args.workload != "step":          # one small case of one kernel family, for profiler captures
        profile_case(args, torch, device)
        return
    link = host_link_peak(torch, device) if (rank == 0 and not args.skip_aux) else None
    w = StepWorkload(args, device, world, args.config)
    cs, synth = w.cs, w.synth
    ctx = dict(world=world, rank=rank, local=local, device=device, barrier=barrier, link=link, hbm_peak=hbm_peak,
               peak_kind=peak_kind, torch=torch)
    out = measure_step_workload(args, w, ctx)
    if args.skip_aux:
        if rank == 0:
            print(json.dumps(out))
        if world > 1:
            dist.destroy_process_group()
        return
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    if not args.no_extras and world == 1:
        out["fused_step"] = fused_step_section(w)
        out["mover_sweep"] = mover_sweep(w, hbm_peak, link)
        w.release()
        del w
        other = "llama70b" if args.config == "llama8b" else "llama8b"
        w2 = StepWorkload(args, device, world, other)
        sub = measure_step_workload(args, w2, ctx)
        sub["cpu_baseline"] = oracle_baseline(other, budget_s=8.0)
        out["second_config"] = sub
        w2.release()
        del w2
        w0 = StepWorkload(args, device, world, "tiny")          # configs[0]: 512-block pool, 2,048-slot host tier, k = 32 / 64
        sub0 = measure_step_workload(args, w0, ctx)
        out["tiny_config"] = {k: sub0[k] for k in ("value", "ms_per_step", "config", "roofline", "roofline_hbm", "e2e", "select",
                                                    "blocks_moved_in_timed_steps", "gpu_launches")}
        w0.release()
        del w0
        out["metadata_scale"] = metadata_scale(torch, cs, synth, device, hbm_peak, calls=args.meta_calls)
        out["exact_survival"] = exact_survival_section(torch, cs, synth, device)
        out["hbm_regime"] = hbm_regime_section(torch, cs, synth, device, hbm_peak)
    out["cpu_baseline"] = oracle_baseline(args.config, budget_s=10.0)     # the oracle, as it stands, on this machine's host cores
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
