#!/usr/bin/env python
"""Benchmark of the GAC hot path (stats + projection + state refresh).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole path over one synthetic gradient list:
gac_stats (fused <g,d>, <g,g>, <d,d>, cosine, regime, gains) followed by
gac_project (in-place rank-one update, stored direction refreshed), in the
projection regime -- the regime that moves the most bytes.

Timing: CUDA events on the launching stream around the two calls of every
step, summed over the K timed steps; between steps a FRESH gradient with the
configured cosine to the stored direction is written into g (as the backward
pass of a training loop would), outside the timed events; that write also
evicts the 126 MB L2.  Prints one JSON line.

--gpus N > 1 without a launcher's environment starts N ranks by itself (one
process per GPU, NCCL, a free port on 127.0.0.1); under an external launcher
(RANK / WORLD_SIZE / LOCAL_RANK set) it is one of those ranks.
"""
from __future__ import annotations

import argparse
import ctypes
import hashlib
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2603_01501_b200 import synth  # noqa: E402

METRIC = "GAC stats+projection params/s"
UNIT = "params/s"
FORCE = dict(c_low=0.05, c_high=2.0)   # legal thresholds that keep every step in the projection regime
NOMINAL_HBM_GBS = 8000.0


# ----------------------------------------------------------------- utilities

def measured_hbm_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def bytes_per_param(g_dtype, d_dtype=torch.float32) -> int:
    sg = 2 if g_dtype == torch.bfloat16 else 4
    sd = 2 if d_dtype == torch.bfloat16 else 4
    return sg + sd


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the
    timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4)}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def nvml_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def recorded_traffic(kernel: str):
    """DRAM bytes per parameter of `kernel` from the committed ncu capture, or
    None when the kernel source changed since the capture."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as fh:
            rec = json.load(fh)
        src = os.path.join(ROOT, "paper_2603_01501_b200", "csrc", "gac_kernels.cuh")
        if hashlib.sha256(open(src, "rb").read()).hexdigest() != rec["source_sha256"]:
            return None
        return rec["kernels"][kernel]
    except Exception:
        return None


def reserve_stdout():
    """Keeps the process's stdout for the one JSON line: returns a file on a duplicate of it and
    points descriptor 1 at stderr, so that what libraries print on stdout (NCCL prints its version
    there) still appears, but not in front of the line."""
    sys.stdout.flush()
    line_out = os.fdopen(os.dup(1), "w")
    os.dup2(2, 1)
    return line_out


# ------------------------------------------------------------------ launcher

def free_port() -> int:
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def rank_environment(n: int, rank: int, port: int, base=None) -> dict:
    """Environment of rank `rank` of an n-rank single-node job, as torch.distributed's
    env:// rendezvous reads it.  Everything else is inherited (NCCL settings included)."""
    env = dict(os.environ if base is None else base)
    env.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(n),
                "LOCAL_WORLD_SIZE": str(n), "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    return env


def spawn_ranks(n: int, argv, worker=None, stdout=None) -> int:
    """Starts n copies of this script (or of `worker`, a command prefix), one per GPU, and waits.
    Rank 0 prints the JSON line on the inherited stdout.  If a rank fails the others are
    terminated and its exit code is returned."""
    worker = worker or [sys.executable, os.path.abspath(__file__)]
    port = free_port()
    procs = [subprocess.Popen(list(worker) + list(argv), env=rank_environment(n, r, port), stdout=stdout)
             for r in range(n)]
    rc = 0
    pending = set(range(n))
    while pending:
        for r in sorted(pending):
            code = procs[r].poll()
            if code is None:
                continue
            pending.discard(r)
            if code != 0 and rc == 0:
                rc = code
                for q in pending:
                    procs[q].terminate()
        time.sleep(0.05)
    return rc


# --------------------------------------------------------------- GPU workload

class Workload:
    def __init__(self, name: str, device, world: int, clip: float = 0.0, sharded: bool = False,
                 peer_exchange: bool = False):
        from paper_2603_01501_b200 import binding as gb
        from paper_2603_01501_b200 import sharding
        self.gb, self.sharding = gb, sharding
        dims_key, self.g_dtype, self.rho, self.config_id = synth.WORKLOADS[name]
        self.name, self.device, self.world = name, device, world
        self.shapes = synth.decoder_tensor_list(synth.DIMS[dims_key])
        self.params = synth.list_numel(self.shapes)
        self.sigma = synth.per_tensor_scales(self.config_id, len(self.shapes))
        self.g, self.d = synth.gradient_list(self.shapes, self.rho, self.config_id, self.g_dtype, device)
        self.d_dtype = synth.WORKLOAD_D_DTYPE.get(name, torch.float32)
        if self.d_dtype != torch.float32:
            self.d = [t.to(self.d_dtype) for t in self.d]
        self.scratch = torch.empty(max(n for _, n in self.shapes), dtype=torch.float32, device=device)
        self.gen = torch.Generator(device=device)
        self.gen.manual_seed(12345 + self.config_id)
        self.ctx = gb.gac_init(self.g, self.d, gb.HParams(clip_max_norm=clip, **FORCE))
        self.step_no = 1      # the stored direction already holds g_{t-1}
        self.sharded = sharded or world > 1     # local sums -> all-reduce -> decision (App. A.1)
        self.sums = torch.zeros(3, dtype=torch.float64, device=device) if self.sharded else None
        self.peer_exchange = bool(peer_exchange and self.sharded)
        if self.peer_exchange:      # the kernels exchange the three sums themselves instead of NCCL
            self.sharding.attach_peer_exchange(gb, self.ctx)

    def refresh(self):
        synth.refresh_gradient_list(self.g, self.d, self.sigma, self.rho, self.gen, self.scratch)

    def step(self, ev=None):
        """stats + project on the current stream; ev = three CUDA events or None."""
        gb = self.gb
        self.step_no += 1
        if ev:
            ev[0].record()
        if self.sharded:
            # sharded form (App. A.1): local sums, ONE all-reduce of three numbers, same decision on every rank
            self.sharding.sharded_step(gb, self.ctx, self.step_no, self.sums,
                                       mark=(ev[1].record if ev else None), peer_exchange=self.peer_exchange)
        else:
            gb.gac_stats(self.ctx, self.step_no, fetch=False)
            if ev:
                ev[1].record()
            gb.gac_project(self.ctx)
        if ev:
            ev[2].record()

    def close(self):
        self.gb.gac_free(self.ctx)
        self.ctx = None
        self.g = self.d = self.scratch = None
        torch.cuda.empty_cache()


def time_steps(wl: Workload, steps: int, warmup: int, sampler=None):
    """Returns (stats_ms list, project_ms list) of the timed steps."""
    for _ in range(warmup):
        wl.refresh()
        wl.step()
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    if wl.world > 1:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    ctxmgr = sampler if sampler is not None else _Null()
    with ctxmgr:
        for i in range(steps):
            wl.refresh()
            wl.step(evs[i])
        torch.cuda.synchronize()
    if wl.world > 1:
        torch.distributed.barrier()
    s_ms = [e[0].elapsed_time(e[1]) for e in evs]
    p_ms = [e[1].elapsed_time(e[2]) for e in evs]
    return s_ms, p_ms


def time_unchanged_regime(wl: Workload, steps: int):
    """The same list under the paper's default thresholds (0.05, 0.3): every
    configured cosine is above c_high, so these are violation steps -- the
    reduction plus the state refresh d' = g with g left alone (a safe step moves
    the same bytes)."""
    gb = wl.gb
    ctx = gb.gac_init(wl.g, wl.d, gb.HParams())
    step_no = 1
    evs = []
    for i in range(3 + steps):
        wl.refresh()
        step_no += 1
        e = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        e[0].record()
        gb.gac_stats(ctx, step_no, fetch=False)
        gb.gac_project(ctx)
        e[1].record()
        if i >= 3:
            evs.append(e)
    res = gb.gac_stats(ctx, step_no + 1)
    gb.gac_project(ctx)
    torch.cuda.synchronize()
    gb.gac_free(ctx)
    ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
    bpp = 2 * bytes_per_param(wl.g_dtype, wl.d_dtype)
    nbytes = wl.params * bpp
    return {"regime": gb.REGIME_NAMES[res.regime], "ms_per_step": ms,
            "value": wl.params / (ms * 1e-3), "unit": UNIT, "bytes_per_param": bpp,
            "hbm_gbs": nbytes / (ms * 1e-3) / 1e9}


def time_exchange_mode(wl: Workload, steps: int):
    """The same list in exchange mode (g and d of one element type): the stored
    direction is refreshed by swapping the roles of the two buffer sets, so a
    projection step reads g and d and writes g' once -- (sg+sd) + (sg+sd+sg)
    bytes per parameter -- and a step that leaves g alone moves only the (sg+sd)
    of the reduction.  Every step's gradient is written into the set that is free."""
    gb = wl.gb
    if wl.g_dtype != wl.d_dtype:
        return {"skipped": "exchange mode needs g and d of one element type"}
    sets = [wl.g, wl.d]
    sg = 2 if wl.g_dtype == torch.bfloat16 else 4
    out = {}
    for label, thr in (("project", FORCE), ("unchanged", {})):
        ctx = gb.gac_init(sets[0], sets[1], gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, **thr))
        step_no, evs = 1, []
        for i in range(3 + steps):
            gi = gb.gac_next_gradient_set(ctx)
            synth.refresh_gradient_list(sets[gi], sets[gi ^ 1], wl.sigma, wl.rho, wl.gen, wl.scratch)
            step_no += 1
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record()
            gb.gac_stats(ctx, step_no, fetch=False)
            e[1].record()
            gb.gac_project(ctx)
            e[2].record()
            if i >= 3:
                evs.append(e)
        gi = gb.gac_next_gradient_set(ctx)
        synth.refresh_gradient_list(sets[gi], sets[gi ^ 1], wl.sigma, wl.rho, wl.gen, wl.scratch)
        res = gb.gac_stats(ctx, step_no + 1)
        gb.gac_project(ctx)
        torch.cuda.synchronize()
        gb.gac_free(ctx)
        s_ms = sum(a.elapsed_time(b) for a, b, _ in evs) / len(evs)
        p_ms = sum(b.elapsed_time(c) for _, b, c in evs) / len(evs)
        proj_bpp = 3 * sg if label == "project" else 0
        roof = None
        if proj_bpp:
            peak, kind = measured_hbm_peak()
            tr = recorded_traffic("gac_project_kernel_exchange")
            key = "f32" if sg == 4 else "bf16_dbf16"
            gbs = wl.params * proj_bpp / (p_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "kernel": "gac_project_kernel (exchange)", "achieved": gbs, "peak": peak,
                    "unit": "GB/s", "frac": gbs / peak, "peak_kind": f"of {kind}",
                    "algorithmic_bytes_per_launch": wl.params * proj_bpp,
                    "traffic": (tr[key] * wl.params if tr and key in tr else None)}
        out[label] = {"roofline": roof,"regime": gb.REGIME_NAMES[res.regime], "cos": res.cos, "ms_per_step": s_ms + p_ms,
                      "stats_ms": s_ms, "project_ms": p_ms, "value": wl.params / ((s_ms + p_ms) * 1e-3),
                      "unit": UNIT, "bytes_per_param": 2 * sg + proj_bpp,
                      "hbm_gbs": wl.params * (2 * sg + proj_bpp) / ((s_ms + p_ms) * 1e-3) / 1e9,
                      "project_kernel_gbs": (wl.params * proj_bpp / (p_ms * 1e-3) / 1e9) if proj_bpp else None}
    # leave the workload as it was found: wl.g holds a gradient, wl.d its stored direction
    synth.refresh_gradient_list(wl.g, wl.d, wl.sigma, wl.rho, wl.gen, wl.scratch)
    return out


def time_fused_adamw(wl: Workload, steps: int, exchange: bool = False, peak=None, peak_kind="measured"):
    """stats + the projection fused with AdamW (Table 2 values): the update goes
    straight into p, m, v and g' is never written.  Moves (sg+sd) + (sg+sd+12) read
    + (sd+12) written bytes per parameter; in exchange mode the stored direction
    is not written either (12 written)."""
    gb = wl.gb
    if exchange and wl.g_dtype != wl.d_dtype:
        return {"skipped": "exchange mode needs g and d of one element type"}
    free, _ = torch.cuda.mem_get_info()
    need = wl.params * 12 + (2 << 30)
    if free < need:
        return {"skipped": f"needs {need} bytes of device memory for p, m, v; {free} free"}
    p = [torch.randn(t.numel(), device=wl.device) * 0.02 for t in wl.g]
    m = [torch.zeros(t.numel(), device=wl.device) for t in wl.g]
    v = [torch.zeros(t.numel(), device=wl.device) for t in wl.g]
    sets = [wl.g, wl.d]
    mode = gb.GAC_STATE_EXCHANGE if exchange else gb.GAC_STATE_RAW
    ctx = gb.gac_init(wl.g, wl.d, gb.HParams(state_mode=mode, **FORCE))
    gb.gac_attach_adamw(ctx, p, m, v, 0)
    opt = gb.AdamW()
    step_no, evs = 1, []
    for i in range(3 + steps + 1):
        gi = gb.gac_next_gradient_set(ctx)          # always the g buffers outside exchange mode
        synth.refresh_gradient_list(sets[gi], sets[gi ^ 1], wl.sigma, wl.rho, wl.gen, wl.scratch)
        if i == 3 + steps:
            break
        step_no += 1
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        gb.gac_stats(ctx, step_no, fetch=False)
        e[1].record()
        gb.gac_project_adamw(ctx, opt)
        e[2].record()
        if i >= 3:
            evs.append(e)
    torch.cuda.synchronize()
    gb.gac_stats(ctx, step_no + 1, fetch=False)
    res = gb.gac_project_adamw(ctx, opt, fetch=True)
    # leave the workload usable by the legs that follow: wl.g a gradient against wl.d
    synth.refresh_gradient_list(wl.g, wl.d, wl.sigma, wl.rho, wl.gen, wl.scratch)
    torch.cuda.synchronize()
    gb.gac_free(ctx)
    s_ms = sum(a.elapsed_time(b) for a, b, _ in evs) / len(evs)
    f_ms = sum(b.elapsed_time(c) for _, b, c in evs) / len(evs)
    sg = 2 if wl.g_dtype == torch.bfloat16 else 4
    sd = 2 if wl.d_dtype == torch.bfloat16 else 4
    bpp = (sg + sd + 12) + (12 if exchange else sd + 12)
    fused_bytes = wl.params * bpp
    del p, m, v
    torch.cuda.empty_cache()
    gbs = fused_bytes / (f_ms * 1e-3) / 1e9
    if peak is None:
        peak, peak_kind = measured_hbm_peak()
    tr = recorded_traffic("gac_adamw_kernel_exchange" if exchange else "gac_adamw_kernel")
    key = dtype_name(wl.g_dtype) + ("_dbf16" if wl.d_dtype != torch.float32 else "")
    return {"ms_per_step": s_ms + f_ms, "stats_ms": s_ms, "fused_ms": f_ms, "steps": len(evs),
            "value": wl.params / ((s_ms + f_ms) * 1e-3), "unit": UNIT,
            "fused_bytes_per_param": bpp,
            "fused_kernel_gbs": gbs,
            "roofline": {"bound": "hbm", "kernel": "gac_adamw_kernel" + (" (exchange)" if exchange else ""),
                         "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                         "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": fused_bytes,
                         "traffic": (tr[key] * wl.params if tr and key in tr else None)},
            "applied_steps": res.applied_steps, "regime": gb.REGIME_NAMES[res.regime]}


class _Null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def check_regime(wl: Workload):
    """One extra (untimed) step that fetches the decision: the timed steps must
    have been projection steps with the configured cosine."""
    wl.refresh()
    gb = wl.gb
    wl.step_no += 1
    if wl.sharded:
        res = wl.sharding.sharded_step(gb, wl.ctx, wl.step_no, wl.sums, fetch=True, peer_exchange=wl.peer_exchange)
    else:
        res = gb.gac_stats(wl.ctx, wl.step_no)
        gb.gac_project(wl.ctx)
    torch.cuda.synchronize()
    return res


def e2e_fits_host(wl: Workload) -> bool:
    """Every rank of the node pins its own host copy of the gradient list: do not
    take more than half of the host's available memory."""
    need = sum(t.numel() * t.element_size() for t in wl.g) * max(1, wl.world)
    try:
        import psutil
        return need <= 0.5 * psutil.virtual_memory().available
    except Exception:
        return True


def time_e2e(wl: Workload, steps: int, warmup: int):
    """Same step through the C ABI with HOST buffers: every step copies the
    gradient list from pinned host memory to the device, runs stats + project,
    and copies the updated gradient list and the decision record back.  Wall
    clock around the whole step, device idle on both sides."""
    gb = wl.gb
    pinned = True
    try:
        host_g = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in wl.g]
    except RuntimeError:
        pinned = False
        host_g = [torch.empty(t.shape, dtype=t.dtype) for t in wl.g]
    h2d = sum(h.numel() * h.element_size() for h in host_g)
    d2h = h2d + ctypes.sizeof(gb.gac_result)      # g' and the decision record
    times = []
    for i in range(warmup + steps):
        wl.refresh()                       # next gradient, staged on the host (untimed)
        for h, t in zip(host_g, wl.g):
            h.copy_(t)
            t.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for h, t in zip(host_g, wl.g):
            t.copy_(h, non_blocking=True)
        wl.step_no += 1
        gb.gac_stats(wl.ctx, wl.step_no, fetch=False)
        gb.gac_project(wl.ctx, fetch=True)          # reads the decision record back
        for h, t in zip(host_g, wl.g):
            h.copy_(t, non_blocking=True)
        torch.cuda.synchronize()
        if i >= warmup:
            times.append((time.perf_counter() - t0) * 1e3)
    ms = sum(times) / len(times)
    return {"value": wl.params * wl.world / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms,
            "steps": steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "pinned": pinned}


# ------------------------------------------------------------- CPU baseline

# Both arms time the oracle on the SAME bounded samples of the workload, so their figures agree:
# all host cores on the first ALL_CORE_SAMPLE parameters after the embedding (the per-layer mix of
# small and large tensors), one thread on the first ONE_THREAD_SAMPLE of those.
ALL_CORE_SAMPLE = 1_000_000_000
ONE_THREAD_SAMPLE = 64_000_000


def host_cores() -> int:
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


def oracle_sample(name: str, target_elems: int):
    """A prefix of the workload's tensor list (whole tensors, the last one cut),
    generated on the CPU with the list's recipe."""
    dims_key, g_dtype, rho, config_id = synth.WORKLOADS[name]
    shapes = synth.decoder_tensor_list(synth.DIMS[dims_key])
    sig = synth.per_tensor_scales(config_id, len(shapes))
    # skip the embedding so that the sample holds the per-layer mix of small and large tensors
    first = 1 if len(shapes) > 1 else 0
    gs, ds, total, used = [], [], 0, 0
    for i in range(first, len(shapes)):
        n = min(shapes[i][1], target_elems - total)
        if n <= 0:
            break
        g, d = synth.gaussian_tensor_pair(n, sig[i], rho, config_id, i, g_dtype, "cpu")
        gs.append(g)
        ds.append(d)
        total += n
        used += 1
    return gs, ds, total, used


def time_oracle_on(sample, name: str, threads: int, steps: int, warmup: int):
    """Wall clock of the oracle's whole step (stats, decision, projection, state refresh) on a sample."""
    from oracle import gac_oracle as orc
    gs, ds, total, used = sample
    hp = orc.HParams(**FORCE)
    times = []
    for i in range(warmup + steps):
        g = [t.clone() for t in gs]
        d = [t.clone() for t in ds]
        t0 = time.perf_counter()
        orc.step(g, d, hp, threads=threads)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    return {"value": total / sec, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"first {used} tensors after the embedding of the {name} list ({total} params, the last "
                      f"tensor cut), stats+project, {steps} timed passes of {sec:.2f} s",
            "seconds_per_pass": sec}


def sample_sizes(name: str):
    dims_key = synth.WORKLOADS[name][0]
    shapes = synth.decoder_tensor_list(synth.DIMS[dims_key])
    avail = synth.list_numel(shapes[1:] if len(shapes) > 1 else shapes)
    return min(ALL_CORE_SAMPLE, avail), min(ONE_THREAD_SAMPLE, avail)


def cpu_baseline(name: str, passes: int = 3):
    """The oracle as it stands on this host: all cores, and one thread on a prefix of the same sample."""
    n_all, n_one = sample_sizes(name)
    sample = oracle_sample(name, n_all)
    cores = host_cores()
    allc = time_oracle_on(sample, name, cores, passes, 1)
    one = time_oracle_on(oracle_sample(name, n_one), name, 1, passes, 1)
    out = {k: allc[k] for k in ("value", "unit", "cores", "kind", "sample")}
    out["single_thread"] = {k: one[k] for k in ("value", "unit", "cores", "sample")}
    return out


def run_reference(args):
    """The CPU oracle as it stands, on the host cores, on the same workload
    definition: every step is one pass over the bounded sample that the library
    arm's `cpu_baseline` uses (shrunk only if K + W passes would not end within
    a few minutes)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    name = args.workload
    cores = host_cores()
    n_all, n_one = sample_sizes(name)
    probe = time_oracle_on(oracle_sample(name, min(n_all, 8_000_000)), name, cores, 1, 0)
    budget_s = 150.0 / max(1, args.steps + args.warmup)
    target = int(min(n_all, max(8_000_000, probe["value"] * budget_s)))
    cb = time_oracle_on(oracle_sample(name, target), name, cores, args.steps, args.warmup)
    one = time_oracle_on(oracle_sample(name, n_one), name, 1, 2, 1)
    config = workload_config(name)
    config["timing"] = "host wall clock (time.perf_counter) around each oracle pass; no GPU is used"
    base = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
    base["single_thread"] = {k: one[k] for k in ("value", "unit", "cores", "sample")}
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": cb["seconds_per_pass"] * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config, "cpu_baseline": base,
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def dtype_name(t) -> str:
    return "bf16" if t == torch.bfloat16 else "f32"


def workload_config(name: str):
    dims_key, g_dtype, rho, config_id = synth.WORKLOADS[name]
    shapes = synth.decoder_tensor_list(synth.DIMS[dims_key])
    d_dtype = synth.WORKLOAD_D_DTYPE.get(name, torch.float32)
    return {"workload": f"{name}: {dims_key} decoder-shaped gradient list, "
                        f"{dtype_name(g_dtype)} g / {dtype_name(d_dtype)} d, target cosine {rho}, "
                        f"projection regime forced with c_low=0.05 c_high=2.0",
            "params_per_gpu": synth.list_numel(shapes), "tensors": len(shapes),
            "bytes_per_param": 3 * bytes_per_param(g_dtype, d_dtype),
            "l2": "inputs larger than L2; a fresh gradient is written between timed steps",
            "timing": "per-step CUDA events around gac_stats+gac_project, summed over the timed steps"}


# ------------------------------------------------------------------- driver

def summarize(wl: Workload, s_ms, p_ms, peak, peak_kind):
    bpp = bytes_per_param(wl.g_dtype, wl.d_dtype)
    s_avg, p_avg = sum(s_ms) / len(s_ms), sum(p_ms) / len(p_ms)
    step_ms = s_avg + p_avg
    proj_bytes = 2 * bpp * wl.params
    stats_bytes = bpp * wl.params
    proj_gbs = proj_bytes / (p_avg * 1e-3) / 1e9
    stats_gbs = stats_bytes / (s_avg * 1e-3) / 1e9
    tr_p, tr_s = recorded_traffic("gac_project_kernel"), recorded_traffic("gac_stats_kernel")
    key = "bf16" if wl.g_dtype == torch.bfloat16 else "f32"
    if wl.d_dtype != torch.float32:
        key += "_dbf16"
    return {
        "ms_per_step": step_ms, "stats_ms": s_avg, "project_ms": p_avg,
        "best_ms_per_step": min(a + b for a, b in zip(s_ms, p_ms)),
        "median_ms_per_step": statistics.median(a + b for a, b in zip(s_ms, p_ms)),
        "hbm_gbs": (proj_bytes + stats_bytes) / (step_ms * 1e-3) / 1e9,
        "roofline": {"bound": "hbm", "kernel": "gac_project_kernel", "achieved": proj_gbs,
                     "peak": peak, "unit": "GB/s", "frac": proj_gbs / peak,
                     "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": proj_gbs / NOMINAL_HBM_GBS,
                     "algorithmic_bytes_per_launch": proj_bytes,
                     "traffic": (tr_p[key] * wl.params if tr_p and key in tr_p else None)},
        "roofline_stats": {"bound": "hbm", "kernel": "gac_stats_kernel", "achieved": stats_gbs,
                           "peak": peak, "unit": "GB/s", "frac": stats_gbs / peak,
                           "peak_kind": f"of {peak_kind}",
                           "algorithmic_bytes_per_launch": stats_bytes,
                           "traffic": (tr_s[key] * wl.params if tr_s and key in tr_s else None)},
    }


def time_graph_replay(wl: Workload, replays: int = 200):
    """One step (both launches, no host read-back) captured in a CUDA graph and replayed:
    what a launch-bound list costs once the launch overhead of two direct calls is gone."""
    gb = wl.gb
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        wl.step()
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        graph.capture_begin()
        wl.step()
        graph.capture_end()
        for _ in range(5):
            graph.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(replays):
            graph.replay()
        b.record()
        side.synchronize()
    torch.cuda.current_stream().wait_stream(side)
    return a.elapsed_time(b) / replays * 1e3     # microseconds per step


def time_other(name: str, device, steps: int, peak: float, adamw: bool = False):
    """A further workload, timed the same way (fewer steps): a compact record."""
    gb_need = synth.list_numel(synth.decoder_tensor_list(synth.DIMS[synth.WORKLOADS[name][0]])) * \
        bytes_per_param(synth.WORKLOADS[name][1], synth.WORKLOAD_D_DTYPE.get(name, torch.float32)) + (6 << 30)
    free, _ = torch.cuda.mem_get_info()
    if free < gb_need:
        return {"skipped": f"needs {gb_need} bytes of device memory, {free} free"}
    wl = Workload(name, device, 1)
    s_ms, p_ms = time_steps(wl, steps, 3)
    res = check_regime(wl)
    bpp = bytes_per_param(wl.g_dtype, wl.d_dtype)
    s_avg, p_avg = sum(s_ms) / len(s_ms), sum(p_ms) / len(p_ms)
    ms = s_avg + p_avg
    out = {"params": wl.params, "steps": steps, "ms_per_step": ms, "stats_ms": s_avg, "project_ms": p_avg,
           "value": wl.params / (ms * 1e-3), "unit": UNIT, "bytes_per_param": 3 * bpp,
           "hbm_gbs": 3 * bpp * wl.params / (ms * 1e-3) / 1e9,
           "stats_gbs": bpp * wl.params / (s_avg * 1e-3) / 1e9,
           "project_gbs": 2 * bpp * wl.params / (p_avg * 1e-3) / 1e9,
           "stats_frac_of_measured_copy": bpp * wl.params / (s_avg * 1e-3) / 1e9 / peak,
           "project_frac_of_measured_copy": 2 * bpp * wl.params / (p_avg * 1e-3) / 1e9 / peak,
           "regime_check": {"cos": res.cos, "regime": wl.gb.REGIME_NAMES[res.regime]}}
    if 3 * bpp * wl.params < (126 << 20):
        out["note"] = ("launch-bound: the whole step moves less than the 126 MB L2 holds, so this is not a "
                       "roofline point")
        out["graph_replay_us_per_step"] = time_graph_replay(wl)
    if adamw:
        out["fused_adamw"] = time_fused_adamw(wl, steps, peak=peak)
        if wl.g_dtype == wl.d_dtype:
            out["fused_adamw_exchange"] = time_fused_adamw(wl, steps, exchange=True, peak=peak)
    wl.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_7b_bf16", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--also", default="cfg5_14b_f32",
                    help="second workload reported under 'also' (1 GPU only); 'none' to skip")
    ap.add_argument("--others", default="cfg1_flat_f32,cfg2_1.5b_f32,cfg3_7b_bf16_dbf16",
                    help="further workloads reported compactly under 'others' (1 GPU only); 'none' to skip")
    ap.add_argument("--clip", type=float, default=0.0,
                    help="fold global-norm clipping with this max norm into the projection pass (0 = off)")
    ap.add_argument("--sharded", action="store_true",
                    help="use the sharded call sequence (local sums, NCCL all-reduce of 3 doubles, decision) "
                         "even on one GPU; always on for --gpus > 1")
    ap.add_argument("--exchange", default="nccl", choices=["nccl", "peer"],
                    help="how the sharded form sums its three numbers across ranks: NCCL's all-reduce (default) or "
                         "the library's own peer stores in the reduction's epilogue (needs symmetric memory)")
    ap.add_argument("--no-adamw", action="store_true",
                    help="skip the legs that time the projection fused with AdamW (1 GPU)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")

    if args.impl == "reference":
        return run_reference(args)

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the GAC path has no CPU fallback")
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        # no launcher around us: become the launcher of one rank per GPU
        have = torch.cuda.device_count()
        if args.gpus > have:
            raise SystemExit(f"--gpus {args.gpus}: only {have} CUDA device(s) are visible")
        return spawn_ranks(args.gpus, sys.argv[1:])

    from paper_2603_01501_b200 import binding as gb
    gb.load_library()
    line_out = reserve_stdout()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1 or args.sharded:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if "MASTER_PORT" not in os.environ:
            if world > 1:
                raise SystemExit("WORLD_SIZE > 1 needs MASTER_PORT from the launcher")
            os.environ["MASTER_PORT"] = str(free_port())
        torch.distributed.init_process_group("nccl", device_id=device, rank=rank, world_size=world)
    peak, peak_kind = measured_hbm_peak()

    wl = Workload(args.workload, device, world, args.clip, args.sharded, args.exchange == "peer")
    sampler = ClockSampler(nvml_index(local_rank))
    wall0 = time.perf_counter()
    s_ms, p_ms = time_steps(wl, args.steps, args.warmup, sampler)
    wall = time.perf_counter() - wall0
    total_ms = sum(s_ms) + sum(p_ms)
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device=device)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        total_ms = float(t.item())
    res = check_regime(wl)
    summ = summarize(wl, s_ms, p_ms, peak, peak_kind)
    ms_per_step = total_ms / args.steps
    info = gb.gac_get_info(wl.ctx)
    line = {"metric": METRIC, "value": wl.params * world / (ms_per_step * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": f"{dtype_name(wl.g_dtype)} g / {dtype_name(wl.d_dtype)} d, f64 sums, f32 fma",
            "data": "synthetic", "config": workload_config(args.workload),
            "hbm_gbs": summ["hbm_gbs"] , "frac_of_nominal_8TBs": summ["hbm_gbs"] / NOMINAL_HBM_GBS,
            "stats_ms": summ["stats_ms"], "project_ms": summ["project_ms"],
            "best_ms_per_step": summ["best_ms_per_step"],
            "median_ms_per_step": summ["median_ms_per_step"],
            "regime_check": {"cos": res.cos, "regime": gb.REGIME_NAMES[res.regime], "alpha": res.alpha,
                             "clip_scale": res.clip_scale},
            "launch": {"grid": info.grid, "threads": info.threads, "chunk_elems": info.chunk_elems,
                       "chunks": info.n_chunks},
            "gpu_launches": (3 if wl.sharded else 2) * args.steps,
            "clocks": sampler.summary(), "roofline": summ["roofline"],
            "roofline_stats": summ["roofline_stats"], "wall_s_timed_loop": wall}
    how = ("the three sums exchanged by peer stores in the reduction's epilogue" if wl.peer_exchange
           else "one NCCL all-reduce of 3 doubles per step")
    if world > 1:
        line["config"]["parallelism"] = f"dp{world}: every rank holds one list as its gradient shard; {how}"
    elif wl.sharded:
        line["config"]["parallelism"] = f"dp1: the sharded call sequence in a one-rank group; {how}"

    few = min(args.steps, 10)
    if world == 1:
        line["unchanged_regime"] = time_unchanged_regime(wl, few)
    if world == 1 and not args.no_adamw:
        line["fused_adamw"] = time_fused_adamw(wl, few, peak=peak, peak_kind=peak_kind)
        if wl.g_dtype == wl.d_dtype:
            line["fused_adamw_exchange"] = time_fused_adamw(wl, few, exchange=True, peak=peak, peak_kind=peak_kind)
    if world == 1 and wl.g_dtype == wl.d_dtype:
        line["exchange_mode"] = time_exchange_mode(wl, few)
    if not args.no_e2e:
        # every rank takes the same branch: the decision to run is agreed on first, and the
        # result is reduced by all ranks whether or not a rank failed
        go = torch.tensor([1.0 if e2e_fits_host(wl) else 0.0], dtype=torch.float64, device=device)
        if world > 1:
            torch.distributed.all_reduce(go, op=torch.distributed.ReduceOp.MIN)
        if float(go.item()) > 0:
            try:
                e2e = time_e2e(wl, min(args.steps, 5), 1)
            except Exception as exc:
                e2e = {"value": None, "unit": UNIT, "error": repr(exc)[:200], "ms_per_step": -1.0}
            if world > 1:
                t = torch.tensor([e2e["ms_per_step"], -e2e["ms_per_step"]], dtype=torch.float64, device=device)
                torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
                if -float(t[1].item()) < 0:       # some rank failed
                    e2e = {"value": None, "unit": UNIT, "error": e2e.get("error", "a rank failed")}
                else:
                    e2e["ms_per_step"] = float(t[0].item())
                    e2e["value"] = wl.params * world / (float(t[0].item()) * 1e-3)
            line["e2e"] = e2e
        else:
            line["e2e"] = {"value": None, "unit": UNIT,
                           "skipped": "the pinned host copies of all ranks would take more than half of the host's memory"}
    wl.close()

    if world == 1 and args.also != "none" and args.also != args.workload:
        free, _ = torch.cuda.mem_get_info()
        dims_key, g_dtype, _, _ = synth.WORKLOADS[args.also]
        need = synth.list_numel(synth.decoder_tensor_list(synth.DIMS[dims_key])) * \
            (bytes_per_param(g_dtype)) + (4 << 30)
        if free > need:
            wl2 = Workload(args.also, device, 1)
            s2, p2 = time_steps(wl2, few, 3)
            r2 = check_regime(wl2)
            also = summarize(wl2, s2, p2, peak, peak_kind)
            also.update({"workload": workload_config(args.also)["workload"],
                         "params": wl2.params, "steps": few,
                         "value": wl2.params / (also["ms_per_step"] * 1e-3), "unit": UNIT,
                         "regime_check": {"cos": r2.cos, "regime": gb.REGIME_NAMES[r2.regime]}})
            if wl2.g_dtype == wl2.d_dtype:
                also["exchange_mode"] = time_exchange_mode(wl2, few)
            line["also"] = also
            wl2.close()
        else:
            line["also"] = {"skipped": f"needs {need} bytes of device memory, {free} free"}

    if world == 1 and args.others != "none":
        line["others"] = {}
        for name in args.others.split(","):
            if name and name != args.workload and name != args.also:
                line["others"][name] = time_other(name, device, few, peak,
                                                  adamw=(not args.no_adamw and name.endswith("_dbf16")))

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(args.workload)

    if world > 1 or args.sharded:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    if rank == 0:
        line_out.write(json.dumps(line) + "\n")
        line_out.flush()
    return 0


if __name__ == "__main__":
    sys.exit(main())
