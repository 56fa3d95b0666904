#!/usr/bin/env python
"""Benchmark of the MOSAIC block-sparse attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one forward layer pass of the workload: block pooling + scoring + top-k selection,
then the block-sparse attention forward (the backward of the same workload is timed beside it
and reported under "stages").  Default workload: the 1.5-degree grid (120x240, 8x8 blocks,
B=1, H=8, d=64, top-k 8) with seeded smooth+noise bf16 inputs.  Rank 0 prints ONE JSON line.

value    effective TFLOP/s over the step: 4*d*b*b FLOP per attended (query block, key block)
         pair, unmasked work only, inputs resident in HBM, L2 flushed between timed iterations,
         device time by CUDA events, max over ranks.
e2e      the same metric with the step's Q, K, V copied from pinned host memory and O copied
         back inside the timed region.
roofline the forward kernel alone against the measured dense bf16 peak of this GPU pool.
cpu_baseline  the fp64 oracle timed on the host cores (reported, never optimised against).
With N > 1 every rank runs the workload on its own GPU (weak scaling, no data-path collective).
`--impl reference` times the oracle (CPU) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2604_16429_b200 import flops, synth

METRIC = "block-sparse attn effective TFLOP/s (select + fwd, ms/layer fwd at 1.5deg grid)"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 256 << 20
MIN_TIMED_SECONDS = 0.5           # the timed region is at least this long, whatever --steps says
OTHER_WORKLOADS = ("c5_0p25deg", "c3_1p5deg_ens24")   # timed beside the default workload (forward only, few steps)
OTHER_STEPS = 5


def kernel_sources_digest() -> str:
    """SHA-256 over the sources of the forward kernel: a stored DRAM-traffic figure is only reported while
    the kernel it was measured on is the kernel that runs."""
    import hashlib
    h = hashlib.sha256()
    for f in ("fwd_tc.cu", "tc_common.cuh", "common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_2604_16429_b200", "csrc", f), "rb").read())
    return h.hexdigest()


def measured_traffic(workload: str):
    """DRAM bytes per launch of the forward kernel from the kept ncu summary of this workload, or None when
    there is none or the kernel has changed since (the summary records the digest of the sources it measured)."""
    import re
    path = os.path.join(ROOT, "profiles", f"fwd_tc_kernel_{workload}.md")
    if not os.path.exists(path):
        return None, "no ncu capture kept for this workload"
    m = re.search(r"kernel_sha256=([0-9a-f]{64})\s+dram_bytes_per_launch=([0-9.eE+]+)", open(path).read())
    if not m:
        return None, "the kept ncu summary carries no traffic record"
    if m.group(1) != kernel_sources_digest():
        return None, "kernel changed since the kept ncu capture"
    return float(m.group(2)), "ncu dram__bytes_read.sum + dram__bytes_write.sum, one launch, kept summary of this workload"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0, "hbm_gbs": FALLBACK_HBM_GBS,
            "source": "fallback"}


class ClockSampler:
    """Samples SM clock and clock-event reasons of one GPU through NVML while a region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, cuda_index: int, period_s: float = 0.002):
        self.samples, self.mask, self.max_mhz = [], 0, None
        self.period, self._stop, self._thr, self.h = period_s, threading.Event(), None, None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID("GPU-" + str(torch.cuda.get_device_properties(cuda_index).uuid))
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    self.mask |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    self.mask |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.h is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self) -> dict:
        if self._thr is not None:
            self._stop.set()
            self._thr.join()
        reasons = [n for bit, n in self.REASONS.items() if self.mask & bit]
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples)}


def describe(w) -> str:
    return (f"{w.name}: {w.nlat}x{w.nlon} grid, {w.bh}x{w.bw} blocks (m={w.m}), B={w.B}, H={w.H}, d={w.d}, "
            + (f"local groups of {w.rlat}x{w.rlon} blocks" if w.local_groups else f"local {2 * w.rlat + 1}x{2 * w.rlon + 1}")
            + f", top-k {w.topk}, {w.kind} bf16 inputs")


# ------------------------------------------------------------------------------------------
def oracle_sample_step(w, x, g, blocks, unit=(0, 0)):
    import oracle
    b, h = unit
    hk = h // (w.H // w.kv_heads)
    idx = oracle.select(g, x["q"][b, h], x["k"][b, hk])
    oracle.fwd(g, x["q"][b, h], x["k"][b, hk], x["v"][b, hk], idx, blocks)
    return idx


def sample_flops(w, g, blocks) -> float:
    import oracle
    pairs = sum(len(oracle.local_set(g, int(i))) + min(w.topk, w.m - len(oracle.local_set(g, int(i)))) for i in blocks)
    return 4.0 * w.d * w.b * w.b * pairs


def cpu_baseline(w, x, idx_gpu, o_gpu, lse_gpu) -> dict:
    """Time the oracle, as it stands, on a bounded sample of the workload (a few seconds to about ten on 16
    host cores): up to 40 whole units for 64-token blocks (the whole 1.5-degree workload has 8), 640 query
    blocks of one unit for larger blocks.  The sample
    doubles as a parity spot check of the launch configuration that was just timed."""
    import oracle
    from oracle import Geom
    oracle.build()
    g = Geom(w.nlat, w.nlon, d=w.d, bh=w.bh, bw=w.bw, rlat=w.rlat, rlon=w.rlon, topk=w.topk, local_groups=w.local_groups)
    rng = np.random.default_rng(0)
    if w.b <= 64:
        units = [(u // w.H, u % w.H) for u in range(min(40, w.U))]
        blocks = np.arange(w.m, dtype=np.int32)
    else:
        units = [(0, 0)]
        blocks = np.sort(rng.choice(w.m, size=min(w.m, 640), replace=False)).astype(np.int32)
    oracle.local_set(g, 0)                                       # load the library before timing
    fl, dt, worst = 0.0, 0.0, 0.0
    for (b, h) in units:
        t0 = time.perf_counter()
        hk = h // (w.H // w.kv_heads)
        idx0 = oracle.select(g, x["q"][b, h], x["k"][b, hk])
        O, L = oracle.fwd(g, x["q"][b, h], x["k"][b, hk], x["v"][b, hk], idx0, blocks)
        dt += time.perf_counter() - t0
        fl += sample_flops(w, g, blocks)
        assert np.array_equal(idx_gpu[b, h].cpu().numpy(), idx0), "selection differs from the oracle"
        tok = np.concatenate([oracle.block_tokens(g, int(j)) for j in blocks])
        err = np.abs(o_gpu[b, h].float().cpu().numpy()[tok] - O.reshape(-1, w.d))
        lerr = np.abs(lse_gpu[b, h].cpu().numpy()[tok] - L.reshape(-1))
        assert err.max() <= 2e-2 and err.mean() <= 2e-3 and lerr.max() <= 2e-3, (err.max(), err.mean(), lerr.max())
        worst = max(worst, float(err.max()))
    sample = (f"selection + forward of {len(units)} unit(s) x {len(blocks)} of {w.m} query blocks, {dt:.2f} s; "
              f"GPU output of the sample within {worst:.2e} of it")
    return {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": sample}


def run_reference(args, w):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from oracle import Geom
    oracle.build()
    g = Geom(w.nlat, w.nlon, d=w.d, bh=w.bh, bw=w.bw, rlat=w.rlat, rlon=w.rlon, topk=w.topk, local_groups=w.local_groups)
    one = synth.Workload(**{**w.__dict__, "B": 1, "H": 1})
    x = synth.make_inputs(one, with_do=False)
    rng = np.random.default_rng(0)
    nb = min(w.m, 64 if w.b <= 64 else 8)
    blocks = np.sort(rng.choice(w.m, size=nb, replace=False)).astype(np.int32)
    fl = sample_flops(w, g, blocks)
    for _ in range(args.warmup):
        oracle_sample_step(w, x, g, blocks)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_sample_step(w, x, g, blocks)
    dt = (time.perf_counter() - t0) / args.steps
    value = fl / dt / 1e12
    sample = f"selection of 1 unit + forward of {nb} of {w.m} query blocks of that unit per step (seed 0)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(w), "sample": sample},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
def forward_only(w, dev, peaks, steps, cuda_index) -> dict:
    """Selection + forward of another workload, timed like the main one (CUDA events per step, L2 flushed
    between steps, clocks sampled during the timed region); host generation of the inputs is outside it."""
    import torch

    from paper_2604_16429_b200 import binding as mb
    x = synth.make_inputs(w, with_do=False)
    dx = {k: torch.from_numpy(v.view(np.int16)).to(dev).view(torch.bfloat16) for k, v in x.items()}
    del x
    p = mb.Params.from_workload(w)
    ws = torch.empty(max(mb.workspace_bytes(p, op) for op in (mb.OP_SELECT, mb.OP_FWD)), dtype=torch.uint8, device=dev)
    idx = torch.empty((w.B, w.H, w.m, w.topk), dtype=torch.int32, device=dev)
    o = torch.empty_like(dx["q"])
    lse = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        mb.mosaic_bsa_select(p, dx["q"], dx["k"], block_idx=idx, ws=ws)
        if ev:
            ev[1].record(stream)
        mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx, o=o, lse=lse, ws=ws)
        if ev:
            ev[2].record(stream)

    for _ in range(3):
        flush_buf.zero_()
        step()
    torch.cuda.synchronize()
    mb.check_status(ws, "warm-up of " + w.name)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    sampler = ClockSampler(cuda_index)
    sampler.start()
    for s in range(steps):
        flush_buf.zero_()
        step(evs[s])
    torch.cuda.synchronize()
    clocks = sampler.stop()
    mb.check_status(ws, "timed region of " + w.name)
    t_sel = sum(e[0].elapsed_time(e[1]) for e in evs) / steps
    t_fwd = sum(e[1].elapsed_time(e[2]) for e in evs) / steps
    fl = flops.fwd_flops(w)
    tf = fl / (t_fwd * 1e-3) / 1e12
    return {"workload": describe(w), "steps": steps, "select_ms": t_sel, "fwd_ms": t_fwd, "ms_layer_fwd": t_sel + t_fwd,
            "fwd_tflops": tf, "step_tflops": fl / ((t_sel + t_fwd) * 1e-3) / 1e12,
            "roofline_frac_of_measured_burst": tf / peaks["bf16_tflops"], "frac_of_nominal_2250": tf / NOMINAL_BF16_TFLOPS,
            "select_pool_gbs_lower_bound": 2.0 * w.U * w.N * w.d * 2 / (t_sel * 1e-3) / 1e9, "clocks": clocks}


def run_ours(args, w):
    import torch

    from paper_2604_16429_b200 import binding as mb
    from paper_2604_16429_b200 import dist as mdist

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank, local_rank, world = mdist.init()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    mb.lib()  # fail loudly if the library is missing

    # every rank runs the same workload on its own members: per-rank noise seeds differ by rank
    wl = synth.Workload(**{**w.__dict__, "cfg": w.cfg + 100 * rank}) if world > 1 else w
    x = synth.make_inputs(wl, with_do=True)
    host = {k: torch.from_numpy(v.view(np.int16)).pin_memory() for k, v in x.items()}
    dx = {k: t.to(dev, non_blocking=True).view(torch.bfloat16) for k, t in host.items()}
    p = mb.Params.from_workload(w)
    ws = torch.empty(max(mb.workspace_bytes(p, op) for op in (mb.OP_SELECT, mb.OP_FWD, mb.OP_BWD)),
                     dtype=torch.uint8, device=dev)
    idx = torch.empty((w.B, w.H, w.m, w.topk), dtype=torch.int32, device=dev)
    o = torch.empty_like(dx["q"])
    lse = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.empty_like(dx["q"]), torch.empty_like(dx["k"]), torch.empty_like(dx["k"])
    flush_buf = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def fwd_step(ev=None):
        if ev:
            ev[0].record(stream)
        mb.mosaic_bsa_select(p, dx["q"], dx["k"], block_idx=idx, ws=ws)
        if ev:
            ev[1].record(stream)
        mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx, o=o, lse=lse, ws=ws)
        if ev:
            ev[2].record(stream)

    def bwd_step():
        mb.mosaic_bsa_bwd(p, dx["q"], dx["k"], dx["v"], o, lse, dx["do"], idx, dq=dq, dk=dk, dv=dv, ws=ws)

    for _ in range(max(args.warmup, 3)):
        flush_buf.zero_()
        fwd_step()
    bwd_step()
    torch.cuda.synchronize()
    mb.check_status(ws, "warm-up")

    # step count: at least --steps, and enough for MIN_TIMED_SECONDS of GPU time (estimated from a short probe)
    probe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    probe[0].record(stream)
    for _ in range(5):
        flush_buf.zero_()
        fwd_step()
    probe[1].record(stream)
    torch.cuda.synchronize()
    K = max(args.steps, min(20000, int(args.min_seconds * 1e3 / max(probe[0].elapsed_time(probe[1]) / 5, 1e-3)) + 1))
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    sampler = ClockSampler(local_rank)
    mdist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    for s in range(K):
        flush_buf.zero_()          # L2 flush, outside the timed interval of the step
        fwd_step(evs[s])
    torch.cuda.synchronize()
    clocks = sampler.stop()
    mdist.barrier()
    t_sel = sum(e[0].elapsed_time(e[1]) for e in evs) / K
    t_fwd = sum(e[1].elapsed_time(e[2]) for e in evs) / K
    t_step = sum(e[0].elapsed_time(e[2]) for e in evs) / K
    mb.check_status(ws, "timed region")

    # backward of the same workload, timed the same way (reported under "stages")
    kb = min(K, 50)
    evb = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(kb)]
    for s in range(kb):
        flush_buf.zero_()
        evb[s][0].record(stream)
        bwd_step()
        evb[s][1].record(stream)
    torch.cuda.synchronize()
    t_bwd = sum(e[0].elapsed_time(e[1]) for e in evb) / kb

    # the paper's three-branch form of the same workload (compression + selection + local, gated), same selection
    gates = torch.randn((w.B, w.H, w.N, 3), dtype=torch.float32, device=dev)
    ws3 = torch.empty(mb.workspace_bytes(p, mb.OP_FWD_BRANCHES), dtype=torch.uint8, device=dev)
    lse_fg, lse_l = torch.empty_like(lse), torch.empty_like(lse)
    k3 = min(K, 50)
    ev3 = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(k3)]
    for s in range(k3 + 2):
        flush_buf.zero_()
        if s >= 2:
            ev3[s - 2][0].record(stream)
        mb.mosaic_bsa_fwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gates, o=dq, lse_fg=lse_fg, lse_l=lse_l, ws=ws3)
        if s >= 2:
            ev3[s - 2][1].record(stream)
    torch.cuda.synchronize()
    mb.check_status(ws3, "three-branch forward")
    t_br = sum(e[0].elapsed_time(e[1]) for e in ev3) / k3
    del ws3, lse_fg, lse_l
    # and its backward (recomputes the forward's intermediates; gradient of the gates included)
    ws3b = torch.empty(mb.workspace_bytes(p, mb.OP_BWD_BRANCHES), dtype=torch.uint8, device=dev)
    dgates = torch.empty_like(gates)
    k3b = min(K, 20)
    ev3b = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(k3b)]
    for s in range(k3b + 2):
        flush_buf.zero_()
        if s >= 2:
            ev3b[s - 2][0].record(stream)
        mb.mosaic_bsa_bwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gates, dx["do"], dq=dq, dk=dk, dv=dv, dgates=dgates, ws=ws3b)
        if s >= 2:
            ev3b[s - 2][1].record(stream)
    torch.cuda.synchronize()
    mb.check_status(ws3b, "three-branch backward")
    t_brb = sum(e[0].elapsed_time(e[1]) for e in ev3b) / k3b
    del ws3b, gates, dgates

    # 2-D rotary position embedding of Q and K (the paper applies it before the operator): an HBM-bound pass
    pos = torch.rand((w.N, 2), dtype=torch.float32, device=dev)
    q_r, k_r = torch.empty_like(dx["q"]), torch.empty_like(dx["k"])
    kr = min(K, 20)
    evr = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(kr)]
    for s in range(kr + 2):
        flush_buf.zero_()
        if s >= 2:
            evr[s - 2][0].record(stream)
        mb.mosaic_bsa_rope(p, dx["q"], dx["k"], pos, q_out=q_r, k_out=k_r)
        if s >= 2:
            evr[s - 2][1].record(stream)
    torch.cuda.synchronize()
    t_rope = sum(e[0].elapsed_time(e[1]) for e in evr) / kr
    rope_gbs = 2 * (dx["q"].numel() + dx["k"].numel()) * 2 / (t_rope * 1e-3) / 1e9
    del pos, q_r, k_r

    # end to end: pinned host -> device, step, device -> pinned host.  The units are independent, so the step runs as
    # a pipeline over groups of units through the same public calls: group c + 1 is copied in (own stream) while group
    # c computes, and group c - 1 is copied out (third stream).  Everything lies between the two timing events.
    ke = min(K, 20)
    o_host = torch.empty(o.shape, dtype=torch.int16).pin_memory()
    ax = 1 if w.B == 1 else 0                       # split the heads of a single sample, else the samples
    extent = w.H if ax == 1 else w.B
    nch = 4 if extent % 4 == 0 else (2 if extent % 2 == 0 else 1)
    if ax == 1 and w.kv_heads != w.H:
        nch = 1                                     # K and V have other head counts: no split by heads
    per = extent // nch
    pch = mb.Params.from_workload(w, **({"H": per} if ax == 1 else {"B": per}))
    sl = [(slice(None), slice(c * per, (c + 1) * per)) if ax == 1 else (slice(c * per, (c + 1) * per),) for c in range(nch)]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(nch)]
    ev_done = [torch.cuda.Event() for _ in range(nch)]
    ev_out = torch.cuda.Event()
    eve = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(ke)]
    for s in range(ke + 1):
        if s:
            eve[s - 1][0].record(stream)
        s_in.wait_stream(stream)                    # the copies start inside the timed region
        s_out.wait_stream(stream)
        for c in range(nch):
            with torch.cuda.stream(s_in):
                for name in ("q", "k", "v"):
                    dx[name][sl[c]].view(torch.int16).copy_(host[name][sl[c]], non_blocking=True)
                ev_in[c].record(s_in)
            stream.wait_event(ev_in[c])
            mb.mosaic_bsa_select(pch, dx["q"][sl[c]], dx["k"][sl[c]], block_idx=idx[sl[c]], ws=ws)
            mb.mosaic_bsa_fwd(pch, dx["q"][sl[c]], dx["k"][sl[c]], dx["v"][sl[c]], idx[sl[c]], o=o[sl[c]], lse=lse[sl[c]], ws=ws)
            ev_done[c].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[c])
                o_host[sl[c]].copy_(o[sl[c]].view(torch.int16), non_blocking=True)
        ev_out.record(s_out)
        stream.wait_event(ev_out)
        if s:
            eve[s - 1][1].record(stream)
    torch.cuda.synchronize()
    mb.check_status(ws, "end-to-end region")
    t_e2e = sum(e[0].elapsed_time(e[1]) for e in eve) / ke
    h2d = 3 * dx["q"].numel() * 2
    d2h = o.numel() * 2

    traffic, traffic_source = measured_traffic(w.name)
    t_step_max = mdist.max_over_ranks(t_step, dev)
    t_e2e_max = mdist.max_over_ranks(t_e2e, dev)
    fl = flops.fwd_flops(w)
    value = world * fl / (t_step_max * 1e-3) / 1e12
    peaks = measured_peaks()
    fwd_tflops = fl / (t_fwd * 1e-3) / 1e12
    pool_bytes = 2.0 * w.U * w.N * w.d * 2

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": K, "steps_requested": args.steps,
        "warmup": max(args.warmup, 3),
        "ms_per_step": t_step_max, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": describe(w), "l2": f"flushed between timed iterations ({L2_FLUSH_BYTES >> 20} MiB write)",
                   "step": "select (pool + top-k) + forward", "parallelism": f"replicas x{world}, no collective"},
        "clocks": clocks,
        "e2e": {"value": world * fl / (t_e2e_max * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": t_e2e_max,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipeline": f"{nch} groups of units: copy in, compute, copy out on three streams"},
        "gpu_launches": 3 * K,
        "roofline": {"kernel": "fwd_tc_kernel", "bound": "tensor", "achieved": fwd_tflops,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": fwd_tflops / peaks["bf16_tflops"],
                     "traffic": traffic, "traffic_source": traffic_source, "peak_source": peaks["source"] + " (burst)",
                     "frac_of_nominal_2250": fwd_tflops / NOMINAL_BF16_TFLOPS, "ms": t_fwd},
        "stages": {"select_ms": t_sel, "fwd_ms": t_fwd, "bwd_ms": t_bwd, "ms_layer_fwd": t_step,
                   "fwd_three_branch_ms": t_br, "bwd_three_branch_ms": t_brb, "rope_ms": t_rope, "rope_gbs": rope_gbs,
                   "fwd_tflops": fwd_tflops, "bwd_tflops": flops.bwd_flops(w) / (t_bwd * 1e-3) / 1e12,
                   "select_pool_gbs_lower_bound": pool_bytes / (t_sel * 1e-3) / 1e9,
                   "pct_of_nominal_peak": 100 * fwd_tflops / NOMINAL_BF16_TFLOPS,
                   "pct_of_measured_peak": 100 * fwd_tflops / peaks["bf16_tflops"]},
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, x, idx, o, lse)
    if world == 1 and args.workload == "c2_1p5deg" and not args.no_other_workloads:
        del dx, host, o, lse, dq, dk, dv, idx, ws, x
        torch.cuda.empty_cache()
        line["other_workloads"] = {name: forward_only(synth.WORKLOADS[name], dev, peaks, OTHER_STEPS, local_rank)
                                   for name in OTHER_WORKLOADS}
    if rank == 0:
        print(json.dumps(line), flush=True)
    mdist.finalize()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="c2_1p5deg", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true")
    ap.add_argument("--min-seconds", type=float, default=MIN_TIMED_SECONDS,
                    help="floor of the timed region in seconds of GPU time (0: exactly --steps steps, for profiler captures)")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
