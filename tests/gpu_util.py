"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI binding and
the oracle on the same seeded bits, and compare."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from oracle import Geom
from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth

FWD_MAX_ABS, FWD_MEAN_ABS = 2e-2, 2e-3      # forward tolerances (bf16 inputs, fp64 oracle)
BWD_MAX_ABS = 5e-2                          # backward tolerance
LSE_ABS = 2e-3                              # fp32 log-sum-exp of fp32-accumulated logits


def geom_of(w, scale=0.0) -> Geom:
    return Geom(w.nlat, w.nlon, d=w.d, bh=w.bh, bw=w.bw, rlat=w.rlat, rlon=w.rlon, topk=w.topk, scale=scale)


def device_inputs(x: dict) -> dict:
    return {k: mb.from_bits(v) for k, v in x.items()}


def oracle_select_all(w, x) -> np.ndarray:
    g = geom_of(w)
    out = np.empty((w.B, w.H, w.m, w.topk), np.int32)
    for b in range(w.B):
        for h in range(w.H):
            out[b, h] = oracle.select(g, x["q"][b, h], x["k"][b, h])
    return out


def gpu_select(w, dx, scale=0.0):
    p = mb.Params.from_workload(w, scale=scale)
    ws = mb.alloc_workspace(p, mb.OP_SELECT)
    idx = mb.mosaic_bsa_select(p, dx["q"], dx["k"], ws=ws)
    mb.check_status(ws, "select")
    return idx


def gpu_fwd(w, dx, idx, scale=0.0):
    p = mb.Params.from_workload(w, scale=scale)
    ws = mb.alloc_workspace(p, mb.OP_FWD)
    o = torch.full_like(dx["q"], float("nan"))
    lse = torch.full((w.B, w.H, w.N), float("nan"), dtype=torch.float32, device="cuda")
    mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx, o=o, lse=lse, ws=ws)
    mb.check_status(ws, "fwd")
    return o, lse


def gpu_bwd(w, dx, o, lse, idx, scale=0.0):
    p = mb.Params.from_workload(w, scale=scale)
    ws = mb.alloc_workspace(p, mb.OP_BWD)
    nan = lambda: torch.full_like(dx["q"], float("nan"))
    dq, dk, dv = mb.mosaic_bsa_bwd(p, dx["q"], dx["k"], dx["v"], o, lse, dx["do"], idx, dq=nan(), dk=nan(),
                                   dv=nan(), ws=ws)
    mb.check_status(ws, "bwd")
    return dq, dk, dv


def compare_fwd_unit(w, x, b, h, idx_unit, o_gpu, lse_gpu, blocks=None, scale=0.0):
    """Compare one unit (all blocks or a sample) with the oracle; returns (max, mean) abs error."""
    g = geom_of(w, scale)
    O, L = oracle.fwd(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], idx_unit, blocks)
    bl = range(w.m) if blocks is None else blocks
    tok = np.concatenate([oracle.block_tokens(g, j) for j in bl])
    og = o_gpu[b, h].float().cpu().numpy().astype(np.float64)[tok]
    lg = lse_gpu[b, h].cpu().numpy().astype(np.float64)[tok]
    assert np.isfinite(og).all() and np.isfinite(lg).all(), "unwritten or non-finite output"
    err = np.abs(og - O.reshape(-1, w.d))
    lerr = np.abs(lg - L.reshape(-1))
    assert err.max() <= FWD_MAX_ABS, f"O max-abs {err.max():.4g} (unit {b},{h})"
    assert err.mean() <= FWD_MEAN_ABS, f"O mean-abs {err.mean():.4g} (unit {b},{h})"
    assert lerr.max() <= LSE_ABS, f"LSE max-abs {lerr.max():.4g} (unit {b},{h})"
    return err.max(), err.mean()
