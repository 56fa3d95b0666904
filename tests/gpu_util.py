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
BWD_MAX_ABS = 5e-2                          # backward tolerance (max-abs, every element)
LSE_ABS = 2e-3                              # fp32 log-sum-exp of fp32-accumulated logits
GUARD = 4096                                # bytes of canary before and after every output and workspace


def assert_bwd_close(name, got, ref):
    gh = got.float().cpu().numpy().astype(np.float64) if torch.is_tensor(got) else np.asarray(got, np.float64)
    assert np.isfinite(gh).all(), f"{name}: unwritten or non-finite gradient"
    err = np.abs(gh - ref)
    assert err.max() <= BWD_MAX_ABS, f"{name}: max-abs {err.max():.4g} at |ref| {np.abs(ref)[np.unravel_index(err.argmax(), err.shape)]:.4g}"
    return float(err.max())


class Guarded:
    """A device buffer with canary bytes on both sides; `check()` fails if a kernel wrote outside it."""
    PATTERN = 0xA5

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((n + 2 * GUARD,), self.PATTERN, dtype=torch.uint8, device="cuda")
        self.t = self.raw[GUARD:GUARD + n].view(dtype).view(*shape)
        self.n = n
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what=""):
        torch.cuda.synchronize()
        lo, hi = self.raw[:GUARD], self.raw[GUARD + self.n:]
        assert bool((lo == self.PATTERN).all()) and bool((hi == self.PATTERN).all()), f"write outside the buffer: {what}"


def geom_of(w, scale=0.0) -> Geom:
    return Geom(w.nlat, w.nlon, d=w.d, bh=w.bh, bw=w.bw, rlat=w.rlat, rlon=w.rlon, topk=w.topk, scale=scale,
                local_groups=getattr(w, "local_groups", False), f16=getattr(w, "f16", False))


def device_inputs(x: dict, f16=False) -> dict:
    return {k: mb.from_bits(v, f16=f16) for k, v in x.items()}


def oracle_select_all(w, x) -> np.ndarray:
    g = geom_of(w)
    out = np.empty((w.B, w.H, w.m, w.topk), np.int32)
    for b in range(w.B):
        for h in range(w.H):
            out[b, h] = oracle.select(g, x["q"][b, h], x["k"][b, h])
    return out


def gpu_select(w, dx, scale=0.0):
    p = mb.Params.from_workload(w, scale=scale)
    ws = Guarded((mb.workspace_bytes(p, mb.OP_SELECT),), torch.uint8)
    idx = Guarded((w.B, w.H, w.m, w.topk), torch.int32, fill=-7)
    mb.mosaic_bsa_select(p, dx["q"], dx["k"], block_idx=idx.t, ws=ws.t)
    mb.check_status(ws.t, "select")
    ws.check("select workspace"); idx.check("block_idx")
    return idx.t.clone()


def gpu_fwd(w, dx, idx, scale=0.0):
    p = mb.Params.from_workload(w, scale=scale)
    ws = Guarded((mb.workspace_bytes(p, mb.OP_FWD),), torch.uint8)
    o = Guarded(tuple(dx["q"].shape), dx["q"].dtype, fill=float("nan"))
    lse = Guarded((w.B, w.H, w.N), torch.float32, fill=float("nan"))
    mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx, o=o.t, lse=lse.t, ws=ws.t)
    mb.check_status(ws.t, "fwd")
    ws.check("fwd workspace"); o.check("o"); lse.check("lse")
    return o.t.clone(), lse.t.clone()


def gpu_bwd(w, dx, o, lse, idx, scale=0.0):
    p = mb.Params.from_workload(w, scale=scale)
    ws = Guarded((mb.workspace_bytes(p, mb.OP_BWD),), torch.uint8)
    outs = [Guarded(tuple(dx[n].shape), dx["q"].dtype, fill=float("nan")) for n in ("q", "k", "k")]
    mb.mosaic_bsa_bwd(p, dx["q"], dx["k"], dx["v"], o, lse, dx["do"], idx, dq=outs[0].t, dk=outs[1].t,
                      dv=outs[2].t, ws=ws.t)
    mb.check_status(ws.t, "bwd")
    ws.check("bwd workspace")
    for name, t in zip(("dq", "dk", "dv"), outs):
        t.check(name)
    return tuple(t.t.clone() for t in outs)


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
