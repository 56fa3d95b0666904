"""GPU parity at the full benchmark sizes, in the launch configuration `bench.py` times (whole workload in
one call).  The oracle cannot compute these sizes whole in seconds, so selection is compared in full for a
few units and attention on sampled query blocks of sampled units; the rest of the output is checked by
properties that hold at any size (everything written, finite, rows of the convex hull of V)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _run_forward(w, x):
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx)
    return dx, idx, o, lse


def _check_units(w, x, idx, o, lse, units, n_blocks, seed):
    rng = np.random.default_rng(seed)
    g = G.geom_of(w)
    idx_h = idx.cpu().numpy()
    for (b, h) in units:
        want = oracle.select(g, x["q"][b, h], x["k"][b, h])
        assert np.array_equal(idx_h[b, h], want), f"selection differs in unit ({b},{h})"
        blocks = np.sort(rng.choice(w.m, size=min(n_blocks, w.m), replace=False)).astype(np.int32)
        blocks[0], blocks[-1] = 0, w.m - 1                      # always include the two polar corners
        G.compare_fwd_unit(w, x, b, h, want, o, lse, blocks=np.unique(blocks))


def _check_properties(w, x, o, lse):
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all(), "unwritten or non-finite output"
    # every output row is a convex combination of value rows: per unit and channel it stays inside V's range
    v = mb.from_bits(x["v"]).float()
    lo, hi = v.amin(dim=2, keepdim=True), v.amax(dim=2, keepdim=True)
    of = o.float()
    assert (of >= lo - 2e-2).all() and (of <= hi + 2e-2).all()


def test_c2_1p5deg_full_size():
    w = synth.WORKLOADS["c2_1p5deg"]
    x = synth.make_inputs(w)
    dx, idx, o, lse = _run_forward(w, x)
    _check_properties(w, x, o, lse)
    _check_units(w, x, idx, o, lse, [(0, 0), (0, 3), (0, 7)], n_blocks=48, seed=2)


def test_c4_training_shape_forward_and_backward():
    w = synth.WORKLOADS["c4_1p5deg_train"]
    x = synth.make_inputs(w)
    dx, idx, o, lse = _run_forward(w, x)
    _check_properties(w, x, o, lse)
    _check_units(w, x, idx, o, lse, [(0, 0), (3, 15)], n_blocks=32, seed=4)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    for t in (dq, dk, dv):
        assert torch.isfinite(t.float()).all()
    g = G.geom_of(w)
    b, h = 2, 5                                                 # one whole unit against the oracle
    want = oracle.select(g, x["q"][b, h], x["k"][b, h])
    dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], x["do"][b, h], want)
    for name, got, ref in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
        err = np.abs(got[b, h].float().cpu().numpy().astype(np.float64) - ref)
        assert err.max() <= G.BWD_MAX_ABS, f"{name} max-abs {err.max():.4g}"


def test_c3_ensemble_full_size():
    w = synth.WORKLOADS["c3_1p5deg_ens24"]
    x = synth.make_inputs(w)
    dx, idx, o, lse = _run_forward(w, x)
    _check_properties(w, x, o, lse)
    _check_units(w, x, idx, o, lse, [(0, 0), (11, 4), (23, 7)], n_blocks=24, seed=3)


def test_c5_0p25deg_full_size():
    w = synth.WORKLOADS["c5_0p25deg"]
    x = synth.make_inputs(w)
    dx, idx, o, lse = _run_forward(w, x)
    _check_properties(w, x, o, lse)
    _check_units(w, x, idx, o, lse, [(0, 1), (0, 6)], n_blocks=6, seed=5)
