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
    _check_units(w, x, idx, o, lse, [(0, 0), (0, 3), (0, 7)], n_blocks=160, seed=2)


def test_c4_training_shape_forward_and_backward():
    w = synth.WORKLOADS["c4_1p5deg_train"]
    x = synth.make_inputs(w)
    dx, idx, o, lse = _run_forward(w, x)
    _check_properties(w, x, o, lse)
    _check_units(w, x, idx, o, lse, [(0, 0), (3, 15)], n_blocks=64, seed=4)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    for t in (dq, dk, dv):
        assert torch.isfinite(t.float()).all()
    g = G.geom_of(w)
    b, h = 2, 5                                                 # one whole unit against the oracle
    want = oracle.select(g, x["q"][b, h], x["k"][b, h])
    dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], x["do"][b, h], want)
    for name, got, ref in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
        G.assert_bwd_close(name, got[b, h], ref)


def test_c3_ensemble_full_size():
    w = synth.WORKLOADS["c3_1p5deg_ens24"]
    x = synth.make_inputs(w)
    dx, idx, o, lse = _run_forward(w, x)
    _check_properties(w, x, o, lse)
    _check_units(w, x, idx, o, lse, [(0, 0), (11, 4), (23, 7)], n_blocks=128, seed=3)


def test_c5_0p25deg_full_size():
    w = synth.WORKLOADS["c5_0p25deg"]
    x = synth.make_inputs(w)
    dx, idx, o, lse = _run_forward(w, x)
    _check_properties(w, x, o, lse)
    _check_units(w, x, idx, o, lse, [(0, 1), (0, 6)], n_blocks=64, seed=5)


def test_c5_0p25deg_backward_sampled_blocks():
    """Backward at the 0.25-degree size (16x16 blocks, four chunks per block): dQ of sampled query blocks and
    dK, dV of sampled key blocks of one unit against the oracle, the most-selected key block of the unit among
    them (its list of connected query blocks is longer than one list buffer of the key-stationary kernel)."""
    w = synth.WORKLOADS["c5_0p25deg"]
    x = synth.make_inputs(w, with_do=True)
    dx, idx, o, lse = _run_forward(w, x)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    for t in (dq, dk, dv):
        assert torch.isfinite(t.float()).all()
    g = G.geom_of(w)
    b, h = 0, 2
    want = oracle.select(g, x["q"][b, h], x["k"][b, h])
    assert np.array_equal(idx.cpu().numpy()[b, h], want)
    indeg = np.bincount(want[want >= 0].ravel(), minlength=w.m)
    popular = int(indeg.argmax())
    assert indeg[popular] + 9 > 64, "no key block with a long list in this unit"
    rng = np.random.default_rng(55)
    qb = np.unique(np.concatenate([[0, w.m - 1], rng.choice(w.m, size=6, replace=False)])).astype(np.int32)
    kb = np.unique(np.concatenate([[popular, 0], rng.choice(w.m, size=2, replace=False)])).astype(np.int32)
    dQ, dK, dV = oracle.bwd_blocks(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], x["do"][b, h], want, qb, kb)
    for n, i in enumerate(qb):
        G.assert_bwd_close(f"dQ block {i}", dq[b, h][oracle.block_tokens(g, int(i))], dQ[n])
    for n, j in enumerate(kb):
        tj = oracle.block_tokens(g, int(j))
        G.assert_bwd_close(f"dK block {j}", dk[b, h][tj], dK[n])
        G.assert_bwd_close(f"dV block {j}", dv[b, h][tj], dV[n])
