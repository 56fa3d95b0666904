"""GPU parity in the paper's own layout: blocks of 128 contiguous tokens of a HEALPix NESTED sequence (a 16-wide
view of the sequence, 8 x 16 blocks), local attention inside aligned groups of blocks (the paper's 1024-token
local blocks), at small sizes element by element and at the paper's three stage shapes."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

SMALL = [
    synth.small_case(256, 16, 8, 16, 3, B=1, H=2, kind="smooth", seed=91, rlat=8, rlon=1, backward=True, local_groups=True),
    synth.small_case(56, 16, 8, 16, 2, B=1, H=1, seed=92, rlat=4, rlon=1, backward=True, local_groups=True),     # 7 blocks: ragged last group, odd pairing
    synth.small_case(40, 48, 8, 8, 2, B=1, H=2, kind="smooth", seed=93, rlat=2, rlon=4, backward=True, local_groups=True),  # 2-D groups, ragged both ways
    synth.small_case(64, 64, 16, 16, 2, B=1, H=1, seed=94, rlat=2, rlon=2, backward=True, local_groups=True),    # 16x16 blocks in 2x2 groups
]


@pytest.mark.parametrize("w", SMALL, ids=lambda w: w.name)
def test_group_mode_select_forward_backward(w):
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    want = G.oracle_select_all(w, x)
    assert np.array_equal(idx.cpu().numpy(), want)
    o, lse = G.gpu_fwd(w, dx, idx)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    g = G.geom_of(w)
    for b in range(w.B):
        for h in range(w.H):
            G.compare_fwd_unit(w, x, b, h, want[b, h], o, lse)
            dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], x["do"][b, h], want[b, h])
            for name, got, ref in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
                G.assert_bwd_close(name, got[b, h], ref)


def test_group_mode_three_branch_form():
    w = SMALL[0]
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    p = mb.Params.from_workload(w)
    gates = np.random.default_rng(95).standard_normal((w.B, w.H, w.N, 3))
    gt = torch.from_numpy(gates.astype(np.float32)).cuda()
    o, lf, ll = mb.mosaic_bsa_fwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gt)
    g = G.geom_of(w)
    idx_h = idx.cpu().numpy()
    for h in range(w.H):
        r = oracle.fwd3(g, x["q"][0, h], x["k"][0, h], x["v"][0, h], idx_h[0, h], gates[0, h].astype(np.float32).astype(np.float64))
        bound = G.FWD_MAX_ABS * np.maximum(1.0, np.abs(gates[0, h]).sum(axis=1, keepdims=True))
        assert (np.abs(o[0, h].float().cpu().numpy() - r["o"]) <= bound).all()
        assert np.abs(ll[0, h].cpu().numpy() - r["lse_l"]).max() <= G.LSE_ABS


@pytest.mark.parametrize("name,units,n_blocks", [("hp_nside16", [(0, 0), (0, 19)], 24), ("hp_nside32", [(0, 3)], 96),
                                                 ("hp_nside64", [(0, 0), (0, 11)], 96)])
def test_paper_stage_shapes(name, units, n_blocks):
    w = synth.WORKLOADS[name]
    x = synth.make_inputs(w, with_do=True)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    assert torch.isfinite(o.float()).all() and all(torch.isfinite(t.float()).all() for t in (dq, dk, dv))
    g = G.geom_of(w)
    idx_h = idx.cpu().numpy()
    rng = np.random.default_rng(w.cfg)
    for (b, h) in units:
        want = oracle.select(g, x["q"][b, h], x["k"][b, h])
        assert np.array_equal(idx_h[b, h], want), f"selection differs in unit ({b},{h})"
        blocks = np.unique(np.concatenate([[0, w.m - 1], rng.choice(w.m, size=min(n_blocks, w.m), replace=False)])).astype(np.int32)
        G.compare_fwd_unit(w, x, b, h, want, o, lse, blocks=blocks)
    b, h = units[0]
    qb = np.array([0, w.m // 2, w.m - 1], np.int32)
    indeg = np.bincount(idx_h[b, h][idx_h[b, h] >= 0].ravel(), minlength=w.m)
    kb = np.unique(np.array([0, int(indeg.argmax()), w.m - 1], np.int32))
    dQ, dK, dV = oracle.bwd_blocks(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], x["do"][b, h], idx_h[b, h], qb, kb)
    for n, i in enumerate(qb):
        G.assert_bwd_close(f"dQ block {i}", dq[b, h][oracle.block_tokens(g, int(i))], dQ[n])
    for n, j in enumerate(kb):
        tj = oracle.block_tokens(g, int(j))
        G.assert_bwd_close(f"dK block {j}", dk[b, h][tj], dK[n])
        G.assert_bwd_close(f"dV block {j}", dv[b, h][tj], dV[n])
