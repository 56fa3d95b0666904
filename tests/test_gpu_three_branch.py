"""GPU parity of the three-branch form (compression + selection + local, gated) against the oracle's
`fwd3`, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _run(w, x, idx, gates, scale=0.0):
    p = mb.Params.from_workload(w, scale=scale)
    dx = G.device_inputs(x)
    ws = G.Guarded((mb.workspace_bytes(p, mb.OP_FWD_BRANCHES),), torch.uint8)
    o = G.Guarded(tuple(dx["q"].shape), torch.bfloat16, fill=float("nan"))
    lf = G.Guarded((w.B, w.H, w.N), torch.float32, fill=float("nan"))
    ll = G.Guarded((w.B, w.H, w.N), torch.float32, fill=float("nan"))
    gt = torch.from_numpy(gates.astype(np.float32)).cuda().contiguous()
    mb.mosaic_bsa_fwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gt, o=o.t, lse_fg=lf.t, lse_l=ll.t, ws=ws.t)
    mb.check_status(ws.t, "fwd_branches")
    for b_, n_ in ((ws, "workspace"), (o, "o"), (lf, "lse_fg"), (ll, "lse_l")):
        b_.check(n_)
    return o.t.float().cpu().numpy().astype(np.float64), lf.t.cpu().numpy().astype(np.float64), ll.t.cpu().numpy().astype(np.float64)


def _compare(w, x, idx_h, gates, got, scale=0.0):
    o, lf, ll = got
    g = G.geom_of(w, scale)
    for b in range(w.B):
        for h in range(w.H):
            r = oracle.fwd3(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], idx_h[b, h], gates[b, h].astype(np.float32).astype(np.float64))
            assert np.isfinite(o[b, h]).all(), "unwritten or non-finite output"
            bound = G.FWD_MAX_ABS * np.maximum(1.0, np.abs(gates[b, h]).sum(axis=1, keepdims=True))
            err = np.abs(o[b, h] - r["o"])
            assert (err <= bound).all(), f"o max-abs {err.max():.4g} (unit {b},{h})"
            assert err.mean() <= G.FWD_MEAN_ABS * max(1.0, np.abs(gates[b, h]).sum(axis=1).mean())
            for name, got_l in (("lse_fg", lf[b, h]), ("lse_l", ll[b, h])):
                inf = np.isneginf(r[name])
                assert np.array_equal(inf, np.isneginf(got_l)), name
                assert inf.all() or np.abs(got_l[~inf] - r[name][~inf]).max() <= G.LSE_ABS, name


CASES = [
    (synth.WORKLOADS["c1_tiny"], 0.0),
    (synth.small_case(40, 56, 8, 8, 5, B=1, H=2, kind="smooth", seed=81), 0.0),      # odd block grid
    (synth.small_case(32, 64, 16, 16, 3, B=1, H=1, kind="smooth", seed=82), 0.0),    # 16x16 blocks
    (synth.small_case(136, 160, 8, 8, 8, B=1, H=1, kind="smooth", seed=83), 0.2),    # m = 340: several key chunks in the compression kernel
]


@pytest.mark.parametrize("w,scale", CASES, ids=lambda a: a.name if hasattr(a, "name") else str(a))
def test_three_branch_forward_matches_oracle(w, scale):
    x = synth.make_inputs(w)
    idx = G.gpu_select(w, G.device_inputs(x))
    rng = np.random.default_rng(w.cfg)
    gates = rng.standard_normal((w.B, w.H, w.N, 3))
    _compare(w, x, idx.cpu().numpy(), gates, _run(w, x, idx, gates, scale), scale)


def test_each_branch_alone_and_empty_selection_rows():
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=1, seed=84)
    x = synth.make_inputs(w)
    idx = G.gpu_select(w, G.device_inputs(x))
    idx[0, 0, 5, :] = -1                                   # a query block that selects nothing
    idx[0, 0, 6, 1:] = -1
    idx_h = idx.cpu().numpy()
    for col in range(3):
        gates = np.zeros((1, 1, w.N, 3)); gates[..., col] = 1.0
        got = _run(w, x, idx, gates)
        _compare(w, x, idx_h, gates, got)
    tok5 = oracle.block_tokens(G.geom_of(w), 5)
    assert np.all(got[0][0, 0][tok5] != 0)                  # local branch of block 5 is alive ...
    gates = np.zeros((1, 1, w.N, 3)); gates[..., 1] = 1.0
    o, lf, _ = _run(w, x, idx, gates)
    assert np.all(o[0, 0][tok5] == 0) and np.all(np.isneginf(lf[0, 0][tok5]))   # ... its selection branch is empty


def test_three_branch_without_selection():
    w = synth.small_case(48, 64, 8, 8, 0, B=1, H=2, seed=85)
    x = synth.make_inputs(w)
    idx = torch.zeros((w.B, w.H, w.m, 0), dtype=torch.int32, device="cuda")
    gates = np.random.default_rng(85).standard_normal((w.B, w.H, w.N, 3))
    _compare(w, x, idx.cpu().numpy(), gates, _run(w, x, idx, gates))


def test_three_branch_at_the_1p5_degree_size_sampled_units():
    w = synth.WORKLOADS["c2_1p5deg"]
    x = synth.make_inputs(w)
    idx = G.gpu_select(w, G.device_inputs(x))
    gates = np.random.default_rng(86).standard_normal((w.B, w.H, w.N, 3))
    o, lf, ll = _run(w, x, idx, gates)
    assert np.isfinite(o).all()
    g = G.geom_of(w)
    idx_h = idx.cpu().numpy()
    for h in (0, 5):
        r = oracle.fwd3(g, x["q"][0, h], x["k"][0, h], x["v"][0, h], idx_h[0, h], gates[0, h].astype(np.float32).astype(np.float64))
        bound = G.FWD_MAX_ABS * np.maximum(1.0, np.abs(gates[0, h]).sum(axis=1, keepdims=True))
        assert (np.abs(o[0, h] - r["o"]) <= bound).all()
        assert np.abs(lf[0, h] - r["lse_fg"]).max() <= G.LSE_ABS and np.abs(ll[0, h] - r["lse_l"]).max() <= G.LSE_ABS


# ---------------------------------------------------------------------------------------------------------
# Backward of the three-branch form against the oracle's `bwd3`.
# Tolerances: dQ, dK, dV are sums of two bf16 branch gradients and the compression branch's fp32 share, rounded to
# bf16 once more: three roundings of 2^-9 relative on values of a few units, on top of the attention backward's own
# error, so the bound is the attention backward's (5e-2) plus 2^-8 of the largest reference magnitude.  The gate
# gradients are dot products of dO with bf16 branch outputs whose own error is bounded by the forward tolerance:
# |error| <= sum_c |dO_c| * err_c, taken here as FWD_MEAN_ABS * sum_c |dO_c| * 4 (errors do not add coherently).
BWD3_CASES = [
    synth.small_case(32, 64, 8, 8, 4, B=1, H=2, seed=91, backward=True),
    synth.small_case(40, 56, 8, 8, 5, B=1, H=1, kind="smooth", seed=92, backward=True),       # odd block grid
    synth.small_case(32, 64, 16, 16, 3, B=1, H=1, kind="smooth", seed=93, backward=True),     # 16x16 blocks
    synth.small_case(256, 16, 8, 16, 3, B=1, H=4, kind="smooth", seed=94, rlat=8, rlon=1, backward=True,
                     local_groups=True, Hkv=2),                                               # the paper's layout, GQA
]


def _run_bwd3(w, x, idx, gates):
    p = mb.Params.from_workload(w)
    dx = G.device_inputs(x)
    ws = G.Guarded((mb.workspace_bytes(p, mb.OP_BWD_BRANCHES),), torch.uint8)
    dq = G.Guarded(tuple(dx["q"].shape), torch.bfloat16, fill=float("nan"))
    dk = G.Guarded(tuple(dx["k"].shape), torch.bfloat16, fill=float("nan"))
    dv = G.Guarded(tuple(dx["k"].shape), torch.bfloat16, fill=float("nan"))
    dg = G.Guarded((w.B, w.H, w.N, 3), torch.float32, fill=float("nan"))
    gt = torch.from_numpy(gates.astype(np.float32)).cuda().contiguous()
    mb.mosaic_bsa_bwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gt, dx["do"], dq=dq.t, dk=dk.t, dv=dv.t, dgates=dg.t, ws=ws.t)
    mb.check_status(ws.t, "bwd_branches")
    for b_, n_ in ((ws, "workspace"), (dq, "dq"), (dk, "dk"), (dv, "dv"), (dg, "dgates")):
        b_.check(n_)
    return [t.t.float().cpu().numpy().astype(np.float64) for t in (dq, dk, dv, dg)]


def _compare_bwd3(w, x, idx_h, gates, got):
    dq, dk, dv, dg = got
    g = G.geom_of(w)
    r = w.H // w.kv_heads
    do_abs = np.abs(synth.bf16_bits_to_f32(x["do"]).astype(np.float64)).sum(axis=-1)     # [B, H, N]
    for b in range(w.B):
        for hk in range(w.kv_heads):
            dK_sum, dV_sum = np.zeros((w.N, w.d)), np.zeros((w.N, w.d))
            for h in range(hk * r, (hk + 1) * r):
                gq = gates[b, h].astype(np.float32).astype(np.float64)
                dQ, dK, dV, dG = oracle.bwd3(g, x["q"][b, h], x["k"][b, hk], x["v"][b, hk], x["do"][b, h], idx_h[b, h], gq)
                tol = G.BWD_MAX_ABS + 2.0 ** -8 * np.abs(dQ).max()
                assert np.isfinite(dq[b, h]).all() and np.abs(dq[b, h] - dQ).max() <= tol, (h, np.abs(dq[b, h] - dQ).max(), tol)
                bound = 4 * G.FWD_MEAN_ABS * do_abs[b, h][:, None] + 1e-3
                assert np.isfinite(dg[b, h]).all() and (np.abs(dg[b, h] - dG) <= bound).all(), (h, np.abs(dg[b, h] - dG).max())
                dK_sum += dK
                dV_sum += dV
            for name, a, ref in (("dK", dk[b, hk], dK_sum), ("dV", dv[b, hk], dV_sum)):
                tol = G.BWD_MAX_ABS + 2.0 ** -8 * np.abs(ref).max()
                assert np.isfinite(a).all() and np.abs(a - ref).max() <= tol, (name, hk, np.abs(a - ref).max(), tol)


@pytest.mark.parametrize("w", BWD3_CASES, ids=lambda w: w.name)
def test_three_branch_backward_matches_oracle(w):
    x = synth.make_inputs(w)
    idx = G.gpu_select(w, G.device_inputs(x))
    gates = np.random.default_rng(w.cfg).standard_normal((w.B, w.H, w.N, 3))
    _compare_bwd3(w, x, idx.cpu().numpy(), gates, _run_bwd3(w, x, idx, gates))


def test_three_branch_backward_one_branch_at_a_time_and_empty_rows():
    """Each gate alone isolates one branch (the compression branch alone reaches every key and value of the unit);
    a query block that selects nothing and key blocks nobody selected get zero from the selection branch."""
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=1, seed=95, backward=True)
    x = synth.make_inputs(w)
    idx = G.gpu_select(w, G.device_inputs(x))
    idx[0, 0, 5, :] = -1
    idx[0, 0, 6, 1:] = -1
    j0 = int(idx[0, 0, 0, 0])
    idx[idx == j0] = -1                                    # a key block that nobody selects
    idx_h = idx.cpu().numpy()
    for col in range(3):
        gates = np.zeros((1, 1, w.N, 3)); gates[..., col] = 1.0
        got = _run_bwd3(w, x, idx, gates)
        _compare_bwd3(w, x, idx_h, gates, got)
        if col == 0:
            assert (np.abs(got[1][0, 0]).max(axis=1) > 0).all() and (np.abs(got[2][0, 0]).max(axis=1) > 0).all()
        if col == 1:
            tok5 = oracle.block_tokens(G.geom_of(w), 5)
            assert np.all(got[0][0, 0][tok5] == 0)
            tu = oracle.block_tokens(G.geom_of(w), j0)
            assert np.all(got[1][0, 0][tu] == 0) and np.all(got[2][0, 0][tu] == 0)


def test_three_branch_backward_at_the_papers_stage_three_shape_in_binary16():
    """The whole stage-3 problem (nside 16: N = 3072, 20 heads, 128-token blocks in 1024-token local groups, 4 selected
    blocks) with the paper's GQA ratio 4 and binary16 storage, as one launch sequence; two heads of two different
    key/value heads against the oracle."""
    base = synth.WORKLOADS["hp_nside16"]
    w = synth.Workload(**{**base.__dict__, "name": "hp_nside16_gqa_f16", "Hkv": 5, "f16": True, "backward": True})
    x = synth.make_inputs(w)
    dx = G.device_inputs(x, f16=True)
    p = mb.Params.from_workload(w)
    idx = G.gpu_select(w, dx)
    idx_h = idx.cpu().numpy()
    gates = np.random.default_rng(96).standard_normal((w.B, w.H, w.N, 3))
    gt = torch.from_numpy(gates.astype(np.float32)).cuda()
    ws = G.Guarded((mb.workspace_bytes(p, mb.OP_BWD_BRANCHES),), torch.uint8)
    dq, dk, dv, dg = mb.mosaic_bsa_bwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gt, dx["do"], ws=ws.t)
    mb.check_status(ws.t, "bwd_branches")
    ws.check("workspace")
    assert all(torch.isfinite(t.float()).all() for t in (dq, dk, dv, dg))
    g = G.geom_of(w)
    r = w.H // w.kv_heads
    for hk in (0, 4):
        dK_sum, dV_sum = np.zeros((w.N, w.d)), np.zeros((w.N, w.d))
        for h in range(hk * r, (hk + 1) * r):
            assert np.array_equal(idx_h[0, h], oracle.select(g, x["q"][0, h], x["k"][0, hk]))
            gq = gates[0, h].astype(np.float32).astype(np.float64)
            dQ, dK, dV, dG = oracle.bwd3(g, x["q"][0, h], x["k"][0, hk], x["v"][0, hk], x["do"][0, h], idx_h[0, h], gq)
            tol = G.BWD_MAX_ABS + 2.0 ** -8 * np.abs(dQ).max()
            assert np.abs(dq[0, h].float().cpu().numpy() - dQ).max() <= tol
            do_abs = np.abs(oracle.widen16(g, x["do"][0, h])).sum(axis=-1)
            assert (np.abs(dg[0, h].cpu().numpy() - dG) <= 4 * G.FWD_MEAN_ABS * do_abs[:, None] + 1e-3).all()
            dK_sum += dK
            dV_sum += dV
        for name, a, ref in (("dK", dk, dK_sum), ("dV", dv, dV_sum)):
            tol = G.BWD_MAX_ABS + 2.0 ** -8 * np.abs(ref).max()
            assert np.abs(a[0, hk].float().cpu().numpy() - ref).max() <= tol, name


def test_three_branch_backward_without_selection_and_at_the_1p5_degree_size():
    """Top-k 0: the selection branch is absent, its gate gradient is zero and the other two branches carry the whole
    gradient.  Then the whole 1.5-degree problem as one launch sequence, two units against the oracle."""
    w0 = synth.small_case(48, 64, 8, 8, 0, B=1, H=2, seed=97, backward=True)
    x0 = synth.make_inputs(w0)
    idx0 = torch.zeros((w0.B, w0.H, w0.m, 0), dtype=torch.int32, device="cuda")
    gates0 = np.random.default_rng(97).standard_normal((w0.B, w0.H, w0.N, 3))
    got0 = _run_bwd3(w0, x0, idx0, gates0)
    _compare_bwd3(w0, x0, idx0.cpu().numpy(), gates0, got0)
    assert np.all(got0[3][..., 1] == 0)

    base = synth.WORKLOADS["c2_1p5deg"]
    w = synth.Workload(**{**base.__dict__, "backward": True})
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    p = mb.Params.from_workload(w)
    idx = G.gpu_select(w, dx)
    idx_h = idx.cpu().numpy()
    gates = np.random.default_rng(98).standard_normal((w.B, w.H, w.N, 3))
    gt = torch.from_numpy(gates.astype(np.float32)).cuda()
    dq, dk, dv, dg = mb.mosaic_bsa_bwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gt, dx["do"])
    assert all(torch.isfinite(t.float()).all() for t in (dq, dk, dv, dg))
    g = G.geom_of(w)
    for h in (1, 6):
        gq = gates[0, h].astype(np.float32).astype(np.float64)
        dQ, dK, dV, dG = oracle.bwd3(g, x["q"][0, h], x["k"][0, h], x["v"][0, h], x["do"][0, h], idx_h[0, h], gq)
        for name, a, ref in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
            tol = G.BWD_MAX_ABS + 2.0 ** -8 * np.abs(ref).max()
            assert np.abs(a[0, h].float().cpu().numpy() - ref).max() <= tol, (name, h)
        do_abs = np.abs(synth.bf16_bits_to_f32(x["do"][0, h]).astype(np.float64)).sum(axis=-1)
        assert (np.abs(dg[0, h].cpu().numpy() - dG) <= 4 * G.FWD_MEAN_ABS * do_abs[:, None] + 1e-3).all()
