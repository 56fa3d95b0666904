"""GPU parity with IEEE binary16 storage (MOSAIC_FLAG_FP16; the paper trains entirely in float16): selection bit for
bit, forward, backward, the three-branch form and the rotary embedding against the oracle decoding the same bits."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

CASES = [
    synth.small_case(32, 64, 8, 8, 4, B=2, H=2, seed=121, backward=True, f16=True),
    synth.small_case(64, 64, 16, 16, 2, B=1, H=2, kind="smooth", seed=122, backward=True, f16=True),
    synth.small_case(256, 16, 8, 16, 3, B=1, H=4, kind="smooth", seed=123, rlat=8, rlon=1, backward=True, local_groups=True,
                     Hkv=2, f16=True),
]


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_select_forward_backward_in_binary16(w):
    x = synth.make_inputs(w)
    dx = G.device_inputs(x, f16=True)
    assert dx["q"].dtype == torch.float16
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    assert o.dtype == torch.float16 and dk.shape == dx["k"].shape
    g = G.geom_of(w)
    assert g.f16
    r = w.H // w.kv_heads
    idx_h = idx.cpu().numpy()
    for b in range(w.B):
        for hk in range(w.kv_heads):
            dK_sum, dV_sum = np.zeros((w.N, w.d)), np.zeros((w.N, w.d))
            for h in range(hk * r, (hk + 1) * r):
                want = oracle.select(g, x["q"][b, h], x["k"][b, hk])
                assert np.array_equal(idx_h[b, h], want), f"selection differs (batch {b}, head {h})"
                O, L = oracle.fwd(g, x["q"][b, h], x["k"][b, hk], x["v"][b, hk], want)
                err = np.abs(o[b, h].float().cpu().numpy().astype(np.float64) - oracle.to_token_order(g, O))
                assert err.max() <= G.FWD_MAX_ABS and err.mean() <= G.FWD_MEAN_ABS
                assert np.abs(lse[b, h].cpu().numpy() - oracle.to_token_order(g, L)).max() <= G.LSE_ABS
                dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][b, h], x["k"][b, hk], x["v"][b, hk], x["do"][b, h], want)
                G.assert_bwd_close(f"dQ head {h}", dq[b, h], dQ)
                dK_sum += dK
                dV_sum += dV
            G.assert_bwd_close(f"dK kv head {hk}", dk[b, hk], dK_sum)
            G.assert_bwd_close(f"dV kv head {hk}", dv[b, hk], dV_sum)


def test_binary16_differs_from_bf16_reading_of_the_same_bits():
    """The flag is honoured: the same bit patterns read as bf16 give another selection input (a guard against a
    path that ignores the flag and happens to pass on symmetric data)."""
    w = CASES[0]
    x = synth.make_inputs(w)
    as_f16 = oracle.widen16(G.geom_of(w), x["q"][0, 0])
    as_bf16 = synth.bf16_bits_to_f32(x["q"][0, 0]).astype(np.float64)
    assert np.abs(as_f16 - as_bf16).max() > 1e-3


def test_three_branch_forward_backward_and_rope_in_binary16():
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=2, seed=124, backward=True, f16=True)
    x = synth.make_inputs(w)
    dx = G.device_inputs(x, f16=True)
    p = mb.Params.from_workload(w)
    idx = G.gpu_select(w, dx)
    idx_h = idx.cpu().numpy()
    gates = np.random.default_rng(125).standard_normal((w.B, w.H, w.N, 3))
    gt = torch.from_numpy(gates.astype(np.float32)).cuda()
    o, lf, ll = mb.mosaic_bsa_fwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gt)
    dq, dk, dv, dg = mb.mosaic_bsa_bwd_branches(p, dx["q"], dx["k"], dx["v"], idx, gt, dx["do"])
    g = G.geom_of(w)
    for h in range(w.H):
        gq = gates[0, h].astype(np.float32).astype(np.float64)
        ref = oracle.fwd3(g, x["q"][0, h], x["k"][0, h], x["v"][0, h], idx_h[0, h], gq)
        bound = G.FWD_MAX_ABS * np.maximum(1.0, np.abs(gq).sum(axis=1, keepdims=True))
        assert (np.abs(o[0, h].float().cpu().numpy() - ref["o"]) <= bound).all()
        dQ, dK, dV, dG = oracle.bwd3(g, x["q"][0, h], x["k"][0, h], x["v"][0, h], x["do"][0, h], idx_h[0, h], gq)
        for name, a, ref_g in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
            tol = G.BWD_MAX_ABS + 2.0 ** -8 * np.abs(ref_g).max()
            assert np.abs(a[0, h].float().cpu().numpy() - ref_g).max() <= tol, name
        do_abs = np.abs(oracle.widen16(g, x["do"][0, h])).sum(axis=-1)
        assert (np.abs(dg[0, h].cpu().numpy() - dG) <= 4 * G.FWD_MEAN_ABS * do_abs[:, None] + 1e-3).all()
    # rotary embedding: binary16 in, binary16 out
    rng = np.random.default_rng(126)
    pos = np.stack([rng.uniform(0, 2 * math.pi, w.N), rng.uniform(-1.5, 1.5, w.N)], axis=1).astype(np.float32)
    qr, kr = mb.mosaic_bsa_rope(p, dx["q"], dx["k"], torch.from_numpy(pos).cuda())
    for name, got, src in (("q", qr, x["q"]), ("k", kr, x["k"])):
        bits = got.view(torch.int16).cpu().numpy().view(np.uint16)
        for h in range(w.H):
            _, want = oracle.rope(g, src[0, h], pos.astype(np.float64))
            a, b_ = bits[0, h].astype(np.int32), want.astype(np.int32)
            oa, ob = np.where(a & 0x8000, -(a & 0x7FFF), a), np.where(b_ & 0x8000, -(b_ & 0x7FFF), b_)
            assert np.abs(oa - ob).max() <= 1 and (oa == ob).mean() >= 0.9999, name
