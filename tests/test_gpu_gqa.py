"""GPU parity with grouped-query attention (the paper's GQA: several query heads share a key/value head):
K, V, dK, dV have Hkv heads, the selection stays per query head, dK and dV sum over the query heads of a group.
The oracle works one (query head, key/value head) unit at a time, so the grouping is written out here."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

CASES = [
    synth.small_case(32, 64, 8, 8, 4, B=2, H=4, seed=101, backward=True, Hkv=2),
    synth.small_case(64, 64, 16, 16, 2, B=1, H=2, kind="smooth", seed=102, backward=True, Hkv=1),
    synth.small_case(256, 16, 8, 16, 3, B=1, H=4, kind="smooth", seed=103, rlat=8, rlon=1, backward=True, local_groups=True, Hkv=1),
]


def _run_all(w, x):
    p = mb.Params.from_workload(w)
    dx = G.device_inputs(x)
    ws = G.Guarded((max(mb.workspace_bytes(p, op) for op in (mb.OP_SELECT, mb.OP_FWD, mb.OP_BWD)),), torch.uint8)
    idx = G.Guarded((w.B, w.H, w.m, w.topk), torch.int32, fill=-7)
    mb.mosaic_bsa_select(p, dx["q"], dx["k"], block_idx=idx.t, ws=ws.t)
    o = G.Guarded(tuple(dx["q"].shape), torch.bfloat16, fill=float("nan"))
    lse = G.Guarded((w.B, w.H, w.N), torch.float32, fill=float("nan"))
    mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx.t, o=o.t, lse=lse.t, ws=ws.t)
    mb.check_status(ws.t, "fwd")
    dq = G.Guarded(tuple(dx["q"].shape), torch.bfloat16, fill=float("nan"))
    dk = G.Guarded(tuple(dx["k"].shape), torch.bfloat16, fill=float("nan"))
    dv = G.Guarded(tuple(dx["k"].shape), torch.bfloat16, fill=float("nan"))
    mb.mosaic_bsa_bwd(p, dx["q"], dx["k"], dx["v"], o.t, lse.t, dx["do"], idx.t, dq=dq.t, dk=dk.t, dv=dv.t, ws=ws.t)
    mb.check_status(ws.t, "bwd")
    for b_, n_ in ((ws, "workspace"), (idx, "block_idx"), (o, "o"), (lse, "lse"), (dq, "dq"), (dk, "dk"), (dv, "dv")):
        b_.check(n_)
    return p, dx, idx.t, o.t, lse.t, dq.t, dk.t, dv.t


@pytest.mark.parametrize("w", CASES, ids=lambda w: w.name)
def test_grouped_query_attention_matches_oracle(w):
    x = synth.make_inputs(w)
    assert x["k"].shape[1] == w.Hkv and x["q"].shape[1] == w.H
    p, dx, idx, o, lse, dq, dk, dv = _run_all(w, x)
    g = G.geom_of(w)
    r = w.H // w.Hkv
    idx_h = idx.cpu().numpy()
    for b in range(w.B):
        for hk in range(w.Hkv):
            dK_sum, dV_sum = np.zeros((w.N, w.d)), np.zeros((w.N, w.d))
            for h in range(hk * r, (hk + 1) * r):
                want = oracle.select(g, x["q"][b, h], x["k"][b, hk])
                assert np.array_equal(idx_h[b, h], want), f"selection differs (batch {b}, head {h})"
                O, L = oracle.fwd(g, x["q"][b, h], x["k"][b, hk], x["v"][b, hk], want)
                og = o[b, h].float().cpu().numpy().astype(np.float64)
                err = np.abs(og - oracle.to_token_order(g, O))
                assert err.max() <= G.FWD_MAX_ABS and err.mean() <= G.FWD_MEAN_ABS
                assert np.abs(lse[b, h].cpu().numpy() - oracle.to_token_order(g, L)).max() <= G.LSE_ABS
                dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][b, h], x["k"][b, hk], x["v"][b, hk], x["do"][b, h], want)
                G.assert_bwd_close(f"dQ head {h}", dq[b, h], dQ)
                dK_sum += dK
                dV_sum += dV
            G.assert_bwd_close(f"dK kv head {hk}", dk[b, hk], dK_sum)
            G.assert_bwd_close(f"dV kv head {hk}", dv[b, hk], dV_sum)


def test_grouped_query_attention_three_branch_and_static_selection():
    w = CASES[0]
    x = synth.make_inputs(w)
    p = mb.Params.from_workload(w)
    dx = G.device_inputs(x)
    idx = mb.mosaic_bsa_select(p, dx["q"], dx["k"])
    assert torch.equal(idx, mb.mosaic_bsa_select_static(p, dx["q"], dx["k"]))
    gates = np.random.default_rng(104).standard_normal((w.B, w.H, w.N, 3))
    o, lf, ll = mb.mosaic_bsa_fwd_branches(p, dx["q"], dx["k"], dx["v"], idx, torch.from_numpy(gates.astype(np.float32)).cuda())
    g = G.geom_of(w)
    r = w.H // w.Hkv
    idx_h = idx.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            ref = oracle.fwd3(g, x["q"][b, h], x["k"][b, h // r], x["v"][b, h // r], idx_h[b, h],
                              gates[b, h].astype(np.float32).astype(np.float64))
            bound = G.FWD_MAX_ABS * np.maximum(1.0, np.abs(gates[b, h]).sum(axis=1, keepdims=True))
            assert (np.abs(o[b, h].float().cpu().numpy() - ref["o"]) <= bound).all()


def test_paper_stage_one_with_gqa_ratio_four_sampled():
    w = synth.WORKLOADS["hp_nside64_gqa"]
    x = synth.make_inputs(w, with_do=True)
    p, dx, idx, o, lse, dq, dk, dv = _run_all(w, x)
    assert all(torch.isfinite(t.float()).all() for t in (o, dq, dk, dv))
    g = G.geom_of(w)
    idx_h = idx.cpu().numpy()
    hk, r = 1, w.H // w.Hkv
    rng = np.random.default_rng(105)
    blocks = np.unique(np.concatenate([[0, w.m - 1], rng.choice(w.m, size=48, replace=False)])).astype(np.int32)
    qb, kb = np.array([0, 200, w.m - 1], np.int32), np.array([5, 300], np.int32)
    dK_sum, dV_sum = np.zeros((kb.size, w.b, w.d)), np.zeros((kb.size, w.b, w.d))
    for h in range(hk * r, (hk + 1) * r):
        want = oracle.select(g, x["q"][0, h], x["k"][0, hk])
        assert np.array_equal(idx_h[0, h], want)
        O, L = oracle.fwd(g, x["q"][0, h], x["k"][0, hk], x["v"][0, hk], want, blocks)
        tok = np.concatenate([oracle.block_tokens(g, int(j)) for j in blocks])
        err = np.abs(o[0, h].float().cpu().numpy().astype(np.float64)[tok] - O.reshape(-1, w.d))
        assert err.max() <= G.FWD_MAX_ABS and err.mean() <= G.FWD_MEAN_ABS
        dQ, dK, dV = oracle.bwd_blocks(g, x["q"][0, h], x["k"][0, hk], x["v"][0, hk], x["do"][0, h], want, qb, kb)
        for n, i in enumerate(qb):
            G.assert_bwd_close(f"dQ head {h} block {i}", dq[0, h][oracle.block_tokens(g, int(i))], dQ[n])
        dK_sum += dK
        dV_sum += dV
    for n, j in enumerate(kb):
        tj = oracle.block_tokens(g, int(j))
        G.assert_bwd_close(f"dK block {j}", dk[0, hk][tj], dK_sum[n])
        G.assert_bwd_close(f"dV block {j}", dv[0, hk][tj], dV_sum[n])
