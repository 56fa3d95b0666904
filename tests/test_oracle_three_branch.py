"""Pins for the oracle's three-branch form (compression + selection + local, gated): each branch against a
textbook routine written here, the gated sum, the link to the union form that the other pins cover, and the
backward against finite differences (including the gradient that reaches the routing scores through the
compression branch)."""
import math

import numpy as np

import oracle
from oracle import Geom
from paper_2604_16429_b200 import synth
from tests.helpers import block_tokens, dense_attention, f64, local_blocks, quantised


def rand_bits(rng, N, d, sigma=1.0):
    return synth.to_bf16_bits((sigma * rng.standard_normal((N, d))).astype(np.float32))


def masked_dense(qf, kf, vf, toks, scale):
    """Softmax attention of the rows of qf over the key/value rows `toks` (textbook, fp64)."""
    o, lse = dense_attention(qf, kf[toks], vf[toks], scale)
    return o, lse


def test_each_branch_matches_a_textbook_routine_and_the_gated_sum():
    rng = np.random.default_rng(31)
    g = Geom(32, 48, d=8, bh=8, bw=8, topk=3)                      # 4 x 6 blocks
    q, k, v = (rand_bits(rng, g.N, g.d) for _ in range(3))
    gates = rng.standard_normal((g.N, 3))
    idx = oracle.select(g, q, k)
    r = oracle.fwd3(g, q, k, v, idx, gates)
    qf, kf, vf = f64(q), f64(k), f64(v)
    sc = 1 / math.sqrt(g.d)
    tok = [block_tokens(g.nlon, g.bh, g.bw, g.nbw, j) for j in range(g.m)]
    # compression: dense attention on the block means, the same vector for every token of a block
    qm, km, vm = (np.stack([x[t].mean(0) for t in tok]) for x in (qf, kf, vf))
    ocg, _ = dense_attention(qm, km, vm, sc)
    x = sc * qm @ km.T
    ab = np.exp(x - x.max(1, keepdims=True)); ab /= ab.sum(1, keepdims=True)
    assert np.abs(r["abar"] - ab).max() < 1e-6 and np.abs(r["abar"].sum(1) - 1).max() < 1e-12
    for i in range(g.m):
        assert np.abs(r["o_cg"][tok[i]] - ocg[i]).max() < 1e-6
        assert np.abs(r["o_cg"][tok[i]] - r["o_cg"][tok[i][0]]).max() == 0.0
        # selection and local: softmax attention over the tokens of the selected / neighbouring blocks
        sel = np.concatenate([tok[j] for j in idx[i] if j >= 0])
        loc = np.concatenate([tok[j] for j in sorted(local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw))])
        for name, lname, toks in (("o_fg", "lse_fg", sel), ("o_l", "lse_l", loc)):
            o, lse = masked_dense(qf[tok[i]], kf, vf, toks, sc)
            assert np.abs(r[name][tok[i]] - o).max() < 1e-12
            assert np.abs(r[lname][tok[i]] - lse).max() < 1e-12
    want = gates[:, :1] * r["o_cg"] + gates[:, 1:2] * r["o_fg"] + gates[:, 2:] * r["o_l"]
    assert np.abs(r["o"] - want).max() < 1e-13
    assert np.abs(r["o_cg"]).max() > 1e-3 and np.abs(r["o_fg"]).max() > 1e-3


def test_link_to_the_union_form_and_special_cases():
    rng = np.random.default_rng(32)
    g = Geom(32, 64, d=8, bh=8, bw=8, topk=4)
    q, k, v = (rand_bits(rng, g.N, g.d) for _ in range(3))
    idx = oracle.select(g, q, k)
    ones = np.ones((g.N, 3))
    r = oracle.fwd3(g, q, k, v, idx, ones)
    # one softmax over the union = the two branch outputs weighted by their normalisers
    O, L = oracle.fwd(g, q, k, v, idx)
    Ou, Lu = oracle.to_token_order(g, O), oracle.to_token_order(g, L)
    zf, zl = np.exp(r["lse_fg"] - Lu), np.exp(r["lse_l"] - Lu)
    assert np.abs(zf + zl - 1).max() < 1e-12
    assert np.abs(zf[:, None] * r["o_fg"] + zl[:, None] * r["o_l"] - Ou).max() < 1e-12
    # gates (0, 0, 1) and nothing selected: the union form with top-k 0
    g0 = Geom(32, 64, d=8, bh=8, bw=8, topk=0)
    idx0 = np.zeros((g0.m, 0), np.int32)
    gl = np.zeros((g.N, 3)); gl[:, 2] = 1.0
    r0 = oracle.fwd3(g0, q, k, v, idx0, gl)
    O0, _ = oracle.fwd(g0, q, k, v, idx0)
    assert np.array_equal(r0["o"], oracle.to_token_order(g0, O0))
    assert np.all(r0["o_fg"] == 0.0) and np.all(np.isneginf(r0["lse_fg"]))
    # top-k covering every non-local block: selection and local together are dense attention
    gd = Geom(16, 24, d=8, bh=8, bw=8, topk=6)
    q, k, v = (rand_bits(rng, gd.N, gd.d) for _ in range(3))
    rd = oracle.fwd3(gd, q, k, v, oracle.select(gd, q, k), np.ones((gd.N, 3)))
    od, ld = dense_attention(f64(q), f64(k), f64(v), 1 / math.sqrt(gd.d))
    zf, zl = np.exp(rd["lse_fg"] - ld), np.exp(rd["lse_l"] - ld)
    assert np.abs(zf[:, None] * rd["o_fg"] + zl[:, None] * rd["o_l"] - od).max() < 1e-12


def _loss3(g, q, k, v, do, idx, gates):
    return float((oracle.fwd3(g, q, k, v, idx, gates)["o"] * f64(do)).sum())


def test_backward_finite_differences_through_all_three_branches():
    rng = np.random.default_rng(33)
    g = Geom(16, 16, d=4, bh=4, bw=4, topk=2)                       # m = 16; sums of 16 multiples of 1/16 are exact in fp32
    q, k, v, do = (quantised((g.N, g.d), rng) for _ in range(4))
    gates = rng.standard_normal((g.N, 3))
    idx = oracle.select(g, q, k)                                   # held constant below
    dQ, dK, dV, dG = oracle.bwd3(g, q, k, v, do, idx, gates)
    args = {"q": q, "k": k, "v": v}
    grads = {"q": dQ, "k": dK, "v": dV}
    for name in ("q", "k", "v"):
        for _ in range(8):
            t, c = int(rng.integers(g.N)), int(rng.integers(g.d))
            est = []
            for h in (1 / 32, 1 / 64):
                vals = {}
                for sgn in (+1, -1):
                    pert = synth.bf16_bits_to_f32(args[name]).copy()
                    pert[t, c] += np.float32(sgn * h)
                    bits = synth.to_bf16_bits(pert)
                    assert np.array_equal(synth.bf16_bits_to_f32(bits), pert)
                    a = dict(args); a[name] = bits
                    vals[sgn] = _loss3(g, a["q"], a["k"], a["v"], do, idx, gates)
                est.append((vals[1] - vals[-1]) / (2 * h))
            fd = (4 * est[1] - est[0]) / 3
            assert abs(fd - grads[name][t, c]) < 2e-5 * max(1.0, abs(fd)), (name, t, c, fd, grads[name][t, c])
    # the output is linear in the gates
    r = oracle.fwd3(g, q, k, v, idx, gates)
    for x, name in enumerate(("o_cg", "o_fg", "o_l")):
        assert np.abs(dG[:, x] - (f64(do) * r[name]).sum(1)).max() < 1e-12
    # only the compression branch open: the gradient reaches every key and value of the unit (routing scores)
    gc = np.zeros((g.N, 3)); gc[:, 0] = 1.0
    dQc, dKc, dVc, _ = oracle.bwd3(g, q, k, v, do, idx, gc)
    assert (np.abs(dKc).max(axis=1) > 0).all() and (np.abs(dVc).max(axis=1) > 0).all()
    t0 = block_tokens(g.nlon, g.bh, g.bw, g.nbw, 5)
    assert np.abs(dKc[t0] - dKc[t0[0]]).max() == 0.0               # the mean spreads it evenly inside a block
