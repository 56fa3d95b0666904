"""Pins for the fp64 oracle: each test checks it against something that is not the oracle
(a textbook routine, brute force, a closed form or an invariant), chosen so that a dropped
term, a wrong sign or index, or a transposed operand fails at least one of them."""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from oracle import Geom
from paper_2604_16429_b200 import flops, synth
from tests.helpers import block_tokens, dense_attention, f64, local_blocks, quantised


def rand_bits(rng, N, d, sigma=1.0):
    return synth.to_bf16_bits((sigma * rng.standard_normal((N, d))).astype(np.float32))


# ------------------------------------------------------------------ geometry (local set)

def test_local_set_interior_polar_and_wrap():
    g = Geom(32, 64, bh=8, bw=8)                     # 4 x 8 blocks
    nbw = g.nbw
    assert sorted(oracle.local_set(g, 1 * nbw + 3)) == sorted(
        [y * nbw + x for y in (0, 1, 2) for x in (2, 3, 4)])
    # polar row: clamping folds the missing row onto the own row -> 6 blocks, each once
    assert sorted(oracle.local_set(g, 0 * nbw + 3)) == sorted([y * nbw + x for y in (0, 1) for x in (2, 3, 4)])
    assert sorted(oracle.local_set(g, 3 * nbw + 3)) == sorted([y * nbw + x for y in (2, 3) for x in (2, 3, 4)])
    # periodic longitude
    assert sorted(oracle.local_set(g, 1 * nbw + 0)) == sorted([y * nbw + x for y in (0, 1, 2) for x in (7, 0, 1)])
    assert sorted(oracle.local_set(g, 1 * nbw + 7)) == sorted([y * nbw + x for y in (0, 1, 2) for x in (6, 7, 0)])


@pytest.mark.parametrize("nlat,nlon,bh,bw,rlat,rlon", [(16, 16, 8, 8, 1, 1), (8, 16, 8, 8, 1, 1),
                                                       (32, 8, 8, 8, 1, 1), (40, 48, 8, 8, 2, 1),
                                                       (24, 24, 8, 8, 0, 0)])
def test_local_set_matches_set_definition(nlat, nlon, bh, bw, rlat, rlon):
    g = Geom(nlat, nlon, bh=bh, bw=bw, rlat=rlat, rlon=rlon)
    for i in range(g.m):
        got = oracle.local_set(g, i)
        assert len(got) == len(set(got))                                       # a set: no repeats
        assert set(got) == local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw, rlat, rlon)


# ------------------------------------------------------------------ pooling and selection

def test_pool_is_block_sum():
    rng = np.random.default_rng(1)
    g = Geom(16, 24, d=8, bh=4, bw=8)
    x = rand_bits(rng, g.N, g.d)
    got = oracle.pool(g, x)
    xf = f64(x)
    for j in range(g.m):
        ref = xf[block_tokens(g.nlon, g.bh, g.bw, g.nbw, j)].sum(axis=0)       # exact in fp64 here
        assert np.array_equal(got[j], ref.astype(np.float32))


@pytest.mark.parametrize("nlat,nlon,bh,bw,topk,d", [(32, 64, 8, 8, 4, 16), (24, 40, 4, 8, 5, 8),
                                                    (16, 32, 8, 8, 3, 64), (32, 32, 8, 8, 30, 8)])
def test_selection_brute_force(nlat, nlon, bh, bw, topk, d):
    rng = np.random.default_rng(nlat * 7 + topk)
    g = Geom(nlat, nlon, d=d, bh=bh, bw=bw, topk=topk)
    q, k = rand_bits(rng, g.N, d), rand_bits(rng, g.N, d)
    idx = oracle.select(g, q, k)
    qf, kf = f64(q), f64(k)
    tok = [block_tokens(nlon, bh, bw, g.nbw, j) for j in range(g.m)]
    pq = [[np.float32(math.fsum(qf[tok[j], c])) for c in range(d)] for j in range(g.m)]
    pk = [[np.float32(math.fsum(kf[tok[j], c])) for c in range(d)] for j in range(g.m)]
    for i in range(g.m):
        loc = local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw)
        cand = []
        for j in range(g.m):
            if j in loc:
                continue
            s = 0.0
            for c in range(d):
                s = s + float(pq[i][c]) * float(pk[j][c])
            cand.append((-s, j))
        cand.sort()
        want = [j for _, j in cand[:topk]] + [-1] * max(0, topk - len(cand))
        assert idx[i].tolist() == want, (i, idx[i], want)


def _blocks_from_pooled(g, pooled):
    """[N,d] bf16 bits whose block sums are `pooled` ([m,d], small integers): the first
    token of each block carries the whole sum, the rest are zero."""
    x = np.zeros((g.N, g.d), np.float32)
    for j in range(g.m):
        x[block_tokens(g.nlon, g.bh, g.bw, g.nbw, j)[0]] = pooled[j]
    return synth.to_bf16_bits(x)


def test_selection_known_winners_and_ties():
    g = Geom(32, 64, d=8, bh=8, bw=8, topk=3)        # 4 x 8 blocks, m = 32
    pq = np.zeros((g.m, g.d), np.float32)
    pk = np.zeros((g.m, g.d), np.float32)
    pq[:, 0] = 1.0                                   # every query block scores key block j by pk[j, 0]
    i = 1 * g.nbw + 1                                # interior block; local = rows 0..2, cols 0..2
    pk[:, 0] = -1.0
    pk[3 * g.nbw + 5, 0] = 5.0                       # clear winner
    pk[0 * g.nbw + 6, 0] = 2.0                       # exact tie ...
    pk[2 * g.nbw + 4, 0] = 2.0                       # ... resolved towards the lower id
    pk[1 * g.nbw + 1, 0] = 9.0                       # own block: best score but local -> never a candidate
    pk[0 * g.nbw + 2, 0] = 8.0                       # neighbour: local too
    idx = oracle.select(g, _blocks_from_pooled(g, pq), _blocks_from_pooled(g, pk))
    assert idx[i].tolist() == [3 * g.nbw + 5, 0 * g.nbw + 6, 2 * g.nbw + 4]
    # a block far from (0,2) and (1,1) sees them as ordinary candidates
    far = 3 * g.nbw + 5
    assert idx[far].tolist() == [1 * g.nbw + 1, 0 * g.nbw + 2, 0 * g.nbw + 6]
    # all scores equal -> the lowest non-local ids, in order
    pk[:, 0] = 1.0
    idx = oracle.select(g, _blocks_from_pooled(g, pq), _blocks_from_pooled(g, pk))
    for i in range(g.m):
        loc = local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw)
        assert idx[i].tolist() == [j for j in range(g.m) if j not in loc][:3]
    # signed zeros compare equal: a -0 score does not lose to +0 with a higher id
    pk[:, 0] = 0.0
    pkb = _blocks_from_pooled(g, pk)
    pkb[block_tokens(g.nlon, g.bh, g.bw, g.nbw, 3)[0], 0] = 0x8000          # -0.0 in block 3
    idx = oracle.select(g, _blocks_from_pooled(g, pq), pkb)
    i = 3 * g.nbw + 6
    loc = local_blocks(3, 6, g.nbh, g.nbw)
    assert idx[i].tolist() == [j for j in range(g.m) if j not in loc][:3]


def test_selection_nan_score_ranks_below_every_number():
    """A key block whose pooled sum is NaN gives a NaN score: it ranks after every finite or infinite
    score (so it is chosen only when fewer than top-k other candidates exist), lower id first among NaNs."""
    g = Geom(32, 64, d=8, bh=8, bw=8, topk=3)        # 4 x 8 blocks, m = 32
    pq = np.zeros((g.m, g.d), np.float32)
    pk = np.zeros((g.m, g.d), np.float32)
    pq[:, 0] = 1.0
    pk[:, 0] = -np.arange(g.m, dtype=np.float32)     # block 0 best, block 31 worst
    i = 1 * g.nbw + 1                                # local = rows 0..2, cols 0..2
    loc = local_blocks(1, 1, g.nbh, g.nbw)
    cand = [j for j in range(g.m) if j not in loc]
    kb = _blocks_from_pooled(g, pk)
    kb[block_tokens(g.nlon, g.bh, g.bw, g.nbw, cand[0])[0], 0] = 0x7FC0      # bf16 NaN in the best candidate
    idx = oracle.select(g, _blocks_from_pooled(g, pq), kb)
    assert idx[i].tolist() == cand[1:4]                                     # the NaN block is passed over
    # -inf is a number: it still ranks above NaN
    g2 = Geom(16, 40, d=8, bh=8, bw=8, topk=4)       # 2 x 5 blocks: 4 candidates per row
    pq2 = np.zeros((g2.m, g2.d), np.float32); pq2[:, 0] = 1.0
    pk2 = np.zeros((g2.m, g2.d), np.float32); pk2[:, 0] = np.arange(g2.m, dtype=np.float32)
    kb2 = _blocks_from_pooled(g2, pk2)
    loc2 = local_blocks(0, 0, g2.nbh, g2.nbw)
    cand2 = [j for j in range(g2.m) if j not in loc2]                        # [2, 3, 7, 8]
    kb2[block_tokens(g2.nlon, g2.bh, g2.bw, g2.nbw, cand2[3])[0], 0] = 0x7FC0   # NaN (would be the best)
    kb2[block_tokens(g2.nlon, g2.bh, g2.bw, g2.nbw, cand2[1])[0], 0] = 0x7FC0   # NaN
    kb2[block_tokens(g2.nlon, g2.bh, g2.bw, g2.nbw, cand2[2])[0], 0] = 0xFF80   # -inf
    idx2 = oracle.select(g2, _blocks_from_pooled(g2, pq2), kb2)
    assert idx2[0].tolist() == [cand2[0], cand2[2], cand2[1], cand2[3]]      # finite, -inf, then NaNs by id


def test_selection_padding_when_few_candidates():
    g = Geom(16, 32, d=8, bh=8, bw=8, topk=4)        # 2 x 4 blocks: local covers 6 of 8
    rng = np.random.default_rng(3)
    idx = oracle.select(g, rand_bits(rng, g.N, g.d), rand_bits(rng, g.N, g.d))
    for i in range(g.m):
        loc = local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw)
        row = idx[i].tolist()
        assert row[2:] == [-1, -1] and set(row[:2]) == set(range(g.m)) - loc


def test_selection_scale_invariance():
    rng = np.random.default_rng(4)
    g = Geom(32, 64, d=16, bh=8, bw=8, topk=4)
    q, k = rand_bits(rng, g.N, g.d), rand_bits(rng, g.N, g.d)
    q4 = synth.to_bf16_bits(synth.bf16_bits_to_f32(q) * np.float32(4.0))       # exact power of two
    assert np.array_equal(oracle.select(g, q, k), oracle.select(g, q4, k))


# ------------------------------------------------------------------ forward

@pytest.mark.parametrize("nlat,nlon,bh,bw,d", [(24, 32, 8, 8, 16), (16, 48, 4, 8, 8)])
def test_forward_equals_dense_when_topk_covers_all(nlat, nlon, bh, bw, d):
    rng = np.random.default_rng(5)
    g = Geom(nlat, nlon, d=d, bh=bh, bw=bw, topk=(nlat // bh) * (nlon // bw))
    q, k, v = (rand_bits(rng, g.N, d) for _ in range(3))
    idx = oracle.select(g, q, k)
    O, L = oracle.fwd(g, q, k, v, idx)
    O, L = oracle.to_token_order(g, O), oracle.to_token_order(g, L)
    Od, Ld = dense_attention(f64(q), f64(k), f64(v), 1 / math.sqrt(d))
    assert np.abs(O - Od).max() < 1e-12 and np.abs(L - Ld).max() < 1e-12


def test_forward_block_diagonal_when_radius_zero_and_no_topk():
    rng = np.random.default_rng(6)
    g = Geom(16, 24, d=8, bh=8, bw=8, rlat=0, rlon=0, topk=0)
    q, k, v = (rand_bits(rng, g.N, g.d) for _ in range(3))
    O, L = oracle.fwd(g, q, k, v, np.zeros((g.m, 0), np.int32))
    for j in range(g.m):
        t = block_tokens(g.nlon, g.bh, g.bw, g.nbw, j)
        Od, Ld = dense_attention(f64(q)[t], f64(k)[t], f64(v)[t], 1 / math.sqrt(g.d))
        assert np.abs(O[j] - Od).max() < 1e-12 and np.abs(L[j] - Ld).max() < 1e-12


def test_forward_matches_masked_dense_and_custom_scale():
    """General case: dense attention with the (local U selected) block mask written out."""
    rng = np.random.default_rng(7)
    g = Geom(32, 48, d=8, bh=8, bw=8, topk=3, scale=0.3)
    q, k, v = (rand_bits(rng, g.N, g.d) for _ in range(3))
    idx = oracle.select(g, q, k)
    O, L = oracle.fwd(g, q, k, v, idx)
    qf, kf, vf = f64(q), f64(k), f64(v)
    for i in range(g.m):
        att = sorted(local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw) | set(idx[i].tolist()))
        tk = np.concatenate([block_tokens(g.nlon, g.bh, g.bw, g.nbw, j) for j in att])
        tq = block_tokens(g.nlon, g.bh, g.bw, g.nbw, i)
        Od, Ld = dense_attention(qf[tq], kf[tk], vf[tk], 0.3)
        assert np.abs(O[i] - Od).max() < 1e-12 and np.abs(L[i] - Ld).max() < 1e-12


def test_closed_forms_zero_query_and_constant_value():
    rng = np.random.default_rng(8)
    g = Geom(32, 32, d=8, bh=8, bw=8, topk=2)
    k, v = rand_bits(rng, g.N, g.d), rand_bits(rng, g.N, g.d)
    q0 = np.zeros((g.N, g.d), np.uint16)
    idx = oracle.select(g, rand_bits(rng, g.N, g.d), k)
    O, L = oracle.fwd(g, q0, k, v, idx)
    vf = f64(v)
    for i in range(g.m):
        att = local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw) | set(idx[i].tolist())
        tk = np.concatenate([block_tokens(g.nlon, g.bh, g.bw, g.nbw, j) for j in sorted(att)])
        assert np.allclose(L[i], math.log(len(tk)), atol=1e-13)                # uniform weights
        assert np.abs(O[i] - vf[tk].mean(axis=0)).max() < 1e-13
    vc = synth.to_bf16_bits(np.full((g.N, g.d), 1.5, np.float32))
    O, _ = oracle.fwd(g, rand_bits(rng, g.N, g.d), k, vc, idx)
    assert np.abs(O - 1.5).max() < 1e-13


def test_weights_row_stochastic_and_convex_hull():
    rng = np.random.default_rng(9)
    g = Geom(32, 64, d=16, bh=8, bw=8, topk=4)
    q, k, v = (rand_bits(rng, g.N, g.d, 2.0) for _ in range(3))
    idx = oracle.select(g, q, k)
    O, _ = oracle.fwd(g, q, k, v, idx)
    vf = f64(v)
    for i, e in itertools.product((0, 5, 13, 31), (0, 17, 63)):
        tok, w = oracle.weights_row(g, q, k, idx, i, e)
        att = local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw) | set(idx[i].tolist())
        assert len(tok) == len(set(tok.tolist())) == len(att) * g.b
        assert set(tok.tolist()) == set(np.concatenate(
            [block_tokens(g.nlon, g.bh, g.bw, g.nbw, j) for j in att]).tolist())
        assert abs(w.sum() - 1.0) < 1e-12 and (w >= 0).all()
        assert np.abs(w @ vf[tok] - O[i, e]).max() < 1e-12
        assert (O[i, e] <= vf[tok].max(axis=0) + 1e-12).all() and (O[i, e] >= vf[tok].min(axis=0) - 1e-12).all()


def test_longitude_roll_equivariance_and_no_latitude_equivariance():
    rng = np.random.default_rng(10)
    g = Geom(32, 64, d=8, bh=8, bw=8, topk=3)
    q, k, v = (rand_bits(rng, g.N, g.d) for _ in range(3))
    idx = oracle.select(g, q, k)
    O, L = oracle.fwd(g, q, k, v, idx)
    O = oracle.to_token_order(g, O).reshape(g.nlat, g.nlon, g.d)

    def roll(x, s, axis):
        return np.ascontiguousarray(np.roll(x.reshape(g.nlat, g.nlon, g.d), s, axis=axis).reshape(g.N, g.d))

    s = 2                                             # two blocks east
    qr, kr, vr = (roll(x, s * g.bw, 1) for x in (q, k, v))
    idx_r = oracle.select(g, qr, kr)
    O_r, _ = oracle.fwd(g, qr, kr, vr, idx_r)
    O_r = oracle.to_token_order(g, O_r).reshape(g.nlat, g.nlon, g.d)
    assert np.abs(O_r - np.roll(O, s * g.bw, axis=1)).max() < 1e-12
    for i in range(g.m):
        by, bx = divmod(i, g.nbw)
        src = idx[by * g.nbw + (bx - s) % g.nbw]
        want = [(j // g.nbw) * g.nbw + (j % g.nbw + s) % g.nbw for j in src]
        assert sorted(idx_r[i].tolist()) == sorted(want)                      # ids move with the blocks
    # latitude is clamped, not periodic: rolling rows changes the result
    ql, kl, vl = (roll(x, g.bh, 0) for x in (q, k, v))
    O_l, _ = oracle.fwd(g, ql, kl, vl, oracle.select(g, ql, kl))
    O_l = oracle.to_token_order(g, O_l).reshape(g.nlat, g.nlon, g.d)
    assert np.abs(O_l - np.roll(O, g.bh, axis=0)).max() > 1e-3


# ------------------------------------------------------------------ backward

def _loss(g, q, k, v, do, idx):
    O, _ = oracle.fwd(g, q, k, v, idx)
    return float((oracle.to_token_order(g, O) * f64(do)).sum())


def test_backward_finite_differences():
    rng = np.random.default_rng(11)
    g = Geom(16, 16, d=4, bh=4, bw=4, topk=2)         # m = 16
    q, k, v, do = (quantised((g.N, g.d), rng) for _ in range(4))
    idx = oracle.select(g, q, k)                      # held constant below
    dQ, dK, dV, _, _ = oracle.bwd(g, q, k, v, do, idx)
    args = {"q": q, "k": k, "v": v}
    grads = {"q": dQ, "k": dK, "v": dV}
    for name in ("q", "k", "v"):
        for _ in range(8):
            t, c = int(rng.integers(g.N)), int(rng.integers(g.d))
            est = []
            for h in (1 / 32, 1 / 64):                # both steps exactly representable in bf16 here
                vals = {}
                for sgn in (+1, -1):
                    pert = synth.bf16_bits_to_f32(args[name]).copy()
                    pert[t, c] += np.float32(sgn * h)
                    bits = synth.to_bf16_bits(pert)
                    assert np.array_equal(synth.bf16_bits_to_f32(bits), pert)
                    a = dict(args); a[name] = bits
                    vals[sgn] = _loss(g, a["q"], a["k"], a["v"], do, idx)
                est.append((vals[1] - vals[-1]) / (2 * h))
            fd = (4 * est[1] - est[0]) / 3            # Richardson: O(h^4)
            assert abs(fd - grads[name][t, c]) < 2e-5 * max(1.0, abs(fd)), (name, t, c, fd, grads[name][t, c])


def test_backward_matches_dense_autograd_formula_when_topk_covers_all():
    """With every block attended the gradients are those of plain softmax attention."""
    rng = np.random.default_rng(12)
    g = Geom(16, 24, d=8, bh=8, bw=8, topk=6)
    q, k, v, do = (rand_bits(rng, g.N, g.d) for _ in range(4))
    idx = oracle.select(g, q, k)
    dQ, dK, dV, O, L = oracle.bwd(g, q, k, v, do, idx)
    qf, kf, vf, dof = f64(q), f64(k), f64(v), f64(do)
    sc = 1 / math.sqrt(g.d)
    x = sc * qf @ kf.T
    P = np.exp(x - x.max(1, keepdims=True)); P /= P.sum(1, keepdims=True)
    Od = P @ vf
    dP = dof @ vf.T
    dS = P * (dP - (dof * Od).sum(1, keepdims=True))
    assert np.abs(O - Od).max() < 1e-12
    assert np.abs(dV - P.T @ dof).max() < 1e-11
    assert np.abs(dQ - sc * dS @ kf).max() < 1e-11
    assert np.abs(dK - sc * dS.T @ qf).max() < 1e-11


def test_backward_visits_only_connected_blocks_and_shift_invariance():
    rng = np.random.default_rng(13)
    g = Geom(32, 64, d=8, bh=8, bw=8, topk=2)
    q, k, v = (rand_bits(rng, g.N, g.d) for _ in range(3))
    idx = oracle.select(g, q, k)
    j = 2 * g.nbw + 4
    connected = [i for i in range(g.m)
                 if j in local_blocks(i // g.nbw, i % g.nbw, g.nbh, g.nbw) or j in idx[i].tolist()]
    assert 9 <= len(connected) < g.m
    do = np.zeros((g.N, g.d), np.float32)
    for i in range(g.m):
        if i not in connected:
            do[block_tokens(g.nlon, g.bh, g.bw, g.nbw, i)] = rng.standard_normal((g.b, g.d))
    dQ, dK, dV, _, _ = oracle.bwd(g, q, k, v, synth.to_bf16_bits(do), idx)
    tj = block_tokens(g.nlon, g.bh, g.bw, g.nbw, j)
    assert np.all(dK[tj] == 0.0) and np.all(dV[tj] == 0.0)                   # exactly zero
    assert np.abs(dK).max() > 1e-3 and np.abs(dV).max() > 1e-3
    # adding one vector to every key shifts all logits of a row equally: sum_t dK_t = 0
    do = rand_bits(rng, g.N, g.d)
    dQ, dK, dV, _, _ = oracle.bwd(g, q, k, v, do, idx)
    assert np.abs(dK.sum(axis=0)).max() < 1e-10 * np.abs(dK).sum()
    # sum_t dV_t = sum_l dO_l because the weights of each row sum to one
    assert np.abs(dV.sum(axis=0) - f64(do).sum(axis=0)).max() < 1e-9


def test_backward_on_block_lists_equals_the_whole_unit_and_the_dense_formula():
    """`bwd_blocks` (gradients of listed blocks only) against the whole-unit backward, which the tests above
    pin, and against the dense softmax-attention gradient written out here when every block is attended."""
    rng = np.random.default_rng(14)
    g = Geom(32, 48, d=8, bh=8, bw=8, topk=3)        # m = 24, sparse pattern
    q, k, v, do = (rand_bits(rng, g.N, g.d) for _ in range(4))
    idx = oracle.select(g, q, k)
    dQ, dK, dV, _, _ = oracle.bwd(g, q, k, v, do, idx)
    qb, kb = [0, 7, 23, 12], [5, 23, 0]
    bQ, bK, bV = oracle.bwd_blocks(g, q, k, v, do, idx, qb, kb)
    for n, i in enumerate(qb):
        assert np.abs(bQ[n] - dQ[block_tokens(g.nlon, g.bh, g.bw, g.nbw, i)]).max() < 1e-12
    for n, j in enumerate(kb):
        tj = block_tokens(g.nlon, g.bh, g.bw, g.nbw, j)
        assert np.abs(bK[n] - dK[tj]).max() < 1e-12 and np.abs(bV[n] - dV[tj]).max() < 1e-12
    assert np.abs(bK).max() > 1e-3 and np.abs(bQ).max() > 1e-3
    # dense case, independent formula
    g = Geom(16, 24, d=8, bh=8, bw=8, topk=6)
    q, k, v, do = (rand_bits(rng, g.N, g.d) for _ in range(4))
    idx = oracle.select(g, q, k)
    qf, kf, vf, dof = f64(q), f64(k), f64(v), f64(do)
    sc = 1 / math.sqrt(g.d)
    x = sc * qf @ kf.T
    P = np.exp(x - x.max(1, keepdims=True)); P /= P.sum(1, keepdims=True)
    dS = P * (dof @ vf.T - (dof * (P @ vf)).sum(1, keepdims=True))
    bQ, bK, bV = oracle.bwd_blocks(g, q, k, v, do, idx, [4], [1, 5])
    assert np.abs(bQ[0] - (sc * dS @ kf)[block_tokens(g.nlon, g.bh, g.bw, g.nbw, 4)]).max() < 1e-11
    for n, j in enumerate([1, 5]):
        tj = block_tokens(g.nlon, g.bh, g.bw, g.nbw, j)
        assert np.abs(bK[n] - (sc * dS.T @ qf)[tj]).max() < 1e-11
        assert np.abs(bV[n] - (P.T @ dof)[tj]).max() < 1e-11


# ------------------------------------------------------------------ cost model

def test_attended_pairs_match_cost_model():
    """Selected + local work is linear in N: N*n*b + N*(local blocks)*b token pairs."""
    for w in (synth.WORKLOADS["c1_tiny"], synth.small_case(40, 48, 8, 8, 5)):
        g = Geom(w.nlat, w.nlon, d=8, bh=w.bh, bw=w.bw, topk=w.topk)
        rng = np.random.default_rng(14)
        idx = oracle.select(g, rand_bits(rng, g.N, 8), rand_bits(rng, g.N, 8))
        pairs = sum(len(oracle.local_set(g, i)) + int((idx[i] >= 0).sum()) for i in range(g.m))
        assert pairs == flops.pairs_per_unit(w)
        interior = g.nbw * (g.nbh - 2) * (9 + w.topk) + 2 * g.nbw * (6 + w.topk)
        assert pairs == interior
    assert flops.pairs_per_unit(synth.WORKLOADS["c2_1p5deg"]) == 7470
    assert flops.pairs_per_unit(synth.WORKLOADS["c5_0p25deg"]) == 100710


def test_golden_fixture_is_reproduced():
    """The stored selection/LSE fixture (written by tests/golden/make_golden.py from the
    oracle alone) still matches: guards the oracle against silent edits."""
    path = os.path.join(os.path.dirname(__file__), "golden", "c1_unit0.txt")
    want_idx, want_lse = [], []
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        tag, *vals = line.split()
        (want_idx if tag == "idx" else want_lse).append(vals)
    w = synth.WORKLOADS["c1_tiny"]
    x = synth.make_inputs(w)
    g = Geom(w.nlat, w.nlon, d=w.d, bh=w.bh, bw=w.bw, topk=w.topk)
    idx = oracle.select(g, x["q"][0, 0], x["k"][0, 0])
    assert idx.tolist() == [[int(t) for t in r] for r in want_idx]
    blocks = [int(r[0]) for r in want_lse]
    _, L = oracle.fwd(g, x["q"][0, 0], x["k"][0, 0], x["v"][0, 0], idx, blocks)
    for n, r in enumerate(want_lse):
        assert np.allclose(L[n, :4], [float(t) for t in r[1:]], rtol=0, atol=1e-12)


# ------------------------------------------------------------------ aligned local groups (the paper's large local blocks)

def test_local_groups_set_and_forward_against_masked_dense():
    """With local_groups the local set is the aligned group of rlat x rlon blocks (ragged at the grid's edge):
    checked against the definition written here, and the forward against masked dense attention."""
    g = Geom(40, 48, d=8, bh=8, bw=8, rlat=2, rlon=4, topk=2, local_groups=True)   # 5 x 6 blocks
    for i in range(g.m):
        by, bx = divmod(i, g.nbw)
        want = [y * g.nbw + x for y in range(by // 2 * 2, min(by // 2 * 2 + 2, g.nbh))
                for x in range(bx // 4 * 4, min(bx // 4 * 4 + 4, g.nbw))]
        assert oracle.local_set(g, i) == want
    # one-column grid: the paper's layout (blocks of contiguous tokens, groups of 8 blocks)
    gh = Geom(256, 16, d=8, bh=8, bw=16, rlat=8, rlon=1, topk=3, local_groups=True)  # 32 blocks of 128 tokens
    assert oracle.local_set(gh, 13) == list(range(8, 16))
    rng = np.random.default_rng(21)
    q, k, v = (rand_bits(rng, gh.N, gh.d) for _ in range(3))
    idx = oracle.select(gh, q, k)
    assert all(j // 8 != i // 8 for i in range(gh.m) for j in idx[i])                # selected blocks are never local
    O, L = oracle.fwd(gh, q, k, v, idx)
    qf, kf, vf = f64(q), f64(k), f64(v)
    for i in (0, 13, 31):
        blocks = list(range(i // 8 * 8, i // 8 * 8 + 8)) + idx[i].tolist()
        toks = np.concatenate([np.arange(j * 128, (j + 1) * 128) for j in blocks])   # block j = tokens 128 j .. 128 j + 127
        od, ld = dense_attention(qf[i * 128:(i + 1) * 128], kf[toks], vf[toks], 1 / math.sqrt(gh.d))
        assert np.abs(O[i] - od).max() < 1e-12 and np.abs(L[i] - ld).max() < 1e-12
