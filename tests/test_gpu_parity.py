"""GPU parity: the CUDA path through the C ABI against the fp64 oracle, element by element,
on sizes the oracle finishes in seconds (several tiles, ragged tails, degenerate cases)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

SELECT_CASES = [
    synth.WORKLOADS["c1_tiny"],
    synth.small_case(136, 160, 8, 8, 8, B=1, H=2, kind="smooth", seed=21),     # m = 340: two key chunks, ragged rows
    synth.small_case(64, 128, 16, 16, 16, B=2, H=1, kind="smooth", seed=22),   # 16x16 blocks, m = 32
    synth.small_case(24, 40, 8, 8, 32, B=1, H=1, seed=23),                      # top-k beyond the candidates -> -1 padding
    synth.small_case(40, 48, 8, 8, 5, B=1, H=3, seed=24, rlat=2, rlon=1),
    synth.small_case(32, 16, 8, 8, 2, B=1, H=1, seed=25),                       # 2 block columns: neighbourhood de-duplicates
    synth.small_case(48, 64, 8, 8, 0, B=1, H=1, seed=26, rlat=0, rlon=0),       # nothing selected
    synth.small_case(240, 320, 8, 8, 8, B=1, H=8, kind="smooth", seed=28),      # m = 1200, 8 units: the 32-rows-per-CTA ranking path
    synth.small_case(32, 64, 8, 16, 3, B=1, H=1, kind="smooth", seed=29),       # 8 x 16 blocks
    synth.small_case(240, 320, 8, 8, 8, B=1, H=5, kind="smooth", seed=30),      # m = 1200, 5 units: the 16-rows-per-CTA ranking path
]


@pytest.mark.parametrize("w", SELECT_CASES, ids=lambda w: w.name)
def test_select_bit_exact(w):
    x = synth.make_inputs(w)
    want = G.oracle_select_all(w, x)
    got = G.gpu_select(w, G.device_inputs(x)).cpu().numpy()
    assert got.shape == want.shape
    assert np.array_equal(got, want), f"{(got != want).sum()} of {want.size} ids differ"


def test_select_ties_go_to_lower_block_id():
    w = synth.small_case(32, 64, 8, 8, 4, seed=27)
    x = synth.make_inputs(w)
    k = x["k"].reshape(1, 1, 32, 64, 64).copy()
    k[:, :, :, 40:48] = k[:, :, :, 8:16]            # block column 5 repeats block column 1 exactly
    k[:, :, :, 56:64] = k[:, :, :, 8:16]
    x["k"] = np.ascontiguousarray(k.reshape(1, 1, -1, 64))
    want = G.oracle_select_all(w, x)
    got = G.gpu_select(w, G.device_inputs(x)).cpu().numpy()
    assert np.array_equal(got, want)
    # the tie is real: some row lists two duplicated blocks in ascending id order
    rows = [r for r in want[0, 0] if any((a % 8, b % 8) in ((1, 5), (1, 7), (5, 7)) and a // 8 == b // 8
                                         for a, b in zip(r[:-1], r[1:]))]
    assert rows


def test_select_near_ties_below_the_screening_resolution():
    """Twenty key blocks whose scores differ by about 1e-6 of their size, far below what an fp32 score can
    resolve: which eight of them a row takes, and in which order, is decided by the exact fp64 chain."""
    w = synth.small_case(120, 160, 8, 8, 8, B=1, H=2, seed=71)                 # m = 300
    x = synth.make_inputs(w)
    kf = synth.bf16_bits_to_f32(x["k"]).reshape(1, 2, 120, 160, 64).copy()
    qf = synth.bf16_bits_to_f32(x["q"]).reshape(1, 2, 120, 160, 64).copy()
    qf[..., 0] = np.abs(qf[..., 0]) + 1.0
    for t in range(20):
        by, bx = (3 * t) % 15, (7 * t) % 20
        blk = kf[:, :, 8 * by:8 * by + 8, 8 * bx:8 * bx + 8]
        blk[...] = 0.0
        blk[..., 0] = 4.0                                                       # pooled channel 0: 256 for all twenty
        blk[:, :, 0, 0, 1] = (1 + t) * 2.0 ** -10                               # the only difference between them
    x["k"] = synth.to_bf16_bits(kf.reshape(1, 2, -1, 64))
    x["q"] = synth.to_bf16_bits(qf.reshape(1, 2, -1, 64))
    want = G.oracle_select_all(w, x)
    got = G.gpu_select(w, G.device_inputs(x)).cpu().numpy()
    assert np.array_equal(got, want), f"{(got != want).sum()} of {want.size} ids differ"
    special = {((3 * t) % 15) * 20 + (7 * t) % 20 for t in range(20)}
    assert np.mean([len(special & set(r.tolist())) for r in want[0, 0]]) > 7    # the rows do choose among them


def test_select_all_scores_tied_takes_the_full_rescoring_path():
    """Every key block identical: all scores of a row tie exactly, nothing can be screened out, and the rows
    fall back to scoring every key; the lowest non-local ids win."""
    w = synth.small_case(120, 160, 8, 8, 6, B=1, H=1, seed=72)                 # m = 300 > survivors a row can hold
    x = synth.make_inputs(w)
    k = x["k"].reshape(1, 1, 15, 8, 20, 8, 64).copy()
    k[...] = k[:, :, :1, :, :1]                                                 # every block repeats block 0
    x["k"] = np.ascontiguousarray(k.reshape(1, 1, -1, 64))
    want = G.oracle_select_all(w, x)
    got = G.gpu_select(w, G.device_inputs(x)).cpu().numpy()
    assert np.array_equal(got, want)
    assert want[0, 0, 150].tolist() == [0, 1, 2, 3, 4, 5]


FWD_CASES = [
    (synth.WORKLOADS["c1_tiny"], 0.0),
    (synth.small_case(24, 40, 8, 8, 3, B=1, H=2, seed=31), 0.0),                # m = 15: last tile holds one block
    (synth.small_case(32, 64, 16, 16, 3, B=1, H=2, kind="smooth", seed=32), 0.0),  # 16x16 blocks: 4 chunks per block
    (synth.small_case(48, 64, 8, 8, 0, B=1, H=1, seed=33, rlat=0, rlon=0), 0.0),   # block-diagonal
    (synth.small_case(40, 48, 8, 8, 6, B=2, H=1, kind="smooth", seed=34, rlat=2, rlon=2), 0.3),
    (synth.small_case(16, 16, 8, 8, 4, B=1, H=1, seed=35), 0.0),                # 2x2 blocks: everything local, all -1
    # every way a 256-row work item is put together
    (synth.small_case(40, 56, 8, 8, 5, B=1, H=2, kind="smooth", seed=51), 0.0),   # 5 x 7 blocks: odd last row (1x4 groups), odd width
    (synth.small_case(32, 64, 8, 16, 3, B=1, H=1, kind="smooth", seed=52), 0.0),  # 128-token blocks (8 x 16): two blocks per item
    (synth.small_case(48, 40, 16, 8, 2, B=1, H=2, seed=53), 0.0),                  # 128-token blocks (16 x 8), 5 block columns: lone block
    (synth.small_case(64, 32, 32, 8, 2, B=1, H=1, seed=54), 0.0),                  # 256-token blocks (32 x 8): one item per block
    (synth.small_case(48, 64, 24, 16, 2, B=1, H=1, kind="smooth", seed=55), 0.0), # 384-token blocks: second item of a block is half empty
]


@pytest.mark.parametrize("w,scale", FWD_CASES, ids=lambda a: a.name if hasattr(a, "name") else str(a))
def test_forward_matches_oracle(w, scale):
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx, scale)
    idx_h = idx.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            G.compare_fwd_unit(w, x, b, h, idx_h[b, h], o, lse, scale=scale)


def test_forward_large_logits_rescale_path():
    """Inputs scaled up so the running maximum jumps by far more than the lazy-rescale threshold."""
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=2, seed=36)
    x = synth.make_inputs(w)
    for n in ("q", "k"):
        x[n] = synth.to_bf16_bits(synth.bf16_bits_to_f32(x[n]) * np.float32(3.0))
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx)
    for h in range(w.H):
        G.compare_fwd_unit(w, x, 0, h, idx.cpu().numpy()[0, h], o, lse)


def test_forward_accepts_caller_block_idx_in_any_order():
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=1, seed=37)
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    o1, l1 = G.gpu_fwd(w, dx, idx)
    rev = torch.flip(idx, dims=[-1]).contiguous()
    rev[..., 0, 0] = -1                                   # drop one id: still valid, different result for row 0
    o2, l2 = G.gpu_fwd(w, dx, rev)
    G.compare_fwd_unit(w, x, 0, 0, rev.cpu().numpy()[0, 0], o2, l2)
    same = oracle.block_tokens(G.geom_of(w), 5)
    assert torch.allclose(o1[0, 0, same].float(), o2[0, 0, same].float(), atol=2e-2)


def test_forward_is_deterministic_and_writes_everything():
    w = synth.WORKLOADS["c1_tiny"]
    dx = G.device_inputs(synth.make_inputs(w))
    idx = G.gpu_select(w, dx)
    o1, l1 = G.gpu_fwd(w, dx, idx)
    o2, l2 = G.gpu_fwd(w, dx, idx)
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(l1, l2)


def test_select_nan_and_infinite_scores():
    """A NaN pooled sum gives NaN scores: that block ranks after every number (also after -inf), and is
    chosen only where fewer than top-k other candidates exist.  Same ids as the oracle, bit for bit."""
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=2, seed=39)
    x = synth.make_inputs(w)
    k = x["k"].copy()
    k[0, 0, 5 * 64 + 17, 3] = 0x7FC0                      # NaN inside key block (0, 2) of unit 0
    k[0, 0, 20 * 64 + 40, 9] = 0xFF80                     # -inf inside key block (2, 5) of unit 0
    k[0, 1, 9 * 64 + 3, 0] = 0x7F80                       # +inf inside key block (1, 0) of unit 1
    x["k"] = k
    want = G.oracle_select_all(w, x)
    got = G.gpu_select(w, G.device_inputs(x)).cpu().numpy()
    assert np.array_equal(got, want), f"{(got != want).sum()} of {want.size} ids differ"
    wn = synth.small_case(16, 40, 8, 8, 4, B=1, H=1, seed=40)          # 4 candidates per row: NaN blocks must be listed last
    xn = synth.make_inputs(wn)
    kn = xn["k"].copy()
    kn[0, 0, 3 * 40 + 20, 1] = 0x7FC0                     # block (0, 2)
    kn[0, 0, 12 * 40 + 30, 1] = 0x7FC0                    # block (1, 3)
    xn["k"] = kn
    want = G.oracle_select_all(wn, xn)
    got = G.gpu_select(wn, G.device_inputs(xn)).cpu().numpy()
    assert np.array_equal(got, want)
    assert (want[0, 0, 0] >= 0).all() and set(want[0, 0, 0][2:].tolist()) == {2, 8}


def test_repeated_and_local_ids_are_skipped_and_reported():
    """A caller's block_idx row that repeats an id or names a block of the row's own neighbourhood: the extra
    entries are ignored (no block is attended twice) in forward and backward, and the status word says so."""
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=1, seed=60, backward=True)
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    clean = idx.clone()
    clean[0, 0, 10, 2:] = -1
    dirty = clean.clone()
    dirty[0, 0, 10, 2] = clean[0, 0, 10, 0]                # repeat of entry 0
    dirty[0, 0, 10, 3] = 11                                # right-hand neighbour of block 10: local
    p = mb.Params.from_workload(w)
    ws = mb.alloc_workspace(p, mb.OP_BWD)
    o1, l1 = mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], clean, ws=ws)
    assert mb.mosaic_bsa_last_status(ws) == 0
    o2, l2 = mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], dirty, ws=ws)
    assert mb.mosaic_bsa_last_status(ws) == -17
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)) and torch.equal(l1, l2)
    G.compare_fwd_unit(w, x, 0, 0, clean.cpu().numpy()[0, 0], o2, l2)
    g1 = mb.mosaic_bsa_bwd(p, dx["q"], dx["k"], dx["v"], o1, l1, dx["do"], clean, ws=ws)
    assert mb.mosaic_bsa_last_status(ws) == 0
    g2 = mb.mosaic_bsa_bwd(p, dx["q"], dx["k"], dx["v"], o1, l1, dx["do"], dirty, ws=ws)
    assert mb.mosaic_bsa_last_status(ws) == -17
    for a, b in zip(g1, g2):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_descriptor_cache_encodes_once_per_tensor():
    w = synth.small_case(56, 88, 8, 8, 4, B=1, H=1, seed=59)    # a grid no other test uses: nothing cached for it yet
    dx = G.device_inputs(synth.make_inputs(w))
    p = mb.Params.from_workload(w)
    ws = mb.alloc_workspace(p, mb.OP_FWD)
    idx = mb.mosaic_bsa_select(p, dx["q"], dx["k"], ws=mb.alloc_workspace(p, mb.OP_SELECT))
    o = torch.empty_like(dx["q"])
    lse = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device="cuda")
    n0 = mb.descriptor_encodes()
    mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx, o=o, lse=lse, ws=ws)
    n1 = mb.descriptor_encodes()
    mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx, o=o, lse=lse, ws=ws)
    n2 = mb.descriptor_encodes()
    assert n1 - n0 == 3 and n2 == n1                       # Q, K, V once; nothing on the second call
    mb.check_status(ws, "fwd")


def test_bad_block_id_is_reported_not_dereferenced():
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=1, seed=38)
    dx = G.device_inputs(synth.make_inputs(w))
    idx = G.gpu_select(w, dx)
    idx[0, 0, 3, 1] = w.m + 5
    p = mb.Params.from_workload(w)
    ws = mb.alloc_workspace(p, mb.OP_FWD)
    o, lse = mb.mosaic_bsa_fwd(p, dx["q"], dx["k"], dx["v"], idx, ws=ws)
    assert mb.mosaic_bsa_last_status(ws) == -17
    assert torch.isfinite(o.float()).all()               # the bad id was skipped, nothing faulted


BWD_CASES = [
    synth.small_case(32, 64, 8, 8, 4, B=1, H=2, seed=41, backward=True),
    synth.small_case(24, 40, 8, 8, 3, B=1, H=1, kind="smooth", seed=42, backward=True),
    synth.small_case(32, 64, 16, 16, 2, B=1, H=1, kind="smooth", seed=43, backward=True),
    synth.small_case(48, 64, 8, 8, 0, B=1, H=1, seed=44, rlat=0, rlon=0, backward=True),
    synth.small_case(32, 64, 8, 16, 3, B=1, H=1, kind="smooth", seed=46, backward=True),   # 128-token blocks
    synth.small_case(40, 56, 8, 8, 5, B=1, H=1, kind="smooth", seed=47, backward=True),    # odd block grid
]


@pytest.mark.parametrize("w", BWD_CASES, ids=lambda w: w.name)
def test_backward_matches_oracle(w):
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    g = G.geom_of(w)
    idx_h = idx.cpu().numpy()
    for b in range(w.B):
        for h in range(w.H):
            dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][b, h], x["k"][b, h], x["v"][b, h], x["do"][b, h], idx_h[b, h])
            for name, got, want in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
                G.assert_bwd_close(name, got[b, h], want)
                gh = got[b, h].float().cpu().numpy().astype(np.float64)
                assert np.abs(gh - want).mean() <= 0.1 * max(np.abs(want).mean(), 1e-3), name


def test_backward_popular_key_blocks_lists_span_several_buffers():
    """Two key blocks that (almost) every query block selects: their lists of connected query blocks are longer
    than one list buffer of the key-stationary kernel, which then continues an item over several buffers."""
    w = synth.small_case(120, 160, 8, 8, 4, B=1, H=1, seed=48, backward=True)      # m = 300
    x = synth.make_inputs(w)
    kf = synth.bf16_bits_to_f32(x["k"]).reshape(1, 1, 120, 160, 64).copy()
    qf = synth.bf16_bits_to_f32(x["q"]).reshape(1, 1, 120, 160, 64).copy()
    qf[..., 0] = np.abs(qf[..., 0]) + 1.0                       # every query likes channel 0 ...
    kf[:, :, 56:64, 72:88, 0] = 6.0                             # ... which two neighbouring key blocks carry
    x["k"] = synth.to_bf16_bits(kf.reshape(1, 1, -1, 64))
    x["q"] = synth.to_bf16_bits(qf.reshape(1, 1, -1, 64))
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    idx_h = idx.cpu().numpy()[0, 0]
    popular = 7 * 20 + 9
    assert (idx_h == popular).any(axis=1).sum() > 260           # in-degree beyond one list buffer (256 entries)
    o, lse = G.gpu_fwd(w, dx, idx)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    dQ, dK, dV, _, _ = oracle.bwd(G.geom_of(w), x["q"][0, 0], x["k"][0, 0], x["v"][0, 0], x["do"][0, 0], idx_h)
    for name, got, want in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
        G.assert_bwd_close(name, got[0, 0], want)


def test_backward_popular_key_block_with_four_chunks_per_block():
    """The same continuation of a long list over several list buffers, with 16x16 blocks (four 64-token chunks
    per block, the 0.25-degree shape): one key block that nearly every query block selects."""
    w = synth.small_case(240, 320, 16, 16, 4, B=1, H=1, seed=50, backward=True)    # 15 x 20 blocks, m = 300
    x = synth.make_inputs(w)
    kf = synth.bf16_bits_to_f32(x["k"]).reshape(1, 1, 240, 320, 64).copy()
    qf = synth.bf16_bits_to_f32(x["q"]).reshape(1, 1, 240, 320, 64).copy()
    qf[..., 0] = np.abs(qf[..., 0]) + 1.0
    kf[:, :, 112:128, 144:160, 0] = 6.0                         # block (7, 9)
    x["k"] = synth.to_bf16_bits(kf.reshape(1, 1, -1, 64))
    x["q"] = synth.to_bf16_bits(qf.reshape(1, 1, -1, 64))
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    idx_h = idx.cpu().numpy()[0, 0]
    g = G.geom_of(w)
    assert np.array_equal(idx_h, oracle.select(g, x["q"][0, 0], x["k"][0, 0]))
    popular = 7 * 20 + 9
    assert (idx_h == popular).any(axis=1).sum() > 260           # in-degree beyond one list buffer (256 entries)
    o, lse = G.gpu_fwd(w, dx, idx)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    qb = np.array([0, popular, 299], np.int32)
    kb = np.array([popular, popular + 1, 0], np.int32)
    dQ, dK, dV = oracle.bwd_blocks(g, x["q"][0, 0], x["k"][0, 0], x["v"][0, 0], x["do"][0, 0], idx_h, qb, kb)
    for n, i in enumerate(qb):
        G.assert_bwd_close(f"dQ block {i}", dq[0, 0][oracle.block_tokens(g, int(i))], dQ[n])
    for n, j in enumerate(kb):
        tj = oracle.block_tokens(g, int(j))
        G.assert_bwd_close(f"dK block {j}", dk[0, 0][tj], dK[n])
        G.assert_bwd_close(f"dV block {j}", dv[0, 0][tj], dV[n])


def test_backward_custom_scale_and_wide_neighbourhood():
    w = synth.small_case(48, 64, 8, 8, 6, B=1, H=2, kind="smooth", seed=49, rlat=2, rlon=1, backward=True)
    scale = 0.2
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx, scale)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx, scale)
    g = G.geom_of(w, scale)
    idx_h = idx.cpu().numpy()
    for h in range(w.H):
        G.compare_fwd_unit(w, x, 0, h, idx_h[0, h], o, lse, scale=scale)
        dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][0, h], x["k"][0, h], x["v"][0, h], x["do"][0, h], idx_h[0, h])
        for name, got, want in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
            G.assert_bwd_close(name, got[0, h], want)


def test_forward_largest_topk_and_16x16_radius_two():
    for w in (synth.small_case(64, 96, 8, 8, 32, B=1, H=1, kind="smooth", seed=56),                    # top-k at its limit
              synth.small_case(96, 96, 16, 16, 5, B=1, H=1, kind="smooth", seed=57, rlat=2, rlon=2)):  # 25 local blocks
        x = synth.make_inputs(w)
        dx = G.device_inputs(x)
        idx = G.gpu_select(w, dx)
        assert np.array_equal(idx.cpu().numpy(), G.oracle_select_all(w, x))
        o, lse = G.gpu_fwd(w, dx, idx)
        G.compare_fwd_unit(w, x, 0, 0, idx.cpu().numpy()[0, 0], o, lse)


@pytest.mark.parametrize("nlat,nlon", [(8, 8), (8, 16), (16, 8), (8, 40)])
def test_degenerate_grids_forward_and_backward(nlat, nlon):
    """One block, one row or one column of blocks: neighbourhoods collapse onto themselves, nothing can be selected."""
    w = synth.small_case(nlat, nlon, 8, 8, 3, B=1, H=2, seed=58 + nlat + nlon, backward=True)
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    want = G.oracle_select_all(w, x)
    assert np.array_equal(idx.cpu().numpy(), want)
    o, lse = G.gpu_fwd(w, dx, idx)
    dq, dk, dv = G.gpu_bwd(w, dx, o, lse, idx)
    g = G.geom_of(w)
    for h in range(w.H):
        G.compare_fwd_unit(w, x, 0, h, want[0, h], o, lse)
        dQ, dK, dV, _, _ = oracle.bwd(g, x["q"][0, h], x["k"][0, h], x["v"][0, h], x["do"][0, h], want[0, h])
        for name, got, ref in (("dQ", dq, dQ), ("dK", dk, dK), ("dV", dv, dV)):
            G.assert_bwd_close(name, got[0, h], ref)


def test_backward_is_deterministic():
    w = BWD_CASES[0]
    dx = G.device_inputs(synth.make_inputs(w))
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx)
    a = G.gpu_bwd(w, dx, o, lse, idx)
    b = G.gpu_bwd(w, dx, o, lse, idx)
    for s, t in zip(a, b):
        assert torch.equal(s.view(torch.int16), t.view(torch.int16))


def test_units_are_independent():
    """Permuting (batch, head) units permutes the outputs bit for bit."""
    w = synth.small_case(32, 64, 8, 8, 4, B=2, H=2, seed=45)
    dx = G.device_inputs(synth.make_inputs(w))
    idx = G.gpu_select(w, dx)
    o, lse = G.gpu_fwd(w, dx, idx)
    perm = {k: torch.flip(v, dims=[0, 1]).contiguous() for k, v in dx.items()}
    idx_p = G.gpu_select(w, perm)
    o_p, lse_p = G.gpu_fwd(w, perm, idx_p)
    assert torch.equal(idx_p, torch.flip(idx, dims=[0, 1]))
    assert torch.equal(o_p.view(torch.int16), torch.flip(o, dims=[0, 1]).view(torch.int16))
    assert torch.equal(lse_p, torch.flip(lse, dims=[0, 1]))
