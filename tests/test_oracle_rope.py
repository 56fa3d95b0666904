"""Pins of the oracle's 2-D rotary position embedding: identity at zero, rotations preserve pair norms, the
inner product of a rotated query and a rotated key depends on the position difference only, agreement with
complex multiplication by numpy's exp(i a), hand values of the frequencies, and the bf16 rounding."""
import math

import numpy as np

import oracle
from oracle import Geom
from paper_2604_16429_b200 import synth


def _case(seed, nlat=8, nlon=16, d=64):
    rng = np.random.default_rng(seed)
    g = Geom(nlat, nlon, d=d, bh=8, bw=8, topk=0)
    x = synth.to_bf16_bits(rng.standard_normal((g.N, g.d)).astype(np.float32))
    pos = np.stack([rng.uniform(0, 2 * math.pi, g.N), rng.uniform(-math.pi / 2, math.pi / 2, g.N)], axis=1)
    return g, x, pos


def test_identity_norms_and_rounding():
    g, x, pos = _case(1)
    out0, bits0 = oracle.rope(g, x, np.zeros_like(pos))
    assert np.array_equal(bits0, x) and np.array_equal(out0, synth.bf16_bits_to_f32(x).astype(np.float64))
    out, bits = oracle.rope(g, x, pos)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    n_in = xf.reshape(g.N, -1, 2) ** 2
    n_out = out.reshape(g.N, -1, 2) ** 2
    assert np.abs(n_in.sum(-1) - n_out.sum(-1)).max() < 1e-12
    assert np.abs(out - xf).max() > 0.1                                   # it did turn something
    assert np.array_equal(bits, synth.to_bf16_bits(out.astype(np.float32)))


def test_matches_complex_multiplication_and_hand_values():
    g, x, pos = _case(2)
    out, _ = oracle.rope(g, x, pos, theta=10000.0)
    xf = synth.bf16_bits_to_f32(x).astype(np.float64)
    D = g.d // 2
    z = xf[:, 0::2] + 1j * xf[:, 1::2]                                    # [N, d/2] pairs, longitude half first
    freq = 10000.0 ** (-np.arange(D // 2) / (D / 2))                      # 1, 10000^(-1/16), ...
    ang = np.concatenate([pos[:, :1] * freq, pos[:, 1:] * freq], axis=1)  # [N, d/2]
    w = z * np.exp(1j * ang)
    assert np.abs(out[:, 0::2] - w.real).max() < 1e-12 and np.abs(out[:, 1::2] - w.imag).max() < 1e-12
    # hand values: a quarter turn of the first longitude pair, and the second pair's frequency 10000^(-1/16)
    g1 = Geom(8, 8, d=64, bh=8, bw=8, topk=0)
    one = np.zeros((g1.N, g1.d), np.float32); one[:, 0] = 1.0; one[:, 2] = 1.0; one[:, 32] = 1.0
    p1 = np.zeros((g1.N, 2)); p1[:, 0] = math.pi / 2; p1[:, 1] = 1.0
    o1, _ = oracle.rope(g1, synth.to_bf16_bits(one), p1)
    assert abs(o1[0, 0]) < 1e-15 and abs(o1[0, 1] - 1.0) < 1e-15
    a = (math.pi / 2) * 0.5623413251903491                                # 10^(-1/4)
    assert abs(o1[0, 2] - math.cos(a)) < 1e-14 and abs(o1[0, 3] - math.sin(a)) < 1e-14
    assert abs(o1[0, 32] - math.cos(1.0)) < 1e-15 and abs(o1[0, 33] - math.sin(1.0)) < 1e-15   # latitude half, angle 1
    # another theta changes every frequency but the first
    o2, _ = oracle.rope(g1, synth.to_bf16_bits(one), p1, theta=100.0)
    assert abs(o2[0, 0] - o1[0, 0]) < 1e-15 and abs(o2[0, 2] - math.cos((math.pi / 2) * 100.0 ** (-1 / 16))) < 1e-14


def test_inner_products_depend_on_the_position_difference_only():
    g, q, pa = _case(3)
    _, k, pb = _case(4)
    rq, _ = oracle.rope(g, q, pa)
    rk, _ = oracle.rope(g, k, pb)
    rd, _ = oracle.rope(g, q, pa - pb)
    kf = synth.bf16_bits_to_f32(k).astype(np.float64)
    assert np.abs((rq * rk).sum(1) - (rd * kf).sum(1)).max() < 1e-11


def test_binary16_storage_decoding_and_rounding_against_numpy():
    """Every binary16 bit pattern decodes as numpy's float16 does, the identity rotation returns the same bits, and
    rotated values round as numpy rounds float32 -> float16."""
    g16 = Geom(8, 16, d=64, bh=8, bw=8, topk=0, f16=True)
    allbits = np.arange(65536, dtype=np.uint16)
    want = allbits.view(np.float16).astype(np.float64)
    got = oracle.widen16(g16, allbits)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and np.array_equal(got[~np.isnan(want)], want[~np.isnan(want)])
    some = allbits[:0x7F80:7]                                             # finite bf16 patterns
    assert np.array_equal(oracle.widen16(Geom(8, 16), some), synth.bf16_bits_to_f32(some).astype(np.float64))
    finite = allbits[np.isfinite(want)]
    x = np.resize(finite, (g16.N, g16.d)).astype(np.uint16)
    _, same = oracle.rope(g16, x, np.zeros((g16.N, 2)))
    assert np.array_equal(same & 0x7FFF, x & 0x7FFF) and np.array_equal(same[(x & 0x7FFF) != 0], x[(x & 0x7FFF) != 0])
    rng = np.random.default_rng(5)
    xs = synth.to_f16_bits((rng.standard_normal((g16.N, g16.d)) * 10.0 ** rng.integers(-7, 5, (g16.N, 1))).astype(np.float32))
    pos = rng.uniform(-3, 3, (g16.N, 2))
    out, bits = oracle.rope(g16, xs, pos)
    with np.errstate(over="ignore"):
        assert np.array_equal(bits, out.astype(np.float32).astype(np.float16).view(np.uint16))
