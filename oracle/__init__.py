"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE, not product code).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It compiles ``mosaic_oracle.c`` with gcc on first use and exposes the
oracle's per-unit functions on numpy arrays.  Inputs are bf16 bit patterns stored
as ``uint16`` arrays of shape ``[N, d]`` (one (batch, head) unit at a time).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mosaic_oracle.c")
_LIB = os.path.join(_HERE, "libmosaic_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2 -fopenmp).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Geom(ctypes.Structure):
    _fields_ = [
        ("nlat", ctypes.c_int32), ("nlon", ctypes.c_int32), ("d", ctypes.c_int32),
        ("bh", ctypes.c_int32), ("bw", ctypes.c_int32),
        ("rlat", ctypes.c_int32), ("rlon", ctypes.c_int32),
        ("topk", ctypes.c_int32),
        ("scale", ctypes.c_double),
        ("local_groups", ctypes.c_int32),
        ("f16", ctypes.c_int32),
    ]


@dataclass(frozen=True)
class Geom:
    nlat: int
    nlon: int
    d: int = 64
    bh: int = 8
    bw: int = 8
    rlat: int = 1
    rlon: int = 1
    topk: int = 0
    scale: float = 0.0
    local_groups: bool = False
    f16: bool = False          # the 16-bit inputs are IEEE binary16 instead of bf16

    @property
    def N(self): return self.nlat * self.nlon
    @property
    def nbh(self): return self.nlat // self.bh
    @property
    def nbw(self): return self.nlon // self.bw
    @property
    def m(self): return self.nbh * self.nbw
    @property
    def b(self): return self.bh * self.bw

    def c(self):
        return _Geom(self.nlat, self.nlon, self.d, self.bh, self.bw, self.rlat, self.rlon,
                     self.topk, float(self.scale), int(self.local_groups), int(self.f16))


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.mo_num_threads.restype = ctypes.c_int
    return _lib


def _p(a, t):
    return a.ctypes.data_as(ctypes.POINTER(t)) if a is not None else None


def _u16(a, g):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16 and a.shape == (g.N, g.d), (a.dtype, a.shape)
    return a


def num_threads() -> int:
    return int(_load().mo_num_threads())


def local_set(g: Geom, i: int) -> list[int]:
    out = np.zeros(256, np.int32)
    gc = g.c()
    n = _load().mo_local_set(ctypes.byref(gc), ctypes.c_int32(i), _p(out, ctypes.c_int32))
    assert n >= 0
    return out[:n].tolist()


def pool(g: Geom, x) -> np.ndarray:
    x = _u16(x, g)
    out = np.zeros((g.m, g.d), np.float32)
    gc = g.c()
    rc = _load().mo_pool_unit(ctypes.byref(gc), _p(x, ctypes.c_uint16), _p(out, ctypes.c_float))
    assert rc == 0
    return out


def select(g: Geom, q, k, return_pooled: bool = False):
    """Selected block ids [m, topk] int32 of one unit (rank order, -1 padded)."""
    q, k = _u16(q, g), _u16(k, g)
    idx = np.full((g.m, max(g.topk, 0)), -1, np.int32)
    pq = np.zeros((g.m, g.d), np.float32)
    pk = np.zeros((g.m, g.d), np.float32)
    gc = g.c()
    rc = _load().mo_select_unit(ctypes.byref(gc), _p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16),
                                _p(idx, ctypes.c_int32), _p(pq, ctypes.c_float), _p(pk, ctypes.c_float))
    assert rc == 0
    return (idx, pq, pk) if return_pooled else idx


def weights_row(g: Geom, q, k, idx, i: int, e_row: int):
    """(token ids, softmax weights) of row e_row of query block i."""
    q, k = _u16(q, g), _u16(k, g)
    idx = np.ascontiguousarray(idx, np.int32).reshape(g.m, g.topk)
    cap = (256 + g.topk) * g.b
    tok = np.zeros(cap, np.int64)
    w = np.zeros(cap, np.float64)
    gc = g.c()
    n = _load().mo_weights_row(ctypes.byref(gc), _p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16),
                               _p(idx, ctypes.c_int32), ctypes.c_int32(i), ctypes.c_int32(e_row),
                               _p(tok, ctypes.c_int64), _p(w, ctypes.c_double))
    assert n >= 0
    return tok[:n].copy(), w[:n].copy()


def fwd(g: Geom, q, k, v, idx, blocks=None):
    """Forward of one unit.  Returns (O [n_blocks, b, d], LSE [n_blocks, b]) in fp64,
    rows in row-major order inside each block; blocks=None means all m blocks."""
    q, k, v = _u16(q, g), _u16(k, g), _u16(v, g)
    idx = np.ascontiguousarray(idx, np.int32).reshape(g.m, g.topk)
    if blocks is None:
        nb, bl = g.m, None
    else:
        bl = np.ascontiguousarray(blocks, np.int32)
        nb = int(bl.size)
    O = np.zeros((nb, g.b, g.d), np.float64)
    L = np.zeros((nb, g.b), np.float64)
    gc = g.c()
    rc = _load().mo_fwd_unit(ctypes.byref(gc), _p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16),
                             _p(v, ctypes.c_uint16), _p(idx, ctypes.c_int32), ctypes.c_int32(nb),
                             _p(bl, ctypes.c_int32), _p(O, ctypes.c_double), _p(L, ctypes.c_double))
    assert rc == 0
    return O, L


def bwd(g: Geom, q, k, v, d_o, idx):
    """Backward of one unit: (dQ, dK, dV, O, LSE), all fp64 in token order."""
    q, k, v, d_o = _u16(q, g), _u16(k, g), _u16(v, g), _u16(d_o, g)
    idx = np.ascontiguousarray(idx, np.int32).reshape(g.m, g.topk)
    dQ = np.zeros((g.N, g.d)); dK = np.zeros((g.N, g.d)); dV = np.zeros((g.N, g.d))
    O = np.zeros((g.N, g.d)); L = np.zeros(g.N)
    gc = g.c()
    rc = _load().mo_bwd_unit(ctypes.byref(gc), _p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16),
                             _p(v, ctypes.c_uint16), _p(d_o, ctypes.c_uint16), _p(idx, ctypes.c_int32),
                             _p(dQ, ctypes.c_double), _p(dK, ctypes.c_double), _p(dV, ctypes.c_double),
                             _p(O, ctypes.c_double), _p(L, ctypes.c_double))
    assert rc == 0
    return dQ, dK, dV, O, L


def bwd_blocks(g: Geom, q, k, v, d_o, idx, qblocks, kblocks):
    """Backward of one unit restricted to lists of blocks: dQ [nq, b, d] of the query blocks in
    `qblocks`, dK and dV [nk, b, d] of the key/value blocks in `kblocks` (fp64, rows in row-major
    order inside each block).  Same arithmetic as `bwd`, for sizes at which a whole unit takes too long."""
    q, k, v, d_o = _u16(q, g), _u16(k, g), _u16(v, g), _u16(d_o, g)
    idx = np.ascontiguousarray(idx, np.int32).reshape(g.m, g.topk)
    qb = np.ascontiguousarray(qblocks, np.int32)
    kb = np.ascontiguousarray(kblocks, np.int32)
    dQ = np.zeros((max(qb.size, 1), g.b, g.d)); dK = np.zeros((max(kb.size, 1), g.b, g.d)); dV = np.zeros_like(dK)
    gc = g.c()
    rc = _load().mo_bwd_blocks(ctypes.byref(gc), _p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16),
                               _p(v, ctypes.c_uint16), _p(d_o, ctypes.c_uint16), _p(idx, ctypes.c_int32),
                               ctypes.c_int32(qb.size), _p(qb, ctypes.c_int32), _p(dQ, ctypes.c_double),
                               ctypes.c_int32(kb.size), _p(kb, ctypes.c_int32), _p(dK, ctypes.c_double),
                               _p(dV, ctypes.c_double))
    assert rc == 0
    return dQ[:qb.size], dK[:kb.size], dV[:kb.size]


def fwd3(g: Geom, q, k, v, idx, gates):
    """Three-branch form of one unit (compression + selection + local, gated).  `gates` is [N, 3] (CG, FG, L).
    Returns a dict of fp64 arrays in token order: o, o_cg, o_fg, o_l [N, d]; lse_fg, lse_l [N]; abar [m, m]."""
    q, k, v = _u16(q, g), _u16(k, g), _u16(v, g)
    idx = np.ascontiguousarray(idx, np.int32).reshape(g.m, g.topk)
    gt = np.ascontiguousarray(gates, np.float64)
    assert gt.shape == (g.N, 3)
    out = {n: np.zeros((g.N, g.d)) for n in ("o", "o_cg", "o_fg", "o_l")}
    out["lse_fg"] = np.zeros(g.N); out["lse_l"] = np.zeros(g.N); out["abar"] = np.zeros((g.m, g.m))
    gc = g.c()
    dp = ctypes.c_double
    rc = _load().mo_fwd3_unit(ctypes.byref(gc), _p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                              _p(idx, ctypes.c_int32), _p(gt, dp), _p(out["o"], dp), _p(out["o_cg"], dp),
                              _p(out["o_fg"], dp), _p(out["o_l"], dp), _p(out["lse_fg"], dp), _p(out["lse_l"], dp),
                              _p(out["abar"], dp))
    assert rc == 0
    return out


def bwd3(g: Geom, q, k, v, d_o, idx, gates):
    """Backward of the three-branch form of one unit: (dQ, dK, dV [N, d], dGates [N, 3]) in fp64, token order."""
    q, k, v, d_o = _u16(q, g), _u16(k, g), _u16(v, g), _u16(d_o, g)
    idx = np.ascontiguousarray(idx, np.int32).reshape(g.m, g.topk)
    gt = np.ascontiguousarray(gates, np.float64)
    assert gt.shape == (g.N, 3)
    dQ = np.zeros((g.N, g.d)); dK = np.zeros((g.N, g.d)); dV = np.zeros((g.N, g.d)); dG = np.zeros((g.N, 3))
    gc = g.c()
    dp = ctypes.c_double
    rc = _load().mo_bwd3_unit(ctypes.byref(gc), _p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                              _p(d_o, ctypes.c_uint16), _p(idx, ctypes.c_int32), _p(gt, dp), _p(dQ, dp), _p(dK, dp),
                              _p(dV, dp), _p(dG, dp))
    assert rc == 0
    return dQ, dK, dV, dG


def rope(g: Geom, x, pos, theta=10000.0):
    """2-D rotary position embedding of one [N, d] tensor (bf16 bits); pos is [N, 2] = (longitude, latitude) in
    radians.  Returns (fp64 unrounded [N, d], bf16 bits [N, d])."""
    x = _u16(x, g)
    pos = np.ascontiguousarray(pos, np.float64)
    assert pos.shape == (g.N, 2)
    out = np.zeros((g.N, g.d))
    bits = np.zeros((g.N, g.d), np.uint16)
    gc = g.c()
    rc = _load().mo_rope_unit(ctypes.byref(gc), _p(x, ctypes.c_uint16), _p(pos, ctypes.c_double), ctypes.c_double(theta),
                              _p(out, ctypes.c_double), _p(bits, ctypes.c_uint16))
    assert rc == 0
    return out, bits


def widen16(g: Geom, bits) -> np.ndarray:
    """The 16-bit storage type's values as fp64 (bf16, or binary16 when g.f16)."""
    bits = np.ascontiguousarray(bits, np.uint16)
    out = np.zeros(bits.shape)
    gc = g.c()
    rc = _load().mo_widen16(ctypes.byref(gc), _p(bits, ctypes.c_uint16), ctypes.c_int64(bits.size), _p(out, ctypes.c_double))
    assert rc == 0
    return out


def block_tokens(g: Geom, j: int) -> np.ndarray:
    """Token ids of block j in row-major order inside the block (layout helper)."""
    by, bx = divmod(j, g.nbw)
    r = np.arange(g.bh)[:, None] + by * g.bh
    c = np.arange(g.bw)[None, :] + bx * g.bw
    return (r * g.nlon + c).reshape(-1)


def to_token_order(g: Geom, per_block: np.ndarray, blocks=None) -> np.ndarray:
    """Scatter a [n_blocks, b, ...] oracle result to token order [N, ...] (NaN elsewhere)."""
    bl = range(g.m) if blocks is None else list(blocks)
    out = np.full((g.N,) + per_block.shape[2:], np.nan)
    for n, j in enumerate(bl):
        out[block_tokens(g, j)] = per_block[n]
    return out
