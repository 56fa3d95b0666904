"""Work counting for the benchmark: attended (query block, key block) pairs and the
effective FLOP they stand for.  Only unmasked work is counted: 4*d*b*b per pair in the
forward (QK^T and PV), 2.5x that in the backward (five products instead of two)."""
from __future__ import annotations


def local_count(by: int, nbh: int, nbw: int, rlat: int, rlon: int) -> int:
    rows = len({min(max(by + dy, 0), nbh - 1) for dy in range(-rlat, rlat + 1)})
    cols = len({dx % nbw for dx in range(-rlon, rlon + 1)})
    return rows * cols


def pairs_per_unit(w) -> int:
    nbh, nbw = w.nlat // w.bh, w.nlon // w.bw
    total = 0
    if getattr(w, "local_groups", False):   # local set = the aligned group of rlat x rlon blocks (ragged at the edges)
        for by in range(nbh):
            for bx in range(nbw):
                nl = (min(nbh, (by // w.rlat + 1) * w.rlat) - (by // w.rlat) * w.rlat) * \
                     (min(nbw, (bx // w.rlon + 1) * w.rlon) - (bx // w.rlon) * w.rlon)
                total += nl + min(w.topk, w.m - nl)
        return total
    for by in range(nbh):
        nl = local_count(by, nbh, nbw, w.rlat, w.rlon)
        total += nbw * (nl + min(w.topk, w.m - nl))
    return total


def fwd_flops(w, units: int | None = None) -> float:
    u = w.U if units is None else units
    return 4.0 * w.d * w.b * w.b * pairs_per_unit(w) * u


def bwd_flops(w, units: int | None = None) -> float:
    return 2.5 * fwd_flops(w, units)
