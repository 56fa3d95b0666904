"""Host-side checks that need no GPU: the library loads, exports every symbol the header
declares, sizes workspaces, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import build as mbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    mbuild.build()


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "mosaic_bsa.h")).read()
    declared = set(re.findall(r"\b(mosaic_bsa_[a-z_]+)\s*\(", header))
    assert declared == set(mb.EXPORTS) and len(declared) >= 6
    L = mb.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_workspace_sizes():
    p = mb.Params(B=1, H=8, nlat=120, nlon=240, topk=8)
    m, U, N = 450, 8, 28800
    assert mb.workspace_bytes(p, mb.OP_FWD) == 256
    sel = mb.workspace_bytes(p, mb.OP_SELECT)
    assert sel >= 256 + 2 * U * m * 64 * 4 and sel % 256 == 0
    bwd = mb.workspace_bytes(p, mb.OP_BWD)
    assert bwd >= 256 + U * N * 4 + U * (m + 1) * 4 + U * m * 8 * 4
    assert mb.workspace_bytes(p, 7) == 0


@pytest.mark.parametrize("kw,code", [
    (dict(nlat=121), -1),            # grid not divisible by the block
    (dict(topk=-1), -1),
    (dict(B=0), -1),
    (dict(flags=4), -1),             # unknown flag bit
    (dict(flags=1, rlat=0), -1),     # group mode needs a group of at least one block
    (dict(flags=1, rlat=8, rlon=8), -2),
    (dict(d=32), -2),                # unsupported head dimension
    (dict(bh=4, bw=4, nlat=120), -2),
    (dict(rlat=3), -2),
    (dict(topk=33), -2),
])
def test_invalid_params_are_rejected(kw, code):
    base = dict(B=1, H=1, nlat=120, nlon=240, topk=8)
    base.update(kw)
    p = mb.Params(**base)
    assert mb.workspace_bytes(p, mb.OP_FWD) == 0
    pc = p.c()
    rc = mb.lib().mosaic_bsa_fwd(ctypes.byref(pc), 256, 256, 256, 256, 256, 256, 256, 1 << 20, None)
    assert rc == code
    assert mb.strerror(rc) not in ("ok", "unknown code")


def test_null_misaligned_and_small_workspace():
    p = mb.Params(B=1, H=1, nlat=32, nlon=64, topk=4)
    pc = p.c()
    L = mb.lib()
    assert L.mosaic_bsa_select(ctypes.byref(pc), None, 256, 256, 256, 1 << 20, None) == -1
    assert L.mosaic_bsa_select(ctypes.byref(pc), 256 + 8, 256, 256, 256, 1 << 20, None) == -4
    assert L.mosaic_bsa_select(ctypes.byref(pc), 256, 256, 256, 256 + 16, 1 << 20, None) == -4
    assert L.mosaic_bsa_select(ctypes.byref(pc), 256, 256, 256, 256, 16, None) == -3
    assert L.mosaic_bsa_bwd(ctypes.byref(pc), 256, 256, 256, 256, 256, 256, 256, 256, 256, None, 256, 1 << 20,
                            None) == -1
    assert L.mosaic_bsa_select(None, 256, 256, 256, 256, 1 << 20, None) == -1
    assert mb.strerror(0) == "ok" and mb.strerror(-16) and mb.strerror(-999) == "unknown code"
