"""The selection entry point that allocates nothing (its scratch is a fixed array inside the library),
for callers that cannot obtain device memory when they need a selection.  Collected last on purpose, so
that a run that stops at the first failure has already run every other test.

Checked through the C ABI against the ordinary entry point, bit for bit (selection ids are integers), on
two calls in a row: the second call is a different, smaller problem, so it meets the first call's
leftovers in the shared array."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import synth

pytestmark = pytest.mark.gpu


def _both(w):
    x = synth.make_inputs(w)
    q, k = mb.from_bits(x["q"]), mb.from_bits(x["k"])
    p = mb.Params.from_workload(w)
    ws = mb.alloc_workspace(p, mb.OP_SELECT)
    want = mb.mosaic_bsa_select(p, q, k, ws=ws)
    mb.check_status(ws, "select")
    out = torch.full((w.B, w.H, w.m, w.topk), -7, dtype=torch.int32, device="cuda")   # allocated by the caller
    got = mb.mosaic_bsa_select_static(p, q, k, block_idx=out)
    torch.cuda.synchronize()
    return got.cpu().numpy(), want.cpu().numpy()


def test_static_scratch_selection_matches_twice_in_a_row():
    first = synth.small_case(136, 160, 8, 8, 8, B=1, H=2, kind="smooth", seed=61)    # m = 340, two units
    second = synth.small_case(32, 64, 8, 8, 4, B=1, H=3, seed=62)                     # smaller: stale sums remain behind it
    for w in (first, second):
        got, want = _both(w)
        assert got.shape == want.shape and (want >= -1).all()
        assert np.array_equal(got, want), f"{(got != want).sum()} of {want.size} ids differ ({w.name})"


def test_static_scratch_rejects_problems_beyond_its_size():
    p = mb.Params(B=24, H=8, nlat=120, nlon=240, topk=8)       # 192 units x 450 blocks: 44 MB of pooled sums
    assert mb.workspace_bytes(p, mb.OP_SELECT) > mb.STATIC_SCRATCH_BYTES
    pc = p.c()
    rc = mb.lib().mosaic_bsa_select_static(ctypes.byref(pc), 256, 256, 256, None)   # never dereferenced: the size check comes first
    assert rc == -3 and "workspace" in mb.strerror(rc)


def test_static_scratch_selection_takes_no_device_memory():
    """Free device memory as the driver reports it is the same before and after a call that has run once before
    (the first call may load the library's module; the caller's tensors exist before the measurement)."""
    w = synth.small_case(32, 64, 8, 8, 4, B=1, H=3, seed=63)
    x = synth.make_inputs(w)
    q, k = mb.from_bits(x["q"]), mb.from_bits(x["k"])
    p = mb.Params.from_workload(w)
    out = torch.empty((w.B, w.H, w.m, w.topk), dtype=torch.int32, device="cuda")
    mb.mosaic_bsa_select_static(p, q, k, block_idx=out)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    mb.mosaic_bsa_select_static(p, q, k, block_idx=out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
