"""The kernels' bounded waits, exercised without faulting anything: a test-only build of the library (short
wait limit, the planner never publishes a CTA's first key list) makes every consumer's wait run out.  The call
must return, report MOSAIC_E_DEVICE_TIMEOUT through the status word, and leave the context usable for the
product library."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2604_16429_b200 import binding as mb
from paper_2604_16429_b200 import build as mbuild
from paper_2604_16429_b200 import synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

TIMEOUT = -16


@pytest.fixture(scope="module")
def waitlib():
    L = ctypes.CDLL(mbuild.build_wait_test())
    vp = ctypes.c_void_p
    L.mosaic_test_wait_probe.restype = ctypes.c_int
    L.mosaic_test_wait_probe.argtypes = [vp, vp, vp]
    L.mosaic_bsa_fwd.restype = ctypes.c_int
    L.mosaic_bsa_fwd.argtypes = [ctypes.POINTER(mb._Params), vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
    L.mosaic_bsa_last_status.restype = ctypes.c_int
    L.mosaic_bsa_last_status.argtypes = [vp, vp]
    return L


def test_wait_on_a_barrier_nothing_arrives_at_gives_up(waitlib):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    assert waitlib.mosaic_test_wait_probe(status.data_ptr(), result.data_ptr(), torch.cuda.current_stream().cuda_stream) == 0
    torch.cuda.synchronize()
    assert int(status.item()) == TIMEOUT
    assert int(result[0].item()) == 0                       # the wait reported failure ...
    assert 1900 <= int(result[1].item()) <= 20000           # ... after its limit of 2e6 cycles (in units of 1024 cycles)


def test_forward_times_out_cleanly_and_the_context_stays_usable(waitlib):
    w = synth.WORKLOADS["c1_tiny"]
    x = synth.make_inputs(w)
    dx = G.device_inputs(x)
    idx = G.gpu_select(w, dx)
    p = mb.Params.from_workload(w)
    pc = p.c()
    ws = torch.zeros(mb.workspace_bytes(p, mb.OP_FWD), dtype=torch.uint8, device="cuda")
    o = torch.zeros_like(dx["q"])
    lse = torch.zeros((w.B, w.H, w.N), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    rc = waitlib.mosaic_bsa_fwd(ctypes.byref(pc), dx["q"].data_ptr(), dx["k"].data_ptr(), dx["v"].data_ptr(),
                                idx.data_ptr(), o.data_ptr(), lse.data_ptr(), ws.data_ptr(), ws.numel(), stream)
    assert rc == 0                                           # the launch itself is fine
    assert waitlib.mosaic_bsa_last_status(ws.data_ptr(), stream) == TIMEOUT
    # the product library on the same context, same buffers: correct results
    o2, lse2 = G.gpu_fwd(w, dx, idx)
    idx_h = idx.cpu().numpy()
    for h in range(w.H):
        G.compare_fwd_unit(w, x, 0, h, idx_h[0, h], o2, lse2)
