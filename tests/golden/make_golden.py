"""Writes tests/golden/c1_unit0.txt from the oracle alone (never from the CUDA path):
the selected block ids of unit 0 of the tiny workload and a few log-sum-exp values.
The paper prints no worked numerical example of the attention, so this fixture only
guards the oracle against silent edits; what pins its mathematics are the tests in
tests/test_oracle_pins.py.  Run: python tests/golden/make_golden.py"""
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))

import oracle
from oracle import Geom
from paper_2604_16429_b200 import synth

w = synth.WORKLOADS["c1_tiny"]
x = synth.make_inputs(w)
g = Geom(w.nlat, w.nlon, d=w.d, bh=w.bh, bw=w.bw, topk=w.topk)
idx = oracle.select(g, x["q"][0, 0], x["k"][0, 0])
blocks = [0, 9, 31]
_, L = oracle.fwd(g, x["q"][0, 0], x["k"][0, 0], x["v"][0, 0], idx, blocks)
out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_unit0.txt")
with open(out, "w") as f:
    f.write("# tiny workload (32x64 grid, 8x8 blocks, top-k 4, N(0,1) bf16 inputs, seeds 1000..1002), unit (b=0,h=0)\n")
    f.write("# idx <4 selected block ids of query block i, i = 0..31>; lse <block> <log-sum-exp of its first 4 rows>\n")
    for r in idx.tolist():
        f.write("idx " + " ".join(str(t) for t in r) + "\n")
    for n, b in enumerate(blocks):
        f.write(f"lse {b} " + " ".join(f"{t:.15f}" for t in L[n, :4]) + "\n")
print("wrote", out)
