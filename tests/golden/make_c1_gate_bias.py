"""Writes tests/golden/c1_gate_bias.txt: the learned gate's bias for the tiny fp32 config (seed 0),
calibrated by the CPU oracle alone so that the mean exit depth of the first two sequences is about
2.5 at threshold 0.5 with the lookahead gate.  Run from the repository root:
    python tests/golden/make_c1_gate_bias.py
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from oracle import cdb_oracle as O                      # noqa: E402
from paper_2608_09444_b200 import synth                 # noqa: E402

dims = synth.TINY
w = synth.weights_to_numpy(synth.make_weights(dims, seed=0, std=0.02))
prompts = synth.make_prompts(8, 32, dims.V, seed=0)


def make(b):
    ww = dict(w)
    ww["b_gate"] = np.array([b], dtype=np.float32)
    return O.Oracle(dims, ww, gate_kind=O.GATE_SIGMOID_CDF, q_or_eps=0.5, lookahead=True)


b, mean = O.calibrate_gate_bias(make, prompts[:2], 16, 2.5, iters=24)
b = float(np.float32(b))
out = make(b)
depths = np.concatenate([out.generate(p, 16)["depths"] for p in prompts])
path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_gate_bias.txt")
with open(path, "w") as f:
    f.write("# gate bias for the tiny fp32 config, written by make_c1_gate_bias.py (CPU oracle only)\n")
    f.write(f"# mean exit depth of sequences 0-1: {mean:.4f}; of all 8 sequences: {depths.mean():.4f}; "
            f"histogram depth 1..4: {np.bincount(depths, minlength=5)[1:].tolist()}\n")
    f.write(f"{b!r}\n")
print(open(path).read())
