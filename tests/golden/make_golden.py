"""Writes the stored expected values under tests/golden/ by calling ONLY the
fp64 oracle on the seeded synthetic inputs (never the CUDA path).

    python tests/golden/make_golden.py

c0_embedding.txt / c1_embedding.txt: the pooled, L2-normalised embedding of
the two smallest benchmark configurations (1-layer 384-d encoder at batch 1,
seq 16, 11 valid tokens; and the 6-layer 384-d encoder of the paper's
Section 8.2 inference benchmark at batch 1, seq 128).  The paper prints no
worked numeric example of any encoder quantity, so these are regression
anchors for the oracle (and ready-made references for the GPU tests), not
values taken from the paper.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import oracle  # noqa: E402
from synth.inputs import CONFIGS, make_inputs  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))

for name in ("c0", "c1"):
    inp = make_inputs(CONFIGS[name])
    out = oracle.encoder_forward(inp.cfg, inp.ids, inp.mask, inp.params, inp.layers)
    path = os.path.join(HERE, f"{name}_embedding.txt")
    with open(path, "w") as f:
        f.write(f"# oracle output for config {name} (seed {inp.cfg.seed}); written by make_golden.py\n")
        f.write(f"# shape {out.shape[0]} x {out.shape[1]}, valid lengths {inp.lengths.tolist()}\n")
        for v in out.reshape(-1):
            f.write(f"{v:.17g}\n")
    print("wrote", path)
