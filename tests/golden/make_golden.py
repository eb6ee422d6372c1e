"""Writes the stored expected values under tests/golden/ by calling only the CPU oracle
(never the CUDA path).  Run from the repository root: ``python tests/golden/make_golden.py``.

c1_actions.txt : final action chunk [16 x 7] of the tiny fp32 configuration (2 layers, width
                 256, 4 Euler steps from t = 1, prefix 64), inputs from the seeded generator.
                 The paper prints no worked example of the expert, so this file guards the
                 oracle against accidental change; it is not a value from the paper.
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import expert_oracle as O            # noqa: E402
from paper_2608_03682_b200 import synth          # noqa: E402


def main():
    cfg = synth.tiny_config()
    W = synth.make_weights(cfg, 1)
    kv, state, noise = synth.make_prefix_kv(cfg, 1, 64), synth.make_state(cfg, 1), synth.make_noise(cfg, 1)
    out = O.denoise(cfg, W, kv, 64, state, noise, 4)
    np.savetxt(os.path.join(os.path.dirname(__file__), "c1_actions.txt"), out, fmt="%.17e",
               header="oracle output, tiny fp32 configuration, 4 Euler steps; written by make_golden.py")


if __name__ == "__main__":
    main()
