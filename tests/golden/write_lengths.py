"""Writes lengths_cfg*.txt: the sequence-length draws of the seeded workload generators.

Calls only the input generator (no oracle, no CUDA).  Run from the repository root:
    python tests/golden/write_lengths.py
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import cf_synth as syn  # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))

if __name__ == "__main__":
    for name, fn in (("cfg2", syn.config2_lengths), ("cfg3", syn.config3_lengths),
                     ("cfg4", syn.config4_lengths), ("cfg5", syn.config5_lengths)):
        np.savetxt(os.path.join(HERE, f"lengths_{name}.txt"), fn(0), fmt="%d")
