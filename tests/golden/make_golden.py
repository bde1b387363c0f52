"""Writes tests/golden/c1_tiny_samples.txt: sampled outputs of the tiny
configuration computed by the CPU oracle alone (no CUDA code is involved).
Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import oracle                                    # noqa: E402
from paper_2304_04237_b200 import synth          # noqa: E402


def main():
    cfg, x = synth.make_config("c1_tiny")
    out = oracle.forward(x["q"], x["k"], x["v"], x["wk"], x["wv"], x["bias"], cfg["ksize"]).reshape(-1)
    idx = np.unique(np.concatenate([np.arange(0, out.size, 397), [0, 31, 32, out.size - 1]]))
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_tiny_samples.txt")
    with open(path, "w") as f:
        f.write("# flat index into out[1,14,14,1,32] and its value; tiny configuration\n"
                "# (B=1, H=W=14, 1 head x 32, k=3, fp32 inputs, seeded synthetic data);\n"
                "# source: the CPU oracle (Eq. 2 with the depthwise keys/values of Eq. 12), float64\n")
        for i in idx:
            f.write(f"{int(i)} {out[i]:.17g}\n")
    print("wrote", path, len(idx), "values")


if __name__ == "__main__":
    main()
