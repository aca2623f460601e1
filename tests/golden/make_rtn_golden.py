"""Writes tests/golden/rtn_groups.txt from the CPU oracle alone (no CUDA code is involved).

The paper prints no worked numeric example of its quantizer, so this fixture is not a pin of the
oracle against the paper: it freezes what the oracle answers today on a small closed-form input, so
that a later change to the oracle's arithmetic or bit layout cannot pass unnoticed (such a change has
to regenerate this file in the same commit and say why).  Run from the repository root:

    python tests/golden/make_rtn_golden.py
"""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
from oracle import rosaq_oracle as orc  # noqa: E402


def closed_form_weights():
    """[256][4] fp32: column 0 a ramp, 1 a sine, 2 all-positive (zero-point clamps), 3 constant."""
    k = np.arange(256, dtype=np.float64)
    W = np.stack([0.001 * (k - 100.0), 0.05 * np.sin(0.37 * k), 0.02 + 0.0003 * k, np.full(256, 0.125)], axis=1)
    return W.astype(np.float32)


def main():
    W = closed_form_weights()
    lines = []
    for bits in (4, 3):
        qd = orc.quantize(W, bits, 128, 128)
        qw = orc.pack(qd["codes"], bits)
        lines.append(f"bits {bits}")
        lines.append("scales " + " ".join(f"{v:04x}" for v in qd["scales"].view(np.uint16).ravel()))
        lines.append("zeros " + " ".join(f"{v:04x}" for v in qd["zeros"].view(np.uint16).ravel()))
        lines.append("salient_row0 " + " ".join(f"{v:04x}" for v in qd["salient"].view(np.uint16)[0]))
        for r in range(qw.shape[0]):
            lines.append(f"qw{r} " + " ".join(f"{v:08x}" for v in qw[r]))
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "rtn_groups.txt"), "w") as f:
        f.write("# oracle.quantize + oracle.pack on closed_form_weights() of make_rtn_golden.py, K = 128, g = 128\n")
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
