"""Writes tests/golden/delta_v1_bits.txt: bit patterns of softplus and delta under the delta-v1 operation
order, for a fixed grid of (z, A), computed by the CPU oracle only. The paper prints no worked numbers for
Eq. (delta_calc); this file guards the build's own fp32 specification against drift.

    python tests/golden/make_delta_golden.py
"""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
import oracle  # noqa: E402


def bits(x):
    return "%08x" % int(np.float32(x).view(np.uint32))


def main():
    zs = [0.0, -0.0, 1e-30, -1e-30, 0.5, -0.5, 1.0, -1.0, 2.5, -2.5, 6.0, -6.0, 20.0, -20.0, 86.9, -86.9,
          0.34657359, -0.34657359, 0.69314718, 1.0397208, 3.1415927, -3.1415927]
    As = [0.5, 1.0, 1.37, 2.0]
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "delta_v1_bits.txt")
    with open(out, "w") as f:
        f.write("# z_bits A_bits softplus_bits delta_bits  (fp32 bit patterns, hex); delta = exp(A*softplus(z)), Eq. (delta_calc)\n")
        for z in zs:
            for a in As:
                sp = np.float32(oracle.softplus_spec(z))
                dl = oracle.exp_spec(np.float32(a) * sp)
                f.write(f"{bits(z)} {bits(a)} {bits(sp)} {bits(dl)}\n")


if __name__ == "__main__":
    main()
