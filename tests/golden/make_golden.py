"""Writes tests/golden/dc_tiny.json from the CPU oracle alone (no CUDA code is involved).

The paper (arXiv 2207.08393) prints no worked numeric example of the data-consistency step
(Eq. 3), so this stored value is a regression guard for the oracle, not a value from the paper.
Run:  python -m tests.golden.make_golden
"""
import json
import os

import numpy as np


def tiny_case():
    from oracle.oracle import Dims, MASK_FULL
    rng = np.random.default_rng(20220808)
    d = Dims(1, 2, 1, 2, (1, 4, 6), 0, MASK_FULL)
    c = lambda shape: ((rng.integers(-8, 9, shape) + 1j * rng.integers(-8, 9, shape)) / 8.0).astype(np.complex64)
    x, y, sens = c(d.image_shape()), c(d.kspace_shape()), c(d.sens_shape())
    mask = (rng.integers(0, 5, d.mask_shape()) / 4.0).astype(np.float32)
    return d, x, y, sens, mask, 0.75


def main():
    from oracle import oracle
    d, x, y, sens, mask, eta = tiny_case()
    f = oracle.dc_forward(x, y, sens, mask, eta, d).ravel()
    v = oracle.dc_vjp(x, sens, mask, eta, d).ravel()
    out = {"source": "oracle/gleam_oracle.c via tests/golden/make_golden.py (Eq. 3; no value printed in the paper)",
           "forward_re": f.real.tolist(), "forward_im": f.imag.tolist(),
           "vjp_re": v.real.tolist(), "vjp_im": v.imag.tolist()}
    with open(os.path.join(os.path.dirname(__file__), "dc_tiny.json"), "w") as fh:
        json.dump(out, fh, indent=0)


if __name__ == "__main__":
    main()
