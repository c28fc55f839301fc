"""Small, seeded invocation of the data-consistency step for profiler captures.

    python -m paper_2207_08393_b200.profile_case knee3d_small    # 8 coils, 20x320x256
    python -m paper_2207_08393_b200.profile_case cine            # 8 coils, 20 frames of 192x160

Runs three forward + VJP pairs through the C ABI on random inputs of the workload's shape and
mask density.  The 3-D case keeps the full 320x256 phase-encode plane (so the kernels and their
launch shapes are those of the full workload) but only 20 readout slabs: about 0.4 GB on the
device, larger than L2, small enough for multi-pass counter collection.
"""
import sys

import numpy as np
import torch

import paper_2207_08393_b200 as g

CASES = {
    "knee3d_small": (1, 8, 1, 3, (20, 320, 256), 1.0 / 12.0),
    "cine": (1, 8, 20, 2, (1, 192, 160), 0.1),
}


def main(name="knee3d_small", reps=3):
    B, C, T, rank, n, density = CASES[name]
    rng = np.random.default_rng(0)
    dev = torch.device("cuda:0")

    def c64(*s):
        a = rng.standard_normal(s, dtype=np.float32) + 1j * rng.standard_normal(s, dtype=np.float32)
        return torch.from_numpy(a.astype(np.complex64)).to(dev)

    x, y, s = c64(B, T, *n), c64(B, C, T, *n), c64(B, C, *n)
    mshape = (B, T, n[2]) if rank == 2 else (B, T, n[1], n[2])
    m = torch.from_numpy((rng.uniform(size=mshape) < density).astype(np.float32)).to(dev)
    dc = g.DataConsistency(B, C, T, rank, n)
    out = torch.empty_like(x)
    for _ in range(reps):
        dc.forward(x, y, s, m, 1.0, out)
        dc.vjp(x, s, m, 1.0, out)
    torch.cuda.synchronize()
    print("ok", name)


if __name__ == "__main__":
    main(*(sys.argv[1:2] or ["knee3d_small"]))
