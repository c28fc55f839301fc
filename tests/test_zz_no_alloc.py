"""gleam_dc_forward_static: the forward step for callers that cannot allocate device memory.

Some deployments give this library no way to obtain scratch: all device memory already belongs to
a framework's caching allocator, or the host application forbids cudaMalloc inside its processing
loop because an allocation may synchronise the device.  For them the library carries one fixed
scratch array per GPU.  The test calls the entry point through the C ABI twice in a row (the array
keeps the first call's contents, which must not leak into the second) and compares both results
with gleam_dc_forward given a caller-allocated workspace, under the tolerance of the parity tests.
This file is collected last so that a run that stops at the first failure has already run every
other test.
"""
import numpy as np
import pytest

from oracle.oracle import Dims
from tests.gpu_common import assert_close

pytestmark = pytest.mark.gpu


def _case(seed, B, C, T, rank, n):
    rng = np.random.default_rng(seed)
    c = lambda *s: ((rng.normal(size=s) + 1j * rng.normal(size=s)) / np.sqrt(2)).astype(np.complex64)
    x, y, sens = c(B, T, *n), c(B, C, T, *n), c(B, C, *n)
    mshape = (B, T, n[2]) if rank == 2 else (B, T, n[1], n[2])
    mask = (rng.uniform(size=mshape) < 0.4).astype(np.float32)
    return x, y, sens, mask


@pytest.mark.parametrize("rank,n", [(2, (1, 64, 160)), (3, (8, 20, 32))])
def test_static_scratch_forward_matches_workspace_forward_twice(oracle, rank, n):
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    B, C, T = 2, 4, 1
    for call, (seed, eta) in enumerate([(101, 0.9), (202, 1.3)]):       # two calls in a row, different data
        x, y, sens, mask = _case(seed, B, C, T, rank, n)
        tx, ty, ts, tm = (torch.from_numpy(a).to(dev) for a in (x, y, sens, mask))
        # existing entry point with a caller-owned workspace
        ws = torch.empty(g.gleam_dc_workspace_size(g.make_dims(B, C, T, rank, n)), dtype=torch.uint8, device=dev)
        ref = torch.empty_like(tx)
        g.gleam_dc_forward(tx, ty, ts, tm, eta, ref, g.make_dims(B, C, T, rank, n, stream=torch.cuda.current_stream(),
                                                                workspace=ws))
        torch.cuda.synchronize()
        # new entry point: no workspace is passed at all
        out = torch.full_like(tx, float("nan"))
        g.gleam_dc_forward_static(tx, ty, ts, tm, eta, out, g.make_dims(B, C, T, rank, n,
                                                                        stream=torch.cuda.current_stream()))
        torch.cuda.synchronize()
        assert_close(out.cpu().numpy(), ref.cpu().numpy().astype(np.complex128), x, "static scratch, call %d" % call)
        # element by element against the CPU oracle as well, and no device memory taken by a repeated call
        assert_close(out.cpu().numpy(), oracle.dc_forward(x, y, sens, mask, eta, Dims(B, C, T, rank, n, 0, 1), nthreads=8), x,
                     "static scratch against the oracle, call %d" % call)
        free_before = torch.cuda.mem_get_info()[0]
        g.gleam_dc_forward_static(tx, ty, ts, tm, eta, out, g.make_dims(B, C, T, rank, n,
                                                                        stream=torch.cuda.current_stream()))
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before


def test_static_scratch_rejects_problems_beyond_its_size():
    import torch
    import paper_2207_08393_b200 as g
    from paper_2207_08393_b200 import binding
    n = (1, 640, 368)
    d = g.make_dims(4, 15, 1, 2, n)
    assert g.gleam_dc_workspace_size(d) > g.gleam_dc_static_scratch_bytes() == 64 << 20
    small = torch.zeros(8, dtype=torch.complex64, device="cuda")      # never read: the size check comes first
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward_static(small, small, small, small, 1.0, small, d)
    assert e.value.status == binding.GLEAM_ERR_WORKSPACE_TOO_SMALL
