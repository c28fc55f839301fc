"""GPU parity of gleam_dc_forward_aty (Eq. 3 in normal-equations form, out = x - eta (A^H A x - aty))
against the CPU oracle on every kernel path that writes the step's output, and its agreement with
gleam_dc_forward when aty is the zero-filled image from gleam_dc_adjoint.  Tolerances as for the
other parity tests: relative L2 <= 2e-5, max abs <= 1e-4 max|x|."""
import numpy as np
import pytest

from oracle.oracle import MASK_FULL, MASK_READOUT_INVARIANT
from paper_2207_08393_b200 import workloads as wl
from tests.gpu_common import assert_close
from tests.test_gpu_parity import crandn, problem, workload_case

pytestmark = pytest.mark.gpu


def run_aty(d, x, aty, sens, mask, eta, in_place=False, alias_aty=False):
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    tx, ts, tm = (torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in (x, sens, mask))
    ta = tx if alias_aty else torch.from_numpy(np.ascontiguousarray(aty)).to(dev)
    dc = g.DataConsistency(d.batch, d.coils, d.frames, d.fft_rank, d.n, d.sens_has_frames, d.mask_kind)
    out = tx if in_place else torch.full_like(tx, float("nan"))
    dc.forward_aty(tx, ta, ts, tm, eta, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


CASES = [
    (2, 2, 5, 3, (1, 24, 160), MASK_READOUT_INVARIANT, 0),      # units numbered across coils, single-warp blocks
    (2, 1, 5, 20, (1, 192, 160), MASK_READOUT_INVARIANT, 1),    # one block per SM, one group split over four warps (1, 1, 1, 2 coils)
    (2, 1, 4, 2, (1, 10, 64), MASK_READOUT_INVARIANT, 1),       # four lines per warp
    (2, 2, 3, 1, (1, 12, 320), MASK_READOUT_INVARIANT, 0),      # one line per warp
    (2, 1, 3, 1, (1, 6, 384), MASK_READOUT_INVARIANT, 0),       # three-stage plan: block-synchronised row kernel
    (2, 1, 3, 2, (1, 8, 368), MASK_READOUT_INVARIANT, 0),
    (2, 2, 3, 1, (1, 12, 16), MASK_FULL, 0),
    (3, 1, 3, 1, (6, 64, 32), MASK_READOUT_INVARIANT, 0),       # row-tile passes
    (3, 1, 2, 2, (4, 10, 12), MASK_READOUT_INVARIANT, 1),       # plain separable passes
    (3, 1, 3, 1, (4, 6, 10), MASK_FULL, 0),
]


@pytest.mark.parametrize("case", CASES)
def test_against_oracle_for_any_image(oracle, case):
    rank, B, C, T, n, kind, shf = case
    d, x, y, sens, mask = problem(rank, B, C, T, n, kind, sens_has_frames=shf, weighted=(kind == MASK_FULL), seed=41 + sum(n))
    aty = crandn(np.random.default_rng(7), *d.image_shape())
    ref = oracle.dc_forward_aty(x, aty, sens, mask, 0.8, d, nthreads=8)
    assert_close(run_aty(d, x, aty, sens, mask, 0.8), ref, x, "forward_aty %s" % (n,))
    assert_close(run_aty(d, x, aty, sens, mask, 0.8, in_place=True), ref, x, "forward_aty in place %s" % (n,))
    ref_alias = oracle.dc_forward_aty(x, x, sens, mask, 0.8, d, nthreads=8)
    assert_close(run_aty(d, x, x, sens, mask, 0.8, alias_aty=True), ref_alias, x, "forward_aty, aty aliases x %s" % (n,))


@pytest.mark.parametrize("name", ["cine", "brain2d"])
def test_workload_with_the_zero_filled_image(oracle, name):
    """aty from gleam_dc_adjoint, then the step: against the oracle's step with y itself (Eq. 3 as written)."""
    import torch
    import paper_2207_08393_b200 as g
    w, d, inp, mask, y = workload_case(oracle, name, MASK_READOUT_INVARIANT)
    dev = torch.device("cuda:0")
    tx, ty, ts, tm = (torch.from_numpy(a).to(dev) for a in (inp["x"], y, inp["sens"], mask))
    dc = g.DataConsistency(w.batch, w.coils, w.frames, w.fft_rank, w.n)
    aty = dc.adjoint(ty, ts, tm)
    out = dc.forward_aty(tx, aty, ts, tm, w.eta)
    ref = oracle.dc_forward(inp["x"], y, inp["sens"], mask, w.eta, d, nthreads=8)
    assert_close(out.cpu().numpy(), ref, inp["x"], name + " forward via A^H y")
    fwd = dc.forward(tx, ty, ts, tm, w.eta)
    assert_close(out.cpu().numpy(), fwd.cpu().numpy().astype(np.complex128), inp["x"], name + " both forms on the GPU")


def test_knee3d_small_volume_with_the_zero_filled_image(oracle):
    import torch
    import paper_2207_08393_b200 as g
    w = wl.scaled(wl.WORKLOADS["knee3d"], n=(8, 128, 64), center=8)
    inp = wl.make_inputs(w)
    from oracle.oracle import Dims
    d = Dims(w.batch, w.coils, w.frames, 3, w.n, 0, MASK_READOUT_INVARIANT)
    y = oracle.apply_A(inp["x_true"], inp["sens"], inp["mask"], d, nthreads=8).astype(np.complex64)
    dev = torch.device("cuda:0")
    tx, ty, ts, tm = (torch.from_numpy(a).to(dev) for a in (inp["x"], y, inp["sens"], inp["mask"]))
    dc = g.DataConsistency(w.batch, w.coils, w.frames, 3, w.n)
    aty = dc.adjoint(ty, ts, tm)
    out = dc.forward_aty(tx, aty, ts, tm, w.eta)
    ref = oracle.dc_forward(inp["x"], y, inp["sens"], inp["mask"], w.eta, d, nthreads=8)
    assert_close(out.cpu().numpy(), ref, inp["x"], "3-D forward via A^H y")


def test_errors():
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    d, x, y, sens, mask = problem(2, 1, 2, 1, (1, 8, 16), MASK_READOUT_INVARIANT)
    tx, ts, tm = (torch.from_numpy(a).to(dev) for a in (x, sens, mask))
    dc = g.DataConsistency(1, 2, 1, 2, (1, 8, 16))
    out = torch.empty_like(tx)
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward_aty(tx, None, ts, tm, 1.0, out, dc.dims())
    assert e.value.status == g.binding.GLEAM_ERR_NULL_POINTER
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward_aty(tx, out, ts, tm, 1.0, out, dc.dims())        # aty overlaps the output
    assert e.value.status == g.binding.GLEAM_ERR_ALIAS
