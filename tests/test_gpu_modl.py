"""GPU parity of the MoDL model inversion (Eq. 7): gleam_modl_cg_forward / gleam_modl_cg_vjp through
the C ABI against the CPU oracle's conjugate-gradient solve, element by element on the same
seeded inputs.

Tolerance: relative L2 <= 2e-5, max abs error <= 1e-4 * max|oracle result| (the bound of the
gradient data-consistency step).  One operator application in single precision deviates by about
1e-7 (relative) from the double-precision one; the conjugate-gradient recurrences amplify
perturbations of their vectors by at most about the condition number of A^H A + mu I
(<= (1 + mu) / mu = 21 for the paper's mu = 0.05 with unit-norm sensitivities), and since the
inner products are accumulated in double precision the steps do not add to it: 21 * 1e-7 = 2e-6
(measured on the full-size workloads: 1.8e-6 after 10 and after 30 steps), a factor 10 of margin.
"""
import numpy as np
import pytest

from oracle.oracle import Dims, MASK_FULL, MASK_READOUT_INVARIANT
from paper_2207_08393_b200 import workloads as wl
from tests.gpu_common import run_gpu_modl
from tests.test_gpu_parity import crandn, workload_case

pytestmark = pytest.mark.gpu

REL_L2_TOL = 2e-5
MAX_ABS_TOL = 1e-4


def close(got, ref, what):
    got = np.asarray(got).astype(np.complex128)
    assert np.isfinite(got.view(np.float64)).all(), what + ": non-finite output"
    scale = max(np.abs(ref).max(), 1e-300)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
    mab = np.abs(got - ref).max() / scale
    assert rel <= REL_L2_TOL, "%s: rel L2 %.3e > %.1e" % (what, rel, REL_L2_TOL)
    assert mab <= MAX_ABS_TOL, "%s: max abs %.3e > %.1e (units of max|result|)" % (what, mab, MAX_ABS_TOL)
    return rel


def problem(rank, B, C, T, n, mask_kind, sens_has_frames=0, weighted=False, seed=0, density=0.4):
    rng = np.random.default_rng(seed)
    d = Dims(B, C, T, rank, tuple(n), sens_has_frames, mask_kind)
    z = crandn(rng, *d.image_shape()); y = crandn(rng, *d.kspace_shape())
    sens = crandn(rng, *d.sens_shape())
    sens = (sens / np.sqrt(np.sum(np.abs(sens) ** 2, axis=1, keepdims=True))).astype(np.complex64)
    if weighted:
        mask = rng.uniform(0, 1, d.mask_shape()).astype(np.float32)
    else:
        mask = (rng.uniform(size=d.mask_shape()) < density).astype(np.float32)
    return d, z, y, sens, mask


def check(oracle, d, z, y, sens, mask, mu, n_iter, what, in_place=False):
    ref = oracle.modl_cg_forward(z, y, sens, mask, mu, n_iter, d, nthreads=8)
    got = run_gpu_modl(z, y, sens, mask, mu, n_iter, d.fft_rank, d.sens_has_frames, d.mask_kind, in_place=in_place)
    close(got, ref, what + " solve")
    refv = oracle.modl_cg_vjp(z, sens, mask, mu, n_iter, d, nthreads=8)
    gotv = run_gpu_modl(z, None, sens, mask, mu, n_iter, d.fft_rank, d.sens_has_frames, d.mask_kind, in_place=in_place)
    close(gotv, refv, what + " vjp")


@pytest.mark.parametrize("n_iter", [1, 2, 3, 10])
@pytest.mark.parametrize("mu", [0.05, 4.0])            # the paper's values for R = 16 and R = 4
def test_rank2_steps_and_mu(oracle, n_iter, mu):
    d, z, y, sens, mask = problem(2, 2, 4, 1, (1, 48, 40), MASK_READOUT_INVARIANT, seed=n_iter)
    check(oracle, d, z, y, sens, mask, mu, n_iter, "rank2 k=%d mu=%g" % (n_iter, mu))


@pytest.mark.parametrize("case", [
    (2, 3, 3, 2, (1, 20, 46), MASK_READOUT_INVARIANT, 1, False),     # per-frame sensitivities, three examples
    (2, 2, 3, 2, (1, 64, 46), MASK_FULL, 0, True),                   # full weighted mask
    (3, 2, 3, 1, (6, 64, 32), MASK_READOUT_INVARIANT, 0, False),     # row-tile 3-D path
    (3, 1, 2, 2, (4, 6, 8), MASK_FULL, 1, False),
    (3, 2, 3, 1, (10, 46, 32), MASK_READOUT_INVARIANT, 0, True),
    (2, 1, 2, 1, (1, 2, 2), MASK_READOUT_INVARIANT, 0, False),       # smallest supported image
    (2, 2, 3, 2, (1, 16, 320), MASK_READOUT_INVARIANT, 0, False),    # three-stage row plan: <p,q> by its own kernel
    (2, 3, 2, 1, (1, 10, 160), MASK_READOUT_INVARIANT, 0, True),     # <p,q> per row from the operator, ragged line groups
])
def test_shapes_and_masks(oracle, case):
    rank, B, C, T, n, kind, shf, weighted = case
    d, z, y, sens, mask = problem(rank, B, C, T, n, kind, sens_has_frames=shf, weighted=weighted, seed=sum(n))
    check(oracle, d, z, y, sens, mask, 0.05, 10, "case %s" % (case,))


def test_in_place_and_determinism(oracle):
    d, z, y, sens, mask = problem(2, 2, 3, 2, (1, 32, 24), MASK_READOUT_INVARIANT, seed=4)
    check(oracle, d, z, y, sens, mask, 0.05, 6, "in place", in_place=True)
    a = run_gpu_modl(z, y, sens, mask, 0.05, 10, 2, 0, MASK_READOUT_INVARIANT)
    b = run_gpu_modl(z, y, sens, mask, 0.05, 10, 2, 0, MASK_READOUT_INVARIANT)
    assert np.array_equal(a.view(np.float32), b.view(np.float32))


def test_examples_are_independent_systems(oracle):
    """An example's result does not depend on the rest of the batch."""
    d, z, y, sens, mask = problem(2, 3, 3, 1, (1, 32, 24), MASK_READOUT_INVARIANT, seed=9)
    z[1] *= 50.0                                         # a very different scale in the middle example
    both = run_gpu_modl(z, y, sens, mask, 0.05, 5, 2, 0, MASK_READOUT_INVARIANT)
    for b in range(3):
        alone = run_gpu_modl(z[b:b + 1], y[b:b + 1], sens[b:b + 1], mask[b:b + 1], 0.05, 5, 2, 0, MASK_READOUT_INVARIANT)
        close(both[b:b + 1], alone.astype(np.complex128), "example %d" % b)


def test_degenerate_inputs():
    d, z, y, sens, mask = problem(2, 2, 2, 1, (1, 8, 8), MASK_READOUT_INVARIANT, seed=1)
    out = run_gpu_modl(np.zeros_like(z), np.zeros_like(y), sens, mask, 0.05, 10, 2, 0, MASK_READOUT_INVARIANT)
    assert np.all(out == 0)                              # zero right-hand side: exactly zero, no NaN
    out = run_gpu_modl(z, y, sens, mask, 0.05, 0, 2, 0, MASK_READOUT_INVARIANT)
    assert np.all(out == 0)                              # no steps: the starting point
    zz = z.copy(); zz[1] = 0; yy = y.copy(); yy[1] = 0   # one example with a zero right-hand side
    out = run_gpu_modl(zz, yy, sens, mask, 0.05, 4, 2, 0, MASK_READOUT_INVARIANT)
    assert np.all(out[1] == 0) and np.isfinite(out.view(np.float32)).all() and np.abs(out[0]).max() > 0


def test_identity_normal_operator():
    """Full mask, unit-norm sensitivities: A^H A = I, so grad_z = mu / (1 + mu) g after one step."""
    d, z, y, sens, mask = problem(2, 2, 4, 1, (1, 64, 46), MASK_READOUT_INVARIANT, seed=3)
    mask[:] = 1.0
    mu = 0.7
    got = run_gpu_modl(z, None, sens, mask, mu, 1, 2, 0, MASK_READOUT_INVARIANT)
    close(got, mu / (1 + mu) * z.astype(np.complex128), "identity")


@pytest.mark.parametrize("name,mu", [("slice64", 0.05), ("knee2d", 0.05), ("knee2d", 4.0), ("cine", 0.05)])
def test_workloads_ten_steps(oracle, name, mu):
    """The paper's MoDL settings: 10 CG steps, mu = 0.05 (R = 16, and the cine network) or 4.0 (R = 4),
    on the knee-like 2-D workload and the cine workload at full size."""
    w, d, inp, mask, y = workload_case(oracle, name)
    ref = oracle.modl_cg_forward(inp["x"], y, inp["sens"], mask, mu, 10, d, nthreads=8)
    got = run_gpu_modl(inp["x"], y, inp["sens"], mask, mu, 10, w.fft_rank, 0, MASK_READOUT_INVARIANT)
    close(got, ref, name + " solve")
    refv = oracle.modl_cg_vjp(inp["g"], inp["sens"], mask, mu, 10, d, nthreads=8)
    gotv = run_gpu_modl(inp["g"], None, inp["sens"], mask, mu, 10, w.fft_rank, 0, MASK_READOUT_INVARIANT)
    close(gotv, refv, name + " vjp")


def test_error_codes():
    import torch
    import paper_2207_08393_b200 as g
    from paper_2207_08393_b200 import binding
    dev = torch.device("cuda:0")
    z = torch.zeros((1, 1, 1, 8, 8), dtype=torch.complex64, device=dev)
    y = torch.zeros((1, 2, 1, 1, 8, 8), dtype=torch.complex64, device=dev)
    s = torch.zeros((1, 2, 1, 8, 8), dtype=torch.complex64, device=dev)
    m = torch.ones((1, 1, 8), dtype=torch.float32, device=dev)
    out = torch.empty_like(z)
    probe = g.make_dims(1, 2, 1, 2, (1, 8, 8))
    nbytes = g.gleam_modl_cg_workspace_size(probe)
    assert nbytes > g.gleam_dc_workspace_size(probe) + 3 * z.numel() * 8
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    d = g.make_dims(1, 2, 1, 2, (1, 8, 8), stream=torch.cuda.current_stream(), workspace=ws)
    for mu, n_iter in ((0.0, 10), (-1.0, 10), (float("nan"), 10), (0.05, -1), (0.05, 1001)):
        with pytest.raises(g.GleamError) as e:
            g.gleam_modl_cg_forward(z, y, s, m, mu, n_iter, out, d)
        assert e.value.status == binding.GLEAM_ERR_BAD_DIMS
    small = g.make_dims(1, 2, 1, 2, (1, 8, 8), workspace=ws.data_ptr(), workspace_bytes=nbytes - 256)
    with pytest.raises(g.GleamError) as e:
        g.gleam_modl_cg_forward(z, y, s, m, 0.05, 10, out, small)
    assert e.value.status == binding.GLEAM_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(g.GleamError) as e:
        g.gleam_modl_cg_forward(z, None, s, m, 0.05, 10, out, d)
    assert e.value.status == binding.GLEAM_ERR_NULL_POINTER
    with pytest.raises(g.GleamError) as e:                       # output inside the workspace
        g.gleam_modl_cg_forward(z, y, s, m, 0.05, 10, ws.data_ptr() + 512, d)
    assert e.value.status == binding.GLEAM_ERR_ALIAS
    g.gleam_modl_cg_forward(z, y, s, m, 0.05, 10, z, d)          # exact alias is allowed
    torch.cuda.synchronize()

