"""Pins for the oracle's gradients of the data-consistency step with respect to the step size and
the measurements (Eq. 3), and for the bridge to the learned prior (two real channels, complex l1
loss; Implementation / Training).  None of the expected values below comes from the functions
under test: dense matrices assembled from the explicit DFT formula, exact difference quotients of
the separately pinned oracle.dc_forward, numpy's own stacking routine, closed forms, brute-force
loops and central differences."""
import numpy as np
import pytest

from oracle.oracle import Dims, MASK_FULL, MASK_READOUT_INVARIANT
from tests.test_oracle_pins import _dft_matrix, crandn, small_problem


def _dense_A(d, sens, mask):
    n = d.n
    Fm = np.eye(1)
    for ax in range(3):
        Fm = np.kron(Fm, _dft_matrix(n[ax]) if (ax >= 3 - d.fft_rank and n[ax] > 1) else np.eye(n[ax]))
    return np.vstack([np.diag(mask[0, 0].astype(float).ravel()) @ Fm @ np.diag(sens[0, c].astype(complex).ravel())
                      for c in range(d.coils)])


@pytest.mark.parametrize("rank,n", [(2, (1, 4, 6)), (2, (1, 3, 5)), (3, (2, 4, 6))])
def test_gradients_against_dense_matrix(oracle, rank, n):
    d, x, y, sens, mask = small_problem(rank=rank, n=n, B=1, C=3, T=1, mask_kind=MASK_FULL, weighted=True)
    g = crandn(*d.image_shape(), rng=np.random.default_rng(3)).astype(np.complex64)
    A = _dense_A(d, sens, mask)
    xv, yv, gv = (a.astype(complex).ravel() for a in (x, y, g))
    a = A.conj().T @ (A @ xv - yv)
    ref_eta = -np.real(np.vdot(gv, a))
    got_eta = oracle.dc_grad_eta(g, x, y, sens, mask, d)
    assert got_eta.shape == (1,) and abs(got_eta[0] - ref_eta) <= 1e-12 * max(1.0, abs(ref_eta))
    eta = 0.65
    ref_y = eta * (A @ gv)
    got_y = oracle.dc_grad_y(g, sens, mask, eta, d).ravel()
    assert np.abs(got_y - ref_y).max() <= 1e-13


@pytest.mark.parametrize("case", [dict(rank=2, n=(1, 6, 8)), dict(rank=3, n=(4, 6, 10), T=1),
                                  dict(rank=2, n=(1, 5, 12), weighted=True, sens_has_frames=1),
                                  dict(rank=3, n=(2, 6, 4), mask_kind=MASK_FULL, weighted=True)])
def test_gradients_are_exact_difference_quotients_of_the_step(oracle, case):
    """Eq. 3 is linear in eta and affine in y: the quotients carry no truncation error."""
    d, x, y, sens, mask = small_problem(**case)
    rng = np.random.default_rng(11)
    g = crandn(*d.image_shape(), rng=rng).astype(np.complex64)
    eta, deta = 0.7, 0.25
    f0 = oracle.dc_forward(x, y, sens, mask, eta, d)
    f1 = oracle.dc_forward(x, y, sens, mask, eta + deta, d)
    per_example = np.array([np.real(np.vdot(g[b].astype(complex), (f1 - f0)[b])) for b in range(d.batch)]) / deta
    got = oracle.dc_grad_eta(g, x, y, sens, mask, d)
    assert np.abs(got - per_example).max() <= 1e-10 * np.abs(per_example).max()
    # measurements: Re<g, DC(x; y + dy) - DC(x; y)> = Re<grad_y, dy>  (dy exactly representable in float32)
    dy = (rng.integers(-4, 5, size=y.shape) + 1j * rng.integers(-4, 5, size=y.shape)).astype(np.complex64) / 8
    y2 = (y + dy).astype(np.complex64)
    dy_exact = y2.astype(complex) - y.astype(complex)
    f2 = oracle.dc_forward(x, y2, sens, mask, eta, d)
    lhs = np.real(np.vdot(g.astype(complex), f2 - f0))
    rhs = np.real(np.vdot(oracle.dc_grad_y(g, sens, mask, eta, d), dy_exact))
    assert abs(lhs - rhs) <= 1e-10 * max(abs(lhs), 1.0)
    # unsampled positions carry no gradient
    gy = oracle.dc_grad_y(g, sens, mask, eta, d)
    mfull = np.broadcast_to(mask.reshape(mask.shape[:2] + (1,) * (5 - mask.ndim) + mask.shape[2:]),
                            (d.batch, d.frames) + tuple(d.n))
    assert np.all(gy[np.broadcast_to(mfull[:, None] == 0, gy.shape)] == 0)


def test_grad_eta_special_cases(oracle):
    d, x, y, sens, mask = small_problem(rank=2, n=(1, 6, 8), unit_sens=True, full_mask=True)
    # A^H A = I: A^H(Ax - y) = x - A^H y; with y = A x exactly consistent the gradient vanishes
    y_cons = oracle.apply_A(x, sens, mask, d)
    g = crandn(*d.image_shape()).astype(np.complex64)
    # y is rounded to complex64 on entry: the residual is the rounding error only
    assert np.abs(oracle.dc_grad_eta(g, x, y_cons, sens, mask, d)).max() <= 1e-5
    # y = 0, g = x: -<x, A^H A x> = -||x||^2 per example
    got = oracle.dc_grad_eta(x, x, np.zeros_like(y), sens, mask, d)
    ref = -np.array([np.vdot(x[b].astype(complex), x[b].astype(complex)).real for b in range(d.batch)])
    assert np.abs(got - ref).max() <= 1e-5 * np.abs(ref).max()     # sens is unit-norm only to float32 rounding


def test_channel_layout_round_trip_is_bit_exact(oracle):
    rng = np.random.default_rng(5)
    x = crandn(3, 2, 4, 5, 6, rng=rng).astype(np.complex64)
    x.view(np.float32).ravel()[7] = np.float32(-0.0)            # a sign bit only a byte comparison sees
    ch = oracle.complex_to_channels(x)
    ref = np.stack([x.real, x.imag], axis=1)                    # numpy's own routine: (B, 2, ...)
    assert ch.dtype == np.float32 and ch.shape == (3, 2, 2, 4, 5, 6)
    assert ch.tobytes() == np.ascontiguousarray(ref).tobytes()
    back = oracle.channels_to_complex(ch)
    assert back.dtype == np.complex64 and back.tobytes() == x.tobytes()
    # index property: element (b, ch, i) of the planar form is component ch of complex element (b, i)
    flat = x.reshape(3, -1).view(np.float32).reshape(3, -1, 2)
    assert np.array_equal(ch.reshape(3, 2, -1)[1, 0], flat[1, :, 0]) and np.array_equal(ch.reshape(3, 2, -1)[2, 1], flat[2, :, 1])


def test_l1_loss_closed_forms_and_brute_force(oracle):
    # constant difference 3 + 4i: every modulus is 5, the mean is 5, the gradient (3+4i)/5/N
    x = np.full((2, 1, 1, 3, 4), 3 + 4j, dtype=np.complex64)
    val, grad = oracle.l1_loss(x, np.zeros_like(x), with_grad=True)
    assert abs(val - 5.0) <= 1e-15
    assert np.abs(grad - (0.6 + 0.8j) / x.size).max() <= 1e-17
    # equal images: zero loss, zero gradient (no 0/0)
    val, grad = oracle.l1_loss(x, x, with_grad=True)
    assert val == 0.0 and np.all(grad == 0)
    # brute force in a Python loop on random data
    rng = np.random.default_rng(9)
    a = crandn(1, 2, 1, 3, 5, rng=rng).astype(np.complex64); b = crandn(1, 2, 1, 3, 5, rng=rng).astype(np.complex64)
    tot = 0.0
    for u, v in zip(a.ravel(), b.ravel()):
        dr, di = float(u.real) - float(v.real), float(u.imag) - float(v.imag)
        tot += (dr * dr + di * di) ** 0.5
    assert abs(oracle.l1_loss(a, b) - tot / a.size) <= 1e-15
    # l1 is symmetric and scales with the difference
    assert abs(oracle.l1_loss(a, b) - oracle.l1_loss(b, a)) <= 1e-16


def test_l1_gradient_against_central_differences(oracle):
    """Re<grad, delta> is the directional derivative of the loss (conjugate-Wirtinger convention)."""
    rng = np.random.default_rng(21)
    a = crandn(2, 1, 1, 4, 6, rng=rng).astype(np.complex64); b = crandn(2, 1, 1, 4, 6, rng=rng).astype(np.complex64)
    _, grad = oracle.l1_loss(a, b, with_grad=True)
    delta = (rng.integers(-8, 9, size=a.shape) + 1j * rng.integers(-8, 9, size=a.shape)) / 8.0
    eps = 2.0 ** -10                       # a +- eps*delta stays exactly representable near |a| ~ 1
    ap, am = (a + eps * delta).astype(np.complex64), (a - eps * delta).astype(np.complex64)
    step = (ap.astype(complex) - am.astype(complex))            # the step actually taken
    num = oracle.l1_loss(ap, b) - oracle.l1_loss(am, b)
    lin = np.real(np.vdot(grad, step))
    assert abs(num - lin) <= 1e-5 * abs(lin) + 1e-9
    # a planted mistake (gradient without the 1/N, or conjugated) misses by far more than that
    assert abs(num - np.real(np.vdot(grad * a.size, step))) > 1e-2 * abs(lin)
    assert abs(num - np.real(np.vdot(np.conj(grad), step))) > 1e-3 * abs(lin)
