"""Pins for the oracle's normal-equations form of the data-consistency step (Eq. 3 with
A^H (A x - y) = A^H A x - A^H y and the zero-filled image aty = A^H y given).  Expected values come
from dense matrices assembled from the explicit DFT formula, from the separately pinned
oracle.dc_forward / oracle.dc_vjp / oracle.apply_AH, and from exact linearity; none from the
function under test."""
import numpy as np
import pytest

from oracle.oracle import MASK_FULL
from tests.test_oracle_bridge import _dense_A
from tests.test_oracle_pins import crandn, small_problem


@pytest.mark.parametrize("rank,n", [(2, (1, 4, 6)), (2, (1, 3, 5)), (3, (2, 4, 6))])
def test_against_dense_matrix(oracle, rank, n):
    d, x, y, sens, mask = small_problem(rank=rank, n=n, B=1, C=3, T=1, mask_kind=MASK_FULL, weighted=True)
    aty = crandn(*d.image_shape(), rng=np.random.default_rng(5)).astype(np.complex64)     # any image, not only A^H y
    A = _dense_A(d, sens, mask)
    xv, av = x.astype(complex).ravel(), aty.astype(complex).ravel()
    eta = 0.8
    ref = xv - eta * (A.conj().T @ (A @ xv) - av)
    got = oracle.dc_forward_aty(x, aty, sens, mask, eta, d).ravel()
    assert np.abs(got - ref).max() <= 1e-13 * max(1.0, np.abs(ref).max())


@pytest.mark.parametrize("case", [dict(rank=2, n=(1, 6, 8)), dict(rank=3, n=(4, 6, 10), T=1),
                                  dict(rank=2, n=(1, 5, 12), weighted=True, sens_has_frames=1, T=3),
                                  dict(rank=3, n=(2, 6, 4), mask_kind=MASK_FULL, weighted=True, B=2)])
def test_equals_the_step_when_aty_is_the_zero_filled_image(oracle, case):
    """With aty = A^H y the two forms of Eq. 3 agree; the only difference is the rounding of aty to single."""
    d, x, y, sens, mask = small_problem(**case)
    aty_exact = oracle.apply_AH(y.astype(np.complex128) * 1.0, sens, mask, d)
    aty = aty_exact.astype(np.complex64)
    eta = 0.6
    ref = oracle.dc_forward(x, y, sens, mask, eta, d)
    got = oracle.dc_forward_aty(x, aty, sens, mask, eta, d)
    rounding = eta * np.abs(aty.astype(np.complex128) - aty_exact).max()
    assert np.abs(got - ref).max() <= rounding + 1e-12
    assert rounding < 1e-6 * max(1.0, np.abs(aty_exact).max())


def test_zero_image_gives_the_vjp_and_the_form_is_linear_in_aty(oracle):
    d, x, y, sens, mask = small_problem(rank=2, n=(1, 6, 10), B=2, C=3, T=2)
    eta = 0.9
    zero = np.zeros(d.image_shape(), np.complex64)
    base = oracle.dc_forward_aty(x, zero, sens, mask, eta, d)
    assert np.abs(base - oracle.dc_vjp(x, sens, mask, eta, d)).max() == 0.0
    rng = np.random.default_rng(9)
    a1 = (rng.integers(-8, 9, size=d.image_shape()) + 1j * rng.integers(-8, 9, size=d.image_shape())).astype(np.complex64) / 4
    got = oracle.dc_forward_aty(x, a1, sens, mask, eta, d)
    assert np.abs((got - base) - eta * a1.astype(np.complex128)).max() <= 1e-13
