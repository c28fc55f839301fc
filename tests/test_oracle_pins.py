"""Pins for the CPU oracle: what the paper's definitions and the mathematics fix, checked without
reference to the oracle's own code path (closed forms, brute force, invariants, an independent
library FFT).  The paper prints no worked numeric example of the data-consistency step, so there is
no printed value to compare with; every pin below is chosen so that a dropped term, a wrong sign,
a transposed operand or a wrong index fails at least one of them.

Citations: sensing model Eq. 1; A = Omega F S (text after Eq. 2); DC step Eq. 3.
"""
import numpy as np
import pytest

from oracle.oracle import Dims, MASK_FULL, MASK_READOUT_INVARIANT

RNG = np.random.default_rng(1234)


def crandn(*shape, rng=RNG):
    return (rng.normal(size=shape) + 1j * rng.normal(size=shape)) / np.sqrt(2)


def inner(a, b):
    return np.vdot(a, b)  # conj(a) . b


def small_problem(rank=2, B=2, C=3, T=2, n=(1, 6, 8), mask_kind=MASK_READOUT_INVARIANT, sens_has_frames=0,
                  unit_sens=False, full_mask=False, weighted=False, seed=7):
    rng = np.random.default_rng(seed)
    d = Dims(B, C, T, rank, tuple(n), sens_has_frames, mask_kind)
    sens = crandn(*d.sens_shape(), rng=rng)
    if unit_sens:
        sens = sens / np.sqrt(np.sum(np.abs(sens) ** 2, axis=1, keepdims=True))
    sens = sens.astype(np.complex64)
    if full_mask:
        mask = np.ones(d.mask_shape(), dtype=np.float32)
    elif weighted:
        mask = rng.uniform(0, 1, d.mask_shape()).astype(np.float32)
    else:
        mask = (rng.uniform(size=d.mask_shape()) < 0.45).astype(np.float32)
    x = crandn(*d.image_shape(), rng=rng).astype(np.complex64)
    y = crandn(*d.kspace_shape(), rng=rng).astype(np.complex64)
    return d, x, y, sens, mask


# ---------------------------------------------------------------------------------------------
# P1  brute force: shift + recursive FFT route == the definition by direct summation
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N", [1, 2, 3, 4, 5, 6, 8, 10, 12, 15, 16, 20, 23, 33, 34, 46, 64, 66, 160, 192, 368])
@pytest.mark.parametrize("sign", [-1, 1])
def test_fft_route_matches_direct_sum_1d(oracle, N, sign):
    v = crandn(N)
    a = oracle.dft_naive_1d(v, sign)
    b = oracle.fft_centered_1d(v, sign)
    assert np.abs(a - b).max() <= 1e-12 * max(1.0, np.abs(a).max())


@pytest.mark.parametrize("shape,rank", [((4, 6), 2), ((3, 5), 2), ((34, 36), 2), ((2, 4, 6), 3), ((34, 3, 40), 3)])
def test_fft_route_matches_direct_sum_nd(oracle, shape, rank):
    v = crandn(2, *shape)
    a = oracle.dftn_naive(v, rank, -1)
    b = oracle.fftn_centered(v, rank, -1)
    assert np.abs(a - b).max() <= 1e-12 * np.abs(a).max()


def test_direct_sum_against_explicit_matrix(oracle):
    """The direct sum against a DFT matrix assembled here from the centred formula."""
    for N in (4, 5, 8, 9):
        o = N // 2
        k = np.arange(N)[:, None]; n = np.arange(N)[None, :]
        Fm = np.exp(-2j * np.pi * (k - o) * (n - o) / N) / np.sqrt(N)
        v = crandn(N)
        assert np.allclose(oracle.dft_naive_1d(v, -1), Fm @ v, atol=1e-13)
        assert np.allclose(oracle.dft_naive_1d(v, +1), Fm.conj().T @ v, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# P2  closed forms: pin centring, scaling and the sign of the exponent
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("N", [4, 6, 7, 64, 160, 368])
def test_delta_at_centre_gives_flat_positive_spectrum(oracle, N):
    v = np.zeros(N, complex); v[N // 2] = 1
    X = oracle.fft_centered_1d(v, -1)
    assert np.allclose(X, 1 / np.sqrt(N), atol=1e-14)


@pytest.mark.parametrize("N", [4, 6, 7, 64, 160, 368])
def test_delta_next_to_centre_gives_negative_phase_ramp(oracle, N):
    o = N // 2
    v = np.zeros(N, complex); v[o + 1] = 1
    X = oracle.fft_centered_1d(v, -1)
    k = np.arange(N)
    assert np.allclose(X, np.exp(-2j * np.pi * (k - o) / N) / np.sqrt(N), atol=1e-13)
    Xh = oracle.fft_centered_1d(v, +1)
    assert np.allclose(Xh, np.exp(+2j * np.pi * (k - o) / N) / np.sqrt(N), atol=1e-13)


@pytest.mark.parametrize("N", [4, 6, 7, 64, 160])
def test_constant_gives_delta_at_centre(oracle, N):
    X = oracle.fft_centered_1d(np.ones(N, complex), -1)
    e = np.zeros(N, complex); e[N // 2] = np.sqrt(N)
    assert np.allclose(X, e, atol=1e-12)


def test_nd_transform_only_touches_trailing_axes(oracle):
    """A rank-2 transform of a stack leaves the leading (frame) axis alone and is separable."""
    v = crandn(3, 6, 8)
    X = oracle.fftn_centered(v, 2, -1)
    for t in range(3):
        rows = np.stack([oracle.fft_centered_1d(v[t, i], -1) for i in range(6)])
        both = np.stack([oracle.fft_centered_1d(rows[:, j], -1) for j in range(8)], axis=1)
        assert np.allclose(X[t], both, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# P12  independent library routine
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape,rank", [((64, 64), 2), ((40, 46), 2), ((6, 10, 12), 3), ((5, 7), 2), ((34, 66), 2)])
def test_against_numpy_fft_with_shifts(oracle, shape, rank):
    v = crandn(2, *shape)
    axes = tuple(range(-rank, 0))
    ref = np.fft.fftshift(np.fft.fftn(np.fft.ifftshift(v, axes=axes), axes=axes, norm="ortho"), axes=axes)
    assert np.allclose(oracle.fftn_centered(v, rank, -1), ref, atol=1e-12)
    refi = np.fft.fftshift(np.fft.ifftn(np.fft.ifftshift(v, axes=axes), axes=axes, norm="ortho"), axes=axes)
    assert np.allclose(oracle.fftn_centered(v, rank, +1), refi, atol=1e-12)


# ---------------------------------------------------------------------------------------------
# P3  unitarity
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape,rank", [((64,), 1), ((46, 40), 2), ((6, 10, 36), 3)])
def test_parseval_and_inverse(oracle, shape, rank):
    v = crandn(*shape)
    X = oracle.fftn_centered(v, rank, -1)
    assert abs(np.linalg.norm(X) - np.linalg.norm(v)) <= 1e-12 * np.linalg.norm(v)
    back = oracle.fftn_centered(X, rank, +1)
    assert np.abs(back - v).max() <= 1e-12


# ---------------------------------------------------------------------------------------------
# P4/P5  adjoint identity, Hermitian PSD normal operator
# ---------------------------------------------------------------------------------------------
CASES = [
    dict(rank=2, n=(1, 6, 8), mask_kind=MASK_READOUT_INVARIANT),
    dict(rank=2, n=(1, 6, 8), mask_kind=MASK_FULL, weighted=True),
    dict(rank=3, n=(4, 6, 10), mask_kind=MASK_READOUT_INVARIANT, sens_has_frames=1),
    dict(rank=3, n=(4, 6, 10), mask_kind=MASK_FULL),
    dict(rank=2, n=(1, 34, 36), mask_kind=MASK_READOUT_INVARIANT, B=1, C=2, T=1),
]


@pytest.mark.parametrize("case", CASES)
def test_adjoint_identity(oracle, case):
    d, x, y, sens, mask = small_problem(**case)
    r = crandn(*d.kspace_shape())
    Ax = oracle.apply_A(x, sens, mask, d)
    AHr = oracle.apply_AH(r, sens, mask, d)
    lhs, rhs = inner(r, Ax), inner(AHr, x.astype(complex))
    assert abs(lhs - rhs) <= 1e-12 * abs(lhs)


@pytest.mark.parametrize("case", CASES)
def test_normal_operator_hermitian_psd(oracle, case):
    d, u, _, sens, mask = small_problem(**case)
    v = crandn(*d.image_shape()).astype(np.complex64)
    N = lambda z: oracle.apply_AH(oracle.apply_A(z, sens, mask, d), sens, mask, d)
    a, b = inner(u.astype(complex), N(v)), inner(v.astype(complex), N(u))
    assert abs(a - np.conj(b)) <= 1e-12 * abs(a)
    q = inner(u.astype(complex), N(u))
    assert q.real >= 0 and abs(q.imag) <= 1e-12 * abs(q.real)


@pytest.mark.parametrize("case", CASES)
def test_dc_is_assembled_from_A_and_AH(oracle, case):
    """Eq. 3 against the separately coded operators: x - eta A^H(Ax - y), A^H applying Omega again."""
    d, x, y, sens, mask = small_problem(**case)
    eta = 0.7
    res = oracle.apply_A(x, sens, mask, d) - y.astype(complex)
    ref = x.astype(complex) - eta * oracle.apply_AH(res, sens, mask, d)
    out = oracle.dc_forward(x, y, sens, mask, eta, d)
    assert np.abs(out - ref).max() <= 1e-13
    refv = x.astype(complex) - eta * oracle.apply_AH(oracle.apply_A(x, sens, mask, d), sens, mask, d)
    assert np.abs(oracle.dc_vjp(x, sens, mask, eta, d) - refv).max() <= 1e-13


def test_A_on_single_voxel_single_coil_closed_form(oracle):
    """One coil, delta image at voxel p: A x = M .* S[p] x[p] * separable centred exponentials."""
    n1, n2 = 6, 8
    d = Dims(1, 1, 1, 2, (1, n1, n2), 0, MASK_FULL)
    rng = np.random.default_rng(3)
    sens = crandn(*d.sens_shape(), rng=rng).astype(np.complex64)
    mask = rng.uniform(0, 1, d.mask_shape()).astype(np.float32)
    x = np.zeros(d.image_shape(), np.complex64)
    p1, p2 = 4, 2
    x[0, 0, 0, p1, p2] = 2 - 1j
    k1 = np.arange(n1)[:, None]; k2 = np.arange(n2)[None, :]
    ph = np.exp(-2j * np.pi * ((k1 - n1 // 2) * (p1 - n1 // 2) / n1 + (k2 - n2 // 2) * (p2 - n2 // 2) / n2))
    ref = mask[0, 0, 0].astype(float) * complex(sens[0, 0, 0, p1, p2]) * (2 - 1j) * ph / np.sqrt(n1 * n2)
    assert np.allclose(oracle.apply_A(x, sens, mask, d)[0, 0, 0, 0], ref, atol=1e-13)


# ---------------------------------------------------------------------------------------------
# P6  full mask and unit-norm sensitivities: A^H A = I
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("rank,n", [(2, (1, 8, 10)), (3, (4, 6, 8))])
def test_full_mask_unit_sens_gives_identity(oracle, rank, n):
    d, x, _, sens, mask = small_problem(rank=rank, n=n, unit_sens=True, full_mask=True)
    x_true = crandn(*d.image_shape()).astype(np.complex64)
    y = oracle.apply_A(x_true, sens, mask, d)              # noiseless
    eta = 0.3
    # complex64 rounding of y and sens limits the match to single precision
    out = oracle.dc_forward(x, y.astype(np.complex64), sens, mask, eta, d)
    assert np.abs(out - ((1 - eta) * x + eta * x_true)).max() <= 2e-6
    out1 = oracle.dc_forward(x, y.astype(np.complex64), sens, mask, 1.0, d)
    assert np.abs(out1 - x_true).max() <= 2e-6
    g = oracle.dc_vjp(x, sens, mask, 1.0, d)
    assert np.abs(g).max() <= 2e-6                         # (I - A^H A) x = 0


# ---------------------------------------------------------------------------------------------
# P7  special cases of the step
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("case", CASES[:4])
def test_special_cases(oracle, case):
    d, x, y, sens, mask = small_problem(**case)
    assert np.array_equal(oracle.dc_forward(x, y, sens, mask, 0.0, d), x.astype(complex))
    zero = np.zeros_like(x)
    aHy = oracle.apply_AH(y.astype(complex), sens, mask, d)
    assert np.abs(oracle.dc_forward(zero, y, sens, mask, 1.0, d) - aHy).max() <= 1e-13
    assert np.abs(oracle.dc_forward(x, np.zeros_like(y), sens, mask, 0.6, d)
                  - oracle.dc_vjp(x, sens, mask, 0.6, d)).max() <= 1e-14


# ---------------------------------------------------------------------------------------------
# P8  affine structure and the exact dot test of the VJP
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("case", CASES[:4])
def test_affine_structure_and_vjp_dot_test(oracle, case):
    d, x, y, sens, mask = small_problem(**case)
    eta = 0.9
    f = lambda z: oracle.dc_forward(z, y, sens, mask, eta, d)
    v = lambda z: oracle.dc_vjp(z, sens, mask, eta, d)
    zero = np.zeros_like(x)
    assert np.abs(f(x) - f(zero) - v(x)).max() <= 1e-13
    g = crandn(*d.image_shape()).astype(np.complex64)
    delta = crandn(*d.image_shape()).astype(np.complex64)
    xp = (x.astype(np.complex128) + delta).astype(np.complex64)
    delta_eff = xp.astype(complex) - x.astype(complex)      # what the rounded inputs really differ by
    lhs = inner(g.astype(complex), f(xp) - f(x)).real
    rhs = inner(v(g), delta_eff).real
    assert abs(lhs - rhs) <= 1e-6 * max(abs(lhs), 1.0)


# ---------------------------------------------------------------------------------------------
# P9  contraction
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("eta", [0.0, 0.5, 1.0, 2.0])
def test_vjp_is_nonexpansive_for_unit_sens(oracle, eta):
    d, g, _, sens, mask = small_problem(unit_sens=True, weighted=True, mask_kind=MASK_FULL)
    out = oracle.dc_vjp(g, sens, mask, eta, d)
    assert np.linalg.norm(out) <= np.linalg.norm(g) * (1 + 1e-6)


# ---------------------------------------------------------------------------------------------
# P10  coil permutation, single unit coil
# ---------------------------------------------------------------------------------------------
def test_coil_permutation_invariance(oracle):
    d, x, y, sens, mask = small_problem()
    perm = np.array([2, 0, 1])
    a = oracle.dc_forward(x, y, sens, mask, 0.8, d)
    b = oracle.dc_forward(x, y[:, perm], sens[:, perm], mask, 0.8, d)
    assert np.abs(a - b).max() <= 1e-13


def test_single_unit_coil_full_mask(oracle):
    d = Dims(1, 1, 1, 2, (1, 6, 8), 0, MASK_FULL)
    x = crandn(*d.image_shape()).astype(np.complex64)
    y = crandn(*d.kspace_shape()).astype(np.complex64)
    sens = np.ones(d.sens_shape(), np.complex64)
    mask = np.ones(d.mask_shape(), np.float32)
    eta = 0.4
    FHy = oracle.fftn_centered(y[:, 0].astype(complex), 2, +1)
    ref = x - eta * (x - FHy)
    assert np.abs(oracle.dc_forward(x, y, sens, mask, eta, d) - ref).max() <= 1e-6


# ---------------------------------------------------------------------------------------------
# P11  readout separability, and equality of the two mask forms
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("rank,n", [(2, (1, 6, 8)), (3, (4, 6, 10))])
def test_readout_invariant_mask_equals_expanded_full_mask(oracle, rank, n):
    d, x, y, sens, mask = small_problem(rank=rank, n=n, mask_kind=MASK_READOUT_INVARIANT)
    dF = Dims(d.batch, d.coils, d.frames, rank, d.n, 0, MASK_FULL)
    if rank == 2:
        full = np.broadcast_to(mask[:, :, None, None, :], dF.mask_shape()).copy()
    else:
        full = np.broadcast_to(mask[:, :, None, :, :], dF.mask_shape()).copy()
    a = oracle.dc_forward(x, y, sens, mask, 1.0, d)
    b = oracle.dc_forward(x, y, sens, full, 1.0, dF)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("rank,n", [(2, (1, 6, 8)), (3, (4, 6, 10))])
def test_readout_separable_formulation(oracle, rank, n):
    """With a readout-invariant mask the readout transform commutes with the mask, so
    A^H(Ax - y) = S^H P^H M (M P S x - R^H y) with P over the phase-encode axes only and R over
    the readout axis.  Checked with transforms of each axis built here from 1-D pieces."""
    d, x, y, sens, mask = small_problem(rank=rank, n=n, B=1, T=1, mask_kind=MASK_READOUT_INVARIANT)
    ro_axis = -2 if rank == 2 else -3

    def pe(a, sign):      # transform the phase-encode axes only
        return oracle.fftn_centered(a, rank - 1, sign)

    def ro(a, sign):      # transform the readout axis only
        moved = np.moveaxis(a, ro_axis, -1)
        return np.moveaxis(oracle.fftn_centered(moved, 1, sign), -1, ro_axis)

    M = mask[0, 0].astype(float)
    if rank == 2:
        M = M[None, :]
    else:
        M = M[None, :, :]
    xs = x[0, 0].astype(complex)
    acc = np.zeros_like(xs)
    for c in range(d.coils):
        S = sens[0, c].astype(complex)
        ytil = ro(y[0, c, 0].astype(complex), +1)
        r = M * (M * pe(S * xs, -1) - ytil)
        acc += np.conj(S) * pe(r, +1)
    ref = xs - 0.75 * acc
    out = oracle.dc_forward(x, y, sens, mask, 0.75, d)[0, 0]
    assert np.abs(out - ref).max() <= 1e-13


# ---------------------------------------------------------------------------------------------
# frames / sens_has_frames / thread count
# ---------------------------------------------------------------------------------------------
def test_frames_are_independent_problems(oracle):
    d, x, y, sens, mask = small_problem(T=3, sens_has_frames=1)
    out = oracle.dc_forward(x, y, sens, mask, 1.0, d)
    for t in range(3):
        d1 = Dims(d.batch, d.coils, 1, 2, d.n, 1, d.mask_kind)
        o1 = oracle.dc_forward(x[:, t:t + 1], y[:, :, t:t + 1], sens[:, :, t:t + 1], mask[:, t:t + 1], 1.0, d1)
        assert np.array_equal(out[:, t:t + 1], o1)


def test_static_sens_broadcasts_over_frames(oracle):
    d, x, y, sens, mask = small_problem(T=3, sens_has_frames=0)
    dT = Dims(d.batch, d.coils, d.frames, 2, d.n, 1, d.mask_kind)
    sensT = np.repeat(sens[:, :, None], 3, axis=2)
    assert np.array_equal(oracle.dc_forward(x, y, sens, mask, 1.0, d), oracle.dc_forward(x, y, sensT, mask, 1.0, dT))


def test_result_independent_of_thread_count(oracle):
    d, x, y, sens, mask = small_problem(C=5)
    a = oracle.dc_forward(x, y, sens, mask, 1.0, d, nthreads=1)
    b = oracle.dc_forward(x, y, sens, mask, 1.0, d, nthreads=4)
    assert np.array_equal(a, b)


def test_golden_tiny_case(oracle):
    """Stored output of a tiny case (written by tests/golden/make_golden.py, which calls only the
    oracle): guards the oracle against silent changes."""
    import json, os
    path = os.path.join(os.path.dirname(__file__), "golden", "dc_tiny.json")
    gold = json.load(open(path))
    from tests.golden.make_golden import tiny_case
    d, x, y, sens, mask, eta = tiny_case()
    out = oracle.dc_forward(x, y, sens, mask, eta, d)
    ref = np.array(gold["forward_re"]) + 1j * np.array(gold["forward_im"])
    assert np.abs(out.ravel() - ref).max() <= 1e-12
    outv = oracle.dc_vjp(x, sens, mask, eta, d)
    refv = np.array(gold["vjp_re"]) + 1j * np.array(gold["vjp_im"])
    assert np.abs(outv.ravel() - refv).max() <= 1e-12


# ---------------------------------------------------------------------------------------------
# dense-matrix brute force: A assembled as an explicit (C V) x V matrix from Kronecker factors
# ---------------------------------------------------------------------------------------------
def _dft_matrix(N):
    o = N // 2
    k = np.arange(N)[:, None]; n = np.arange(N)[None, :]
    return np.exp(-2j * np.pi * (k - o) * (n - o) / N) / np.sqrt(N)


@pytest.mark.parametrize("rank,n", [(2, (1, 4, 6)), (2, (1, 3, 5)), (3, (2, 4, 6))])
def test_dense_matrix_brute_force(oracle, rank, n):
    d, x, y, sens, mask = small_problem(rank=rank, n=n, B=1, C=3, T=1, mask_kind=MASK_FULL, weighted=True)
    V = d.V
    Fm = np.eye(1)
    for ax in range(3):
        Fm = np.kron(Fm, _dft_matrix(n[ax]) if (ax >= 3 - rank and n[ax] > 1) else np.eye(n[ax]))
    blocks = []
    for c in range(d.coils):
        S = np.diag(sens[0, c].astype(complex).ravel())
        M = np.diag(mask[0, 0].astype(float).ravel())
        blocks.append(M @ Fm @ S)
    A = np.vstack(blocks)                                   # (C V) x V, coil-major rows like y
    xv = x.astype(complex).ravel(); yv = y.astype(complex).ravel()
    eta = 0.65
    ref = xv - eta * (A.conj().T @ (A @ xv - yv))
    out = oracle.dc_forward(x, y, sens, mask, eta, d).ravel()
    assert np.abs(out - ref).max() <= 1e-13
    refv = xv - eta * (A.conj().T @ (A @ xv))
    assert np.abs(oracle.dc_vjp(x, sens, mask, eta, d).ravel() - refv).max() <= 1e-13
