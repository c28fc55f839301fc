"""Pins for the oracle's MoDL model inversion (Eq. 7, second line):

    x = (A^H A + mu I)^{-1} (A^H y + mu z)   by a fixed number of conjugate-gradient steps.

The paper prints neither a CG listing nor a worked example, so the pins are what the mathematics
fixes, computed here without the oracle's operator code: a dense matrix of A assembled from the
explicit centred-DFT formula, numpy's dense solver for the converged result, and the Krylov-space
characterisation of the k-th CG iterate (the minimiser of the H-norm error over
span{b, Hb, ..., H^(k-1) b}) for the truncated iteration.
"""
import numpy as np
import pytest

from oracle.oracle import Dims, MASK_FULL, MASK_READOUT_INVARIANT


def crandn(rng, *shape):
    return (rng.normal(size=shape) + 1j * rng.normal(size=shape)) / np.sqrt(2)


def dft_matrix(N):
    o = N // 2
    k = np.arange(N)[:, None] - o
    n = np.arange(N)[None, :] - o
    return np.exp(-2j * np.pi * k * n / N) / np.sqrt(N)


def dense_A(d, sens, mask, t=0, b=0):
    """Dense (C*V, V) matrix of A = Omega F S for one example and frame, from the definitions."""
    n0, n1, n2 = d.n
    if d.fft_rank == 2:
        F = np.kron(np.eye(n0), np.kron(dft_matrix(n1), dft_matrix(n2)))
    else:
        F = np.kron(dft_matrix(n0), np.kron(dft_matrix(n1), dft_matrix(n2)))
    V = n0 * n1 * n2
    if d.mask_kind == MASK_FULL:
        m = mask[b, t].reshape(V).astype(np.float64)
    elif d.fft_rank == 2:
        m = np.broadcast_to(mask[b, t][None, None, :], (n0, n1, n2)).reshape(V).astype(np.float64)
    else:
        m = np.broadcast_to(mask[b, t][None, :, :], (n0, n1, n2)).reshape(V).astype(np.float64)
    rows = []
    for c in range(d.coils):
        s = (sens[b, c, t] if d.sens_has_frames else sens[b, c]).reshape(V).astype(np.complex128)
        rows.append(m[:, None] * F * s[None, :])
    return np.vstack(rows)


def problem(seed, rank=2, B=1, C=2, T=1, n=(1, 4, 4), mask_kind=MASK_READOUT_INVARIANT, weighted=False,
            sens_has_frames=0):
    rng = np.random.default_rng(seed)
    d = Dims(B, C, T, rank, tuple(n), sens_has_frames, mask_kind)
    sens = crandn(rng, *d.sens_shape()).astype(np.complex64)
    if weighted:
        mask = rng.uniform(0.1, 1.0, d.mask_shape()).astype(np.float32)
    else:
        mask = (rng.uniform(size=d.mask_shape()) < 0.5).astype(np.float32)
    z = crandn(rng, *d.image_shape()).astype(np.complex64)
    y = crandn(rng, *d.kspace_shape()).astype(np.complex64)
    g = crandn(rng, *d.image_shape()).astype(np.complex64)
    return d, z, y, g, sens, mask


def dense_system(d, z, y, sens, mask, mu, b=0, t=0):
    A = dense_A(d, sens, mask, t=t, b=b)
    V = A.shape[1]
    H = A.conj().T @ A + mu * np.eye(V)
    yv = np.concatenate([y[b, c, t].reshape(V) for c in range(d.coils)]).astype(np.complex128)
    rhs = A.conj().T @ yv + mu * z[b, t].reshape(V).astype(np.complex128)
    return H, rhs


def krylov_minimiser(H, b, k):
    """argmin over span{b, Hb, ..., H^(k-1) b} of the H-norm error: solve the projected system."""
    cols = [b]
    for _ in range(k - 1):
        cols.append(H @ cols[-1])
    Q, _ = np.linalg.qr(np.stack(cols, axis=1))
    c = np.linalg.solve(Q.conj().T @ H @ Q, Q.conj().T @ b)
    return Q @ c


@pytest.mark.parametrize("rank,n,mask_kind,weighted", [
    (2, (1, 4, 4), MASK_READOUT_INVARIANT, False),
    (2, (1, 4, 6), MASK_FULL, True),
    (3, (2, 2, 4), MASK_READOUT_INVARIANT, True),
    (3, (2, 3, 2), MASK_FULL, False),
])
def test_converged_cg_equals_dense_solve(oracle, rank, n, mask_kind, weighted):
    d, z, y, g, sens, mask = problem(11, rank=rank, n=n, mask_kind=mask_kind, weighted=weighted)
    mu = 0.3
    H, rhs = dense_system(d, z, y, sens, mask, mu)
    want = np.linalg.solve(H, rhs)
    got = oracle.modl_cg_forward(z, y, sens, mask, mu, 3 * H.shape[0], d).reshape(-1)
    assert np.abs(got - want).max() <= 1e-10 * np.abs(want).max()
    # VJP with respect to z: mu H^{-1} g
    want_g = mu * np.linalg.solve(H, g.reshape(-1).astype(np.complex128))
    got_g = oracle.modl_cg_vjp(g, sens, mask, mu, 3 * H.shape[0], d).reshape(-1)
    assert np.abs(got_g - want_g).max() <= 1e-10 * np.abs(want_g).max()


@pytest.mark.parametrize("k", [1, 2, 3, 5, 8])
def test_truncated_cg_is_the_krylov_minimiser(oracle, k):
    d, z, y, g, sens, mask = problem(5, rank=2, C=3, n=(1, 4, 6))
    mu = 0.05
    H, rhs = dense_system(d, z, y, sens, mask, mu)
    want = krylov_minimiser(H, rhs, k)
    got = oracle.modl_cg_forward(z, y, sens, mask, mu, k, d).reshape(-1)
    assert np.abs(got - want).max() <= 1e-8 * np.abs(want).max()
    want_g = krylov_minimiser(H, mu * g.reshape(-1).astype(np.complex128), k)
    got_g = oracle.modl_cg_vjp(g, sens, mask, mu, k, d).reshape(-1)
    assert np.abs(got_g - want_g).max() <= 1e-8 * np.abs(want_g).max()


def test_identity_normal_operator_closed_form(oracle):
    """Full mask and sum_c |S_c|^2 = 1 give A^H A = I: one CG step is exact and
    x = (x_true + mu z) / (1 + mu) for noiseless y = A x_true."""
    rng = np.random.default_rng(3)
    d = Dims(2, 3, 2, 2, (1, 6, 8), 0, MASK_READOUT_INVARIANT)
    sens = crandn(rng, *d.sens_shape())
    sens = (sens / np.sqrt(np.sum(np.abs(sens) ** 2, axis=1, keepdims=True))).astype(np.complex64)
    mask = np.ones(d.mask_shape(), dtype=np.float32)
    x_true = crandn(rng, *d.image_shape()).astype(np.complex64)
    z = crandn(rng, *d.image_shape()).astype(np.complex64)
    y = oracle.apply_A(x_true, sens, mask, d).astype(np.complex64)
    mu = 0.7
    for n_iter in (1, 4):
        got = oracle.modl_cg_forward(z, y, sens, mask, mu, n_iter, d)
        want = (x_true.astype(np.complex128) + mu * z) / (1 + mu)
        assert np.abs(got - want).max() <= 5e-6       # y and S are rounded to single precision
    got_g = oracle.modl_cg_vjp(z, sens, mask, mu, 1, d)
    assert np.abs(got_g - mu / (1 + mu) * z).max() <= 5e-6


def test_examples_and_frames(oracle):
    """Each batch example is its own system; the frames of one example are solved jointly."""
    d, z, y, g, sens, mask = problem(21, rank=2, B=2, C=2, T=2, n=(1, 4, 4), sens_has_frames=1)
    mu, k = 0.1, 3
    got = oracle.modl_cg_forward(z, y, sens, mask, mu, k, d)
    for b in range(2):
        d1 = Dims(1, d.coils, d.frames, d.fft_rank, d.n, d.sens_has_frames, d.mask_kind)
        alone = oracle.modl_cg_forward(z[b:b + 1], y[b:b + 1], sens[b:b + 1], mask[b:b + 1], mu, k, d1)
        assert np.abs(got[b] - alone[0]).max() <= 1e-13 * np.abs(alone).max()
        # joint over the frames: block-diagonal dense system of the example
        Hs, rs = zip(*[dense_system(d, z, y, sens, mask, mu, b=b, t=t) for t in range(2)])
        V = Hs[0].shape[0]
        H = np.zeros((2 * V, 2 * V), dtype=np.complex128)
        H[:V, :V], H[V:, V:] = Hs
        want = krylov_minimiser(H, np.concatenate(rs), k)
        assert np.abs(got[b].reshape(-1) - want).max() <= 1e-8 * np.abs(want).max()


def test_linear_in_z_and_vjp_is_its_adjoint(oracle):
    """Converged: x(z) is affine in z with Jacobian mu H^{-1} (Hermitian), so
    Re<g, x(z + dz) - x(z)> = Re<vjp(g), dz>."""
    d, z, y, g, sens, mask = problem(8, rank=2, C=2, n=(1, 4, 4))
    rng = np.random.default_rng(9)
    dz = crandn(rng, *d.image_shape()).astype(np.complex64)
    mu, k = 0.2, 60
    x0 = oracle.modl_cg_forward(z, y, sens, mask, mu, k, d)
    x1 = oracle.modl_cg_forward((z + dz).astype(np.complex64), y, sens, mask, mu, k, d)
    v = oracle.modl_cg_vjp(g, sens, mask, mu, k, d)
    zz = (z + dz).astype(np.complex64).astype(np.complex128) - z.astype(np.complex128)
    lhs = np.vdot(g.astype(np.complex128), x1 - x0).real
    rhs = np.vdot(v, zz).real
    assert abs(lhs - rhs) <= 1e-9 * max(1.0, abs(lhs))


def test_zero_right_hand_side_and_zero_steps(oracle):
    d, z, y, g, sens, mask = problem(2)
    out = oracle.modl_cg_forward(np.zeros_like(z), np.zeros_like(y), sens, mask, 0.05, 10, d)
    assert np.all(out == 0)
    out = oracle.modl_cg_forward(z, y, sens, mask, 0.05, 0, d)
    assert np.all(out == 0)


def test_planted_mistakes_are_caught():
    """The Krylov pin separates the method from near misses: a dropped mu term in H, a missing
    mu in the right-hand side, or steepest descent instead of CG all miss by far more than the
    pin's tolerance."""
    d, z, y, g, sens, mask = problem(5, rank=2, C=3, n=(1, 4, 6))
    mu, k = 0.05, 3
    H, rhs = dense_system(d, z, y, sens, mask, mu)
    want = krylov_minimiser(H, rhs, k)
    A = dense_A(d, sens, mask)
    wrong_H = krylov_minimiser(A.conj().T @ A + 1e-12 * np.eye(H.shape[0]), rhs, k)
    wrong_rhs = krylov_minimiser(H, rhs - mu * z.reshape(-1), k)
    xs, r = np.zeros_like(rhs), rhs.copy()
    for _ in range(k):                                  # steepest descent
        a = np.vdot(r, r).real / np.vdot(r, H @ r).real
        xs, r = xs + a * r, r - a * (H @ r)
    for wrong in (wrong_H, wrong_rhs, xs):
        assert np.abs(wrong - want).max() > 1e-4 * np.abs(want).max()
