"""ctypes binding of the CPU oracle (TEST INFRASTRUCTURE — never imported by the CUDA library).

Builds ``oracle/libgleam_oracle.so`` from ``gleam_oracle.c`` with gcc on first use and exposes
numpy wrappers.  All results are complex128 (float64); inputs are rounded to complex64/float32
first, because those are the arrays the GPU path sees.

Operators follow the GLEAM paper: A = Omega F S (text after Eq. 2), DC(x) = x - eta A^H(Ax - y)
(Eq. 3, eta = 2t), VJP(g) = g - eta A^H A g.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gleam_oracle.c")
_LIB = os.path.join(_HERE, "libgleam_oracle.so")
_lib = None

MASK_FULL = 0
MASK_READOUT_INVARIANT = 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, p, dbl, i32 = ctypes.c_int64, ctypes.c_void_p, ctypes.c_double, ctypes.c_int
        lib.oracle_dft_naive_1d.argtypes = [p, p, i64, i32]
        lib.oracle_dft_naive_1d.restype = None
        lib.oracle_fft_centered_1d.argtypes = [p, p, i64, i32]
        lib.oracle_fft_centered_1d.restype = i32
        lib.oracle_fftn_centered.argtypes = [p, i64, p, i32, i32, i32]
        lib.oracle_fftn_centered.restype = i32
        lib.oracle_dftn_naive.argtypes = [p, i64, p, i32, i32]
        lib.oracle_dftn_naive.restype = i32
        lib.oracle_apply_A.argtypes = [p, p, p, p, p, i32]
        lib.oracle_apply_A.restype = i32
        lib.oracle_apply_AH.argtypes = [p, p, p, p, p, i32]
        lib.oracle_apply_AH.restype = i32
        lib.oracle_dc.argtypes = [p, p, p, p, dbl, p, p, i32]
        lib.oracle_dc.restype = i32
        lib.oracle_dc_aty.argtypes = [p, p, p, p, dbl, p, p, i32]
        lib.oracle_dc_aty.restype = i32
        lib.oracle_modl_cg.argtypes = [p, p, p, p, dbl, i32, p, p, i32]
        lib.oracle_modl_cg.restype = i32
        lib.oracle_modl_cg_vjp.argtypes = [p, p, p, dbl, i32, p, p, i32]
        lib.oracle_modl_cg_vjp.restype = i32
        lib.oracle_dc_grad_eta.argtypes = [p, p, p, p, p, p, p, i32]
        lib.oracle_dc_grad_eta.restype = i32
        lib.oracle_dc_grad_y.argtypes = [p, p, p, dbl, p, p, i32]
        lib.oracle_dc_grad_y.restype = i32
        lib.oracle_complex_to_channels.argtypes = [p, i64, i64, p]
        lib.oracle_complex_to_channels.restype = None
        lib.oracle_channels_to_complex.argtypes = [p, i64, i64, p]
        lib.oracle_channels_to_complex.restype = None
        lib.oracle_l1_loss.argtypes = [p, p, i64, p]
        lib.oracle_l1_loss.restype = dbl
        lib.oracle_max_threads.argtypes = []
        lib.oracle_max_threads.restype = i32
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


@dataclass(frozen=True)
class Dims:
    """Problem shape.  spatial = (n0, n1, n2) with n0 = 1 for fft_rank 2."""
    batch: int
    coils: int
    frames: int
    fft_rank: int
    n: tuple
    sens_has_frames: int = 0
    mask_kind: int = MASK_READOUT_INVARIANT

    @property
    def V(self) -> int:
        return int(self.n[0]) * int(self.n[1]) * int(self.n[2])

    def image_shape(self):
        return (self.batch, self.frames) + tuple(self.n)

    def kspace_shape(self):
        return (self.batch, self.coils, self.frames) + tuple(self.n)

    def sens_shape(self):
        if self.sens_has_frames:
            return (self.batch, self.coils, self.frames) + tuple(self.n)
        return (self.batch, self.coils) + tuple(self.n)

    def mask_shape(self):
        if self.mask_kind == MASK_FULL:
            return (self.batch, self.frames) + tuple(self.n)
        if self.fft_rank == 2:
            return (self.batch, self.frames, self.n[2])
        return (self.batch, self.frames, self.n[1], self.n[2])

    def as_array(self) -> np.ndarray:
        return np.array([self.batch, self.coils, self.frames, self.fft_rank, self.n[0], self.n[1],
                         self.n[2], self.sens_has_frames, self.mask_kind], dtype=np.int64)


def _c64(a, shape=None):
    a = np.ascontiguousarray(a, dtype=np.complex64)
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _f32(a, shape=None):
    a = np.ascontiguousarray(a, dtype=np.float32)
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def dft_naive_1d(v, sign: int = -1) -> np.ndarray:
    """Centred orthonormal 1-D DFT by direct summation (the definition)."""
    a = np.ascontiguousarray(v, dtype=np.complex128)
    out = np.empty_like(a)
    _load().oracle_dft_naive_1d(_ptr(a), _ptr(out), a.size, sign)
    return out


def fft_centered_1d(v, sign: int = -1) -> np.ndarray:
    """Centred orthonormal 1-D DFT through the shift + recursive FFT route."""
    a = np.ascontiguousarray(v, dtype=np.complex128)
    out = np.empty_like(a)
    rc = _load().oracle_fft_centered_1d(_ptr(a), _ptr(out), a.size, sign)
    assert rc == 0, rc
    return out


def _as_volumes(a, rank):
    a = np.array(a, dtype=np.complex128, order="C", copy=True)
    sp = a.shape[-rank:]
    n = np.array((1,) * (3 - rank) + tuple(sp), dtype=np.int64)
    outer = int(np.prod(a.shape[:-rank], dtype=np.int64)) if a.ndim > rank else 1
    return a, n, outer


def fftn_centered(a, rank: int, sign: int = -1, nthreads: int = 1) -> np.ndarray:
    """Centred orthonormal DFT over the trailing ``rank`` axes (FFT route)."""
    a, n, outer = _as_volumes(a, rank)
    rc = _load().oracle_fftn_centered(_ptr(a), outer, _ptr(n), rank, sign, nthreads)
    assert rc == 0, rc
    return a


def dftn_naive(a, rank: int, sign: int = -1) -> np.ndarray:
    """Centred orthonormal DFT over the trailing ``rank`` axes by direct summation."""
    a, n, outer = _as_volumes(a, rank)
    rc = _load().oracle_dftn_naive(_ptr(a), outer, _ptr(n), rank, sign)
    assert rc == 0, rc
    return a


def apply_A(x, sens, mask, d: Dims, nthreads: int = 1) -> np.ndarray:
    """k = Omega F S x, shape (B, C, T, n0, n1, n2)."""
    x = _c64(x, d.image_shape()); sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    k = np.empty(d.kspace_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_apply_A(_ptr(x), _ptr(sens), _ptr(mask), _ptr(dd), _ptr(k), nthreads)
    assert rc == 0, rc
    return k


def apply_AH(k, sens, mask, d: Dims, nthreads: int = 1) -> np.ndarray:
    """img = S^H F^H Omega k, shape (B, T, n0, n1, n2).  k is complex128 (not rounded)."""
    k = np.array(k, dtype=np.complex128, order="C", copy=True)
    assert k.shape == d.kspace_shape()
    sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    img = np.empty(d.image_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_apply_AH(_ptr(k), _ptr(sens), _ptr(mask), _ptr(dd), _ptr(img), nthreads)
    assert rc == 0, rc
    return img


def dc_forward(x, y, sens, mask, eta: float, d: Dims, nthreads: int = 1) -> np.ndarray:
    """Eq. 3: out = x - eta A^H (A x - y)."""
    x = _c64(x, d.image_shape()); y = _c64(y, d.kspace_shape())
    sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    out = np.empty(d.image_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_dc(_ptr(x), _ptr(y), _ptr(sens), _ptr(mask), float(eta), _ptr(dd), _ptr(out), nthreads)
    assert rc == 0, rc
    return out


def dc_forward_aty(x, aty, sens, mask, eta: float, d: Dims, nthreads: int = 1) -> np.ndarray:
    """Eq. 3 in normal-equations form: out = x - eta (A^H A x - aty), aty = A^H y given as complex64."""
    x = _c64(x, d.image_shape()); aty = _c64(aty, d.image_shape())
    sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    out = np.empty(d.image_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_dc_aty(_ptr(x), _ptr(aty), _ptr(sens), _ptr(mask), float(eta), _ptr(dd), _ptr(out), nthreads)
    assert rc == 0, rc
    return out


def dc_vjp(g, sens, mask, eta: float, d: Dims, nthreads: int = 1) -> np.ndarray:
    """Vector-Jacobian product of Eq. 3: grad_in = g - eta A^H A g."""
    g = _c64(g, d.image_shape()); sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    out = np.empty(d.image_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_dc(_ptr(g), None, _ptr(sens), _ptr(mask), float(eta), _ptr(dd), _ptr(out), nthreads)
    assert rc == 0, rc
    return out


def modl_cg_forward(z, y, sens, mask, mu: float, n_iter: int, d: Dims, nthreads: int = 1) -> np.ndarray:
    """Eq. 7: x = (A^H A + mu I)^{-1} (A^H y + mu z) by n_iter conjugate-gradient steps from zero."""
    z = _c64(z, d.image_shape()); y = _c64(y, d.kspace_shape())
    sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    out = np.empty(d.image_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_modl_cg(_ptr(z), _ptr(y), _ptr(sens), _ptr(mask), float(mu), int(n_iter), _ptr(dd),
                                _ptr(out), nthreads)
    assert rc == 0, rc
    return out


def modl_cg_vjp(g, sens, mask, mu: float, n_iter: int, d: Dims, nthreads: int = 1) -> np.ndarray:
    """grad_z = mu (A^H A + mu I)^{-1} g by n_iter conjugate-gradient steps from zero."""
    g = _c64(g, d.image_shape()); sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    out = np.empty(d.image_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_modl_cg_vjp(_ptr(g), _ptr(sens), _ptr(mask), float(mu), int(n_iter), _ptr(dd), _ptr(out),
                                    nthreads)
    assert rc == 0, rc
    return out


def dc_grad_eta(g, x, y, sens, mask, d: Dims, nthreads: int = 1) -> np.ndarray:
    """Gradient of Eq. 3 with respect to the step size for a cotangent g of the output, one value
    per batch example: -Re<g_b, A^H(A x - y)_b>."""
    g = _c64(g, d.image_shape()); x = _c64(x, d.image_shape()); y = _c64(y, d.kspace_shape())
    sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    out = np.empty(d.batch, dtype=np.float64)
    dd = d.as_array()
    rc = _load().oracle_dc_grad_eta(_ptr(g), _ptr(x), _ptr(y), _ptr(sens), _ptr(mask), _ptr(dd), _ptr(out), nthreads)
    assert rc == 0, rc
    return out


def dc_grad_y(g, sens, mask, eta: float, d: Dims, nthreads: int = 1) -> np.ndarray:
    """Gradient of Eq. 3 with respect to the measurements: eta Omega F S g, shape of y."""
    g = _c64(g, d.image_shape()); sens = _c64(sens, d.sens_shape()); mask = _f32(mask, d.mask_shape())
    out = np.empty(d.kspace_shape(), dtype=np.complex128)
    dd = d.as_array()
    rc = _load().oracle_dc_grad_y(_ptr(g), _ptr(sens), _ptr(mask), float(eta), _ptr(dd), _ptr(out), nthreads)
    assert rc == 0, rc
    return out


def complex_to_channels(x) -> np.ndarray:
    """complex64 (B, ...) -> float32 (B, 2, ...): channel 0 the real part, channel 1 the imaginary part."""
    x = np.ascontiguousarray(x, dtype=np.complex64)
    out = np.empty((x.shape[0], 2) + x.shape[1:], dtype=np.float32)
    inner = int(np.prod(x.shape[1:], dtype=np.int64))
    _load().oracle_complex_to_channels(_ptr(x), x.shape[0], inner, _ptr(out))
    return out


def channels_to_complex(ch) -> np.ndarray:
    """float32 (B, 2, ...) -> complex64 (B, ...)."""
    ch = np.ascontiguousarray(ch, dtype=np.float32)
    assert ch.shape[1] == 2
    out = np.empty((ch.shape[0],) + ch.shape[2:], dtype=np.complex64)
    inner = int(np.prod(ch.shape[2:], dtype=np.int64))
    _load().oracle_channels_to_complex(_ptr(ch), ch.shape[0], inner, _ptr(out))
    return out


def l1_loss(x, ref, with_grad: bool = False):
    """mean |x - ref| over all complex elements; with_grad also returns (x - ref)/|x - ref|/N."""
    x = np.ascontiguousarray(x, dtype=np.complex64); ref = _c64(ref, x.shape)
    grad = np.empty(x.shape, dtype=np.complex128) if with_grad else None
    val = float(_load().oracle_l1_loss(_ptr(x), _ptr(ref), x.size, _ptr(grad) if with_grad else None))
    return (val, grad) if with_grad else val
