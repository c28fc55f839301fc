"""Seeded synthetic inputs shaped like the paper's workloads (numpy only).

This module holds no arithmetic of the reconstruction method: it draws images, coil sensitivity
maps, sampling masks and noise.  It applies no Fourier transform and no forward model.  Both the
CPU oracle's tests and the CUDA path's tests and benchmark take their inputs from here.

The five workloads stand in for the data sets the paper trains on (3-D FSE knee volumes of
320x320x256 with 8 coils and Poisson-disc masks; multi-coil brain slices with 1-D random masks and
a fully sampled centre; 20-frame cardiac cine with k-t variable-density masks — Experiments /
Datasets section), which are not available offline.

Conventions: arrays are row-major, last index fastest; the last spatial axis is the phase-encode
axis of 2-D problems; 3-D problems are (readout, ky, kz).  CN(0, s^2) is a circular complex normal
with E|z|^2 = s^2.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

MASK_FULL = 0
MASK_READOUT_INVARIANT = 1

BASE_SEED = 20220808


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # 1-based position in the list of configurations
    batch: int
    coils: int
    frames: int
    fft_rank: int
    n: tuple                   # (n0, n1, n2); n0 = 1 for fft_rank 2
    eta: float
    chain: int = 1             # unrolled iterations chained in the timed run
    mask_recipe: str = "random1d"
    accel: float = 4.0
    center: float = 8.0        # centre lines (count if >= 1, fraction of the axis if < 1)
    x_is_noise: bool = False   # iterate ~ CN(0,1) instead of a phantom
    phantom_noise: float = 0.05
    noise_sigma: float = 0.01
    description: str = ""

    @property
    def V(self) -> int:
        return self.n[0] * self.n[1] * self.n[2]

    @property
    def voxel_coils(self) -> int:
        return self.batch * self.coils * self.frames * self.V

    def image_shape(self):
        return (self.batch, self.frames) + tuple(self.n)

    def kspace_shape(self):
        return (self.batch, self.coils, self.frames) + tuple(self.n)

    def sens_shape(self):
        return (self.batch, self.coils) + tuple(self.n)   # static over frames

    def mask_shape(self, mask_kind=MASK_READOUT_INVARIANT):
        if mask_kind == MASK_FULL:
            return (self.batch, self.frames) + tuple(self.n)
        if self.fft_rank == 2:
            return (self.batch, self.frames, self.n[2])
        return (self.batch, self.frames, self.n[1], self.n[2])


WORKLOADS = {
    w.name: w for w in [
        Workload("slice64", 1, 1, 8, 1, 2, (1, 64, 64), 1.0, 1, "random1d", 4.0, 8, x_is_noise=True,
                 description="2D single slice, 8 coils, 64x64, 4x random phase-encode lines + 8 centre lines"),
        Workload("knee2d", 2, 4, 15, 1, 2, (1, 640, 368), 0.5, 1, "equispaced1d", 8.0, 0.04,
                 description="2D knee-like, batch 4, 15 coils, 640x368, 8x equispaced + 4% centre"),
        Workload("brain2d", 3, 8, 16, 1, 2, (1, 640, 320), 1.0, 10, "random1d", 4.0, 0.08,
                 description="2D brain-like, batch 8, 16 coils, 640x320, 4x random + 8% centre, 10 chained iterations"),
        Workload("knee3d", 4, 1, 8, 1, 3, (320, 320, 256), 1.0, 1, "poisson2d", 12.0, 24,
                 description="3D knee-like, 8 coils, 320x320x256, 12x Poisson-disc ky-kz + 24x24 centre"),
        Workload("cine", 5, 1, 8, 20, 2, (1, 192, 160), 1.0, 8, "ktvd1d", 10.0, 6,
                 description="2D+time cine-like, 8 coils, 192x160x20 frames, 10x k-t variable density + 6 centre lines, 8 chained iterations"),
    ]
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (used for reduced-size parity cases)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(kw)
    return Workload(**d)


def _rng(w: Workload, k: int, seed_offset: int = 0):
    return np.random.default_rng(BASE_SEED + 1000 * w.index + k + 100000 * seed_offset)


def cnormal(rng, shape, sigma=1.0):
    s = sigma / np.sqrt(2.0)
    return rng.normal(0.0, s, shape) + 1j * rng.normal(0.0, s, shape)


def _coords(n):
    """Per-axis coordinates in [-1, 1)."""
    return [(-1.0 + 2.0 * np.arange(m) / m) if m > 1 else np.zeros(1) for m in n]


# ----------------------------------------------------------------------------------------------
# coil sensitivities
# ----------------------------------------------------------------------------------------------
def make_sens(w: Workload, rng) -> np.ndarray:
    """Smooth maps: Gaussian magnitude blobs around the object times a random quadratic phase,
    normalised so that sum_c |S_c|^2 = 1 at every voxel."""
    n0, n1, n2 = w.n
    u0, u1, u2 = _coords(w.n)
    out = np.empty((w.batch, w.coils) + tuple(w.n), dtype=np.complex64)
    three_d = w.fft_rank == 3
    for b in range(w.batch):
        maps = np.empty((w.coils,) + tuple(w.n), dtype=np.complex128)
        for c in range(w.coils):
            ang = 2 * np.pi * c / w.coils + rng.uniform(-0.2, 0.2)
            sig = rng.uniform(0.6, 0.9)
            c1, c2 = 1.1 * np.cos(ang), 1.1 * np.sin(ang)
            c0 = (0.5 if c % 2 == 0 else -0.5) if three_d else 0.0
            coef = rng.uniform(-np.pi, np.pi, 10)
            d0 = (u0 - c0)[:, None, None]; d1 = (u1 - c1)[None, :, None]; d2 = (u2 - c2)[None, None, :]
            mag = np.exp(-(d1 ** 2 + d2 ** 2 + (d0 ** 2 if three_d else 0.0)) / (2 * sig ** 2))
            a0 = u0[:, None, None]; a1 = u1[None, :, None]; a2 = u2[None, None, :]
            ph = (coef[0] + coef[1] * a1 + coef[2] * a2 + coef[3] * a1 * a2 + coef[4] * a1 ** 2 + coef[5] * a2 ** 2)
            if three_d:
                ph = ph + coef[6] * a0 + coef[7] * a0 * a1 + coef[8] * a0 * a2 + coef[9] * a0 ** 2
            maps[c] = mag * np.exp(1j * ph)
        rss = np.sqrt(np.sum(np.abs(maps) ** 2, axis=0))
        out[b] = (maps / rss[None]).astype(np.complex64)
    return out


# ----------------------------------------------------------------------------------------------
# phantoms
# ----------------------------------------------------------------------------------------------
def make_phantom(w: Workload, rng, n_shapes: int = 50) -> np.ndarray:
    """Sum of random ellipses (3-D: ellipsoids) with complex amplitudes; cine: radii pulse over
    the frames.  Shape (B, T, n0, n1, n2), float64 complex."""
    n0, n1, n2 = w.n
    u0, u1, u2 = _coords(w.n)
    three_d = w.fft_rank == 3
    img = np.zeros((w.batch, w.frames) + tuple(w.n), dtype=np.complex128)
    for b in range(w.batch):
        for _ in range(n_shapes):
            ctr = rng.uniform(-0.6, 0.6, 3)
            ax = rng.uniform(0.05, 0.4, 3)
            th = rng.uniform(0, np.pi)
            amp = rng.uniform(0.1, 1.0) * np.exp(1j * rng.uniform(-np.pi, np.pi))
            phi = rng.uniform(0, 2 * np.pi)
            for t in range(w.frames):
                s = 1.0 + (0.15 * np.sin(2 * np.pi * t / max(w.frames, 1) + phi) if w.frames > 1 else 0.0)
                r = ax * s
                rmax = float(r.max())
                # bounding box in index space (keeps the 3-D case cheap)
                sl = []
                for a, (u, m) in enumerate(zip((u0, u1, u2), w.n)):
                    if m == 1:
                        sl.append(slice(0, 1)); continue
                    lo = int(np.floor((ctr[a] - rmax + 1.0) * m / 2.0)); hi = int(np.ceil((ctr[a] + rmax + 1.0) * m / 2.0)) + 1
                    sl.append(slice(max(lo, 0), min(hi, m)))
                if any(s_.stop <= s_.start for s_ in sl):
                    continue
                d0 = (u0[sl[0]] - (ctr[0] if three_d else 0.0))[:, None, None]
                d1 = (u1[sl[1]] - ctr[1])[None, :, None]
                d2 = (u2[sl[2]] - ctr[2])[None, None, :]
                e1 = np.cos(th) * d1 + np.sin(th) * d2
                e2 = -np.sin(th) * d1 + np.cos(th) * d2
                q = (e1 / r[1]) ** 2 + (e2 / r[2]) ** 2
                if three_d:
                    q = q + (d0 / r[0]) ** 2
                else:
                    q = q + 0.0 * d0
                img[b, t][sl[0], sl[1], sl[2]] += amp * (q <= 1.0)
    return img


# ----------------------------------------------------------------------------------------------
# sampling masks (phase-encode patterns).  Returned as float32 0/1 arrays in readout-invariant
# form: (B, T, n2) for fft_rank 2, (B, T, n1, n2) for fft_rank 3.
# ----------------------------------------------------------------------------------------------
def _center_count(w: Workload, n: int) -> int:
    return int(round(w.center * n)) if w.center < 1 else int(w.center)


def _mask_random1d(n, n_center, n_total, rng):
    m = np.zeros(n, dtype=np.float32)
    lo = n // 2 - n_center // 2
    m[lo:lo + n_center] = 1
    rest = np.flatnonzero(m == 0)
    extra = max(n_total - n_center, 0)
    m[rng.choice(rest, size=min(extra, rest.size), replace=False)] = 1
    return m


def _mask_equispaced1d(n, n_center, step, rng):
    m = np.zeros(n, dtype=np.float32)
    m[int(rng.integers(0, step))::step] = 1
    lo = n // 2 - n_center // 2
    m[lo:lo + n_center] = 1
    return m


def _mask_ktvd1d(n, n_center, n_total, rng):
    m = np.zeros(n, dtype=np.float32)
    lo = n // 2 - n_center // 2
    m[lo:lo + n_center] = 1
    rest = np.flatnonzero(m == 0)
    k = rest - n // 2
    wgt = (1.0 - np.abs(k) / (n / 2.0)) ** 2 + 1e-6
    wgt /= wgt.sum()
    m[rng.choice(rest, size=max(n_total - n_center, 0), replace=False, p=wgt)] = 1
    return m


def _poisson_disc(n1, n2, radius, rng, throws):
    """Dart throwing on the integer ky-kz grid with a minimum distance."""
    cell = max(radius / np.sqrt(2.0), 1.0)
    g1, g2 = int(np.ceil(n1 / cell)), int(np.ceil(n2 / cell))
    grid = -np.ones((g1, g2), dtype=np.int64)
    pts = []
    cand = np.stack([rng.integers(0, n1, throws), rng.integers(0, n2, throws)], axis=1)
    r2 = radius * radius
    for p1, p2 in cand:
        c1, c2 = int(p1 / cell), int(p2 / cell)
        ok = True
        for a in range(max(c1 - 2, 0), min(c1 + 3, g1)):
            for bb in range(max(c2 - 2, 0), min(c2 + 3, g2)):
                j = grid[a, bb]
                if j >= 0:
                    q = pts[j]
                    if (q[0] - p1) ** 2 + (q[1] - p2) ** 2 < r2:
                        ok = False
                        break
            if not ok:
                break
        if ok:
            grid[c1, c2] = len(pts)
            pts.append((int(p1), int(p2)))
    return pts


def _mask_poisson2d(n1, n2, calib, accel, rng):
    target = n1 * n2 / accel
    radius = np.sqrt(0.62 * accel)           # dart throwing saturates near this density
    seed = int(rng.integers(0, 2 ** 31))
    best = None
    lo, hi = 0.6 * radius, 1.6 * radius
    for _ in range(7):
        r = 0.5 * (lo + hi)
        pts = _poisson_disc(n1, n2, r, np.random.default_rng(seed), throws=int(12 * target))
        m = np.zeros((n1, n2), dtype=np.float32)
        if pts:
            pa = np.array(pts)
            m[pa[:, 0], pa[:, 1]] = 1
        a, b = n1 // 2 - calib // 2, n2 // 2 - calib // 2
        m[a:a + calib, b:b + calib] = 1
        cnt = float(m.sum())
        if best is None or abs(cnt - target) < abs(best[0] - target):
            best = (cnt, m)
        if abs(cnt - target) <= 0.02 * target:
            break
        if cnt > target:
            lo = r
        else:
            hi = r
    return best[1]


def make_mask(w: Workload, rng) -> np.ndarray:
    n0, n1, n2 = w.n
    if w.fft_rank == 3:
        out = np.empty((w.batch, w.frames, n1, n2), dtype=np.float32)
        for b in range(w.batch):
            for t in range(w.frames):
                if w.mask_recipe == "poisson2d":
                    out[b, t] = _mask_poisson2d(n1, n2, min(_center_count(w, n1), n1, n2), w.accel, rng)
                else:
                    raise ValueError(w.mask_recipe)
        return out
    out = np.empty((w.batch, w.frames, n2), dtype=np.float32)
    nc = min(_center_count(w, n2), n2)
    tot = max(int(round(n2 / w.accel)), nc)
    for b in range(w.batch):
        for t in range(w.frames):
            if w.mask_recipe == "random1d":
                out[b, t] = _mask_random1d(n2, nc, tot, rng)
            elif w.mask_recipe == "equispaced1d":
                out[b, t] = _mask_equispaced1d(n2, nc, int(round(w.accel)), rng)
            elif w.mask_recipe == "ktvd1d":
                out[b, t] = _mask_ktvd1d(n2, nc, tot, rng)
            else:
                raise ValueError(w.mask_recipe)
    return out


def expand_mask(w: Workload, mask_ri: np.ndarray) -> np.ndarray:
    """Readout-invariant mask -> full (B, T, n0, n1, n2) float32 array with the same values."""
    if w.fft_rank == 2:
        full = np.broadcast_to(mask_ri[:, :, None, None, :], w.mask_shape(MASK_FULL))
    else:
        full = np.broadcast_to(mask_ri[:, :, None, :, :], w.mask_shape(MASK_FULL))
    return np.ascontiguousarray(full, dtype=np.float32)


# ----------------------------------------------------------------------------------------------
# whole input sets
# ----------------------------------------------------------------------------------------------
def make_inputs(w: Workload, seed_offset: int = 0) -> dict:
    """Everything except the measurements y (which need the forward model; the tests build them
    with the oracle's operator, the benchmark with ``standin_kspace``).

    Returns complex64 / float32 arrays: x_true, x (the iterate), g (a cotangent), sens,
    mask (readout-invariant form), noise (k-space noise, unmasked)."""
    sens = make_sens(w, _rng(w, 0, seed_offset))
    if w.x_is_noise:
        x_true = cnormal(_rng(w, 1, seed_offset), w.image_shape())
        x = cnormal(_rng(w, 2, seed_offset), w.image_shape())
    else:
        x_true = make_phantom(w, _rng(w, 1, seed_offset)) + cnormal(_rng(w, 5, seed_offset), w.image_shape(), w.phantom_noise)
        # the iterate: a damped, perturbed copy of the object (stands in for the zero-filled image)
        x = 0.8 * x_true + cnormal(_rng(w, 2, seed_offset), w.image_shape(), w.phantom_noise)
    g = cnormal(_rng(w, 3, seed_offset), w.image_shape())
    mask = make_mask(w, _rng(w, 4, seed_offset))
    return {
        "x_true": x_true.astype(np.complex64),
        "x": x.astype(np.complex64),
        "g": g.astype(np.complex64),
        "sens": sens,
        "mask": mask,
    }


def make_noise(w: Workload, seed_offset: int = 0) -> np.ndarray:
    """k-space noise CN(0, sigma^2), shape of y, complex64 (to be masked by the caller)."""
    rng = _rng(w, 6, seed_offset)
    out = np.empty(w.kspace_shape(), dtype=np.complex64)
    s = w.noise_sigma / np.sqrt(2.0)
    flat = out.reshape(w.batch * w.coils, -1)
    for i in range(flat.shape[0]):       # chunked: the 3-D case is 1.7 GB
        m = flat.shape[1]
        flat[i] = (rng.standard_normal(m, dtype=np.float32) * s + 1j * rng.standard_normal(m, dtype=np.float32) * s)
    return out


def standin_kspace(w: Workload, mask_ri: np.ndarray, seed_offset: int = 0) -> np.ndarray:
    """Measurements for timing runs, drawn without any transform: masked complex Gaussian samples
    under a centre-weighted power-law envelope (k-space energy of an image concentrates at the
    centre).  Values do not influence the run time; the sampling pattern does and is the real one."""
    rng = _rng(w, 7, seed_offset)
    env = np.ones(w.n, dtype=np.float32)
    for a, m in enumerate(w.n):
        if m == 1:
            continue
        k = (np.arange(m) - m // 2) / (m / 2.0)
        shape = [1, 1, 1]; shape[a] = m
        env = env * (1.0 / (1.0 + 30.0 * k.reshape(shape) ** 2)).astype(np.float32)
    full = expand_mask(w, mask_ri)                       # (B,T,n0,n1,n2)
    out = np.empty(w.kspace_shape(), dtype=np.complex64)
    s = 1.0 / np.sqrt(2.0)
    for b in range(w.batch):
        for c in range(w.coils):
            for t in range(w.frames):
                z = rng.standard_normal(w.n, dtype=np.float32) * s + 1j * rng.standard_normal(w.n, dtype=np.float32) * s
                out[b, c, t] = (z * env * full[b, t]).astype(np.complex64)
    return out
