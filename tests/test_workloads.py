"""Host-side checks of the seeded synthetic input generators (no method arithmetic in there)."""
import numpy as np
import pytest

from paper_2207_08393_b200 import workloads as wl


@pytest.mark.parametrize("name", ["slice64", "cine"])
def test_shapes_dtypes_and_determinism(name):
    w = wl.WORKLOADS[name]
    a = wl.make_inputs(w)
    b = wl.make_inputs(w)
    assert a["x"].shape == w.image_shape() and a["x"].dtype == np.complex64
    assert a["sens"].shape == w.sens_shape() and a["sens"].dtype == np.complex64
    assert a["mask"].shape == w.mask_shape() and a["mask"].dtype == np.float32
    for k in a:
        assert np.array_equal(a[k], b[k]), k
    assert np.allclose(np.sum(np.abs(a["sens"]) ** 2, axis=1), 1.0, atol=1e-5)


def test_mask_recipes_have_the_stated_density():
    w = wl.WORKLOADS["slice64"]
    m = wl.make_inputs(w)["mask"]
    assert m.sum() == 16 and m[0, 0, 28:36].all()
    w = wl.scaled(wl.WORKLOADS["knee2d"], batch=1, n=(1, 16, 368))
    m = wl.make_mask(w, np.random.default_rng(0))
    assert m[0, 0, 184 - 7:184 + 8].all() and 46 <= m.sum() <= 61
    w = wl.scaled(wl.WORKLOADS["brain2d"], batch=2, n=(1, 16, 320))
    m = wl.make_mask(w, np.random.default_rng(0))
    assert (m.sum(axis=-1) == 80).all()
    w = wl.WORKLOADS["cine"]
    m = wl.make_mask(w, np.random.default_rng(0))
    assert (m.sum(axis=-1) == 16).all() and m[0, :, 77:83].all()
    assert len({tuple(r) for r in m[0]}) > 1          # re-randomised per frame


def test_poisson_disc_mask_density_and_calibration():
    w = wl.scaled(wl.WORKLOADS["knee3d"], n=(4, 96, 80), center=12)
    m = wl.make_mask(w, np.random.default_rng(0))[0, 0]
    target = 96 * 80 / 12.0
    assert abs(m.sum() - target) <= 0.25 * target
    assert m[48 - 6:48 + 6, 40 - 6:40 + 6].all()


def test_expand_mask_and_standin_kspace():
    w = wl.scaled(wl.WORKLOADS["cine"], frames=3, n=(1, 12, 16), coils=2)
    m = wl.make_mask(w, np.random.default_rng(0))
    full = wl.expand_mask(w, m)
    assert full.shape == w.mask_shape(wl.MASK_FULL)
    assert np.array_equal(full[0, 1, 0, 5], m[0, 1])
    y = wl.standin_kspace(w, m)
    assert y.shape == w.kspace_shape() and y.dtype == np.complex64
    assert np.all(y[:, :, :, :, :, :][..., m[0, 0] == 0][:, :, 0] == 0)
