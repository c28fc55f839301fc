"""The C-ABI library loads, exports every symbol that include/gleam.h declares, and its host-side
argument checks work without a GPU (no kernel is launched here)."""
import ctypes
import os
import re

import pytest

import paper_2207_08393_b200 as g
from paper_2207_08393_b200 import binding, _build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    _build.build()
    return g.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gleam.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return re.findall(r"GLEAM_API\s+[\w\s\*]+?\b(gleam_\w+)\s*\(", text)


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 6
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.EXPORTS) <= set(names)


def test_version_and_status_strings(lib):
    assert g.gleam_version() == 1
    assert g.gleam_status_string(0) == "ok"
    for code in range(-9, 0):
        assert g.gleam_status_string(code) not in ("ok", "unknown status")
    assert g.gleam_status_string(-99) == "unknown status"


def test_dims_struct_matches_header_layout():
    d = g.gleam_dims
    assert ctypes.sizeof(d) == 4 * 10 + 3 * 8
    assert d.stream.offset == 40 and d.workspace.offset == 48 and d.workspace_bytes.offset == 56


def test_supported_lengths(lib):
    for n in (64, 160, 192, 256, 320, 368, 640):
        assert g.gleam_dc_length_supported(n)
    for n in (1, 3, 7, 63, 1000003):
        assert not g.gleam_dc_length_supported(n)


def test_workspace_size_formula(lib):
    # readout-invariant 2-D: mask table + z table
    d = g.make_dims(4, 15, 1, 2, (1, 640, 368))
    ws = g.gleam_dc_workspace_size(d)
    assert ws >= 4 * 15 * 640 * 368 * 8
    # full mask: one coil-volume workspace
    d = g.make_dims(1, 8, 1, 3, (320, 320, 256), mask_kind=g.GLEAM_MASK_FULL)
    assert g.gleam_dc_workspace_size(d) >= 8 * 320 * 320 * 256 * 8


@pytest.mark.parametrize("kw,code", [
    (dict(batch=0), binding.GLEAM_ERR_BAD_DIMS),
    (dict(coils=0), binding.GLEAM_ERR_BAD_DIMS),
    (dict(fft_rank=4), binding.GLEAM_ERR_BAD_DIMS),
    (dict(n=(2, 64, 64)), binding.GLEAM_ERR_BAD_DIMS),           # rank 2 needs n0 == 1
    (dict(mask_kind=7), binding.GLEAM_ERR_BAD_DIMS),
    (dict(n=(1, 64, 63)), binding.GLEAM_ERR_UNSUPPORTED_SIZE),   # odd length
    (dict(n=(1, 14, 64)), binding.GLEAM_ERR_UNSUPPORTED_SIZE),   # no plan for 14
])
def test_bad_dims_are_rejected_on_the_host(lib, kw, code):
    base = dict(batch=1, coils=2, frames=1, fft_rank=2, n=(1, 64, 64))
    base.update(kw)
    d = g.make_dims(**base)
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_workspace_size(d)
    assert e.value.status == code
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward(1 << 20, 2 << 20, 3 << 20, 4 << 20, 1.0, 5 << 20, d)   # never dereferenced
    assert e.value.status == code


def test_null_pointers_and_small_workspace(lib):
    d = g.make_dims(1, 2, 1, 2, (1, 64, 64))
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward(None, 8, 8, 8, 1.0, 8, d)
    assert e.value.status == binding.GLEAM_ERR_NULL_POINTER
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward(8, None, 8, 8, 1.0, 8, d)            # forward needs y
    assert e.value.status == binding.GLEAM_ERR_NULL_POINTER
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward(1 << 20, 2 << 20, 3 << 20, 4 << 20, 1.0, 5 << 20, d)   # no workspace given
    assert e.value.status == binding.GLEAM_ERR_NULL_POINTER
    d = g.make_dims(1, 2, 1, 2, (1, 64, 64), workspace=1 << 30, workspace_bytes=16)
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward(1 << 20, 2 << 20, 3 << 20, 4 << 20, 1.0, 5 << 20, d)
    assert e.value.status == binding.GLEAM_ERR_WORKSPACE_TOO_SMALL


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library(str(tmp_path / "nope.so"))


def test_every_eligible_extent_pair_has_row_tile_kernels(lib):
    """The separable 3-D path has contiguous row-tile passes for every (n1, n2) whose plans allow them: the
    library's table against the eligibility rule evaluated here from sizes.def (two-stage split of n1 whose
    first radix is a multiple of the lines a warp holds of n2; two-stage warp-resident plan of n2; shared memory)."""
    import importlib.util
    spec = importlib.util.spec_from_file_location("gen_pairs", os.path.join(ROOT, "paper_2207_08393_b200", "csrc", "gen_pairs.py"))
    gp = importlib.util.module_from_spec(spec); spec.loader.exec_module(gp)
    P = gp.plans()
    listed = set()
    for line in open(os.path.join(ROOT, "paper_2207_08393_b200", "csrc", "pairs.def")):
        m = re.match(r"GLEAM_PAIR\((\d+), (\d+), (\d+), (\d+),", line)
        if m:
            listed.add((int(m.group(1)), int(m.group(4)), int(m.group(2))))
    assert len(listed) >= 300
    count = 0
    for n1 in P:
        for n2 in P:
            ry = g.gleam_dc_rowtile_split(n1, n2)
            hit = [t for t in listed if t[0] == n1 and t[1] == n2]
            assert (ry > 0) == bool(hit), (n1, n2)
            if hit:
                assert hit[0][2] == ry and n1 % ry == 0
                count += 1
    assert count == len(listed)
    assert g.gleam_dc_rowtile_split(320, 256) == 16 and g.gleam_dc_rowtile_split(128, 128) > 0
    assert g.gleam_dc_rowtile_split(640, 256) == 0            # three-stage plan: general middle pass
