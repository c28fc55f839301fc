"""GPU parity: gleam_dc_forward / gleam_dc_vjp through the C ABI against the CPU oracle, element
by element on the same seeded inputs.  Tolerances: relative L2 <= 2e-5 and max abs error
<= 1e-4 * max|x| (x = the call's image-domain input)."""
import numpy as np
import pytest

from oracle.oracle import Dims, MASK_FULL, MASK_READOUT_INVARIANT
from paper_2207_08393_b200 import workloads as wl
from tests.gpu_common import assert_close, run_gpu

pytestmark = pytest.mark.gpu


def crandn(rng, *shape):
    return ((rng.normal(size=shape) + 1j * rng.normal(size=shape)) / np.sqrt(2)).astype(np.complex64)


def problem(rank, B, C, T, n, mask_kind, sens_has_frames=0, weighted=False, seed=0, density=0.4):
    rng = np.random.default_rng(seed)
    d = Dims(B, C, T, rank, tuple(n), sens_has_frames, mask_kind)
    x = crandn(rng, *d.image_shape()); y = crandn(rng, *d.kspace_shape()); sens = crandn(rng, *d.sens_shape())
    if weighted:
        mask = rng.uniform(0, 1, d.mask_shape()).astype(np.float32)
    else:
        mask = (rng.uniform(size=d.mask_shape()) < density).astype(np.float32)
    return d, x, y, sens, mask


def check(oracle, d, x, y, sens, mask, eta, in_place=False, what=""):
    ref_f = oracle.dc_forward(x, y, sens, mask, eta, d, nthreads=8)
    got_f = run_gpu(x, y, sens, mask, eta, d.fft_rank, d.sens_has_frames, d.mask_kind, in_place=in_place)
    assert_close(got_f, ref_f, x, what + " forward")
    ref_v = oracle.dc_vjp(x, sens, mask, eta, d, nthreads=8)
    got_v = run_gpu(x, None, sens, mask, eta, d.fft_rank, d.sens_has_frames, d.mask_kind, in_place=in_place)
    assert_close(got_v, ref_v, x, what + " vjp")


# every compiled transform length on each axis role, small batches, ragged tiles
LENGTHS = [2, 4, 6, 8, 10, 12, 16, 20, 24, 32, 40, 46, 48, 64, 80, 92, 96, 120, 128, 160, 184, 192, 240, 256, 320,
           368, 384, 512, 640]


@pytest.mark.parametrize("n2", LENGTHS)
def test_rank2_separable_every_length_as_phase_encode_axis(oracle, n2):
    d, x, y, sens, mask = problem(2, 2, 3, 1, (1, 10, n2), MASK_READOUT_INVARIANT, seed=n2)
    check(oracle, d, x, y, sens, mask, 0.9, what="n2=%d" % n2)


@pytest.mark.parametrize("n1", LENGTHS)
def test_rank2_separable_every_length_as_readout_axis(oracle, n1):
    d, x, y, sens, mask = problem(2, 1, 2, 2, (1, n1, 12), MASK_READOUT_INVARIANT, seed=1000 + n1)
    check(oracle, d, x, y, sens, mask, 1.1, what="n1=%d" % n1)


@pytest.mark.parametrize("n", [(1, 6, 8), (1, 10, 6), (1, 64, 46), (1, 46, 64), (1, 20, 160), (1, 96, 40)])
@pytest.mark.parametrize("weighted", [False, True])
def test_rank2_full_mask(oracle, n, weighted):
    d, x, y, sens, mask = problem(2, 2, 3, 2, n, MASK_FULL, weighted=weighted, seed=sum(n))
    check(oracle, d, x, y, sens, mask, 0.8, what="full %s" % (n,))


@pytest.mark.parametrize("n", [(4, 6, 10), (2, 2, 2), (6, 10, 2), (16, 12, 20), (10, 46, 32), (32, 20, 64),
                               (6, 64, 16), (4, 128, 24), (4, 32, 64), (6, 64, 32), (2, 320, 64)])   # (6, 64, 16): dense weighted mask, more sampled entries per tile than the staging area
@pytest.mark.parametrize("mask_kind", [MASK_READOUT_INVARIANT, MASK_FULL])
def test_rank3_small(oracle, n, mask_kind):
    d, x, y, sens, mask = problem(3, 2, 3, 1, n, mask_kind, weighted=(n[0] == 6), seed=sum(n) + mask_kind)
    check(oracle, d, x, y, sens, mask, 1.0, what="rank3 %s kind %d" % (n, mask_kind))


@pytest.mark.parametrize("n", [(4, 128, 128), (6, 192, 160), (4, 256, 192), (4, 92, 46), (2, 240, 120), (4, 184, 96), (6, 48, 24)])
def test_rank3_row_tile_pairs_beyond_the_benchmark_shape(oracle, n):
    """Extent pairs that used the general strided middle pass before every eligible pair got row-tile kernels."""
    import paper_2207_08393_b200 as g
    assert g.gleam_dc_rowtile_split(n[1], n[2]) > 0
    d, x, y, sens, mask = problem(3, 1, 3, 1, n, MASK_READOUT_INVARIANT, seed=sum(n), density=0.25)
    check(oracle, d, x, y, sens, mask, 1.0, what="row-tile pair %s" % (n,))


def test_rank3_separable_spans_several_chunks(oracle):
    # workspace chunking: 48 MB / (units * n1 * n2 * 8 B) slabs per chunk -> more than one chunk
    d, x, y, sens, mask = problem(3, 1, 8, 1, (12, 320, 256), MASK_READOUT_INVARIANT, seed=5, density=0.1)
    check(oracle, d, x, y, sens, mask, 1.0, what="rank3 chunks")


@pytest.mark.parametrize("mask_kind", [MASK_READOUT_INVARIANT, MASK_FULL])
def test_frames_and_per_frame_sensitivities(oracle, mask_kind):
    d, x, y, sens, mask = problem(2, 2, 3, 3, (1, 12, 16), mask_kind, sens_has_frames=1, seed=11)
    check(oracle, d, x, y, sens, mask, 0.7, what="frames")
    d, x, y, sens, mask = problem(3, 1, 2, 2, (4, 6, 8), mask_kind, sens_has_frames=1, seed=12)
    check(oracle, d, x, y, sens, mask, 0.7, what="frames3d")


@pytest.mark.parametrize("mask_kind", [MASK_READOUT_INVARIANT, MASK_FULL])
def test_in_place_output(oracle, mask_kind):
    d, x, y, sens, mask = problem(2, 1, 4, 1, (1, 20, 32), mask_kind, seed=3)
    check(oracle, d, x, y, sens, mask, 1.0, in_place=True, what="in place")


def test_degenerate_masks_and_eta(oracle):
    d, x, y, sens, mask = problem(2, 1, 3, 1, (1, 16, 24), MASK_READOUT_INVARIANT, seed=4)
    check(oracle, d, x, y, sens, np.zeros_like(mask), 1.0, what="empty mask")        # out == x
    check(oracle, d, x, y, sens, np.ones_like(mask), 1.0, what="full sampling")
    check(oracle, d, x, y, sens, mask, 0.0, what="eta 0")
    got = run_gpu(x, y, sens, np.zeros_like(mask), 1.0, 2, 0, MASK_READOUT_INVARIANT)
    assert np.array_equal(got, x)


def test_single_coil_single_everything(oracle):
    d, x, y, sens, mask = problem(2, 1, 1, 1, (1, 2, 2), MASK_FULL, seed=6, density=1.0)
    check(oracle, d, x, y, sens, mask, 0.5, what="2x2")


@pytest.mark.parametrize("rank,n", [(2, (1, 16, 24)), (3, (6, 10, 12))])
@pytest.mark.parametrize("mask_kind", [MASK_READOUT_INVARIANT, MASK_FULL])
def test_unsampled_measurements_are_never_read(oracle, rank, n, mask_kind):
    """y may hold anything (here NaN) wherever the mask is zero, for both mask kinds and ranks."""
    d, x, y, sens, mask = problem(rank, 1, 3, 1, n, mask_kind, seed=8 + rank + mask_kind)
    dfull = Dims(1, 3, 1, rank, n, 0, MASK_FULL)
    mfull = np.broadcast_to(mask.reshape(mask.shape[:2] + (1,) * (5 - mask.ndim) + mask.shape[2:]), dfull.mask_shape())
    y_clean = y * mfull[:, None]
    ref = oracle.dc_forward(x, y_clean, sens, mask, 1.0, d)
    y_bad = y.copy()
    y_bad[np.broadcast_to(mfull[:, None] == 0, y.shape)] = np.nan
    got = run_gpu(x, y_bad, sens, mask, 1.0, rank, 0, mask_kind)
    assert_close(got, ref, x, "NaN in unsampled y")


@pytest.mark.parametrize("case", [
    (2, 2, 8, 1, (1, 64, 160), MASK_READOUT_INVARIANT),      # one-pass 2-D kernel
    (2, 1, 6, 20, (1, 192, 160), MASK_READOUT_INVARIANT),    # the same, one block per SM with a group split by coils
    (3, 1, 4, 1, (8, 64, 32), MASK_READOUT_INVARIANT),       # separable 3-D path
    (3, 1, 3, 1, (6, 20, 24), MASK_FULL),                    # general path
])
def test_deterministic_across_repeats(case):
    """No float atomics anywhere: 20 repeats give the same bits (forward and VJP)."""
    rank, B, C, T, n, kind = case
    d, x, y, sens, mask = problem(rank, B, C, T, n, kind, seed=9)
    first = run_gpu(x, y, sens, mask, 1.0, rank, 0, kind)
    first_v = run_gpu(x, None, sens, mask, 1.0, rank, 0, kind)
    for _ in range(20):
        assert np.array_equal(first, run_gpu(x, y, sens, mask, 1.0, rank, 0, kind))
        assert np.array_equal(first_v, run_gpu(x, None, sens, mask, 1.0, rank, 0, kind))


def test_cross_export_identities():
    """forward(x; y) - forward(0; y) = vjp(x) - ... affine structure through the library itself."""
    d, x, y, sens, mask = problem(2, 1, 4, 1, (1, 32, 48), MASK_READOUT_INVARIANT, seed=10)
    f_x = run_gpu(x, y, sens, mask, 0.9, 2, 0, 1).astype(np.complex128)
    f_0 = run_gpu(np.zeros_like(x), y, sens, mask, 0.9, 2, 0, 1).astype(np.complex128)
    v_x = run_gpu(x, None, sens, mask, 0.9, 2, 0, 1).astype(np.complex128)
    assert np.linalg.norm(f_x - f_0 - v_x) <= 1e-5 * np.linalg.norm(v_x)
    full = np.broadcast_to(mask[:, :, None, None, :], (1, 1, 1, 32, 48)).copy()
    f_full = run_gpu(x, y, sens, full, 0.9, 2, 0, 0).astype(np.complex128)
    assert np.linalg.norm(f_full - f_x) <= 1e-5 * np.linalg.norm(f_x)


def test_non_default_stream(oracle):
    import torch
    d, x, y, sens, mask = problem(2, 1, 3, 1, (1, 16, 32), MASK_READOUT_INVARIANT, seed=13)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        got = run_gpu(x, y, sens, mask, 1.0, 2, 0, 1, stream=st)
    assert_close(got, oracle.dc_forward(x, y, sens, mask, 1.0, d), x, "stream")


def test_error_codes_on_device_buffers():
    import torch
    import paper_2207_08393_b200 as g
    from paper_2207_08393_b200 import binding
    x = torch.zeros((1, 1, 1, 64, 64), dtype=torch.complex64, device="cuda")
    y = torch.zeros((1, 2, 1, 1, 64, 64), dtype=torch.complex64, device="cuda")
    s = torch.zeros((1, 2, 1, 64, 64), dtype=torch.complex64, device="cuda")
    m = torch.ones((1, 1, 64), dtype=torch.float32, device="cuda")
    ws = torch.empty(g.gleam_dc_workspace_size(g.make_dims(1, 2, 1, 2, (1, 64, 64))), dtype=torch.uint8, device="cuda")
    d = g.make_dims(1, 2, 1, 2, (1, 64, 64), workspace=ws)
    host = torch.zeros((1, 1, 1, 64, 64), dtype=torch.complex64)
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward(host, y, s, m, 1.0, x, d)
    assert e.value.status == binding.GLEAM_ERR_NOT_DEVICE_POINTER
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_forward(x, y, s, m, 1.0, y, d)               # out overlaps y
    assert e.value.status == binding.GLEAM_ERR_ALIAS
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_vjp(x, s, m, 1.0, x.view(torch.float32)[..., 4:].data_ptr(), d)   # partial overlap
    assert e.value.status == binding.GLEAM_ERR_ALIAS
    g.gleam_dc_forward(x, y, s, m, 1.0, x, d)                  # exact alias is allowed
    torch.cuda.synchronize()
    # a call that returns an argument error has enqueued nothing: an adjoint whose out overlaps y
    # must leave both untouched (it clears out only after every check has passed)
    y.fill_(3.0)
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_adjoint(y, s, m, y.view(torch.float32)[0, 1].data_ptr(), d)
    assert e.value.status == binding.GLEAM_ERR_ALIAS
    torch.cuda.synchronize()
    assert bool((y == 3.0).all())


# ----------------------------------------------------------------------------------------------
# the five workloads at full size
# ----------------------------------------------------------------------------------------------
def workload_case(oracle, name, mask_kind=MASK_READOUT_INVARIANT):
    w = wl.WORKLOADS[name]
    inp = wl.make_inputs(w)
    d = Dims(w.batch, w.coils, w.frames, w.fft_rank, w.n, 0, mask_kind)
    mask = inp["mask"] if mask_kind == MASK_READOUT_INVARIANT else wl.expand_mask(w, inp["mask"])
    dri = Dims(w.batch, w.coils, w.frames, w.fft_rank, w.n, 0, MASK_READOUT_INVARIANT)
    y = oracle.apply_A(inp["x_true"], inp["sens"], inp["mask"], dri, nthreads=8)
    noise = wl.make_noise(w)
    y = (y + noise * wl.expand_mask(w, inp["mask"])[:, None]).astype(np.complex64)
    return w, d, inp, mask, y


@pytest.mark.parametrize("name", ["slice64", "knee2d", "brain2d", "cine"])
@pytest.mark.parametrize("mask_kind", [MASK_READOUT_INVARIANT, MASK_FULL])
def test_workload_full_size(oracle, name, mask_kind):
    w, d, inp, mask, y = workload_case(oracle, name, mask_kind)
    ref = oracle.dc_forward(inp["x"], y, inp["sens"], mask, w.eta, d, nthreads=8)
    got = run_gpu(inp["x"], y, inp["sens"], mask, w.eta, w.fft_rank, 0, mask_kind)
    assert_close(got, ref, inp["x"], name + " forward")
    refv = oracle.dc_vjp(inp["g"], inp["sens"], mask, w.eta, d, nthreads=8)
    gotv = run_gpu(inp["g"], None, inp["sens"], mask, w.eta, w.fft_rank, 0, mask_kind)
    assert_close(gotv, refv, inp["g"], name + " vjp")


def test_workload_knee3d_full_size(oracle):
    """320x320x256, 8 coils: the oracle evaluates the full 3-D definition in double precision."""
    w, d, inp, mask, y = workload_case(oracle, "knee3d")
    got = run_gpu(inp["x"], y, inp["sens"], mask, w.eta, 3, 0, MASK_READOUT_INVARIANT)
    ref = oracle.dc_forward(inp["x"], y, inp["sens"], mask, w.eta, d, nthreads=8)
    assert_close(got, ref, inp["x"], "knee3d forward")
    del ref, got
    gotv = run_gpu(inp["g"], None, inp["sens"], mask, w.eta, 3, 0, MASK_READOUT_INVARIANT)
    refv = oracle.dc_vjp(inp["g"], inp["sens"], mask, w.eta, d, nthreads=8)
    assert_close(gotv, refv, inp["g"], "knee3d vjp")


def test_workload_knee3d_full_size_general_mask(oracle):
    """The same volume with its mask handed over as a general (B, T, n0, n1, n2) array: the arbitrary-mask
    path (three transformed axes on a coil-volume workspace) at full size."""
    w, d, inp, mask, y = workload_case(oracle, "knee3d", MASK_FULL)
    got = run_gpu(inp["x"], y, inp["sens"], mask, w.eta, 3, 0, MASK_FULL)
    ref = oracle.dc_forward(inp["x"], y, inp["sens"], mask, w.eta, d, nthreads=8)
    assert_close(got, ref, inp["x"], "knee3d forward, general mask")
    del ref, got
    gotv = run_gpu(inp["g"], None, inp["sens"], mask, w.eta, 3, 0, MASK_FULL)
    refv = oracle.dc_vjp(inp["g"], inp["sens"], mask, w.eta, d, nthreads=8)
    assert_close(gotv, refv, inp["g"], "knee3d vjp, general mask")


def test_chained_iterations_match_oracle(oracle):
    """Unrolled chain as the cine workload runs it: x_{i+1} = DC(x_i), then g_i = VJP(g_{i+1})."""
    w = wl.scaled(wl.WORKLOADS["cine"], frames=4, n=(1, 48, 40), chain=4)
    inp = wl.make_inputs(w)
    d = Dims(w.batch, w.coils, w.frames, 2, w.n, 0, MASK_READOUT_INVARIANT)
    y = oracle.apply_A(inp["x_true"], inp["sens"], inp["mask"], d).astype(np.complex64)
    xg, xo = inp["x"], inp["x"]
    for _ in range(w.chain):
        xg = run_gpu(xg, y, inp["sens"], inp["mask"], w.eta, 2, 0, MASK_READOUT_INVARIANT)
        xo = oracle.dc_forward(xo, y, inp["sens"], inp["mask"], w.eta, d).astype(np.complex64)
    assert_close(xg, xo, inp["x"], "chain forward")
    gg, go = inp["g"], inp["g"]
    for _ in range(w.chain):
        gg = run_gpu(gg, None, inp["sens"], inp["mask"], w.eta, 2, 0, MASK_READOUT_INVARIANT)
        go = oracle.dc_vjp(go, inp["sens"], inp["mask"], w.eta, d).astype(np.complex64)
    assert_close(gg, go, inp["g"], "chain vjp")


def test_rank3_chunked_workspace_matches_whole_volume(oracle, tmp_path):
    """The 3-D separable path can process the readout slabs in chunks (GLEAM_CHUNK_MB, read once per
    process): a child process with a 1 MB chunk target must give the same bits as the default
    whole-volume run, and both must match the oracle."""
    import os
    import subprocess
    import sys
    import paper_2207_08393_b200 as g
    d, x, y, sens, mask = problem(3, 1, 4, 1, (12, 64, 48), MASK_READOUT_INVARIANT, seed=21, density=0.15)
    whole = run_gpu(x, y, sens, mask, 0.9, 3, 0, MASK_READOUT_INVARIANT)
    assert_close(whole, oracle.dc_forward(x, y, sens, mask, 0.9, d), x, "whole volume")
    np.savez(tmp_path / "in.npz", x=x, y=y, sens=sens, mask=mask)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import sys, numpy as np; sys.path.insert(0, %r)\n"
        "from tests.gpu_common import run_gpu\n"
        "import paper_2207_08393_b200 as g\n"
        "z = np.load(%r)\n"
        "ws = g.gleam_dc_workspace_size(g.make_dims(1, 4, 1, 3, (12, 64, 48)))\n"
        "out = run_gpu(z['x'], z['y'], z['sens'], z['mask'], 0.9, 3, 0, 1)\n"
        "np.savez(%r, out=out, ws=ws)\n"
    ) % (root, str(tmp_path / "in.npz"), str(tmp_path / "out.npz"))
    # 4 coils x 64 x 48 x 8 B = 98 KB per slab: a 1 MB target gives 10 slabs per chunk, two chunks for 12 slabs
    subprocess.run([sys.executable, "-c", code], check=True, env=dict(os.environ, GLEAM_CHUNK_MB="1"), timeout=600)
    res = np.load(tmp_path / "out.npz")
    assert int(res["ws"]) < g.gleam_dc_workspace_size(g.make_dims(1, 4, 1, 3, (12, 64, 48)))
    assert np.array_equal(res["out"], whole)


def _in_place_chain(x, y, sens, mask, eta, iters):
    """iters forward calls, then iters VJP calls, all in place on one buffer and enqueued back to
    back with no synchronisation in between; returns the buffer after each half."""
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    tx, ty, ts, tm = (torch.from_numpy(a).to(dev) for a in (x, y, sens, mask))
    B, T, C, n = x.shape[0], x.shape[1], sens.shape[1], x.shape[2:]
    dc = g.DataConsistency(B, C, T, 2, n, 0, MASK_READOUT_INVARIANT)
    for _ in range(iters):
        dc.forward(tx, ty, ts, tm, eta, tx)
    after_fwd = tx.clone()
    for _ in range(iters):
        dc.vjp(tx, ts, tm, eta, tx)
    torch.cuda.synchronize()
    return after_fwd.cpu().numpy(), tx.cpu().numpy()


def test_overlapped_launches_equal_serialised_launches(oracle, tmp_path):
    """One-round launches of the one-pass row kernel start while the launch before them drains and
    wait for it on the device.  A chain of in-place calls (every call reads what the call before it
    wrote, and overwrites what that call read) must give the bits of a child process in which
    every launch is fully serialised (GLEAM_NO_OVERLAP=1, read once per process), and both must
    match the oracle."""
    import os
    import subprocess
    import sys
    d, x, y, sens, mask = problem(2, 1, 4, 6, (1, 48, 160), MASK_READOUT_INVARIANT, seed=5, density=0.2)
    eta, iters = 0.2, 6
    fwd, vjp = _in_place_chain(x, y, sens, mask, eta, iters)
    xo = x
    for _ in range(iters):
        xo = oracle.dc_forward(xo, y, sens, mask, eta, d).astype(np.complex64)
    assert_close(fwd, xo, x, "in-place forward chain")
    np.savez(tmp_path / "in.npz", x=x, y=y, sens=sens, mask=mask)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import sys, numpy as np; sys.path.insert(0, %r)\n"
        "from tests.test_gpu_parity import _in_place_chain\n"
        "z = np.load(%r)\n"
        "fwd, vjp = _in_place_chain(z['x'], z['y'], z['sens'], z['mask'], %r, %d)\n"
        "np.savez(%r, fwd=fwd, vjp=vjp)\n"
    ) % (root, str(tmp_path / "in.npz"), eta, iters, str(tmp_path / "out.npz"))
    subprocess.run([sys.executable, "-c", code], check=True, env=dict(os.environ, GLEAM_NO_OVERLAP="1"), timeout=600)
    res = np.load(tmp_path / "out.npz")
    assert np.array_equal(res["fwd"], fwd)
    assert np.array_equal(res["vjp"], vjp)


@pytest.mark.parametrize("case", [
    (2, 2, 3, 2, (1, 20, 46), MASK_READOUT_INVARIANT),
    (2, 1, 4, 1, (1, 64, 320), MASK_READOUT_INVARIANT),      # three-stage plan on the contiguous axis (fallback row kernel)
    (3, 2, 3, 1, (6, 64, 32), MASK_READOUT_INVARIANT),       # row-tile 3-D path
    (3, 1, 2, 1, (10, 46, 32), MASK_READOUT_INVARIANT),      # general 3-D path
    (2, 2, 3, 1, (1, 12, 16), MASK_FULL),                    # nothing to prepare
])
def test_prepared_forward_equals_forward(oracle, case):
    """gleam_dc_prepare + gleam_dc_forward_prepared (unrolled iterations with the same y and mask)
    give the bits of gleam_dc_forward, iteration after iteration, and match the oracle."""
    import torch
    import paper_2207_08393_b200 as g
    rank, B, C, T, n, kind = case
    d, x, y, sens, mask = problem(rank, B, C, T, n, kind, seed=77 + sum(n))
    dev = torch.device("cuda:0")
    tx, ty, ts, tm = (torch.from_numpy(a).to(dev) for a in (x, y, sens, mask))
    dc_a = g.DataConsistency(B, C, T, rank, n, 0, kind)
    dc_b = g.DataConsistency(B, C, T, rank, n, 0, kind)
    dc_b.prepare(ty, tm)
    xa, xb, xo = tx, tx, x
    for it in range(3):
        xa = dc_a.forward(xa, ty, ts, tm, 0.6)
        xb = dc_b.forward_prepared(xb, ty, ts, tm, 0.6)
        torch.cuda.synchronize()
        assert torch.equal(xa, xb), "iteration %d differs" % it
        xo = oracle.dc_forward(xo, y, sens, mask, 0.6, d).astype(np.complex64)
    assert_close(xb.cpu().numpy(), xo, x, "prepared chain")
    with pytest.raises(g.GleamError):
        g.gleam_dc_prepare(None, tm, dc_b.dims())


@pytest.mark.parametrize("case", [
    (2, 2, 3, 2, (1, 20, 46), MASK_READOUT_INVARIANT, False),
    (2, 2, 3, 1, (1, 12, 16), MASK_FULL, True),
    (3, 1, 3, 1, (6, 64, 32), MASK_READOUT_INVARIANT, True),
])
def test_adjoint_is_the_zero_filled_image(oracle, case):
    """gleam_dc_adjoint = A^H y against the oracle's adjoint operator (pinned by the adjoint identity)."""
    import torch
    import paper_2207_08393_b200 as g
    rank, B, C, T, n, kind, weighted = case
    d, x, y, sens, mask = problem(rank, B, C, T, n, kind, weighted=weighted, seed=5 + sum(n))
    dev = torch.device("cuda:0")
    ty, ts, tm = (torch.from_numpy(a).to(dev) for a in (y, sens, mask))
    dc = g.DataConsistency(B, C, T, rank, n, 0, kind)
    got = dc.adjoint(ty, ts, tm).cpu().numpy()
    ref = oracle.apply_AH(y, sens, mask, d)
    got = got.astype(np.complex128)
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= 2e-5 and np.abs(got - ref).max() <= 1e-4 * np.abs(ref).max(), rel


# ----------------------------------------------------------------------------------------------
# single-round launches of the one-pass kernel with numbered k-space units: one block per SM, with and
# without groups split by coils over four warps
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("C,T,R", [
    (8, 18, 192),      # 12 groups per SM on 148 SMs: whole groups only, also for the call with z
    (6, 14, 192),      # 10 groups per SM: two groups per SM split over four warps each; coils not a multiple of four
    (5, 20, 192),      # 13 groups per SM: one split group, quarters of 1, 1, 1 and 2 coils
    (4, 12, 160),      # 7 groups per SM: single-warp blocks
])
def test_one_pass_kernel_block_shapes(oracle, C, T, R):
    d, x, y, sens, mask = problem(2, 1, C, T, (1, R, 160), MASK_READOUT_INVARIANT, sens_has_frames=1, seed=C + T, density=0.14)
    check(oracle, d, x, y, sens, mask, 0.7, what="one-pass kernel, %d coils, %d frames of %d rows" % (C, T, R))
