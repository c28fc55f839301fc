"""The persistent kernel of the separable 3-D path (n2 = 256, n1 a compiled multiple of 16): parity
with the CPU oracle over several ring turns, odd coil counts, batches and frames; bit-identical
repeats; and the bounded waits between blocks (a withheld work item must end in GLEAM_ERR_TIMEOUT,
never in a hang)."""
import numpy as np
import pytest

from oracle.oracle import Dims, MASK_READOUT_INVARIANT
from tests.gpu_common import assert_close, run_gpu
from tests.test_gpu_parity import problem

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def fused_on():
    """The persistent kernel is opt-in; every test here selects it and restores the default afterwards."""
    import paper_2207_08393_b200 as g
    g.gleam_dc_set_fused(True)
    yield
    g.gleam_dc_set_fused(False)


@pytest.mark.parametrize("B,C,T,n", [
    (1, 2, 1, (4, 64, 256)),        # fewer slabs than ring slots
    (1, 3, 1, (40, 64, 256)),       # odd coil count (groups of 2 and 1 coils), several ring turns
    (2, 1, 2, (6, 128, 256)),       # one coil: the second compute group only joins the coil sum; batch and frames
    (1, 8, 1, (12, 320, 256)),      # the knee3d phase-encode plane
])
def test_fused_path_matches_oracle(oracle, B, C, T, n):
    d, x, y, sens, mask = problem(3, B, C, T, n, MASK_READOUT_INVARIANT, seed=sum(n) + C, density=0.2)
    ref_v = oracle.dc_vjp(x, sens, mask, 0.9, d, nthreads=8)
    got_v = run_gpu(x, None, sens, mask, 0.9, 3, 0, MASK_READOUT_INVARIANT)
    assert_close(got_v, ref_v, x, "fused vjp %s" % (n,))
    # the forward call of the same dims and workspace layout (its k-space pass is not part of the persistent kernel)
    ref_f = oracle.dc_forward(x, y, sens, mask, 0.9, d, nthreads=8)
    got_f = run_gpu(x, y, sens, mask, 0.9, 3, 0, MASK_READOUT_INVARIANT)
    assert_close(got_f, ref_f, x, "forward %s" % (n,))


def test_fused_path_knee3d_full_size_vjp(oracle):
    """The whole 320 x 320 x 256 volume with 8 coils through the persistent kernel (320 slabs, 20 turns of the default
    ring of 16 slabs), element by element against the oracle; the status word stays clear."""
    import torch
    import paper_2207_08393_b200 as g
    from oracle.oracle import Dims
    from paper_2207_08393_b200 import workloads as wl
    w = wl.WORKLOADS["knee3d"]
    inp = wl.make_inputs(w)
    d = Dims(w.batch, w.coils, w.frames, 3, w.n, 0, MASK_READOUT_INVARIANT)
    dev = torch.device("cuda:0")
    tg, ts, tm = (torch.from_numpy(inp[k]).to(dev) for k in ("g", "sens", "mask"))
    dc = g.DataConsistency(w.batch, w.coils, w.frames, 3, w.n)
    got = dc.vjp(tg, ts, tm, w.eta)
    assert g.gleam_dc_check_status(dc.dims()) == 0
    waits = g.gleam_dc_fused_wait_stats(dc.dims())
    assert set(waits) == set(g.binding.FUSED_WAIT_KINDS)
    got = got.cpu().numpy()
    del tg, ts, tm, dc
    torch.cuda.empty_cache()
    ref = oracle.dc_vjp(inp["g"], inp["sens"], inp["mask"], w.eta, d, nthreads=8)
    assert_close(got, ref, inp["g"], "knee3d vjp through the persistent kernel")


def test_fused_path_weighted_mask_in_place_and_per_frame_sens(oracle):
    d, x, y, sens, mask = problem(3, 1, 4, 2, (6, 64, 256), MASK_READOUT_INVARIANT, sens_has_frames=1, weighted=True, seed=3)
    ref = oracle.dc_vjp(x, sens, mask, 1.1, d, nthreads=8)
    got = run_gpu(x, None, sens, mask, 1.1, 3, 1, MASK_READOUT_INVARIANT, in_place=True)
    assert_close(got, ref, x, "fused vjp in place")
    ref = oracle.dc_forward(x, y, sens, mask, 1.1, d, nthreads=8)
    got = run_gpu(x, y, sens, mask, 1.1, 3, 1, MASK_READOUT_INVARIANT, in_place=True)
    assert_close(got, ref, x, "fused forward in place")


def test_fused_path_is_deterministic():
    """Work items are handed out dynamically; every output element is still computed by one item in
    a fixed order, so repeats give the same bits."""
    d, x, y, sens, mask = problem(3, 1, 5, 1, (16, 64, 256), MASK_READOUT_INVARIANT, seed=4, density=0.15)
    first = run_gpu(x, None, sens, mask, 1.0, 3, 0, MASK_READOUT_INVARIANT)
    first_f = run_gpu(x, y, sens, mask, 1.0, 3, 0, MASK_READOUT_INVARIANT)
    for _ in range(20):
        assert np.array_equal(first, run_gpu(x, None, sens, mask, 1.0, 3, 0, MASK_READOUT_INVARIANT))
        assert np.array_equal(first_f, run_gpu(x, y, sens, mask, 1.0, 3, 0, MASK_READOUT_INVARIANT))


@pytest.mark.parametrize("n", [(16, 64, 256), (12, 128, 256)])
def test_fused_path_repeats_with_a_small_middle_radix(oracle, n):
    """Planes of 64 and 128 rows (middle radix 4 and 8, below the 16 rows of a tile): the mask rows of a middle-pass
    item share a buffer with nothing else that is live.  A block that goes from a third-pass item straight to a
    middle-pass item whose dependency is already met is the case that once wrote them over live partial sums, now
    and then: ten runs each, every one against the oracle."""
    d, x, y, sens, mask = problem(3, 1, 5, 1, n, MASK_READOUT_INVARIANT, seed=sum(n), density=0.15)
    ref = oracle.dc_vjp(x, sens, mask, 1.0, d, nthreads=8)
    for i in range(10):
        got = run_gpu(x, None, sens, mask, 1.0, 3, 0, MASK_READOUT_INVARIANT)
        assert_close(got, ref, x, "fused vjp %s, run %d" % (n, i))


def test_status_is_ok_after_a_normal_call():
    import torch
    import paper_2207_08393_b200 as g
    d, x, y, sens, mask = problem(3, 1, 2, 1, (4, 64, 256), MASK_READOUT_INVARIANT, seed=6)
    dev = torch.device("cuda:0")
    tx, ts, tm = (torch.from_numpy(a).to(dev) for a in (x, sens, mask))
    dc = g.DataConsistency(1, 2, 1, 3, (4, 64, 256))
    dc.vjp(tx, ts, tm, 1.0)
    assert g.gleam_dc_check_status(dc.dims()) == 0
    # a problem class without inter-block waits only synchronises
    dc2 = g.DataConsistency(1, 2, 1, 2, (1, 16, 32))
    assert g.gleam_dc_check_status(dc2.dims()) == 0


def test_withheld_item_ends_in_timeout_not_in_a_hang():
    """One first-pass item is drawn but never run nor counted: every block that depends on it gives
    up after the (shortened) limit, the kernel returns, the status call reports GLEAM_ERR_TIMEOUT,
    and the next normal call on the same workspace works."""
    import time
    import torch
    import paper_2207_08393_b200 as g
    from paper_2207_08393_b200 import binding
    d, x, y, sens, mask = problem(3, 1, 4, 1, (8, 64, 256), MASK_READOUT_INVARIANT, seed=7, density=0.2)
    dev = torch.device("cuda:0")
    tx, ts, tm = (torch.from_numpy(a).to(dev) for a in (x, sens, mask))
    dc = g.DataConsistency(1, 4, 1, 3, (8, 64, 256))
    good = dc.vjp(tx, ts, tm, 0.7).clone()
    assert g.gleam_dc_check_status(dc.dims()) == 0
    per_period = 4 + 16 + 4                      # BY third-pass, 16 middle-pass, BY first-pass items (BY = 64 / 16)
    try:
        g.gleam_dc_debug_fused(2 * per_period + 4 + 16 + 1, 50_000_000)      # a first-pass item of slab 2; 50 ms limit
        t0 = time.time()
        dc.vjp(tx, ts, tm, 0.7)
        status = g.gleam_dc_check_status(dc.dims())
        elapsed = time.time() - t0
    finally:
        g.gleam_dc_debug_fused(-1, 0)
    assert status == binding.GLEAM_ERR_TIMEOUT
    assert elapsed < 20.0
    again = dc.vjp(tx, ts, tm, 0.7)
    assert g.gleam_dc_check_status(dc.dims()) == 0
    assert torch.equal(again, good)
