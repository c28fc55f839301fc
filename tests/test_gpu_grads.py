"""gleam_dc_grad_eta / gleam_dc_grad_y (gradients of Eq. 3 with respect to the step size and the
measurements) through the C ABI against the CPU oracle, element by element."""
import numpy as np
import pytest

from oracle.oracle import MASK_FULL, MASK_READOUT_INVARIANT
from paper_2207_08393_b200 import workloads as wl
from tests.test_gpu_parity import crandn, problem

pytestmark = pytest.mark.gpu


def run_grads(d, g_in, x, y, sens, mask, eta):
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    tg, tx, ty, ts, tm = (torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in (g_in, x, y, sens, mask))
    probe = g.make_dims(d.batch, d.coils, d.frames, d.fft_rank, d.n, d.sens_has_frames, d.mask_kind)
    nbytes = g.gleam_dc_grad_workspace_size(probe)
    ws = torch.empty(nbytes + 512, dtype=torch.uint8, device=dev)
    ws[nbytes:] = 0xA5
    dims = g.make_dims(d.batch, d.coils, d.frames, d.fft_rank, d.n, d.sens_has_frames, d.mask_kind,
                       stream=torch.cuda.current_stream(), workspace=ws.data_ptr(), workspace_bytes=nbytes)
    ge = torch.full((d.batch,), float("nan"), dtype=torch.float64, device=dev)
    gy = torch.full_like(ty, float("nan"))
    g.gleam_dc_grad_eta(tg, tx, ty, ts, tm, ge, dims)
    g.gleam_dc_grad_y(tg, ts, tm, eta, gy, dims)
    torch.cuda.synchronize()
    assert bool((ws[nbytes:] == 0xA5).all()), "workspace overrun"
    return ge.cpu().numpy(), gy.cpu().numpy()


CASES = [
    (2, 2, 3, 2, (1, 20, 46), MASK_READOUT_INVARIANT, 0, False),
    (2, 1, 4, 1, (1, 64, 320), MASK_READOUT_INVARIANT, 0, True),
    (2, 2, 3, 1, (1, 12, 16), MASK_FULL, 0, True),
    (3, 2, 3, 1, (6, 64, 32), MASK_READOUT_INVARIANT, 0, False),
    (3, 1, 2, 2, (10, 46, 32), MASK_READOUT_INVARIANT, 1, False),
    (3, 1, 3, 1, (6, 10, 12), MASK_FULL, 0, True),
    (3, 1, 2, 1, (2, 6, 10), MASK_FULL, 0, False),          # extents that are 2 mod 4: the global sign of the centred transform
]


@pytest.mark.parametrize("case", CASES)
def test_gradients_match_oracle(oracle, case):
    rank, B, C, T, n, kind, shf, weighted = case
    d, x, y, sens, mask = problem(rank, B, C, T, n, kind, sens_has_frames=shf, weighted=weighted, seed=31 + sum(n))
    g_in = crandn(np.random.default_rng(5), *d.image_shape())
    eta = 0.8
    ge, gy = run_grads(d, g_in, x, y, sens, mask, eta)
    ref_e = oracle.dc_grad_eta(g_in, x, y, sens, mask, d, nthreads=8)
    ref_y = oracle.dc_grad_y(g_in, sens, mask, eta, d, nthreads=8)
    # grad_eta is an inner product of O(N) terms of size |g||a|: tolerance relative to that scale
    a_norm = np.array([np.linalg.norm((x[b].astype(complex) - oracle.dc_forward(x, y, sens, mask, 1.0, d)[b]).ravel()) for b in range(B)])
    g_norm = np.array([np.linalg.norm(g_in[b].ravel()) for b in range(B)])
    assert np.all(np.abs(ge - ref_e) <= 2e-5 * a_norm * g_norm), (ge, ref_e)
    rel = np.linalg.norm(gy - ref_y) / max(np.linalg.norm(ref_y), 1e-300)
    assert np.isfinite(gy.view(np.float32)).all() and rel <= 2e-5, rel
    assert np.abs(gy - ref_y).max() <= 1e-4 * np.abs(g_in).max() * max(1.0, np.abs(ref_y).max() / np.abs(g_in).max())
    # exactly zero where the mask is zero
    mfull = np.broadcast_to(mask.reshape(mask.shape[:2] + (1,) * (5 - mask.ndim) + mask.shape[2:]), (B, T) + tuple(n))
    assert np.all(gy[np.broadcast_to(mfull[:, None] == 0, gy.shape)] == 0)


def test_gradients_on_the_cine_workload(oracle):
    w = wl.WORKLOADS["cine"]
    inp = wl.make_inputs(w)
    from oracle.oracle import Dims
    d = Dims(w.batch, w.coils, w.frames, 2, w.n, 0, MASK_READOUT_INVARIANT)
    y = oracle.apply_A(inp["x_true"], inp["sens"], inp["mask"], d, nthreads=8).astype(np.complex64)
    ge, gy = run_grads(d, inp["g"], inp["x"], y, inp["sens"], inp["mask"], w.eta)
    ref_e = oracle.dc_grad_eta(inp["g"], inp["x"], y, inp["sens"], inp["mask"], d, nthreads=8)
    ref_y = oracle.dc_grad_y(inp["g"], inp["sens"], inp["mask"], w.eta, d, nthreads=8)
    scale = np.linalg.norm(inp["g"].ravel()) * np.linalg.norm((inp["x"].astype(complex) - oracle.dc_forward(inp["x"], y, inp["sens"], inp["mask"], 1.0, d, nthreads=8)).ravel())
    assert abs(ge[0] - ref_e[0]) <= 2e-5 * scale
    assert np.linalg.norm(gy - ref_y) <= 2e-5 * np.linalg.norm(ref_y)
