"""Bridge to the learned prior on the GPU: the two-real-channel layout read and written inside the
data-consistency kernels (bit-exact against the oracle's layout conversion applied to the plain call)
and the complex l1 loss with its gradient (against the oracle)."""
import numpy as np
import pytest

from oracle.oracle import MASK_FULL, MASK_READOUT_INVARIANT
from tests.gpu_common import assert_close
from tests.test_gpu_parity import problem

pytestmark = pytest.mark.gpu

CASES = [
    (2, 2, 3, 2, (1, 20, 48), MASK_READOUT_INVARIANT),      # one-pass 2-D kernel
    (2, 1, 2, 1, (1, 12, 46), MASK_READOUT_INVARIANT),      # line length 2 mod 4
    (2, 1, 4, 1, (1, 16, 320), MASK_READOUT_INVARIANT),     # one line per warp, k-space units numbered across coils
    (2, 1, 5, 20, (1, 192, 160), MASK_READOUT_INVARIANT),   # one block per SM with a group split by coils
    (2, 1, 3, 1, (1, 8, 384), MASK_READOUT_INVARIANT),      # block-synchronised row kernel (three-stage plan)
    (2, 2, 3, 1, (1, 12, 16), MASK_FULL),
    (3, 2, 3, 1, (6, 64, 32), MASK_READOUT_INVARIANT),      # row-tile 3-D path
    (3, 1, 2, 2, (4, 46, 32), MASK_READOUT_INVARIANT),      # general 3-D path
    (3, 1, 3, 1, (6, 10, 12), MASK_FULL),
]


def _run(d, x_arr, y, sens, mask, eta, layout, in_place=False):
    """x_arr: complex64 (B,T,...) or float32 (B,2,T,...) according to layout; returns the output array as stored."""
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    tx = torch.from_numpy(np.ascontiguousarray(x_arr)).to(dev)
    ts, tm = torch.from_numpy(sens).to(dev), torch.from_numpy(mask).to(dev)
    ty = None if y is None else torch.from_numpy(y).to(dev)
    dc = g.DataConsistency(d.batch, d.coils, d.frames, d.fft_rank, d.n, d.sens_has_frames, d.mask_kind)
    if in_place:
        out = tx
    elif layout & g.GLEAM_OUT_CHANNELS:
        out = torch.full((d.batch, 2, d.frames) + tuple(d.n), float("nan"), dtype=torch.float32, device=dev)
    else:
        out = torch.full((d.batch, d.frames) + tuple(d.n), float("nan"), dtype=torch.complex64, device=dev)
    if ty is not None:
        g.gleam_dc_forward_layout(tx, ty, ts, tm, eta, out, dc.dims(), layout)
    else:
        g.gleam_dc_vjp_layout(tx, ts, tm, eta, out, dc.dims(), layout)
    torch.cuda.synchronize()
    return out.cpu().numpy()


@pytest.mark.parametrize("case", CASES)
def test_two_channel_layout_is_bit_exact(oracle, case):
    """Reading x and writing out in (B, 2, T, ...) form changes where the same float values live,
    nothing else: every layout combination gives the bytes of the complex call, re-laid by the oracle."""
    import paper_2207_08393_b200 as g
    rank, B, C, T, n, kind = case
    d, x, y, sens, mask = problem(rank, B, C, T, n, kind, seed=41 + sum(n))
    x_ch = oracle.complex_to_channels(x)
    for yy in (y, None):
        plain = _run(d, x, yy, sens, mask, 0.9, 0)
        ref = oracle.dc_forward(x, yy, sens, mask, 0.9, d) if yy is not None else oracle.dc_vjp(x, sens, mask, 0.9, d)
        assert_close(plain, ref, x, "plain call")
        plain_ch = oracle.complex_to_channels(plain)
        assert _run(d, x_ch, yy, sens, mask, 0.9, g.GLEAM_X_CHANNELS).tobytes() == plain.tobytes()
        assert _run(d, x, yy, sens, mask, 0.9, g.GLEAM_OUT_CHANNELS).tobytes() == plain_ch.tobytes()
        assert _run(d, x_ch, yy, sens, mask, 0.9, g.GLEAM_X_CHANNELS | g.GLEAM_OUT_CHANNELS).tobytes() == plain_ch.tobytes()
        assert _run(d, x_ch, yy, sens, mask, 0.9, g.GLEAM_X_CHANNELS | g.GLEAM_OUT_CHANNELS, in_place=True).tobytes() == plain_ch.tobytes()


def test_mixed_layouts_in_place_are_rejected():
    import torch
    import paper_2207_08393_b200 as g
    from paper_2207_08393_b200 import binding
    d, x, y, sens, mask = problem(2, 1, 2, 1, (1, 12, 16), MASK_READOUT_INVARIANT, seed=2)
    dev = torch.device("cuda:0")
    tx, ts, tm = (torch.from_numpy(a).to(dev) for a in (x, sens, mask))
    dc = g.DataConsistency(1, 2, 1, 2, (1, 12, 16))
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_vjp_layout(tx, ts, tm, 1.0, tx, dc.dims(), g.GLEAM_OUT_CHANNELS)
    assert e.value.status == binding.GLEAM_ERR_ALIAS
    with pytest.raises(g.GleamError) as e:
        g.gleam_dc_vjp_layout(tx, ts, tm, 1.0, tx, dc.dims(), 8)
    assert e.value.status == binding.GLEAM_ERR_BAD_DIMS


@pytest.mark.parametrize("shape", [(2, 3, 1, 12, 16), (1, 20, 1, 192, 160), (1, 1, 4, 6, 10)])
def test_l1_loss_and_gradient_match_oracle(oracle, shape):
    import torch
    import paper_2207_08393_b200 as g
    rng = np.random.default_rng(sum(shape))
    x = ((rng.normal(size=shape) + 1j * rng.normal(size=shape))).astype(np.complex64)
    r = ((rng.normal(size=shape) + 1j * rng.normal(size=shape))).astype(np.complex64)
    r.ravel()[::7] = x.ravel()[::7]                     # exact zeros of the difference
    ref_loss, ref_grad = oracle.l1_loss(x, r, with_grad=True)
    dev = torch.device("cuda:0")
    B, T = shape[0], shape[1]
    n = shape[2:]
    rank = 3 if n[0] > 1 else 2
    ws = torch.empty(g.gleam_l1_loss_workspace_size(), dtype=torch.uint8, device=dev)
    dims = g.make_dims(B, 1, T, rank, n, stream=torch.cuda.current_stream(), workspace=ws)
    tr = torch.from_numpy(r).to(dev)
    for layout in (0, g.GLEAM_X_CHANNELS, g.GLEAM_OUT_CHANNELS, g.GLEAM_X_CHANNELS | g.GLEAM_OUT_CHANNELS):
        tx = torch.from_numpy(oracle.complex_to_channels(x) if layout & g.GLEAM_X_CHANNELS else x).to(dev)
        loss = torch.full((1,), float("nan"), dtype=torch.float64, device=dev)
        if layout & g.GLEAM_OUT_CHANNELS:
            grad = torch.full((B, 2, T) + tuple(n), float("nan"), dtype=torch.float32, device=dev)
        else:
            grad = torch.full(shape, float("nan"), dtype=torch.complex64, device=dev)
        g.gleam_l1_loss(tx, tr, loss, grad, dims, layout)
        torch.cuda.synchronize()
        assert abs(float(loss[0]) - ref_loss) <= 1e-6 * ref_loss
        got = grad.cpu().numpy()
        if layout & g.GLEAM_OUT_CHANNELS:
            got = oracle.channels_to_complex(got)
        assert np.isfinite(got.view(np.float32)).all()
        assert np.abs(got - ref_grad).max() <= 1e-5 / x.size          # |grad| = 1/N per element
        assert np.all(got.ravel()[::7] == 0)
        g.gleam_l1_loss(tx, tr, loss, None, dims, layout)              # loss alone
        torch.cuda.synchronize()
        assert abs(float(loss[0]) - ref_loss) <= 1e-6 * ref_loss
