"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI on numpy inputs and
compare with the CPU oracle under the stated tolerances."""
import numpy as np

REL_L2_TOL = 2e-5      # relative L2 error against the oracle
MAX_ABS_TOL = 1e-4     # max abs error, in units of max|input image|


def to_oracle_dims(oracle_mod, batch, coils, frames, fft_rank, n, sens_has_frames, mask_kind):
    return oracle_mod.Dims(batch, coils, frames, fft_rank, tuple(n), sens_has_frames, mask_kind)


def run_gpu(x, y, sens, mask, eta, fft_rank, sens_has_frames, mask_kind, in_place=False, stream=None):
    """forward if y is given, else vjp.  Returns a complex64 numpy array."""
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    B, T = x.shape[0], x.shape[1]
    C = sens.shape[1]
    n = x.shape[2:]
    tx = torch.from_numpy(np.ascontiguousarray(x, dtype=np.complex64)).to(dev)
    ts = torch.from_numpy(np.ascontiguousarray(sens, dtype=np.complex64)).to(dev)
    tm = torch.from_numpy(np.ascontiguousarray(mask, dtype=np.float32)).to(dev)
    ty = None if y is None else torch.from_numpy(np.ascontiguousarray(y, dtype=np.complex64)).to(dev)
    probe = g.make_dims(B, C, T, fft_rank, n, sens_has_frames, mask_kind)
    nbytes = g.gleam_dc_workspace_size(probe)
    ws = torch.empty(nbytes + 512, dtype=torch.uint8, device=dev)
    ws[nbytes:] = 0xA5                                   # canary behind the workspace
    out = tx if in_place else torch.full_like(tx, float("nan"))
    st = stream if stream is not None else torch.cuda.current_stream()
    d = g.make_dims(B, C, T, fft_rank, n, sens_has_frames, mask_kind, stream=st, workspace=ws.data_ptr(),
                    workspace_bytes=nbytes)
    if ty is not None:
        g.gleam_dc_forward(tx, ty, ts, tm, eta, out, d)
    else:
        g.gleam_dc_vjp(tx, ts, tm, eta, out, d)
    torch.cuda.synchronize()
    assert bool((ws[nbytes:] == 0xA5).all()), "workspace overrun"
    return out.cpu().numpy()


def assert_close(got, ref, x_in, what=""):
    ref = np.asarray(ref)
    got = np.asarray(got).astype(np.complex128)
    assert np.isfinite(got.view(np.float64)).all(), what + ": non-finite output"
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300)
    mab = np.abs(got - ref).max() / max(np.abs(x_in).max(), 1e-300)
    assert rel <= REL_L2_TOL, "%s: rel L2 %.3e > %.1e" % (what, rel, REL_L2_TOL)
    assert mab <= MAX_ABS_TOL, "%s: max abs %.3e > %.1e (units of max|x|)" % (what, mab, MAX_ABS_TOL)
    return rel, mab


def run_gpu_modl(z, y, sens, mask, mu, n_iter, fft_rank, sens_has_frames, mask_kind, in_place=False):
    """MoDL model inversion (y given) or its VJP (y None) through the C ABI.  Returns complex64 numpy."""
    import torch
    import paper_2207_08393_b200 as g
    dev = torch.device("cuda:0")
    B, T = z.shape[0], z.shape[1]
    C = sens.shape[1]
    n = z.shape[2:]
    tz = torch.from_numpy(np.ascontiguousarray(z, dtype=np.complex64)).to(dev)
    ts = torch.from_numpy(np.ascontiguousarray(sens, dtype=np.complex64)).to(dev)
    tm = torch.from_numpy(np.ascontiguousarray(mask, dtype=np.float32)).to(dev)
    ty = None if y is None else torch.from_numpy(np.ascontiguousarray(y, dtype=np.complex64)).to(dev)
    probe = g.make_dims(B, C, T, fft_rank, n, sens_has_frames, mask_kind)
    nbytes = g.gleam_modl_cg_workspace_size(probe)
    ws = torch.empty(nbytes + 512, dtype=torch.uint8, device=dev)
    ws[nbytes:] = 0xA5                                   # canary behind the workspace
    out = tz if in_place else torch.full_like(tz, float("nan"))
    d = g.make_dims(B, C, T, fft_rank, n, sens_has_frames, mask_kind, stream=torch.cuda.current_stream(),
                    workspace=ws.data_ptr(), workspace_bytes=nbytes)
    if ty is not None:
        g.gleam_modl_cg_forward(tz, ty, ts, tm, mu, n_iter, out, d)
    else:
        g.gleam_modl_cg_vjp(tz, ts, tm, mu, n_iter, out, d)
    torch.cuda.synchronize()
    assert bool((ws[nbytes:] == 0xA5).all()), "workspace overrun"
    return out.cpu().numpy()
