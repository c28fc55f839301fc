"""ctypes binding of ``libgleam_dc.so`` (C ABI: include/gleam.h).

Argument marshalling only: every arithmetic step runs in the CUDA library.  The functions carry
the same names and argument order as the C entry points and accept torch CUDA tensors (or raw
integer device addresses).  There is no CPU fallback: if the shared library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libgleam_dc.so")

GLEAM_OK = 0
GLEAM_ERR_NULL_POINTER = -1
GLEAM_ERR_BAD_DIMS = -2
GLEAM_ERR_UNSUPPORTED_SIZE = -3
GLEAM_ERR_NOT_DEVICE_POINTER = -4
GLEAM_ERR_WORKSPACE_TOO_SMALL = -5
GLEAM_ERR_ALIAS = -6
GLEAM_ERR_CUDA = -7
GLEAM_ERR_UNIMPLEMENTED = -8
GLEAM_ERR_TIMEOUT = -9

GLEAM_X_CHANNELS = 1
GLEAM_OUT_CHANNELS = 2

GLEAM_MASK_FULL = 0
GLEAM_MASK_READOUT_INVARIANT = 1

EXPORTS = ["gleam_dc_forward", "gleam_dc_vjp", "gleam_dc_workspace_size", "gleam_dc_length_supported",
           "gleam_status_string", "gleam_version", "gleam_dc_forward_host", "gleam_dc_vjp_host",
           "gleam_dc_host_arena_size", "gleam_dc_launch_count", "gleam_dc_profile_begin", "gleam_dc_profile_end",
           "gleam_dc_forward_static", "gleam_dc_static_scratch_bytes",
           "gleam_modl_cg_forward", "gleam_modl_cg_vjp", "gleam_modl_cg_workspace_size",
           "gleam_dc_prepare", "gleam_dc_forward_prepared", "gleam_dc_forward_aty", "gleam_dc_adjoint",
           "gleam_dc_check_status", "gleam_dc_debug_fused", "gleam_dc_fused_wait_stats", "gleam_dc_set_fused",
           "gleam_dc_grad_eta", "gleam_dc_grad_y", "gleam_dc_grad_workspace_size",
           "gleam_dc_forward_layout", "gleam_dc_vjp_layout", "gleam_l1_loss", "gleam_l1_loss_workspace_size",
           "gleam_measure_fp32_peak", "gleam_dc_rowtile_split"]

KERNEL_CLASSES = ["zmap", "col_z", "row_fused", "row_fwd", "col_mid_sep", "row_inv", "col_mid_full", "col_fwd",
                  "col_inv", "cg_vec", "fused3d"]


class gleam_dims(ctypes.Structure):
    _fields_ = [
        ("struct_version", ctypes.c_int32),
        ("batch", ctypes.c_int32),
        ("coils", ctypes.c_int32),
        ("frames", ctypes.c_int32),
        ("fft_rank", ctypes.c_int32),
        ("n", ctypes.c_int32 * 3),
        ("sens_has_frames", ctypes.c_int32),
        ("mask_kind", ctypes.c_int32),
        ("stream", ctypes.c_void_p),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_uint64),
    ]


class GleamError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__("gleam status %d: %s" % (status, text))
        self.status = status


_lib = None


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(path):
            raise RuntimeError(
                "%s is missing: build it with `python -m paper_2207_08393_b200._build` "
                "(there is no CPU fallback)" % path)
        lib = ctypes.CDLL(path)
        vp, f32, i32 = ctypes.c_void_p, ctypes.c_float, ctypes.c_int
        dp = ctypes.POINTER(gleam_dims)
        lib.gleam_dc_forward.argtypes = [vp, vp, vp, vp, f32, vp, dp]
        lib.gleam_dc_forward.restype = i32
        lib.gleam_dc_vjp.argtypes = [vp, vp, vp, f32, vp, dp]
        lib.gleam_dc_vjp.restype = i32
        lib.gleam_dc_workspace_size.argtypes = [dp, ctypes.POINTER(ctypes.c_uint64)]
        lib.gleam_dc_workspace_size.restype = i32
        lib.gleam_dc_length_supported.argtypes = [ctypes.c_int32]
        lib.gleam_dc_length_supported.restype = i32
        lib.gleam_status_string.argtypes = [i32]
        lib.gleam_status_string.restype = ctypes.c_char_p
        lib.gleam_version.argtypes = []
        lib.gleam_version.restype = i32
        u64 = ctypes.c_uint64
        lib.gleam_dc_forward_host.argtypes = [vp, vp, vp, vp, f32, vp, dp, vp, u64]
        lib.gleam_dc_forward_host.restype = i32
        lib.gleam_dc_vjp_host.argtypes = [vp, vp, vp, f32, vp, dp, vp, u64]
        lib.gleam_dc_vjp_host.restype = i32
        lib.gleam_dc_host_arena_size.argtypes = [dp, ctypes.POINTER(u64)]
        lib.gleam_dc_host_arena_size.restype = i32
        lib.gleam_dc_forward_static.argtypes = [vp, vp, vp, vp, f32, vp, dp]
        lib.gleam_dc_forward_static.restype = i32
        lib.gleam_dc_static_scratch_bytes.argtypes = []
        lib.gleam_dc_static_scratch_bytes.restype = u64
        lib.gleam_dc_adjoint.argtypes = [vp, vp, vp, vp, dp]
        lib.gleam_dc_adjoint.restype = i32
        lib.gleam_dc_prepare.argtypes = [vp, vp, dp]
        lib.gleam_dc_prepare.restype = i32
        lib.gleam_dc_forward_prepared.argtypes = [vp, vp, vp, vp, f32, vp, dp]
        lib.gleam_dc_forward_prepared.restype = i32
        lib.gleam_dc_forward_aty.argtypes = [vp, vp, vp, vp, f32, vp, dp]
        lib.gleam_dc_forward_aty.restype = i32
        lib.gleam_modl_cg_forward.argtypes = [vp, vp, vp, vp, f32, ctypes.c_int32, vp, dp]
        lib.gleam_modl_cg_forward.restype = i32
        lib.gleam_modl_cg_vjp.argtypes = [vp, vp, vp, f32, ctypes.c_int32, vp, dp]
        lib.gleam_modl_cg_vjp.restype = i32
        lib.gleam_modl_cg_workspace_size.argtypes = [dp, ctypes.POINTER(u64)]
        lib.gleam_modl_cg_workspace_size.restype = i32
        lib.gleam_dc_check_status.argtypes = [dp]
        lib.gleam_dc_check_status.restype = i32
        lib.gleam_dc_fused_wait_stats.argtypes = [dp, ctypes.POINTER(u64), ctypes.c_int32]
        lib.gleam_dc_fused_wait_stats.restype = i32
        lib.gleam_dc_grad_eta.argtypes = [vp, vp, vp, vp, vp, vp, dp]
        lib.gleam_dc_grad_eta.restype = i32
        lib.gleam_dc_grad_y.argtypes = [vp, vp, vp, f32, vp, dp]
        lib.gleam_dc_grad_y.restype = i32
        lib.gleam_dc_grad_workspace_size.argtypes = [dp, ctypes.POINTER(u64)]
        lib.gleam_dc_grad_workspace_size.restype = i32
        u32 = ctypes.c_uint32
        lib.gleam_dc_forward_layout.argtypes = [vp, vp, vp, vp, f32, vp, dp, u32]
        lib.gleam_dc_forward_layout.restype = i32
        lib.gleam_dc_vjp_layout.argtypes = [vp, vp, vp, f32, vp, dp, u32]
        lib.gleam_dc_vjp_layout.restype = i32
        lib.gleam_l1_loss.argtypes = [vp, vp, vp, vp, dp, u32]
        lib.gleam_l1_loss.restype = i32
        lib.gleam_l1_loss_workspace_size.argtypes = []
        lib.gleam_l1_loss_workspace_size.restype = u64
        lib.gleam_measure_fp32_peak.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double)]
        lib.gleam_measure_fp32_peak.restype = i32
        lib.gleam_dc_rowtile_split.argtypes = [ctypes.c_int32, ctypes.c_int32]
        lib.gleam_dc_rowtile_split.restype = ctypes.c_int32
        lib.gleam_dc_set_fused.argtypes = [ctypes.c_int32]
        lib.gleam_dc_set_fused.restype = None
        lib.gleam_dc_debug_fused.argtypes = [ctypes.c_int32, u64]
        lib.gleam_dc_debug_fused.restype = None
        lib.gleam_dc_launch_count.argtypes = []
        lib.gleam_dc_launch_count.restype = u64
        lib.gleam_dc_profile_begin.argtypes = []
        lib.gleam_dc_profile_begin.restype = i32
        lib.gleam_dc_profile_end.argtypes = [ctypes.POINTER(f32), ctypes.POINTER(ctypes.c_uint32), ctypes.c_int32]
        lib.gleam_dc_profile_end.restype = i32
        _lib = lib
    return _lib


def gleam_status_string(status: int) -> str:
    return load_library().gleam_status_string(int(status)).decode()


def gleam_version() -> int:
    return int(load_library().gleam_version())


def gleam_dc_length_supported(n: int) -> bool:
    return load_library().gleam_dc_length_supported(int(n)) == GLEAM_OK


def _addr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return int(t.data_ptr())


def _check(status: int):
    if status != GLEAM_OK:
        raise GleamError(status, gleam_status_string(status))


def make_dims(batch, coils, frames, fft_rank, n, sens_has_frames=0, mask_kind=GLEAM_MASK_READOUT_INVARIANT,
              stream=None, workspace=None, workspace_bytes=0) -> gleam_dims:
    """Fills a ``gleam_dims``.  ``stream`` is a torch.cuda.Stream, a raw handle or None (legacy
    default stream); ``workspace`` a torch uint8 CUDA tensor or a raw address."""
    d = gleam_dims()
    d.struct_version = 1
    d.batch, d.coils, d.frames, d.fft_rank = int(batch), int(coils), int(frames), int(fft_rank)
    d.n[0], d.n[1], d.n[2] = int(n[0]), int(n[1]), int(n[2])
    d.sens_has_frames, d.mask_kind = int(sens_has_frames), int(mask_kind)
    if stream is not None and not isinstance(stream, int):
        stream = stream.cuda_stream
    d.stream = stream or None
    if workspace is not None and not isinstance(workspace, int):
        workspace_bytes = workspace.numel() * workspace.element_size()
        workspace = workspace.data_ptr()
    d.workspace = workspace or None
    d.workspace_bytes = int(workspace_bytes)
    return d


def gleam_dc_workspace_size(dims: gleam_dims) -> int:
    out = ctypes.c_uint64(0)
    _check(load_library().gleam_dc_workspace_size(ctypes.byref(dims), ctypes.byref(out)))
    return int(out.value)


def gleam_dc_forward(x, y, sens, mask, eta, out, dims: gleam_dims) -> None:
    """out = x - eta A^H (A x - y)  (Eq. 3, eta = 2t).  Enqueues on dims.stream and returns."""
    _check(load_library().gleam_dc_forward(_addr(x), _addr(y), _addr(sens), _addr(mask), float(eta), _addr(out),
                                            ctypes.byref(dims)))


def gleam_dc_vjp(grad_out, sens, mask, eta, grad_in, dims: gleam_dims) -> None:
    """grad_in = grad_out - eta A^H A grad_out  (VJP of Eq. 3 with respect to x)."""
    _check(load_library().gleam_dc_vjp(_addr(grad_out), _addr(sens), _addr(mask), float(eta), _addr(grad_in),
                                        ctypes.byref(dims)))


def gleam_dc_adjoint(y, sens, mask, out, dims: gleam_dims) -> None:
    """out = A^H y, the zero-filled SENSE image."""
    _check(load_library().gleam_dc_adjoint(_addr(y), _addr(sens), _addr(mask), _addr(out), ctypes.byref(dims)))


def gleam_dc_prepare(y, mask, dims: gleam_dims) -> None:
    """Computes what Eq. 3 needs from y and the mask alone into dims.workspace (kept by the caller
    until the last gleam_dc_forward_prepared)."""
    _check(load_library().gleam_dc_prepare(_addr(y), _addr(mask), ctypes.byref(dims)))


def gleam_dc_forward_aty(x, aty, sens, mask, eta, out, dims: gleam_dims) -> None:
    """Eq. 3 in normal-equations form: out = x - eta (A^H A x - aty) with aty = A^H y given as an image."""
    _check(load_library().gleam_dc_forward_aty(_addr(x), _addr(aty), _addr(sens), _addr(mask), float(eta),
                                               _addr(out), ctypes.byref(dims)))


def gleam_dc_forward_prepared(x, y, sens, mask, eta, out, dims: gleam_dims) -> None:
    """gleam_dc_forward with the tables of an earlier gleam_dc_prepare(y, mask, dims)."""
    _check(load_library().gleam_dc_forward_prepared(_addr(x), _addr(y), _addr(sens), _addr(mask), float(eta),
                                                     _addr(out), ctypes.byref(dims)))


def gleam_dc_check_status(dims: gleam_dims) -> int:
    """Synchronises dims.stream and returns the device-side status of the work enqueued with these
    dims and workspace: GLEAM_OK or GLEAM_ERR_TIMEOUT (a bounded wait between blocks ran out)."""
    return int(load_library().gleam_dc_check_status(ctypes.byref(dims)))


FUSED_WAIT_KINDS = ["ring_slot", "first_pass_done", "middle_pass_done", "sens_tile", "workspace_tile"]


def gleam_dc_fused_wait_stats(dims: gleam_dims) -> dict:
    """{kind: (microseconds summed over all blocks, waits that had to spin)} of the last persistent-kernel call."""
    n = len(FUSED_WAIT_KINDS)
    buf = (ctypes.c_uint64 * (2 * n))()
    _check(load_library().gleam_dc_fused_wait_stats(ctypes.byref(dims), buf, n))
    return {FUSED_WAIT_KINDS[i]: (buf[2 * i] * 1e-3, int(buf[2 * i + 1])) for i in range(n)}


def gleam_dc_grad_workspace_size(dims: gleam_dims) -> int:
    out = ctypes.c_uint64(0)
    _check(load_library().gleam_dc_grad_workspace_size(ctypes.byref(dims), ctypes.byref(out)))
    return int(out.value)


def gleam_dc_grad_eta(grad_out, x, y, sens, mask, grad_eta, dims: gleam_dims) -> None:
    """grad_eta[b] = -Re<g_b, A^H(A x - y)_b> (device float64, one value per batch example)."""
    _check(load_library().gleam_dc_grad_eta(_addr(grad_out), _addr(x), _addr(y), _addr(sens), _addr(mask),
                                             _addr(grad_eta), ctypes.byref(dims)))


def gleam_dc_grad_y(grad_out, sens, mask, eta, grad_y, dims: gleam_dims) -> None:
    """grad_y = eta Omega F S grad_out (complex64, layout of y)."""
    _check(load_library().gleam_dc_grad_y(_addr(grad_out), _addr(sens), _addr(mask), float(eta), _addr(grad_y),
                                           ctypes.byref(dims)))


def gleam_dc_forward_layout(x, y, sens, mask, eta, out, dims: gleam_dims, layout: int) -> None:
    """gleam_dc_forward with x and / or out in the two-real-channel layout (B, 2, T, n0, n1, n2) float32."""
    _check(load_library().gleam_dc_forward_layout(_addr(x), _addr(y), _addr(sens), _addr(mask), float(eta), _addr(out),
                                                   ctypes.byref(dims), int(layout)))


def gleam_dc_vjp_layout(grad_out, sens, mask, eta, grad_in, dims: gleam_dims, layout: int) -> None:
    _check(load_library().gleam_dc_vjp_layout(_addr(grad_out), _addr(sens), _addr(mask), float(eta), _addr(grad_in),
                                               ctypes.byref(dims), int(layout)))


def gleam_l1_loss_workspace_size() -> int:
    return int(load_library().gleam_l1_loss_workspace_size())


def gleam_l1_loss(x, ref, loss, grad, dims: gleam_dims, layout: int = 0) -> None:
    """loss (device float64 scalar) = mean |x - ref|; grad (optional) = (x - ref)/|x - ref|/N."""
    _check(load_library().gleam_l1_loss(_addr(x), _addr(ref), _addr(loss), _addr(grad), ctypes.byref(dims), int(layout)))


def gleam_measure_fp32_peak(scratch, stream=None) -> float:
    """Measured FP32 FMA peak of the current device in TFLOP/s (independent FMA chains, no memory traffic)."""
    out = ctypes.c_double(0.0)
    if stream is not None and not isinstance(stream, int):
        stream = stream.cuda_stream
    _check(load_library().gleam_measure_fp32_peak(_addr(scratch), stream or None, ctypes.byref(out)))
    return float(out.value)


def gleam_dc_rowtile_split(n1: int, n2: int) -> int:
    """Rows per block of the row-tile kernels for phase-encode extents (n1, n2), 0 if the pair has none."""
    return int(load_library().gleam_dc_rowtile_split(int(n1), int(n2)))


def gleam_dc_set_fused(on: bool) -> None:
    """Selects the persistent kernel of the separable 3-D path (off by default); call before sizing workspaces."""
    load_library().gleam_dc_set_fused(1 if on else 0)


def gleam_dc_debug_fused(withhold_item: int = -1, wait_limit_ns: int = 0) -> None:
    """Test aid: withhold one item of the persistent 3-D kernel and / or shorten its wait limit."""
    load_library().gleam_dc_debug_fused(int(withhold_item), int(wait_limit_ns))


def gleam_dc_host_arena_size(dims: gleam_dims) -> int:
    out = ctypes.c_uint64(0)
    _check(load_library().gleam_dc_host_arena_size(ctypes.byref(dims), ctypes.byref(out)))
    return int(out.value)


def gleam_dc_forward_host(x, y, sens, mask, eta, out, dims: gleam_dims, arena, arena_bytes=None) -> None:
    """Host-buffer variant: x, y, sens, mask, out are host tensors (pinned for asynchronous copies);
    arena is a device uint8 tensor of gleam_dc_host_arena_size(dims) bytes."""
    if arena_bytes is None:
        arena_bytes = arena.numel() * arena.element_size()
    _check(load_library().gleam_dc_forward_host(_addr(x), _addr(y), _addr(sens), _addr(mask), float(eta), _addr(out),
                                                 ctypes.byref(dims), _addr(arena), int(arena_bytes)))


def gleam_dc_vjp_host(grad_out, sens, mask, eta, grad_in, dims: gleam_dims, arena, arena_bytes=None) -> None:
    if arena_bytes is None:
        arena_bytes = arena.numel() * arena.element_size()
    _check(load_library().gleam_dc_vjp_host(_addr(grad_out), _addr(sens), _addr(mask), float(eta), _addr(grad_in),
                                             ctypes.byref(dims), _addr(arena), int(arena_bytes)))


def gleam_dc_static_scratch_bytes() -> int:
    return int(load_library().gleam_dc_static_scratch_bytes())


def gleam_dc_forward_static(x, y, sens, mask, eta, out, dims: gleam_dims) -> None:
    """gleam_dc_forward with the library's own fixed scratch array instead of dims.workspace, for
    callers that cannot allocate device memory.  Calls whose GPU work overlaps race on that array."""
    _check(load_library().gleam_dc_forward_static(_addr(x), _addr(y), _addr(sens), _addr(mask), float(eta),
                                                   _addr(out), ctypes.byref(dims)))


def gleam_dc_launch_count() -> int:
    return int(load_library().gleam_dc_launch_count())


def gleam_dc_profile_begin() -> None:
    _check(load_library().gleam_dc_profile_begin())


def gleam_dc_profile_end() -> dict:
    """Returns {kernel class: (milliseconds, launches)} accumulated since gleam_dc_profile_begin()."""
    n = len(KERNEL_CLASSES)
    ms = (ctypes.c_float * n)()
    cnt = (ctypes.c_uint32 * n)()
    _check(load_library().gleam_dc_profile_end(ms, cnt, n))
    return {KERNEL_CLASSES[i]: (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i]}


class DataConsistency:
    """Convenience holder: dims + a workspace tensor for one problem shape on the current device
    and stream.  ``forward`` / ``vjp`` allocate their output unless one is passed."""

    def __init__(self, batch, coils, frames, fft_rank, n, sens_has_frames=0,
                 mask_kind=GLEAM_MASK_READOUT_INVARIANT, stream=None):
        import torch
        self._torch = torch
        probe = make_dims(batch, coils, frames, fft_rank, n, sens_has_frames, mask_kind)
        nbytes = gleam_dc_workspace_size(probe)
        self.workspace = torch.empty(max(nbytes, 256), dtype=torch.uint8, device="cuda")
        self.shape = (batch, frames) + tuple(int(v) for v in n)
        self._args = (batch, coils, frames, fft_rank, n, sens_has_frames, mask_kind)
        self.stream = stream

    def dims(self) -> gleam_dims:
        torch = self._torch
        st = self.stream if self.stream is not None else torch.cuda.current_stream()
        return make_dims(*self._args, stream=st, workspace=self.workspace)

    def forward(self, x, y, sens, mask, eta, out=None):
        if out is None:
            out = self._torch.empty_like(x)
        gleam_dc_forward(x, y, sens, mask, eta, out, self.dims())
        return out

    def vjp(self, grad_out, sens, mask, eta, grad_in=None):
        if grad_in is None:
            grad_in = self._torch.empty_like(grad_out)
        gleam_dc_vjp(grad_out, sens, mask, eta, grad_in, self.dims())
        return grad_in

    def adjoint(self, y, sens, mask, out=None):
        """A^H y, shape (B, T, n0, n1, n2)."""
        if out is None:
            out = self._torch.empty(self.shape, dtype=y.dtype, device=y.device)
        gleam_dc_adjoint(y, sens, mask, out, self.dims())
        return out

    def prepare(self, y, mask):
        """For unrolled iterations with the same y and mask: fills the workspace once; follow with
        forward_prepared calls only (forward and vjp of this object would overwrite it)."""
        gleam_dc_prepare(y, mask, self.dims())

    def forward_aty(self, x, aty, sens, mask, eta, out=None):
        """The step with the zero-filled image aty = A^H y (``adjoint``) given instead of y."""
        if out is None:
            out = self._torch.empty_like(x)
        gleam_dc_forward_aty(x, aty, sens, mask, eta, out, self.dims())
        return out

    def forward_prepared(self, x, y, sens, mask, eta, out=None):
        if out is None:
            out = self._torch.empty_like(x)
        gleam_dc_forward_prepared(x, y, sens, mask, eta, out, self.dims())
        return out


def gleam_modl_cg_workspace_size(dims: gleam_dims) -> int:
    out = ctypes.c_uint64(0)
    _check(load_library().gleam_modl_cg_workspace_size(ctypes.byref(dims), ctypes.byref(out)))
    return int(out.value)


def gleam_modl_cg_forward(z, y, sens, mask, mu, n_iter, out, dims: gleam_dims) -> None:
    """out = (A^H A + mu I)^{-1} (A^H y + mu z) by n_iter conjugate-gradient steps (Eq. 7)."""
    _check(load_library().gleam_modl_cg_forward(_addr(z), _addr(y), _addr(sens), _addr(mask), float(mu), int(n_iter),
                                                 _addr(out), ctypes.byref(dims)))


def gleam_modl_cg_vjp(grad_out, sens, mask, mu, n_iter, grad_z, dims: gleam_dims) -> None:
    """grad_z = mu (A^H A + mu I)^{-1} grad_out by n_iter conjugate-gradient steps."""
    _check(load_library().gleam_modl_cg_vjp(_addr(grad_out), _addr(sens), _addr(mask), float(mu), int(n_iter),
                                             _addr(grad_z), ctypes.byref(dims)))


class ModlCG(DataConsistency):
    """Holder of dims + workspace for the MoDL model inversion of one problem shape."""

    def __init__(self, batch, coils, frames, fft_rank, n, sens_has_frames=0,
                 mask_kind=GLEAM_MASK_READOUT_INVARIANT, stream=None):
        super().__init__(batch, coils, frames, fft_rank, n, sens_has_frames, mask_kind, stream)
        probe = make_dims(batch, coils, frames, fft_rank, n, sens_has_frames, mask_kind)
        nbytes = gleam_modl_cg_workspace_size(probe)
        self.workspace = self._torch.empty(max(nbytes, 256), dtype=self._torch.uint8, device="cuda")

    def solve(self, z, y, sens, mask, mu, n_iter=10, out=None):
        if out is None:
            out = self._torch.empty_like(z)
        gleam_modl_cg_forward(z, y, sens, mask, mu, n_iter, out, self.dims())
        return out

    def solve_vjp(self, grad_out, sens, mask, mu, n_iter=10, grad_z=None):
        if grad_z is None:
            grad_z = self._torch.empty_like(grad_out)
        gleam_modl_cg_vjp(grad_out, sens, mask, mu, n_iter, grad_z, self.dims())
        return grad_z
