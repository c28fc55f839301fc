"""Greedy module-wise training loop of GLEAM (Alg. 1) on one GPU, around the CUDA data-consistency step.

The unrolled network is split into M modules; module m maps x^(m-1) to x^(m) = f_theta_m(DC(x^(m-1)))
(iterated N/M times inside the module), is trained against its own local loss (complex l1 against the
reference image), and hands a detached x^(m) to the next module: no activation of an earlier module is
kept, so the peak memory is that of one module (Eq. 10 and the text around Alg. 1).

Only the orchestration and the learned prior live here, in PyTorch.  Every data-consistency step, its
vector-Jacobian product and the loss run in the CUDA library through the C ABI, directly on the
two-real-channel tensors the prior takes and returns (gleam_dc_forward_layout / gleam_dc_vjp_layout /
gleam_l1_loss): there is no layout conversion pass and no CPU fallback.
"""
from __future__ import annotations

import torch
import torch.nn as nn

from . import binding as _b


class _DCFunction(torch.autograd.Function):
    """out = x - eta A^H (A x - y) on (B, 2, T, n0, n1, n2) float32 tensors; backward = the library's VJP."""

    @staticmethod
    def forward(ctx, x_ch, step):
        out = torch.empty_like(x_ch)
        _b.gleam_dc_forward_layout(x_ch, step.y, step.sens, step.mask, step.eta, out, step.dc.dims(),
                                   _b.GLEAM_X_CHANNELS | _b.GLEAM_OUT_CHANNELS)
        ctx.step = step
        return out

    @staticmethod
    def backward(ctx, grad_out):
        step = ctx.step
        grad_out = grad_out.contiguous()
        grad_in = torch.empty_like(grad_out)
        _b.gleam_dc_vjp_layout(grad_out, step.sens, step.mask, step.eta, grad_in, step.dc.dims(),
                               _b.GLEAM_X_CHANNELS | _b.GLEAM_OUT_CHANNELS)
        return grad_in, None


class _L1Function(torch.autograd.Function):
    """mean |x - ref| of a two-channel image against a complex64 reference; the gradient comes from the same kernel."""

    @staticmethod
    def forward(ctx, x_ch, step):
        loss = torch.empty(1, dtype=torch.float64, device=x_ch.device)
        grad = torch.empty_like(x_ch)
        _b.gleam_l1_loss(x_ch, step.ref, loss, grad, step.l1_dims(), _b.GLEAM_X_CHANNELS | _b.GLEAM_OUT_CHANNELS)
        ctx.save_for_backward(grad)
        return loss[0].to(torch.float32)

    @staticmethod
    def backward(ctx, g):
        (grad,) = ctx.saved_tensors
        return grad * g, None


class DataConsistencyStep:
    """One measurement setting (y, sens, mask, eta, reference) bound to the CUDA library for a problem shape."""

    def __init__(self, y, sens, mask, eta, ref, fft_rank=2, mask_kind=_b.GLEAM_MASK_READOUT_INVARIANT):
        B, C, T = y.shape[0], y.shape[1], y.shape[2]
        n = tuple(y.shape[3:])
        self.y, self.sens, self.mask, self.eta, self.ref = y, sens, mask, float(eta), ref
        self.shape = (B, C, T, fft_rank, n)
        self.dc = _b.DataConsistency(B, C, T, fft_rank, n, 0, mask_kind)
        self._l1_ws = torch.empty(max(_b.gleam_l1_loss_workspace_size(), 256), dtype=torch.uint8, device=y.device)

    def l1_dims(self):
        B, C, T, rank, n = self.shape
        return _b.make_dims(B, 1, T, rank, n, stream=torch.cuda.current_stream(), workspace=self._l1_ws)

    def apply(self, x_ch):
        return _DCFunction.apply(x_ch, self)

    def loss(self, x_ch):
        return _L1Function.apply(x_ch, self)


class ResidualPrior(nn.Module):
    """The learned proximal block: residual blocks of two (ReLU -> 3x3 convolution) pairs, no normalisation,
    on the two real channels of a 2-D image (frames are folded into the batch)."""

    def __init__(self, features=16, blocks=2):
        super().__init__()
        self.head = nn.Conv2d(2, features, 3, padding=1)
        self.blocks = nn.ModuleList([
            nn.Sequential(nn.ReLU(), nn.Conv2d(features, features, 3, padding=1),
                          nn.ReLU(), nn.Conv2d(features, features, 3, padding=1)) for _ in range(blocks)])
        self.tail = nn.Conv2d(features, 2, 3, padding=1)

    def forward(self, x_ch):                      # (B, 2, T, 1, n1, n2)
        B, _, T, n0, n1, n2 = x_ch.shape
        h = x_ch.permute(0, 2, 3, 1, 4, 5).reshape(B * T * n0, 2, n1, n2)
        f = self.head(h)
        for blk in self.blocks:
            f = f + blk(f)
        h = h + self.tail(f)
        return h.reshape(B, T, n0, 2, n1, n2).permute(0, 3, 1, 2, 4, 5).contiguous()


class GleamModule(nn.Module):
    """`iterations` unrolled steps x <- f_theta_i(DC(x)) that are trained together (one greedy module)."""

    def __init__(self, iterations=1, features=16, blocks=2):
        super().__init__()
        self.priors = nn.ModuleList([ResidualPrior(features, blocks) for _ in range(iterations)])

    def forward(self, x_ch, step: DataConsistencyStep):
        for prior in self.priors:
            x_ch = prior(step.apply(x_ch))
        return x_ch


def greedy_step(modules, optimizers, x0_ch, step: DataConsistencyStep):
    """One mini-batch of Alg. 1: every module is run forward from the detached output of the module before,
    scored by its own loss, back-propagated and updated; returns the local losses and the final image."""
    losses = []
    x = x0_ch.detach()
    for module, opt in zip(modules, optimizers):
        opt.zero_grad(set_to_none=True)
        out = module(x, step)
        loss = step.loss(out)
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
        x = out.detach()                          # activations of this module are dropped here
    return losses, x


def end_to_end_step(modules, optimizer, x0_ch, step: DataConsistencyStep):
    """The conventional baseline (Eq. 9): one loss at the end, back-propagated through all modules."""
    optimizer.zero_grad(set_to_none=True)
    x = x0_ch.detach()
    for module in modules:
        x = module(x, step)
    loss = step.loss(x)
    loss.backward()
    optimizer.step()
    return float(loss.detach()), x.detach()
