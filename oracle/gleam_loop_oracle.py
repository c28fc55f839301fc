"""CPU double-precision restatement of one mini-batch of GLEAM's greedy training (Alg. 1) — TEST
INFRASTRUCTURE, never imported by the CUDA library or its binding.

Module m computes x^(m) = f_theta_m(DC(x^(m-1))) (its unrolled iterations in sequence), is scored by
the complex l1 loss against the reference, back-propagated on its own, updated, and passes a detached
x^(m) on (Eq. 10, Alg. 1).  The data-consistency step and its vector-Jacobian product are the oracle's
(oracle.dc_forward / oracle.dc_vjp, Eq. 3); the prior is a plain float64 torch CPU network written
here: residual blocks of two (ReLU -> 3x3 convolution) pairs without normalisation, on the real and
imaginary channels (Implementation / Training).  Images are complex (B, T, 1, n1, n2) arrays.
"""
import numpy as np
import torch
import torch.nn as nn

from . import oracle as _o


class _DC(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, prob):                     # x: complex128 (B, T, 1, n1, n2)
        ctx.prob = prob
        out = _o.dc_forward(x.numpy().astype(np.complex64), prob["y"], prob["sens"], prob["mask"], prob["eta"], prob["d"])
        return torch.from_numpy(out)

    @staticmethod
    def backward(ctx, g):
        prob = ctx.prob
        out = _o.dc_vjp(g.numpy().astype(np.complex64), prob["sens"], prob["mask"], prob["eta"], prob["d"])
        return torch.from_numpy(out), None


class Prior(nn.Module):
    def __init__(self, features, blocks):
        super().__init__()
        self.head = nn.Conv2d(2, features, 3, padding=1)
        self.blocks = nn.ModuleList([
            nn.Sequential(nn.ReLU(), nn.Conv2d(features, features, 3, padding=1),
                          nn.ReLU(), nn.Conv2d(features, features, 3, padding=1)) for _ in range(blocks)])
        self.tail = nn.Conv2d(features, 2, 3, padding=1)

    def forward(self, x):                          # complex (B, T, 1, n1, n2)
        B, T, n0, n1, n2 = x.shape
        h = torch.stack([x.real, x.imag], dim=-3).reshape(B * T * n0, 2, n1, n2)
        f = self.head(h)
        for blk in self.blocks:
            f = f + blk(f)
        h = h + self.tail(f)
        h = h.reshape(B, T, n0, 2, n1, n2)
        return torch.complex(h[:, :, :, 0], h[:, :, :, 1])


class Module(nn.Module):
    def __init__(self, iterations, features, blocks):
        super().__init__()
        self.priors = nn.ModuleList([Prior(features, blocks) for _ in range(iterations)])

    def forward(self, x, prob):
        for p in self.priors:
            x = p(_DC.apply(x, prob))
        return x


def l1(x, ref):
    return (x - ref).abs().mean()


def greedy_step(modules, optimizers, x0, prob, ref):
    """One mini-batch of Alg. 1 in float64 on the CPU.  The float32 rounding of the image entering each
    data-consistency step (the oracle's input precision) is the only departure from double."""
    losses, x = [], x0.detach()
    for m, opt in zip(modules, optimizers):
        opt.zero_grad(set_to_none=True)
        out = m(x, prob)
        loss = l1(out, ref)
        loss.backward()
        opt.step()
        losses.append(float(loss.detach()))
        x = out.detach()
    return losses, x
