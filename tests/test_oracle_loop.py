"""Pins for the CPU restatement of GLEAM's greedy mini-batch (Alg. 1): its data-consistency node
back-propagates the adjoint (exact dot test, Eq. 3 is affine), modules are decoupled (the update of a
module is the one obtained by training it alone on the detached output of the module before), and with
a single module the greedy step is ordinary back-propagation (Eq. 10 reduces to Eq. 9)."""
import copy

import numpy as np
import torch

from oracle import gleam_loop_oracle as loop
from oracle.oracle import Dims, MASK_READOUT_INVARIANT
from tests.test_oracle_pins import crandn


def _problem(oracle, seed=0):
    rng = np.random.default_rng(seed)
    d = Dims(1, 3, 2, 2, (1, 8, 12), 0, MASK_READOUT_INVARIANT)
    sens = crandn(*d.sens_shape(), rng=rng).astype(np.complex64)
    mask = (rng.uniform(size=d.mask_shape()) < 0.5).astype(np.float32)
    xt = crandn(*d.image_shape(), rng=rng).astype(np.complex64)
    y = oracle.apply_A(xt, sens, mask, d).astype(np.complex64)
    prob = dict(y=y, sens=sens, mask=mask, eta=0.7, d=d)
    x0 = torch.from_numpy(oracle.apply_AH(y, sens, mask, d).astype(np.complex64).astype(np.complex128))
    return prob, x0, torch.from_numpy(xt.astype(np.complex128))


def test_dc_node_backpropagates_the_adjoint(oracle):
    prob, x0, ref = _problem(oracle)
    rng = np.random.default_rng(1)
    x = x0.clone().requires_grad_(True)
    out = loop._DC.apply(x, prob)
    g = torch.from_numpy(crandn(*x0.shape, rng=rng).astype(np.complex64).astype(np.complex128))
    out.backward(g)
    delta = (rng.integers(-4, 5, size=x0.shape) + 1j * rng.integers(-4, 5, size=x0.shape)) / 8.0
    x2 = torch.from_numpy((x0.numpy().astype(np.complex64) + delta.astype(np.complex64)).astype(np.complex128))
    step = (x2 - x0).numpy()
    lhs = np.real(np.vdot(g.numpy(), (loop._DC.apply(x2, prob) - out.detach()).numpy()))
    rhs = np.real(np.vdot(x.grad.numpy(), step))
    assert abs(lhs - rhs) <= 1e-9 * max(1.0, abs(lhs))


def test_modules_are_decoupled_and_one_module_is_plain_backprop(oracle):
    prob, x0, ref = _problem(oracle)
    torch.manual_seed(0)
    mods = [loop.Module(1, 4, 1).double() for _ in range(3)]
    alone = copy.deepcopy(mods)
    opts = [torch.optim.SGD(m.parameters(), lr=0.1) for m in mods]
    losses, x_fin = loop.greedy_step(mods, opts, x0, prob, ref)
    # the same three updates, one module at a time, each on the detached output of the (old) module before
    x = x0
    for k, m in enumerate(alone):
        old = copy.deepcopy(m)
        opt = torch.optim.SGD(m.parameters(), lr=0.1)
        out = m(x, prob)
        loss = loop.l1(out, ref)
        assert abs(float(loss) - losses[k]) <= 1e-12
        opt.zero_grad(); loss.backward(); opt.step()
        for p, q in zip(m.parameters(), mods[k].parameters()):
            assert torch.equal(p, q)
        x = old(x, prob).detach()
    assert torch.equal(x, x_fin)
    assert losses[0] > 0 and all(np.isfinite(losses))
