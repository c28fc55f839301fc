"""Greedy module-wise training (Alg. 1) around the CUDA data-consistency step: one mini-batch against a
CPU double-precision restatement (oracle DC + float64 prior), and the memory claim the method rests on
(activations of one module at a time)."""
import numpy as np
import pytest

from oracle.oracle import Dims, MASK_READOUT_INVARIANT

pytestmark = pytest.mark.gpu


def _setup(oracle, n=(1, 32, 48), B=1, C=4, T=2, seed=3):
    import torch
    from paper_2207_08393_b200 import workloads as wl
    w = wl.scaled(wl.WORKLOADS["cine"], batch=B, coils=C, frames=T, n=n)
    inp = wl.make_inputs(w)
    d = Dims(B, C, T, 2, n, 0, MASK_READOUT_INVARIANT)
    y = oracle.apply_A(inp["x_true"], inp["sens"], inp["mask"], d).astype(np.complex64)
    x0 = oracle.apply_AH(y, inp["sens"], inp["mask"], d).astype(np.complex64)          # zero-filled SENSE image
    return w, d, inp, y, x0


def test_one_greedy_minibatch_matches_cpu_double(oracle):
    import torch
    from oracle import gleam_loop_oracle as ref_loop
    from paper_2207_08393_b200 import gleam_loop as gl
    w, d, inp, y, x0 = _setup(oracle)
    dev = torch.device("cuda:0")
    torch.manual_seed(0)
    M, iters, feat = 3, 2, 8
    mods = [gl.GleamModule(iters, feat, 2).to(dev) for _ in range(M)]
    refs = [ref_loop.Module(iters, feat, 2).double() for _ in range(M)]
    for a, b in zip(mods, refs):
        b.load_state_dict({k: v.detach().cpu().double() for k, v in a.state_dict().items()})
    opts = [torch.optim.Adam(m.parameters(), lr=1e-3, betas=(0.9, 0.999)) for m in mods]
    ropts = [torch.optim.Adam(m.parameters(), lr=1e-3, betas=(0.9, 0.999)) for m in refs]
    step = gl.DataConsistencyStep(torch.from_numpy(y).to(dev), torch.from_numpy(inp["sens"]).to(dev),
                                  torch.from_numpy(inp["mask"]).to(dev), w.eta, torch.from_numpy(inp["x_true"]).to(dev))
    x0_ch = torch.from_numpy(oracle.complex_to_channels(x0)).to(dev)
    losses, x_fin = gl.greedy_step(mods, opts, x0_ch, step)
    prob = dict(y=y, sens=inp["sens"], mask=inp["mask"], eta=w.eta, d=d)
    rlosses, rx = ref_loop.greedy_step(refs, ropts, torch.from_numpy(x0.astype(np.complex128)), prob,
                                       torch.from_numpy(inp["x_true"].astype(np.complex128)))
    assert np.allclose(losses, rlosses, rtol=2e-4), (losses, rlosses)
    got = oracle.channels_to_complex(x_fin.cpu().numpy())
    assert np.linalg.norm(got - rx.numpy()) <= 1e-3 * np.linalg.norm(rx.numpy())
    # the first Adam update moves every parameter by lr * sign(gradient): compare the updated parameters
    for a, b in zip(mods, refs):
        for (ka, va), (kb, vb) in zip(a.state_dict().items(), b.state_dict().items()):
            assert ka == kb
            diff = (va.detach().cpu().double() - vb).abs().max().item()
            assert diff <= 2.5e-3, (ka, diff)          # 2 lr at most, where a tiny gradient changes sign in float32


def test_gradient_through_the_step_is_the_library_vjp(oracle):
    """Back-propagation through DataConsistencyStep.apply = gleam_dc_vjp on the two-channel tensors."""
    import torch
    from paper_2207_08393_b200 import gleam_loop as gl
    w, d, inp, y, x0 = _setup(oracle)
    dev = torch.device("cuda:0")
    step = gl.DataConsistencyStep(torch.from_numpy(y).to(dev), torch.from_numpy(inp["sens"]).to(dev),
                                  torch.from_numpy(inp["mask"]).to(dev), w.eta, torch.from_numpy(inp["x_true"]).to(dev))
    x_ch = torch.from_numpy(oracle.complex_to_channels(x0)).to(dev).requires_grad_(True)
    g = inp["g"]
    out = step.apply(x_ch)
    out.backward(torch.from_numpy(oracle.complex_to_channels(g)).to(dev))
    got = oracle.channels_to_complex(x_ch.grad.cpu().numpy())
    ref = oracle.dc_vjp(g, inp["sens"], inp["mask"], w.eta, d)
    assert np.linalg.norm(got - ref) <= 2e-5 * np.linalg.norm(ref)
    fwd = oracle.channels_to_complex(out.detach().cpu().numpy())
    assert np.linalg.norm(fwd - oracle.dc_forward(x0, y, inp["sens"], inp["mask"], w.eta, d)) <= 2e-5 * np.linalg.norm(fwd)


def test_greedy_training_holds_one_module_of_activations(oracle):
    """Peak memory of a greedy mini-batch stays near that of one module while end-to-end back-propagation
    grows with the number of modules (the paper's memory claim, here for 6 modules)."""
    import torch
    from paper_2207_08393_b200 import gleam_loop as gl
    w, d, inp, y, x0 = _setup(oracle, n=(1, 96, 80), T=4)
    dev = torch.device("cuda:0")
    step = gl.DataConsistencyStep(torch.from_numpy(y).to(dev), torch.from_numpy(inp["sens"]).to(dev),
                                  torch.from_numpy(inp["mask"]).to(dev), w.eta, torch.from_numpy(inp["x_true"]).to(dev))
    x0_ch = torch.from_numpy(oracle.complex_to_channels(x0)).to(dev)

    def peak(fn, M):
        torch.manual_seed(1)
        mods = [gl.GleamModule(1, 32, 2).to(dev) for _ in range(M)]
        torch.cuda.synchronize(); torch.cuda.reset_peak_memory_stats()
        base = torch.cuda.memory_allocated()
        fn(mods)
        torch.cuda.synchronize()
        return torch.cuda.max_memory_allocated() - base

    def run_greedy(mods):
        gl.greedy_step(mods, [torch.optim.SGD(m.parameters(), lr=1e-3) for m in mods], x0_ch, step)

    def run_e2e(mods):
        gl.end_to_end_step(mods, torch.optim.SGD([p for m in mods for p in m.parameters()], lr=1e-3), x0_ch, step)

    g1, g6, e6 = peak(run_greedy, 1), peak(run_greedy, 6), peak(run_e2e, 6)
    assert g6 <= 1.3 * g1 + (1 << 20)
    assert e6 >= 3.0 * g6
