"""Benchmark of the SENSE data-consistency step (forward + VJP) on B200.

    python bench.py --gpus N --steps K --warmup W [--workload knee3d] [--impl reference]

One step = the workload's unrolled iterations: `chain` gleam_dc_forward calls chained as
x_{i+1} = DC(x_i), then `chain` gleam_dc_vjp calls chained backwards, all on the same y, S and mask
(chain = 1 for knee3d, knee2d and slice64; 10 for brain2d; 8 for cine).  Every call runs all rows
of the hot path: sensitivity multiply, FFT, mask + residual, inverse FFT, coil sum, update.
`value` is voxel*coils per second with every input resident in HBM; `e2e` is the same metric
through the host-buffer C-ABI calls (one forward + one VJP per step) with pinned host inputs, the
host->device copies and the device->host copy of the results inside the timed region.

N > 1 runs N independent replicas (the path has no exchange step); the time is the max over ranks.
`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "dc_step_fwd_plus_vjp_throughput"
UNIT = "voxel*coils/s"

# FP32 ALU peak: 148 SMs x 128 FP32 lanes x 2 flop (FMA) x SM clock
SM_COUNT, FP32_LANES = 148, 128


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


def fp32_peak_tflops(sm_mhz):
    return SM_COUNT * FP32_LANES * 2 * sm_mhz * 1e6 / 1e12


# ------------------------------------------------------------------------------------------------
# roofline bookkeeping (algorithmic bytes / flops; N log2 N counting of the transforms)
# ------------------------------------------------------------------------------------------------
def call_roofline(w, with_y):
    """min bytes = x + S + (y) + mask + out;  flops = 2 B C T transforms x 5 N log2 N, N = points
    per full transform."""
    img = w.batch * w.frames * w.V * 8
    sens = w.batch * w.coils * w.V * 8
    ksp = w.batch * w.coils * w.frames * w.V * 8
    pe = w.n[2] if w.fft_rank == 2 else w.n[1] * w.n[2]
    mask = w.batch * w.frames * pe * 4
    nbytes = 2 * img + sens + mask + (ksp if with_y else 0)
    npts = w.V
    flops = 2 * w.batch * w.coils * w.frames * 5 * npts * math.log2(npts)
    return nbytes, flops


def kernel_work(cls, w, launches_per_call, density=1.0):
    """Algorithmic (bytes, flops) of ONE launch of a kernel class for workload w.
    Per voxel*coil figures are listed beside each case; density = sampled fraction of the
    phase-encode positions (the readout transform of y runs at those only)."""
    W = w.voxel_coils / launches_per_call        # voxel*coils one launch processes
    C = w.coils
    l2 = math.log2
    if cls == "row_fwd":        # read S (8) + x (8/C), write W (8)
        return W * (16 + 8 / C), W * (5 * l2(w.n[2]) + 6)
    if cls == "row_inv":        # read W (8) + S (8) + x (8/C), write out (8/C)
        return W * (16 + 16 / C), W * (5 * l2(w.n[2]) + 8)
    if cls == "col_mid_sep":    # read + write W (16), tables
        return W * 16, W * (10 * l2(w.n[1]) + 4)
    if cls == "row_fused":      # read S (8) [+ z (8) in the forward call, averaged] + x/out (16/C)
        return W * (8 + 4 + 16 / C), W * (10 * l2(w.n[2]) + 20)
    if cls == "col_z":          # read y (8), write z (8), at the sampled positions only
        nro = w.n[1] if w.fft_rank == 2 else w.n[0]
        return W * 16 * density, W * (5 * l2(nro)) * density
    if cls == "col_mid_full":
        nro = w.n[1] if w.fft_rank == 2 else w.n[0]
        return W * 24, W * (10 * l2(nro) + 6)
    if cls in ("col_fwd", "col_inv"):
        return W * 16, W * (5 * l2(w.n[1]))
    if cls == "fused3d":        # one launch = the whole call: read S (8) + x (8/C), write out (8/C); both transforms over (n1, n2)
        return W * (8 + 16 / C), W * (10 * l2(w.n[1] * w.n[2]) + 20)
    if cls == "cg_vec":         # image-sized vector kernels of the CG solve: on average 3.7 passes of 8 B
        return W * (3.7 * 8 / C), W * (8.0 / C)     # per voxel (init 5, dot 2, step 6, dir 3 passes)
    return 0.0, 0.0


# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken between the wall-clock times t_begin and t_end (the timed
        region); if the region was too short to catch one, of all samples of the run under load."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "timed region"}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        rows = [r.strip().split(",") for r in open(self.tmp.name) if r.strip()]
        os.unlink(self.tmp.name)

        def stamp(r):
            try:
                return datetime.datetime.strptime(r[0].strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
            except ValueError:
                return None
        if t_begin is not None:
            inside = [r[1:] for r in rows if (stamp(r) is not None and t_begin - 0.05 <= stamp(r) <= t_end + 0.05)]
            if inside:
                rows = [[None] + r for r in inside]
            else:
                out["window"] = "whole run (timed region shorter than the sampling interval)"
        rows = [r[1:] for r in rows]
        sm, names = [], ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in rows:
            try:
                sm.append(float(r[0])); out["sm_max_mhz"] = float(r[1])
            except (ValueError, IndexError):
                continue
            for nme, v in zip(names, r[3:7]):
                if v.strip().lower().startswith("active"):
                    reasons.add(nme)
        if sm:
            busy = [v for v in sm if v >= 0.5 * max(sm)] or sm
            out["sm_mhz"] = statistics.median(busy)
        out["reasons"] = sorted(reasons)
        out["samples"] = len(sm)
        return out


def dist_setup(n_gpus):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def aggregate(local_ms, local_units, world, dist=None, device=None):
    """Whole-job numbers from per-rank ones: time = max over ranks, units = sum over ranks.
    With world == 1 no process group is needed."""
    if world == 1 or dist is None:
        return local_ms, local_units
    import torch
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ------------------------------------------------------------------------------------------------
def reference_sample(w, cores=None):
    """Bounded sample of a workload for the CPU oracle: same kind of problem, fewer units.  With at
    least 8 host threads the whole workload is the sample (knee3d: about 10 s per step).  A smaller
    knee3d sample keeps 40 readout slabs, so that the readout axis still goes through the oracle's
    FFT route (lengths above 32) like the full volume, not through its direct sum."""
    from paper_2207_08393_b200 import workloads as wl
    if cores is None:
        from oracle import oracle
        cores = oracle.max_threads()
    if w.name == "knee3d":
        if cores >= 8:
            return w, "whole workload"
        return wl.scaled(w, n=(40, w.n[1], w.n[2])), "8 coils, 40 of 320 readout slabs (40x320x256)"
    if w.name in ("knee2d", "brain2d") and cores < 8:
        return wl.scaled(w, batch=1), "batch 1 of %d" % w.batch
    return w, "whole workload"


def make_problem(w, seed_offset=0):
    from paper_2207_08393_b200 import workloads as wl
    inp = wl.make_inputs(w, seed_offset)
    y = wl.standin_kspace(w, inp["mask"], seed_offset)
    return inp, y


def run_reference(args, w):
    """Times the CPU oracle, as it stands, on a bounded sample (rank 0 only)."""
    rank, world, _ = dist_setup(args.gpus)
    if rank != 0:
        return
    from oracle import oracle
    oracle.build()
    cores = oracle.max_threads()
    ws, sample_txt = reference_sample(w, cores)
    inp, y = make_problem(ws)
    d = oracle.Dims(ws.batch, ws.coils, ws.frames, ws.fft_rank, ws.n, 0, oracle.MASK_READOUT_INVARIANT)

    def step():
        oracle.dc_forward(inp["x"], y, inp["sens"], inp["mask"], ws.eta, d, nthreads=cores)
        oracle.dc_vjp(inp["g"], inp["sens"], inp["mask"], ws.eta, d, nthreads=cores)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = ws.voxel_coils * args.steps / dt
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "description": w.description, "sample": sample_txt,
                   "step": "%d gleam_dc_forward + %d gleam_dc_vjp evaluated by the oracle" % (1, 1),
                   "voxel_coils_per_step": ws.voxel_coils},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args, w):
    import numpy as np
    import torch
    import paper_2207_08393_b200 as g

    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    g.load_library()
    peaks = load_peaks()

    from paper_2207_08393_b200 import workloads as wl
    inp, y = make_problem(w, seed_offset=rank)
    full_mask = args.mask == "full"
    mask_kind = g.GLEAM_MASK_FULL if full_mask else g.GLEAM_MASK_READOUT_INVARIANT
    density = float(np.count_nonzero(inp["mask"])) / inp["mask"].size
    if full_mask:        # the same sampling pattern handed over as a general (B, T, n0, n1, n2) mask
        inp = dict(inp, mask=wl.expand_mask(w, inp["mask"]))
    tx, tg, ts, tm, ty = (torch.from_numpy(a).to(dev) for a in (inp["x"], inp["g"], inp["sens"], inp["mask"], y))
    dc = g.DataConsistency(w.batch, w.coils, w.frames, w.fft_rank, w.n, mask_kind=mask_kind)
    out = torch.empty_like(tx)
    gin = torch.empty_like(tg)
    stream = torch.cuda.current_stream()

    chain = max(1, w.chain)
    out2 = torch.empty_like(tx) if chain > 1 else None
    gin2 = torch.empty_like(tg) if chain > 1 else None

    def forward_chain():
        """x_{i+1} = DC(x_i): `chain` unrolled iterations with the same y, S and mask (the learned
        prior between them is outside this library)."""
        src = tx
        for i in range(chain):
            dst = out if i % 2 == 0 else out2
            dc.forward(src, ty, ts, tm, w.eta, dst)
            src = dst

    def vjp_chain():
        """g_i = VJP(g_{i+1}) through the same `chain` iterations."""
        src = tg
        for i in range(chain):
            dst = gin if i % 2 == 0 else gin2
            dc.vjp(src, ts, tm, w.eta, dst)
            src = dst

    def step():
        if args.calls != "vjp":
            forward_chain()
        if args.calls != "forward":
            vjp_chain()

    flush = None
    inputs_bytes = sum(t.numel() * t.element_size() for t in (tx, tg, ts, tm, ty))
    if inputs_bytes < 256 << 20:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # L2 is 126 MB

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3 if sampler else 0.0)       # let the sampler start before the GPU gets busy
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # ---- the launches of a step, captured once as a CUDA graph and replayed (the calls are a few tens of
    # microseconds each, so enqueueing them one by one from Python would be part of the measurement) ----
    use_graph = args.launch == "graph" and not args.kernels_only
    graph_pool = []

    def replayed(fn):
        """fn's launches as a CUDA graph on the current stream; fn itself when graphs are off or the capture fails."""
        if not use_graph:
            return fn, None
        try:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                fn()                                   # first use on this stream outside the capture
                torch.cuda.synchronize()
                n0 = g.gleam_dc_launch_count()
                gr = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gr, stream=side):
                    fn()
                n1 = g.gleam_dc_launch_count()
            stream.wait_stream(side)
            torch.cuda.synchronize()
            graph_pool.append(gr)
            return gr.replay, int(n1 - n0)
        except Exception as e:                         # noqa: BLE001
            sys.stderr.write("graph capture failed (%s): launching eagerly\n" % e)
            return fn, None

    step_eager = step
    step, step_launches = replayed(step_eager)
    for _ in range(3):
        step()
    barrier()

    # ---- device-resident timed region -------------------------------------------------------
    launches0 = g.gleam_dc_launch_count()
    t_begin = time.time()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        barrier()
        local_ms = e0.elapsed_time(e1)
    else:
        # small workloads: flush L2 between steps, time each step with its own event pair
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        barrier()
        for a, b in evs:
            flush.fill_(1)
            a.record(stream)
            step()
            b.record(stream)
        barrier()
        local_ms = sum(a.elapsed_time(b) for a, b in evs)
    launches = g.gleam_dc_launch_count() - launches0 if step_launches is None else step_launches * args.steps
    t_end = time.time()
    total_ms, total_units = aggregate(local_ms, w.voxel_coils * chain * args.steps, world, dist, dev)
    value = total_units / (total_ms * 1e-3)
    if args.kernels_only:
        if sampler:
            sampler.stop()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "workload": w.name, "calls": args.calls, "steps": args.steps,
                              "ms_per_step": total_ms / args.steps, "gpu_launches": int(launches), "profiler_run": True,
                              "fused_wait_us_last_call": g.gleam_dc_fused_wait_stats(dc.dims())}))
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- per-kernel pass (CUDA events around every launch, on the launching stream) ----------
    prof_steps = min(args.steps, 5)
    g.gleam_dc_profile_begin()
    for _ in range(prof_steps):
        if flush is not None:
            flush.fill_(1)
        step_eager()
    prof = g.gleam_dc_profile_end()
    kernels = {}
    for cls, (ms, cnt) in prof.items():
        calls = (1.0 if cls in ("zmap", "col_z") else 2.0) * chain * prof_steps    # zmap, col_z: forward calls only
        per_call = cnt / calls
        nbytes, flops = kernel_work(cls, w, max(per_call, 1e-9), density)
        avg_s = ms * 1e-3 / cnt
        kernels[cls] = {"launches_per_step": cnt / prof_steps, "ms_per_step": ms / prof_steps, "avg_us": avg_s * 1e6,
                        "gbs": nbytes / avg_s / 1e9, "tflops": flops / avg_s / 1e12}
    # forward / vjp split (events around whole calls)
    ef = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    split = [0.0, 0.0]
    forward_chain_r, _ = replayed(forward_chain)
    vjp_chain_r, _ = replayed(vjp_chain)
    for _ in range(prof_steps):
        if flush is not None:
            flush.fill_(1)
        ef[0].record(stream); forward_chain_r()
        ef[1].record(stream); vjp_chain_r()
        ef[2].record(stream); torch.cuda.synchronize()
        split[0] += ef[0].elapsed_time(ef[1]) / prof_steps / chain      # per call
        split[1] += ef[1].elapsed_time(ef[2]) / prof_steps / chain

    # ---- cost of reading and writing the image in the prior's two-real-channel layout inside the kernels ----
    g_ch = torch.stack([tg.real, tg.imag], dim=1).contiguous()
    gin_ch = [torch.empty_like(g_ch), torch.empty_like(g_ch)]
    both = g.GLEAM_X_CHANNELS | g.GLEAM_OUT_CHANNELS

    def vjp_chain_channels():
        src = g_ch
        for i in range(chain):
            g.gleam_dc_vjp_layout(src, ts, tm, w.eta, gin_ch[i % 2], dc.dims(), both)
            src = gin_ch[i % 2]

    lay = [0.0, 0.0]
    for _ in range(prof_steps):
        for k, fn in enumerate((vjp_chain_r, replayed(vjp_chain_channels)[0])):
            if flush is not None:
                flush.fill_(1)
            ef[0].record(stream); fn()
            ef[1].record(stream); torch.cuda.synchronize()
            lay[k] += ef[0].elapsed_time(ef[1]) / prof_steps / chain
    layout_cost = {"vjp_us_complex64": lay[0] * 1e3, "vjp_us_two_channel_in_and_out": lay[1] * 1e3,
                   "relative_cost": lay[1] / lay[0] - 1.0}
    del g_ch, gin_ch

    # ---- the same chain with the y-dependent tables computed once per step (gleam_dc_prepare) ----
    prepared = None
    if chain > 1 and not full_mask:
        def forward_chain_prepared():
            dc.prepare(ty, tm)
            src = tx
            for i in range(chain):
                dst = out if i % 2 == 0 else out2
                dc.forward_prepared(src, ty, ts, tm, w.eta, dst)
                src = dst

        forward_chain(); ref_last = (out if (chain - 1) % 2 == 0 else out2).clone()
        forward_chain_prepared(); torch.cuda.synchronize()
        assert torch.equal(ref_last, out if (chain - 1) % 2 == 0 else out2), "prepared chain differs"
        pf = 0.0
        forward_chain_prepared_r, _ = replayed(forward_chain_prepared)
        for _ in range(prof_steps):
            if flush is not None:
                flush.fill_(1)
            ef[0].record(stream); forward_chain_prepared_r()
            ef[1].record(stream); torch.cuda.synchronize()
            pf += ef[0].elapsed_time(ef[1]) / prof_steps
        step_ms = pf + split[1] * chain
        prepared = {"forward_us_per_call": pf / chain * 1e3, "ms_per_step": step_ms,
                    "value": w.voxel_coils * chain / (step_ms * 1e-3), "unit": UNIT,
                    "what": "1 gleam_dc_prepare + %d gleam_dc_forward_prepared per step, VJP chain as in the main number" % chain}

    # ---- the same chain in normal-equations form: A^H y once per step, then steps that cost a VJP call ----
    aty_chain = None
    if True:
        aty_buf = torch.empty_like(tx)

        def forward_chain_aty():
            dc.adjoint(ty, ts, tm, aty_buf)
            src = tx
            for i in range(chain):
                dst = out if i % 2 == 0 else out2
                dc.forward_aty(src, aty_buf, ts, tm, w.eta, dst)
                src = dst

        forward_chain(); torch.cuda.synchronize()
        ref_last = (out if (chain - 1) % 2 == 0 else out2).clone()
        forward_chain_aty(); torch.cuda.synchronize()
        got_last = out if (chain - 1) % 2 == 0 else out2
        dev_rel = float((got_last - ref_last).abs().pow(2).sum().sqrt() / ref_last.abs().pow(2).sum().sqrt())
        assert dev_rel < 2e-5 * chain, "normal-equations chain differs from the plain chain: %g" % dev_rel
        af, ad = 0.0, 0.0

        def aty_steps():
            src = tx
            for i in range(chain):
                dst = out if i % 2 == 0 else out2
                dc.forward_aty(src, aty_buf, ts, tm, w.eta, dst)
                src = dst

        adjoint_r, _ = replayed(lambda: dc.adjoint(ty, ts, tm, aty_buf))
        aty_steps_r, _ = replayed(aty_steps)
        for _ in range(prof_steps):
            if flush is not None:
                flush.fill_(1)
            ef[0].record(stream); adjoint_r()
            ef[1].record(stream); aty_steps_r()
            ef[2].record(stream); torch.cuda.synchronize()
            ad += ef[0].elapsed_time(ef[1]) / prof_steps
            af += ef[1].elapsed_time(ef[2]) / prof_steps
        step_ms = ad + af + split[1] * chain
        aty_chain = {"adjoint_us": ad * 1e3, "forward_us_per_call": af / chain * 1e3, "ms_per_step": step_ms,
                     "value": w.voxel_coils * chain / (step_ms * 1e-3), "unit": UNIT,
                     "rel_l2_against_plain_chain": dev_rel,
                     "what": "1 gleam_dc_adjoint (A^H y) + %d gleam_dc_forward_aty per step, VJP chain as in the main number" % chain}
        del aty_buf

    # ---- the same steps without the L2 flush (problems that fit in L2: both figures are reported) ----
    warm = None
    if flush is not None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        step(); torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream); torch.cuda.synchronize()
        wms = e0.elapsed_time(e1) / args.steps
        warm = {"ms_per_step": wms, "value": w.voxel_coils * chain / (wms * 1e-3), "unit": UNIT,
                "what": "steps back to back, inputs and tables left in L2 by the step before (rank 0)"}

    clocks = sampler.stop(t_begin, t_end) if sampler else None

    # ---- end to end through the host-buffer entry points --------------------------------------
    e2e_steps = max(1, min(args.steps, 3 if inputs_bytes > (1 << 30) else 10))
    hx, hg, hs, hm, hy = (torch.from_numpy(a).pin_memory() for a in (inp["x"], inp["g"], inp["sens"], inp["mask"], y))
    hout, hgin = torch.empty_like(hx).pin_memory(), torch.empty_like(hg).pin_memory()
    d_host = g.make_dims(w.batch, w.coils, w.frames, w.fft_rank, w.n, mask_kind=mask_kind, stream=stream)
    arena = torch.empty(g.gleam_dc_host_arena_size(d_host), dtype=torch.uint8, device=dev)

    def step_host():
        g.gleam_dc_forward_host(hx, hy, hs, hm, w.eta, hout, d_host, arena)
        g.gleam_dc_vjp_host(hg, hs, hm, w.eta, hgin, d_host, arena)

    dc.forward(tx, ty, ts, tm, w.eta, out)      # single calls on the device-resident inputs: the
    dc.vjp(tg, ts, tm, w.eta, gin)              # results the host-buffer path has to reproduce
    step_host()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        step_host()
    e1.record(stream)
    barrier()
    e2e_ms, e2e_units = aggregate(e0.elapsed_time(e1), w.voxel_coils * e2e_steps, world, dist, dev)
    nb = lambda t: t.numel() * t.element_size()
    h2d = nb(hx) + nb(hy) + 2 * nb(hs) + 2 * nb(hm) + nb(hg)
    d2h = nb(hout) + nb(hgin)
    # the host path must give the same result as the device path
    assert torch.equal(hout.to(dev), out) and torch.equal(hgin.to(dev), gin), "host-buffer path differs"

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline --------------------------------------------------------------------------------
    sm_mhz = peaks["sm_max_mhz"]
    alu_peak = fp32_peak_tflops(sm_mhz)
    alu_measured = g.gleam_measure_fp32_peak(out, stream)      # independent FMA chains, best of four launches
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    kd = kernels[dom]
    t_hbm = kd["gbs"] / peaks["hbm_gbs"]
    t_alu = kd["tflops"] / alu_peak
    if t_hbm >= t_alu:
        roof = {"bound": "hbm", "achieved": kd["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": t_hbm}
    else:
        roof = {"bound": "alu", "achieved": kd["tflops"], "peak": alu_peak, "unit": "TFLOP/s", "frac": t_alu}
    roof.update({"kernel": dom, "peak_source": peaks["source"] + (" copy bandwidth" if roof["bound"] == "hbm" else
                 " sm_max_mhz x 148 SMs x 128 lanes x 2"), "traffic": measured_traffic(w.name, dom),
                 "share_of_step": kd["ms_per_step"] / sum(k["ms_per_step"] for k in kernels.values())})
    ns = {}
    for name, with_y, ms in (("forward", True, split[0]), ("vjp", False, split[1])):
        nbytes, flops = call_roofline(w, with_y)
        t_b, t_f = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (alu_peak * 1e12)
        ns[name] = {"min_bytes": nbytes, "fft_flops": flops, "hbm_us": t_b * 1e6, "fp32_us": t_f * 1e6,
                    "measured_us": ms * 1e3, "frac": max(t_b, t_f) / (ms * 1e-3),
                    "frac_with_measured_fp32_peak": max(t_b, flops / (alu_measured * 1e12)) / (ms * 1e-3)}

    if aty_chain is not None:       # x, A^H y, S, mask in; out: no measurements are read
        nbytes, flops = call_roofline(w, False)
        nbytes += w.batch * w.frames * w.V * 8
        t_b, t_f = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (alu_peak * 1e12)
        ms = aty_chain["forward_us_per_call"] * 1e-3
        ns["forward_aty"] = {"min_bytes": nbytes, "fft_flops": flops, "hbm_us": t_b * 1e6, "fp32_us": t_f * 1e6,
                             "measured_us": ms * 1e3, "frac": max(t_b, t_f) / (ms * 1e-3),
                             "frac_with_measured_fp32_peak": max(t_b, flops / (alu_measured * 1e12)) / (ms * 1e-3)}

    # ---- CPU baseline: the oracle, once, on the host cores of the machine ---------------------------
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import oracle
        oracle.build()
        cores = oracle.max_threads()
        wsamp, sample_txt = (w, "whole workload, 1 step") if w.name != "knee3d" or cores >= 8 else reference_sample(w, cores)
        if wsamp is not w:
            inp_c, y_c = make_problem(wsamp)
            if full_mask:
                inp_c = dict(inp_c, mask=wl.expand_mask(wsamp, inp_c["mask"]))
        else:
            inp_c, y_c = inp, y
        d = oracle.Dims(wsamp.batch, wsamp.coils, wsamp.frames, wsamp.fft_rank, wsamp.n, 0,
                        oracle.MASK_FULL if full_mask else oracle.MASK_READOUT_INVARIANT)
        t0 = time.perf_counter()
        oracle.dc_forward(inp_c["x"], y_c, inp_c["sens"], inp_c["mask"], wsamp.eta, d, nthreads=cores)
        oracle.dc_vjp(inp_c["g"], inp_c["sens"], inp_c["mask"], wsamp.eta, d, nthreads=cores)
        dt = time.perf_counter() - t0
        cpu = {"value": wsamp.voxel_coils / dt, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample_txt,
               "seconds": dt}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "description": w.description, "step": "%d chained gleam_dc_forward + %d chained gleam_dc_vjp" % (chain, chain),
                   "launch": "one CUDA graph per step, captured from the same C-ABI calls and replayed" if step_launches is not None else "eager, call by call",
                   "voxel_coils_per_step": w.voxel_coils * chain, "e2e_step": "1 forward + 1 vjp with host buffers", "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "l2": "inputs exceed L2" if flush is None else "256 MB L2 flush before every step (chain)",
                   "mask": "general (B,T,n0,n1,n2) array" if full_mask else "readout-invariant"},
        "ms_per_iteration": total_ms / args.steps / chain,
        "clocks": clocks,
        "e2e": {"value": e2e_units / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": int(launches),
        "roofline": roof,
        "call_roofline": ns,
        "fp32_peak": {"derived_tflops": alu_peak, "measured_tflops": alu_measured,
                      "how": "derived: 148 SMs x 128 lanes x 2 flop x sm_max_mhz; measured: independent FMA chains, no memory traffic"},
        "prepared_chain": prepared,
        "normal_equations_chain": aty_chain,
        "warm_l2": warm,
        "two_channel_layout": layout_cost,
        "kernels": kernels,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


MODL_METRIC = "modl_cg_solve_plus_vjp_throughput"


def run_modl(args, w):
    """MoDL model inversion (Eq. 7): one step = gleam_modl_cg_forward + gleam_modl_cg_vjp, each with
    --cg-steps conjugate-gradient steps.  `value` counts voxel*coils per application of the normal
    operator A^H A (the solve applies it cg_steps + 1 times counting the right-hand side A^H y, the
    VJP cg_steps times), so it is comparable with the data-consistency metric."""
    import numpy as np
    import torch
    n_iter, mu = args.cg_steps, args.mu
    ops_per_step = 2 * n_iter + 1
    if args.impl == "reference":
        rank, world, _ = dist_setup(args.gpus)
        if rank != 0:
            return
        from oracle import oracle
        oracle.build()
        ws, sample_txt = reference_sample(w)
        inp, y = make_problem(ws)
        d = oracle.Dims(ws.batch, ws.coils, ws.frames, ws.fft_rank, ws.n, 0, oracle.MASK_READOUT_INVARIANT)
        cores = oracle.max_threads()
        for _ in range(args.warmup):
            oracle.modl_cg_forward(inp["x"], y, inp["sens"], inp["mask"], mu, 1, d, nthreads=cores)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            oracle.modl_cg_forward(inp["x"], y, inp["sens"], inp["mask"], mu, n_iter, d, nthreads=cores)
            oracle.modl_cg_vjp(inp["g"], inp["sens"], inp["mask"], mu, n_iter, d, nthreads=cores)
        dt = time.perf_counter() - t0
        value = ws.voxel_coils * ops_per_step * args.steps / dt
        print(json.dumps({
            "impl": "reference", "metric": MODL_METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "description": w.description, "sample": sample_txt, "mu": mu, "cg_steps": n_iter},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample_txt},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))
        return

    import paper_2207_08393_b200 as g
    rank, world, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    g.load_library()
    peaks = load_peaks()
    inp, y = make_problem(w, seed_offset=rank)
    tz, tg, ts, tm, ty = (torch.from_numpy(a).to(dev) for a in (inp["x"], inp["g"], inp["sens"], inp["mask"], y))
    cg = g.ModlCG(w.batch, w.coils, w.frames, w.fft_rank, w.n)
    out, gz = torch.empty_like(tz), torch.empty_like(tg)
    stream = torch.cuda.current_stream()

    def step():
        cg.solve(tz, ty, ts, tm, mu, n_iter, out)
        cg.solve_vjp(tg, ts, tm, mu, n_iter, gz)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)       # L2 is 126 MB
    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.3 if sampler else 0.0)
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    launches0 = g.gleam_dc_launch_count()
    t_begin = time.time()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    for a, b in evs:
        flush.fill_(1)
        a.record(stream)
        step()
        b.record(stream)
    barrier()
    local_ms = sum(a.elapsed_time(b) for a, b in evs)
    launches = g.gleam_dc_launch_count() - launches0
    t_end = time.time()
    total_ms, total_units = aggregate(local_ms, w.voxel_coils * ops_per_step * args.steps, world, dist, dev)
    value = total_units / (total_ms * 1e-3)
    clocks = sampler.stop(t_begin, t_end) if sampler else None

    # ---- per-kernel pass (CUDA events around every launch) -------------------------------------
    prof_steps = min(args.steps, 3)
    g.gleam_dc_profile_begin()
    for _ in range(prof_steps):
        flush.fill_(1)
        step()
    prof = g.gleam_dc_profile_end()
    kernels = {}
    for cls, (ms, cnt) in prof.items():
        nbytes, flops = kernel_work(cls, w, 1.0, float(np.count_nonzero(inp["mask"])) / inp["mask"].size)   # every launch covers the whole problem
        avg_s = ms * 1e-3 / cnt
        kernels[cls] = {"launches_per_step": cnt / prof_steps, "ms_per_step": ms / prof_steps, "avg_us": avg_s * 1e6,
                        "gbs": nbytes / avg_s / 1e9, "tflops": flops / avg_s / 1e12}

    # ---- end to end: pinned host inputs copied in, results copied out, every step ----------------
    e2e_steps = max(1, min(args.steps, 5))
    hz, hg, hs, hm, hy = (torch.from_numpy(a).pin_memory() for a in (inp["x"], inp["g"], inp["sens"], inp["mask"], y))
    hout, hgz = torch.empty_like(hz).pin_memory(), torch.empty_like(hg).pin_memory()

    def step_host():
        dz, dg, ds, dm, dy = (t.to(dev, non_blocking=True) for t in (hz, hg, hs, hm, hy))
        cg.solve(dz, dy, ds, dm, mu, n_iter, out)
        cg.solve_vjp(dg, ds, dm, mu, n_iter, gz)
        hout.copy_(out, non_blocking=True)
        hgz.copy_(gz, non_blocking=True)

    step_host()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(e2e_steps):
        step_host()
    e1.record(stream)
    barrier()
    e2e_ms, e2e_units = aggregate(e0.elapsed_time(e1), w.voxel_coils * ops_per_step * e2e_steps, world, dist, dev)
    nb = lambda t: t.numel() * t.element_size()
    h2d, d2h = sum(nb(t) for t in (hz, hg, hs, hm, hy)), nb(hout) + nb(hgz)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    alu_peak = fp32_peak_tflops(peaks["sm_max_mhz"])
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    kd = kernels[dom]
    t_hbm, t_alu = kd["gbs"] / peaks["hbm_gbs"], kd["tflops"] / alu_peak
    if t_hbm >= t_alu:
        roof = {"bound": "hbm", "achieved": kd["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": t_hbm}
    else:
        roof = {"bound": "alu", "achieved": kd["tflops"], "peak": alu_peak, "unit": "TFLOP/s", "frac": t_alu}
    roof.update({"kernel": dom, "peak_source": peaks["source"] + (" copy bandwidth" if roof["bound"] == "hbm" else
                 " sm_max_mhz x 148 SMs x 128 lanes x 2"), "traffic": None,
                 "share_of_step": kd["ms_per_step"] / sum(k["ms_per_step"] for k in kernels.values())})
    # whole step against the operator's own roofline: ops_per_step applications of A^H A at their VJP bound
    nbytes, flops = call_roofline(w, False)
    bound_s = ops_per_step * max(nbytes / (peaks["hbm_gbs"] * 1e9), flops / (alu_peak * 1e12))
    step_roof = {"operator_applications": ops_per_step, "bound_us": bound_s * 1e6,
                 "measured_us": total_ms / args.steps * 1e3, "frac": bound_s / (total_ms / args.steps * 1e-3)}

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import oracle
        oracle.build()
        cores = oracle.max_threads()
        wsamp, sample_txt = reference_sample(w)
        inp_c, y_c = (inp, y) if wsamp is w else make_problem(wsamp)
        d = oracle.Dims(wsamp.batch, wsamp.coils, wsamp.frames, wsamp.fft_rank, wsamp.n, 0, oracle.MASK_READOUT_INVARIANT)
        t0 = time.perf_counter()
        oracle.modl_cg_forward(inp_c["x"], y_c, inp_c["sens"], inp_c["mask"], mu, n_iter, d, nthreads=cores)
        oracle.modl_cg_vjp(inp_c["g"], inp_c["sens"], inp_c["mask"], mu, n_iter, d, nthreads=cores)
        dt = time.perf_counter() - t0
        cpu = {"value": wsamp.voxel_coils * ops_per_step / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": sample_txt + ", 1 step", "seconds": dt}

    print(json.dumps({
        "metric": MODL_METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "description": w.description, "mu": mu, "cg_steps": n_iter,
                   "step": "1 gleam_modl_cg_forward + 1 gleam_modl_cg_vjp; value counts voxel*coils per application "
                           "of A^H A (%d per step)" % ops_per_step,
                   "parallelism": "replicas only" if world > 1 else "1 gpu", "l2": "256 MB L2 flush before every step"},
        "clocks": clocks,
        "e2e": {"value": e2e_units / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": int(launches), "roofline": roof, "step_roofline": step_roof, "kernels": kernels, "cpu_baseline": cpu}))
    if dist is not None:
        dist.destroy_process_group()

def kernel_sources_digest():
    """SHA-256 over the CUDA sources of the library: identifies the kernels a counter capture was taken on."""
    import hashlib
    csrc = os.path.join(ROOT, "paper_2207_08393_b200", "csrc")
    h = hashlib.sha256()
    for name in sorted(os.listdir(csrc)):
        h.update(name.encode())
        h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()


def measured_traffic(workload, kernel):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of a kernel class from the
    recorded ncu captures; None when there is no capture or the kernel sources have changed since."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    rec = json.load(open(path))
    digest = kernel_sources_digest()
    for e in rec.get("captures", []):
        if e.get("workload") == workload and e.get("kernel") == kernel and e.get("sources_sha256") == digest:
            return float(e["dram_bytes_per_launch"])
    return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="knee3d")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--mask", default="invariant", choices=["invariant", "full"],
                    help="invariant: the mask is handed over in readout-invariant form (separable path); full: the same "
                         "pattern as a general (B,T,n0,n1,n2) array (arbitrary-mask path)")
    ap.add_argument("--kernels-only", action="store_true",
                    help="profiler run: warm-up and timed steps only, then a short JSON line (no per-kernel pass, no "
                         "end-to-end leg, no CPU baseline)")
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"],
                    help="graph: the step's launches are captured once and replayed; eager: enqueued call by call")
    ap.add_argument("--calls", default="both", choices=["both", "forward", "vjp"], help="which calls a step makes")
    ap.add_argument("--print-sources-digest", action="store_true", help="print the digest that keys profiles/dram_traffic.json")
    ap.add_argument("--method", default="dc", choices=["dc", "modl"],
                    help="dc: the gradient data-consistency step (Eq. 3); modl: the model inversion of Eq. 7 "
                         "by 10 conjugate-gradient steps (use with --workload knee2d or cine)")
    ap.add_argument("--mu", type=float, default=0.05)
    ap.add_argument("--cg-steps", type=int, default=10)
    args = ap.parse_args()
    from paper_2207_08393_b200 import workloads as wl
    if args.print_sources_digest:
        print(kernel_sources_digest())
        return
    if args.workload == "knee3d_small":
        # profiler case: the full 320 x 256 phase-encode plane of knee3d (same kernels and launch shapes), 20 of
        # the 320 readout slabs: 0.4 GB on the device, larger than L2, small enough for multi-pass counter captures
        w = wl.scaled(wl.WORKLOADS["knee3d"], name="knee3d_small", n=(20, 320, 256),
                      description="profiler case: knee3d with 20 of 320 readout slabs (8 coils, 20x320x256)")
    else:
        w = wl.WORKLOADS[args.workload]
    if args.method == "modl":
        run_modl(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
