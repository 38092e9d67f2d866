#!/usr/bin/env python
"""Benchmark of the composed forward (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload all|c1..c9]

A step is one composed forward of the workload's module (every submodule of its default
decomposition) over one batch of seeded synthetic input.  With no --workload the run covers the
five modules of the workload list in one invocation: the line's top level describes C5, the
largest (the 4-layer decoder; --steps K times exactly K of its forwards), and its `workloads`
object carries the same measurements of C1-C4, each with the step count it used.  `value` is the whole-job throughput in
TFLOP/s of algorithmic work with inputs resident in HBM; `e2e` repeats the measurement with the
step's inputs copied from pinned host memory and its result copied back inside the timed region.
Each step works on a different copy of the inputs and outputs (a rotation larger than L2), so no
step finds its operands in L2 from the step before.

Under torchrun every rank runs the same workload on its own GPU (independent batches, no
collective on the data path: weak scaling); times are device times, max over ranks.

`--impl reference` times the fp64 CPU oracle, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "composed-module fwd latency, TFLOP/s & GB/s as % of B200 roofline, per subkernel"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (null where no capture of that workload's dominant kernel exists).
# c4: the attention kernel was captured on 2 of the 16 batch elements (52.2 MB; its traffic is
# proportional to the batch) and is scaled by 8 here.
# c5: average over the 32 GEMM launches of two captured steps (16 per step, four shapes).
NCU_TRAFFIC_BYTES = {"c2": 89.9e6,            # profiles/gemm_tc2_c2.md
                     "c3": 26.25e6,            # profiles/conv3x3_tc2_groupnorm_c3.md (conv; its output stays in L2)
                     "c4": 8 * 52.2e6,         # profiles/attention_tc2_c4.md
                     "c5": 259.7e6}            # profiles/gemm_tc2_decoder_c5.md

DEFAULT_STEPS = {"c1": 2000, "c2": 200, "c3": 400, "c4": 100, "c5": 50, "c6": 100, "c7": 400, "c8": 200, "c9": 200}


def full_workload(name, seed=0, batch=None, only_ops=None):
    """The named workload at its full size.  `batch` (a smaller leading batch dimension) and `only_ops` (the
    first N operators alone) cut out small cases of the same kernels for profiler captures."""
    import workloads as W
    kw = {}
    if batch is not None:
        kw = {"c1": {"M": batch}, "c2": {"M": batch}, "c3": {"NB": batch}, "c4": {"B": batch}, "c5": {"B": batch},
              "c6": {"B": batch}, "c7": {"NB": batch}, "c8": {"M": batch}, "c9": {"NB": batch}}[name]
    w = W.generate.WORKLOADS[name](seed, **kw)
    if only_ops is not None:
        w.ops = w.ops[:only_ops]
        w.partitions = {"fused": [0], "per_op": list(range(len(w.ops)))}
        w.flops = None          # recomputed from the operators once the module exists
    return w


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ----------------------------------------------------------------------------------------------------
# clocks: sampled on a thread while the timed region runs (read-only NVML queries)
# ----------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._t = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _once(self):
        try:
            self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            try:
                r = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
            except Exception:
                r = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            for bit, name in self.REASONS.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._once()
            self._stop.wait(0.02)

    def start(self):
        if self.nv:
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()

    def stop(self):
        if self._t:
            self._once()
            self._stop.set()
            self._t.join()
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ----------------------------------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------------------------------
def oracle_sample(name, w, budget_s=12.0):
    """Time the fp64 oracle on a bounded sample of the workload: a leading block of independent
    rows / images / batch elements, sized from a short probe to take about `budget_s` seconds.
    Returns (flops_done, seconds, description)."""
    import numpy as np
    from oracle import modules as OM

    def sub(frac_units):
        import copy
        s = copy.copy(w)
        s.inputs = dict(w.inputs)
        s.ops = [dict(o, attrs=dict(o["attrs"])) for o in w.ops]
        from workloads.generate import Tensor
        if name in ("c1", "c2"):
            rows = frac_units
            s.inputs["x"] = Tensor("x", w.dtype, w.inputs["x"].store[:rows])
            total = w.inputs["x"].shape[0]
            what = f"first {rows} of {total} rows of X"
        elif name == "c8":
            rows = frac_units
            for k in ("xq", "sx"):
                s.inputs[k] = Tensor(k, w.inputs[k].dtype, w.inputs[k].store[:rows])
            total = w.inputs["xq"].shape[0]
            what = f"first {rows} of {total} rows of X"
        elif name in ("c3", "c7", "c9"):
            s.inputs["x"] = Tensor("x", w.dtype, w.inputs["x"].store[:frac_units])
            total = w.inputs["x"].shape[0]
            what = f"first {frac_units} of {total} images"
        elif name == "c4":
            b_total, h, sq, d = w.inputs["q"].shape
            for k in ("q", "k", "v"):
                s.inputs[k] = Tensor(k, w.dtype, w.inputs[k].store[:frac_units])
            s.inputs["r"] = Tensor("r", w.dtype, w.inputs["r"].store[: frac_units * sq])
            total = b_total
            what = f"first {frac_units} of {total} batch elements"
        else:
            attn = [o for o in w.ops if o["kind"] in ("attention_causal", "attention")][0]["attrs"]
            sq, total = attn["seq"], attn["batch"]
            s.inputs["x"] = Tensor("x", w.dtype, w.inputs["x"].store[: frac_units * sq])
            for o in s.ops:
                if o["kind"] in ("attention_causal", "attention"):
                    o["attrs"]["batch"] = frac_units
            what = f"first {frac_units} of {total} batch elements"
        return s, total, what

    probe_units = {"c1": 64, "c2": 64, "c3": 1, "c4": 1, "c5": 1, "c6": 1, "c7": 1, "c8": 64, "c9": 1}[name]
    s, total, _ = sub(probe_units)
    t0 = time.perf_counter()
    OM.run_workload(s, [0])
    probe = max(time.perf_counter() - t0, 1e-4)
    units = int(min(total, max(probe_units, probe_units * budget_s / probe)))
    if units > probe_units:
        s, total, what = sub(units)
        t0 = time.perf_counter()
        OM.run_workload(s, [0])
        secs = time.perf_counter() - t0
    else:
        s, total, what = sub(probe_units)
        units, secs = probe_units, probe
    return w.flops * units / total, secs, what


def submodule_work(w, module):
    """Algorithmic flops and minimum bytes of every submodule of the module's current decomposition:
    flops of the contractions inside it; bytes = its contract inputs + outputs + the parameters its
    operators read (each counted once)."""
    import numpy as np
    esz = {0: 4, 1: 2}
    cuts = module.decomposition() + [len(w.ops)]
    out = []
    for s_ in range(len(cuts) - 1):
        fl = 0.0
        by = 0.0
        ins, outs = module.contract(s_)
        for _, (dt_, shape, _) in ins + outs:
            by += float(np.prod(shape)) * esz[dt_]
        for j in range(cuts[s_], cuts[s_ + 1]):
            op = w.ops[j]
            for pn in op["params"].values():
                if pn is not None:
                    by += w.params[pn].nbytes()
            _, xs, _ = module.value_spec(op["in"][0])
            _, ys, _ = module.value_spec(op["out"])
            if op["kind"] in ("linear", "linear_fp8"):
                fl += 2.0 * float(np.prod(xs)) * op["attrs"]["n"]
            elif op["kind"] == "conv2d_3x3":
                fl += 2.0 * xs[0] * xs[1] * xs[2] * 9 * xs[3] * op["attrs"]["c_out"]
            elif op["kind"] in ("attention_causal", "attention"):
                a = op["attrs"]
                if a["layout"] == "bhsd":
                    b_, h_, sq, d_ = xs
                else:
                    b_, sq, h_, d_ = a["batch"], a["seq"], a["heads"], a["head_dim"]
                # causal: the exact j <= i triangle; unmasked: every (query, key) pair
                fl += 4.0 * b_ * h_ * d_ * (sq * (sq + 1) / 2 if op["kind"] == "attention_causal" else sq * sq)
        out.append((fl, by))
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = full_workload(args.workload)
    t_all = []
    flops = 0.0
    what = ""
    budget = max(2.0, min(12.0, 120.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        f, s, what = oracle_sample(args.workload, w, budget_s=budget)
        if i >= args.warmup:
            t_all.append(s)
            flops = f
    mean_s = sum(t_all) / len(t_all)
    val = flops / mean_s / 1e12
    cores = os.cpu_count()
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean_s * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "sample": what},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                         "blas": "numpy fp64, contractions through the BLAS numpy links (multi-threaded)", "sample": what},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------------------
# nominal B200 figures, for the second column the metric asks for (context, not the denominator of `frac`)
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}


def roofline_of(name, launches_per_step, dominant, achieved, peak, pk, kernel_ms, t_roof_ms, ms_per_step, min_step_ms,
                median_step_ms=None, t_roof_nominal_ms=None, peak_scale=1.0):
    """Roofline object of the dominant kernel.  A one-launch step is timed directly by the per-step
    event pairs; in a multi-kernel step the dominant kernel's duration comes from the per-submodule
    event pairs of mk_module_profile (mean over its launches)."""
    r = {"bound": "tensor" if peak > 100 else "alu", "unit": "TFLOP/s", "peak": peak, "peak_source": pk["_source"] if peak > 100 else "derived",
         "traffic": NCU_TRAFFIC_BYTES.get(name), "module_t_roof_ms": t_roof_ms, "module_frac": t_roof_ms / ms_per_step,
         "min_step_ms": min_step_ms, "median_step_ms": median_step_ms,
         "module_frac_of_nominal": (t_roof_nominal_ms / ms_per_step) if t_roof_nominal_ms else None}
    if peak > 100:
        # both denominators side by side: the burst figure suits a timed region of a few milliseconds, the
        # sustained one a step timed inside a run long enough for the power cap to act (see `sustained`)
        fl = t_roof_ms * 1e-3 * peak      # algorithmic TFLOP of the module when it is tensor-bound
        for key in ("bf16_tflops", "bf16_tflops_sustained"):
            if key in pk:
                r["module_frac_of_" + ("burst" if key == "bf16_tflops" else "sustained") + "_peak"] = (fl / (pk[key] * peak_scale)) / (ms_per_step * 1e-3)
    if launches_per_step == 1 or dominant is None:
        r.update({"kernel": "whole step (one launch)", "achieved": achieved, "frac": achieved / peak, "kernel_ms": kernel_ms})
    else:
        k, a = dominant
        ach = a["flops"] / (a["ms"] * 1e-3) / 1e12
        r.update({"kernel": k, "achieved": ach, "frac": ach / peak, "kernel_ms": a["ms"] / a["launches"],
                  "launches_per_step": a["launches"]})
    return r


def measure_one(name, args, steps, ctx, rank, local, world, cpu_seconds):
    """All measurements of one workload; returns the line's fields on rank 0, None elsewhere."""
    import torch
    from paper_2607_20501_b200 import dist as D
    from paper_2607_20501_b200.runner import DeviceWorkload

    w = full_workload(name, batch=args.batch, only_ops=args.only_ops)
    # rotation: enough independent copies that a pass over all of them exceeds L2 (126 MB) twice over
    per_copy = sum(t.nbytes() for t in w.inputs.values()) + sum(t.nbytes() for t in w.params.values())
    rot = int(max(2, min(8, -(-300e6 // max(per_copy, 1)))))
    sets = [DeviceWorkload(ctx, w, device=f"cuda:{local}") for _ in range(rot)]
    part = args.decomposition or ("fused" if "fused" in w.partitions else None)
    for dw in sets:
        if part:
            dw.module.set_decomposition(w.partitions[part])
        dw.ensure_workspace()
    impls = [sets[0].module.bound_impl(s) for s in range(sets[0].module.n_sub())]
    if w.flops is None:
        work = submodule_work(w, sets[0].module)
        w.flops = sum(f for f, _ in work)
        w.min_bytes = sum(b for _, b in work)
    stream = torch.cuda.current_stream()

    def barrier():
        D.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        sets[i % rot].forward()
    barrier()
    launches_per_step = sets[0].module.launch_count()

    # ---- timed region: K steps, device time, per-step event pairs for the kernel duration
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    t_begin.record(stream)
    for i in range(steps):
        ev[i][0].record(stream)
        sets[i % rot].forward()
        ev[i][1].record(stream)
    t_end.record(stream)
    barrier()
    clocks = sampler.stop()
    ctx.check()
    total_ms = t_begin.elapsed_time(t_end)
    step_ms = sorted(a.elapsed_time(b) for a, b in ev)
    kernel_ms = sum(step_ms) / len(step_ms)

    # ---- short steps: below about 0.1 ms the Python loop above (ctypes call + two event records per step) cannot
    # keep the GPU fed, and up to 0.2 ms it still leaves gaps now and then (C2: 103.7 us from the loop against
    # 98.8 us of device time, the same kernels, the same box).  For every step shorter than 0.2 ms the same K
    # steps are replayed from a CUDA graph (one node per kernel launch, the rotation over input sets unrolled
    # into it) and THAT time is reported, with the loop's time beside it; a graph of as many one-element
    # kernels gives the launch floor.
    graph_info = None
    sustained = None
    if args.timed_only:
        # profiler captures: the warm-up and the K timed steps are all that is launched
        if rank == 0:
            print(json.dumps({"timed_only": True, "workload": name, "steps": steps, "ms_per_step": total_ms / steps,
                              "launches_per_step": launches_per_step}))
        return None
    if kernel_ms < 1.0:
        gstream = torch.cuda.Stream()
        gstream.wait_stream(stream)
        reps = max(1, steps // rot)
        with torch.cuda.stream(gstream):
            for dw in sets:
                dw.forward()            # launch plans for this stream exist before capture
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=gstream):
                for dw in sets:
                    dw.forward()
            for _ in range(3):
                g.replay()
            torch.cuda.synchronize()
            if kernel_ms < 0.2:
                tiny = torch.zeros(1, device=f"cuda:{local}")
                gf = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gf, stream=gstream):
                    for _ in range(rot * launches_per_step):
                        tiny.add_(1.0)
                for _ in range(3):
                    gf.replay()
                torch.cuda.synchronize()
                g0, g1, g2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                g0.record(gstream)
                for _ in range(reps):
                    g.replay()
                g1.record(gstream)
                for _ in range(reps):
                    gf.replay()
                g2.record(gstream)
                torch.cuda.synchronize()
                graph_info = {"ms_per_step": g0.elapsed_time(g1) / (reps * rot), "steps": reps * rot,
                              "launch_floor_ms_per_step": g1.elapsed_time(g2) / (reps * rot),
                              "eager_ms_per_step": total_ms / steps}
            # ---- the sustained regime: a sub-millisecond step timed over K steps is a burst measurement (the
            # whole timed region can be shorter than the power controller's reaction); the same graph replayed
            # back to back for at least half a second, with the clocks sampled beside it, gives the figure a
            # long-running job would see
            n_rep = int(max(1, -(-500.0 // max(kernel_ms * rot, 1e-3))))
            s_sampler = ClockSampler(local)
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            s_sampler.start()
            q0.record(gstream)
            for _ in range(n_rep):
                g.replay()
            q1.record(gstream)
            torch.cuda.synchronize()
            s_clocks = s_sampler.stop()
            sustained = {"ms_per_step": q0.elapsed_time(q1) / (n_rep * rot), "steps": n_rep * rot,
                         "seconds": q0.elapsed_time(q1) * 1e-3, "timing": "CUDA graph replay, back to back",
                         "clocks": s_clocks}
        ctx.check()
        if graph_info:
            total_ms = graph_info["ms_per_step"] * steps
            kernel_ms = graph_info["ms_per_step"]
    else:
        # a step of a millisecond or more keeps the GPU fed from the Python loop; the sustained figure is the
        # same loop run for at least half a second
        n_rep = int(max(steps, -(-500.0 // kernel_ms)))
        s_sampler = ClockSampler(local)
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        s_sampler.start()
        q0.record(stream)
        for i in range(n_rep):
            sets[i % rot].forward()
        q1.record(stream)
        torch.cuda.synchronize()
        s_clocks = s_sampler.stop()
        ctx.check()
        sustained = {"ms_per_step": q0.elapsed_time(q1) / n_rep, "steps": n_rep, "seconds": q0.elapsed_time(q1) * 1e-3,
                     "timing": "stream order from the host loop, back to back", "clocks": s_clocks}

    # ---- end to end: pinned host inputs in, result out, every step
    host_in = {k: torch.empty(t.shape, dtype=sets[0].inputs[k].dtype).pin_memory() for k, t in w.inputs.items()}
    for k in host_in:
        host_in[k].copy_(sets[0].inputs[k].cpu())
    host_out = [torch.empty(sets[0].out.shape, dtype=sets[0].out.dtype).pin_memory() for _ in range(rot)]
    h2d = sum(t.numel() * t.element_size() for t in host_in.values())
    d2h = host_out[0].numel() * host_out[0].element_size()
    e2e_steps = max(3, min(steps, 50))

    # Every step copies its inputs in, runs the forward and copies its result out; the three legs run on three
    # streams, so that step i's copy out, step i + 1's forward and step i + 2's copy in overlap (PCIe carries
    # both directions at once).  A buffer set is reused only when the step that used it last has let go of it.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(rot)]
    ev_fwd = [torch.cuda.Event() for _ in range(rot)]
    ev_out = [torch.cuda.Event() for _ in range(rot)]
    used = [False] * rot

    def e2e_step(i):
        k_set = i % rot
        dw = sets[k_set]
        if used[k_set]:
            s_in.wait_event(ev_fwd[k_set])      # the forward that read these inputs last
        with torch.cuda.stream(s_in):
            for k in host_in:
                dw.inputs[k].copy_(host_in[k], non_blocking=True)
            ev_in[k_set].record(s_in)
        stream.wait_event(ev_in[k_set])
        if used[k_set]:
            stream.wait_event(ev_out[k_set])    # the copy out that read this output last
        dw.forward()
        ev_fwd[k_set].record(stream)
        s_out.wait_event(ev_fwd[k_set])
        with torch.cuda.stream(s_out):
            host_out[k_set].copy_(dw.out, non_blocking=True)
            ev_out[k_set].record(s_out)
        used[k_set] = True

    for i in range(rot):
        e2e_step(i)
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    s_in.wait_event(e0)
    s_out.wait_event(e0)
    for i in range(e2e_steps):
        e2e_step(i)
    stream.wait_event(ev_out[(e2e_steps - 1) % rot])
    stream.wait_stream(s_out)
    stream.wait_stream(s_in)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    k_last = (e2e_steps - 1) % rot
    if not torch.equal(host_out[k_last].view(torch.uint8), sets[k_last].out.cpu().view(torch.uint8)):
        raise RuntimeError("end-to-end leg: the result copied to the host differs from the device result")

    # ---- per-subkernel breakdown: every submodule of the decomposition that names each kernel once
    # (time, share, algorithmic work, roofline fraction of that subkernel)
    breakdown = None
    dominant = None
    split_name = {"c1": "split", "c2": "split", "c3": "split2", "c4": "split3", "c5": "fused_tails", "c6": "fused_tails", "c7": "split2", "c9": "split3"}.get(name)
    if rank == 0 and split_name in w.partitions:
        pk_ = peaks()
        dw = sets[0]
        dw.module.set_decomposition(w.partitions[split_name])
        dw.ensure_workspace()
        dw.forward()
        torch.cuda.synchronize()
        ev_ms = dw.profile(iters=20)
        # The event pairs of mk_module_profile include the gap between two kernels in a stream (several microseconds:
        # a third of a 20 us row kernel).  Each submodule is therefore also timed ALONE: mk_module_forward_sub of that
        # submodule, over the rotating buffer sets (their boundary tensors kept from one whole forward each), replayed
        # back to back from a CUDA graph.  `ms` is that device time; `event_ms` the event-pair figure.
        n_sub = dw.module.n_sub()
        for d_ in sets:
            d_.module.set_decomposition(w.partitions[split_name])
            d_.module.keep_intermediates(True)
            d_.ensure_workspace()
            d_.forward()
        torch.cuda.synchronize()
        ms = []
        bs = torch.cuda.Stream()
        bs.wait_stream(stream)
        with torch.cuda.stream(bs):
            for s_ in range(n_sub):
                reps_in = max(1, 8 // rot)
                for d_ in sets:
                    d_.forward_sub(s_)
                torch.cuda.synchronize()
                gsub = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gsub, stream=bs):
                    for _ in range(reps_in):
                        for d_ in sets:
                            d_.forward_sub(s_)
                gsub.replay()
                torch.cuda.synchronize()
                n_rep = int(max(2, min(50, 2.0 // max(ev_ms[s_] * reps_in * rot, 1e-3))))     # about 2 ms per submodule
                b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                b0.record(bs)
                for _ in range(n_rep):
                    gsub.replay()
                b1.record(bs)
                torch.cuda.synchronize()
                ms.append(b0.elapsed_time(b1) / (n_rep * reps_in * rot))
                del gsub
        ctx.check()
        tot = sum(ms)
        work = submodule_work(w, dw.module)
        rows, agg, agg_ev = [], {}, {}
        for s_, (t_, (fl, by)) in enumerate(zip(ms, work)):
            impl = dw.module.bound_impl(s_)
            ae = agg_ev.setdefault(impl, {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "launches": 0})
            ae["ms"] += ev_ms[s_]; ae["flops"] += fl; ae["bytes"] += by; ae["launches"] += 1
            t_roof = max(fl / (pk_["bf16_tflops"] * 1e12), by / (pk_["hbm_gbs"] * 1e9)) * 1e3
            rows.append({"sub": s_, "impl": impl, "ms": round(t_, 5), "event_ms": round(ev_ms[s_], 5), "tflops": round(fl / (t_ * 1e-3) / 1e12, 1),
                         "gbs": round(by / (t_ * 1e-3) / 1e9, 1), "roof_frac": round(t_roof / t_, 3),
                         "bound": "tensor" if fl / (pk_["bf16_tflops"] * 1e12) >= by / (pk_["hbm_gbs"] * 1e9) else "hbm"})
            a = agg.setdefault(impl, {"ms": 0.0, "flops": 0.0, "bytes": 0.0, "launches": 0})
            a["ms"] += t_; a["flops"] += fl; a["bytes"] += by; a["launches"] += 1
        breakdown = {"decomposition": split_name, "ms_total": tot, "event_ms_total": sum(ev_ms),
                     "timing": "each submodule alone (mk_module_forward_sub) by CUDA graph replay over the rotating buffer sets; event_ms: mk_module_profile's event pairs",
                     "share": {k: round(v["ms"] / tot, 4) for k, v in agg.items()},
                     "per_kernel": {k: {"ms": round(v["ms"], 5), "launches": v["launches"],
                                        "tflops": round(v["flops"] / (v["ms"] * 1e-3) / 1e12, 1),
                                        "gbs": round(v["bytes"] / (v["ms"] * 1e-3) / 1e9, 1)} for k, v in agg.items()},
                     "submodules": rows if len(rows) <= 12 else rows[:12]}
        # the roofline object describes the dominant kernel as it ran INSIDE whole forwards (the event-pair figures, taken
        # at the clocks of a long step); the per-submodule device times above are short bursts of one kernel alone
        dk = max(agg_ev, key=lambda k: agg_ev[k]["ms"])
        dominant = (dk, agg_ev[dk])
        if graph_info:
            # launch-bound module: the split decomposition's step by graph replay too (the fused / split comparison)
            gs = torch.cuda.Stream()
            gs.wait_stream(stream)
            with torch.cuda.stream(gs):
                dw.forward()
                torch.cuda.synchronize()
                gsp = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gsp, stream=gs):
                    for _ in range(8):
                        dw.forward()
                for _ in range(3):
                    gsp.replay()
                torch.cuda.synchronize()
                s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                nrep = max(1, steps // 8)
                s0.record(gs)
                for _ in range(nrep):
                    gsp.replay()
                s1.record(gs)
                torch.cuda.synchronize()
            ctx.check()
            breakdown["graph_ms_per_step"] = s0.elapsed_time(s1) / (nrep * 8)
            breakdown["launches_per_step"] = dw.module.launch_count()

    # ---- max over ranks
    total_ms, kernel_ms, e2e_ms = D.max_over_ranks([total_ms, kernel_ms, e2e_ms], device=f"cuda:{local}")

    if rank == 0:
        pk = peaks()
        ms_per_step = total_ms / steps
        value = world * w.flops / (ms_per_step * 1e-3) / 1e12
        achieved = w.flops / (kernel_ms * 1e-3) / 1e12
        peak = pk["bf16_tflops"] if ms_per_step < 1.0 else pk.get("bf16_tflops_sustained", pk["bf16_tflops"])
        fp8 = any(t.dtype == "fp8" for t in w.inputs.values())
        if fp8:
            # the contraction's own peak: the measured bf16 figure times the nominal fp8 : bf16 ratio of the tensor cores (2)
            peak *= 2.0
        if w.dtype == "f32":
            # plain fp32 FMA units: 148 SMs x 128 lanes x 2 flop x 1.965 GHz (no fp32 tensor path at this tolerance)
            peak = 148 * 128 * 2 * 1.965e9 / 1e12
        t_roof_ms = max(w.flops / (peak * 1e12), w.min_bytes / (pk["hbm_gbs"] * 1e9)) * 1e3
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8" if fp8 else ("bf16" if w.dtype == "bf16" else "f32"), "data": "synthetic",
            "config": {"workload": name, "decomposition": part, "impls": impls,
                       "l2": (f"rotation over {rot} independent input/output sets ({rot * per_copy / 1e6:.0f} MB > L2)" if rot * per_copy > 126e6 else
                              f"rotation over {rot} independent input/output sets ({rot * per_copy / 1e6:.1f} MB in all: the whole problem is "
                              "smaller than L2 and bound by launch latency, so L2 residency is part of the measurement)"),
                       "shapes": {k: list(t.shape) for k, t in w.inputs.items()},
                       **({"cut": {"batch": args.batch, "only_ops": args.only_ops}} if (args.batch or args.only_ops) else {})},
            "roofline": roofline_of(name, launches_per_step, dominant, achieved, peak, pk, kernel_ms, t_roof_ms, ms_per_step, step_ms[0],
                                    median_step_ms=step_ms[len(step_ms) // 2], peak_scale=2.0 if fp8 else 1.0,
                                    t_roof_nominal_ms=(None if w.dtype == "f32" else
                                                       max(w.flops / (NOMINAL["bf16_tflops"] * (2 if fp8 else 1) * 1e12), w.min_bytes / (NOMINAL["hbm_gbs"] * 1e9)) * 1e3)),
            "e2e": {"value": world * w.flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                    "pipeline": f"copy in / forward / copy out on three streams over {rot} buffer sets"},
            "gpu_launches": launches_per_step * steps,
            "clocks": clocks,
            "per_subkernel": breakdown,
        }
        if graph_info:
            line["config"]["timing"] = "CUDA graph replay (step shorter than 0.2 ms; the Python loop's time is kept beside it in `graph`)"
            line["graph"] = graph_info
        if sustained:
            ps = pk.get("bf16_tflops_sustained", pk["bf16_tflops"]) * (2.0 if fp8 else 1.0) if w.dtype != "f32" else peak
            t_roof_s = max(w.flops / (ps * 1e12), w.min_bytes / (pk["hbm_gbs"] * 1e9)) * 1e3
            sustained.update({"value": w.flops / (sustained["ms_per_step"] * 1e-3) / 1e12, "unit": "TFLOP/s", "peak": ps,
                              "module_t_roof_ms": t_roof_s, "module_frac": t_roof_s / sustained["ms_per_step"]})
            line["sustained"] = sustained
        if not args.no_cpu and world == 1:
            f, s, what = oracle_sample(name, w, budget_s=cpu_seconds)
            line["cpu_baseline"] = {"value": f / s / 1e12, "unit": "TFLOP/s", "cores": os.cpu_count(), "kind": "oracle",
                                    "blas": "numpy fp64, contractions through the BLAS numpy links (multi-threaded)",
                                    "sample": what, "seconds": s}
        else:
            line["cpu_baseline"] = None
    return line if rank == 0 else None


SUITE = ["c1", "c2", "c3", "c4", "c5"]      # the workload list's five modules; the last one is the headline
SUITE_KEYS = ("ms_per_step", "value", "unit", "steps", "dtype", "config", "roofline", "sustained", "graph", "e2e", "gpu_launches",
              "clocks", "per_subkernel", "cpu_baseline")


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2607_20501_b200 import dist as D

    rank, local, world = D.env_world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    D.init("nccl", torch.device("cuda", local))
    from paper_2607_20501_b200 import Context
    ctx = Context(local)

    if args.workload != "all":
        steps = args.steps if args.steps is not None else DEFAULT_STEPS[args.workload]
        line = measure_one(args.workload, args, steps, ctx, rank, local, world, args.cpu_seconds)
    else:
        import gc
        # C1-C4 first, each with its own step count (their steps are 7 us to 0.5 ms long: the default counts make
        # every timed region tens of milliseconds), then the headline C5 with exactly --steps K steps.
        others = {}
        for name in SUITE[:-1]:
            r = measure_one(name, args, DEFAULT_STEPS[name], ctx, rank, local, world, min(args.cpu_seconds, 4.0))
            if r is not None:
                others[name] = {k: r[k] for k in SUITE_KEYS if k in r}
                others[name]["module_frac"] = r["roofline"]["module_frac"]
            gc.collect()                 # the workload's device buffers go before the next one is uploaded
            torch.cuda.empty_cache()
        steps = args.steps if args.steps is not None else DEFAULT_STEPS[SUITE[-1]]
        line = measure_one(SUITE[-1], args, steps, ctx, rank, local, world, args.cpu_seconds)
        if line is not None:
            line["workloads"] = others
            fr = {k: round(v["module_frac"], 4) for k, v in others.items()}
            fr[SUITE[-1]] = round(line["roofline"]["module_frac"], 4)
            line["module_frac"] = fr
            line["gpu_launches_all_workloads"] = line["gpu_launches"] + sum(v["gpu_launches"] for v in others.values())
    if rank == 0 and line is not None:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=["all", "c1", "c2", "c3", "c4", "c5", "c6", "c7", "c8", "c9"],
                    help="default: all five modules of the workload list for the GPU arm (headline C5), c5 for the reference arm")
    ap.add_argument("--decomposition", default=None)
    ap.add_argument("--batch", type=int, default=None, help="smaller leading batch dimension (profiler captures)")
    ap.add_argument("--only-ops", type=int, default=None, help="run the first N operators alone (profiler captures)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle leg")
    ap.add_argument("--timed-only", action="store_true",
                    help="launch only the warm-up and the K timed steps (profiler captures of one workload)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 3
        if args.workload in (None, "all"):
            args.workload = "c5"
        run_reference(args)
    else:
        if args.workload is None:
            args.workload = "all" if (args.batch is None and args.only_ops is None) else "c2"
        run_ours(args)


if __name__ == "__main__":
    main()
