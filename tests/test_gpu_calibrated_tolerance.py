"""Per-stage calibrated tolerances and the feasibility gap (paper, the section on verification with
calibrated tolerances and its bug-detection tables), run as a protocol on the composed C4 block at reduced size.

Calibration: over several seeds, every submodule of the three-way decomposition is checked LOCALLY - the
GPU stage's output against the fp64 oracle of that stage applied to the very tensors the GPU stage read -
and its tolerance is set to max + 3 sigma of the observed maximum absolute error (no relative part).  The
module's output gets the same treatment (global check).  Then subtly wrong subkernels are emulated by
handing the GPU a perturbed description of one stage (the oracle keeps the true one):

  * the local check of the perturbed stage, with its calibrated tolerance, must flag every one of them, and
    the local checks of the other stages must stay green (errors are localised);
  * the module-level check with the fixed bf16 tolerance (rtol 2e-2, atol 2e-2) lets some of them through:
    that is the feasibility gap the decomposition closes."""
import copy

import numpy as np
import pytest

import workloads as W
from workloads import generate as G
from oracle import modules as OM
from oracle.compare import check_close
from paper_2607_20501_b200.runner import to_host_f64
from tests.parity import run_gpu

pytestmark = pytest.mark.gpu

SHAPE = dict(B=2, H=4, S=256, D=128)
STAGES = [("a", 0, 1), ("h", 1, 3), ("y", 3, 4)]     # boundary value, first op, one past the last op


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_20501_b200 import Context
    return Context(0)


def _local_errors(ctx, w_gpu, w_true):
    """Max abs error of every stage against the oracle of that stage on the GPU stage's own inputs, and of
    the module output against the oracle of the whole true module."""
    dw, out = run_gpu(ctx, w_gpu, w_gpu.partitions["split3"], keep=True)
    have = {k: t.f64() for k, t in w_true.inputs.items()}
    params = {k: t.f64() for k, t in w_true.params.items()}
    errs = {}
    for name, lo, hi in STAGES:
        ref, _ = OM.run_module(w_true.ops[lo:hi], {k: have[k] for op in w_true.ops[lo:hi] for k in op["in"] if k in have}, params)
        got = out if name == "y" else to_host_f64(dw.intermediate(name))
        errs[name] = float(np.abs(got - ref).max())
        have[name] = got                       # the next stage is judged on what it was actually given
    ref_all, _ = OM.run_workload(w_true, [0])
    return errs, float(np.abs(out - ref_all).max()), check_close(out, ref_all, "bf16")["ok"]


def test_calibrated_local_checks_catch_what_the_global_tolerance_lets_through(ctx):
    seeds = range(8)
    runs = []
    for s in seeds:
        w = W.c4(s, **SHAPE)
        errs, gerr, gok = _local_errors(ctx, w, w)
        assert gok
        runs.append((errs, gerr))
    tol = {n: float(np.max([r[0][n] for r in runs]) + 3 * np.std([r[0][n] for r in runs])) for n, _, _ in STAGES}
    gtol = float(np.max([r[1] for r in runs]) + 3 * np.std([r[1] for r in runs]))
    assert all(t > 0 for t in tol.values())

    def mutant(kind):
        w = W.c4(100, **SHAPE)
        m = copy.copy(w)
        m.inputs, m.params = dict(w.inputs), dict(w.params)
        m.ops = [dict(o, attrs=dict(o["attrs"])) for o in w.ops]
        if kind == "attention: logits 5 % too large":
            m.inputs["q"] = G.make("q", "bf16", (1.05 * w.inputs["q"].f64()).astype(np.float32))
            stage = "a"
        elif kind == "projection: one output column 30 % off":
            wo = w.params["Wo"].f64().copy()
            wo[:, 7] *= 1.3
            m.params["Wo"] = G.make("Wo", "bf16", wo.astype(np.float32))
            stage = "h"
        else:
            m.ops[3]["attrs"]["eps"] = 3e-2
            stage = "y"
        return w, m, stage

    evaded_global = 0
    for kind in ("attention: logits 5 % too large", "projection: one output column 30 % off", "rmsnorm: eps 3e-2 instead of 1e-6"):
        w_true, w_mut, stage = mutant(kind)
        errs, gerr, gok_fixed = _local_errors(ctx, w_mut, w_true)
        assert errs[stage] > tol[stage], f"{kind}: local error {errs[stage]:.3g} within calibrated {tol[stage]:.3g}"
        for n, _, _ in STAGES:
            if n != stage:
                assert errs[n] <= tol[n], f"{kind}: stage {n} flagged although only {stage} is wrong"
        evaded_global += int(gok_fixed)
    # at least one of these subtle faults passes the fixed module-level tolerance
    assert evaded_global >= 1
    assert gtol < 0.2
