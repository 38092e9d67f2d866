"""fp64 CPU oracle: composed modules.

TEST INFRASTRUCTURE ONLY (see oracle/ops.py).  A module is an operator
sequence; a decomposition is a contiguous partition of that sequence into
submodules, each with a fixed input/output contract (paper, Methodology: the
codebase is a set of subkernels plus one top-level module that only chains
them).  `run_module` evaluates the sequence submodule by submodule, handing a
submodule nothing but its contract inputs, so that a decomposition whose
contract misses a tensor fails here as it would in the composed kernel.
No value is rounded at a boundary: every decomposition of a module therefore
gives the same result, which tests/test_oracle_modules.py asserts.
"""
from __future__ import annotations

from . import ops as O


def apply_op(op, vals, params):
    """Evaluate one operator description against named fp64 values."""
    kind = op["kind"]
    ins = [vals[n] for n in op["in"]]
    p = {k: (params[v] if v is not None else None) for k, v in op["params"].items()}
    a = op["attrs"]
    if kind == "linear":
        return O.linear(ins[0], p["w"])
    if kind == "linear_fp8":
        return O.linear_fp8_block(ins[0], ins[1], p["w"], p["sw"])
    if kind == "conv2d_3x3":
        return O.conv2d_3x3_nhwc(ins[0], p["w"])
    if kind == "bias_add":
        return O.bias_add(ins[0], p["b"])
    if kind == "relu":
        return O.relu(ins[0])
    if kind == "gelu_tanh":
        return O.gelu_tanh(ins[0])
    if kind == "gelu_erf":
        return O.gelu_erf(ins[0])
    if kind == "silu":
        return O.silu(ins[0])
    if kind == "scale":
        return O.scale(ins[0], a["s"])
    if kind == "clamp":
        return O.clamp(ins[0], a["lo"], a["hi"])
    if kind == "residual_add":
        return O.residual_add(ins[0], ins[1])
    if kind == "swiglu":
        return O.swiglu(ins[0])
    if kind == "layernorm":
        return O.layernorm(ins[0], p.get("gamma"), p.get("beta"), a["eps"])
    if kind == "rmsnorm":
        return O.rmsnorm(ins[0], p.get("gamma"), a["eps"])
    if kind == "softmax":
        return O.softmax(ins[0])
    if kind == "groupnorm":
        return O.groupnorm_nhwc(ins[0], p.get("gamma"), p.get("beta"), a["groups"], a["eps"])
    if kind == "attention_causal":
        if a["layout"] == "bhsd":
            return O.attention_causal_bhsd(ins[0], ins[1], ins[2])
        return O.attention_causal_packed(ins[0], a["batch"], a["seq"], a["heads"], a["head_dim"])
    if kind == "avgpool":
        return O.avgpool_nhwc(ins[0], a["k"], a["stride"])
    if kind == "maxpool":
        return O.maxpool_nhwc(ins[0], a["k"], a["stride"])
    if kind == "lppool":
        return O.lppool_nhwc(ins[0], a["k"], a["stride"], a["p"])
    if kind == "attention":
        if a["layout"] == "bhsd":
            return O.attention_bhsd(ins[0], ins[1], ins[2])
        return O.attention_packed(ins[0], a["batch"], a["seq"], a["heads"], a["head_dim"])
    raise ValueError(f"unknown operator kind {kind!r}")


def contracts(ops, input_names, partition):
    """Per submodule: (names read from outside, names produced for outside).

    The last op's value is the module output.  Every op belongs to exactly
    one submodule (the partition is a list of first-op indices, starting at 0
    and strictly increasing)."""
    n = len(ops)
    cuts = list(partition)
    if not cuts or cuts[0] != 0 or any(b <= a for a, b in zip(cuts, cuts[1:])) or cuts[-1] >= n:
        raise ValueError("partition must start at 0 and increase strictly inside the op list")
    bounds = cuts + [n]
    out = []
    for s in range(len(cuts)):
        lo, hi = bounds[s], bounds[s + 1]
        made = {ops[i]["out"] for i in range(lo, hi)}
        reads = []
        for i in range(lo, hi):
            for name in ops[i]["in"]:
                if name not in made and name not in reads:
                    reads.append(name)
        later = set()
        for i in range(hi, n):
            later.update(ops[i]["in"])
        writes = [ops[i]["out"] for i in range(lo, hi)
                  if ops[i]["out"] in later or i == n - 1]
        out.append((reads, writes))
    return out


def run_module(ops, inputs, params, partition=None):
    """Evaluate the module.  Returns (output, boundary) where `boundary` maps
    each submodule-boundary value name to its fp64 tensor (with the per-op
    partition that is every intermediate)."""
    if partition is None:
        partition = list(range(len(ops)))
    cons = contracts(ops, list(inputs), partition)
    bounds = list(partition) + [len(ops)]
    outer = dict(inputs)          # what the top-level module holds
    boundary = {}
    for s, (reads, writes) in enumerate(cons):
        local = {name: outer[name] for name in reads}   # contract inputs only
        for i in range(bounds[s], bounds[s + 1]):
            local[ops[i]["out"]] = apply_op(ops[i], local, params)
        for name in writes:
            outer[name] = local[name]
            boundary[name] = local[name]
    return outer[ops[-1]["out"]], boundary


def run_workload(w, partition=None):
    """Widen a workload's stored tensors to fp64 and evaluate it."""
    inputs = {k: t.f64() for k, t in w.inputs.items()}
    params = {k: t.f64() for k, t in w.params.items()}
    return run_module(w.ops, inputs, params, partition)
