"""Acceptance predicate of the parity tests.  TEST INFRASTRUCTURE ONLY.

Element-wise |out - ref| <= atol + rtol * |ref|, every element must pass and
any NaN/Inf fails (paper, appendix "Modular Kernel Generation Enables Better
Correctness Checking", the allclose criterion).  Tolerances: fp32 rtol 1e-4 /
atol 1e-5, bf16 rtol 2e-2 / atol 2e-2.
"""
from __future__ import annotations

import numpy as np

TOL = {"f32": (1e-4, 1e-5), "bf16": (2e-2, 2e-2)}


def check_close(out, ref, dtype=None, rtol=None, atol=None):
    """Return a dict: ok, n_bad, max_abs, max_rel_excess, worst index."""
    if rtol is None or atol is None:
        rtol, atol = TOL[dtype]
    out = np.asarray(out, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if out.shape != ref.shape:
        return {"ok": False, "why": f"shape {out.shape} vs {ref.shape}", "n_bad": out.size,
                "max_abs": float("inf")}
    finite = np.isfinite(out)
    err = np.abs(out - ref)
    bound = atol + rtol * np.abs(ref)
    bad = ~finite | ~(err <= bound)
    n_bad = int(bad.sum())
    res = {"ok": n_bad == 0, "n_bad": n_bad, "size": int(out.size),
           "max_abs": float(np.nanmax(np.where(finite, err, np.nan))) if finite.any() else float("inf"),
           "rtol": rtol, "atol": atol}
    if n_bad:
        idx = np.unravel_index(int(np.argmax(np.where(bad, np.where(finite, err, np.inf), -1.0))), out.shape)
        res["worst"] = (tuple(int(i) for i in idx), float(out[idx]), float(ref[idx]))
    return res
