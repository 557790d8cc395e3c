"""Comparison gates shared by the parity tests (host arithmetic only, no kernels, no oracle)."""
from __future__ import annotations

import numpy as np

# bf16 inputs / fp32 accumulation / bf16 output, and the fp32 path.
GATES = {
    "bf16": dict(max_abs=2e-2, mean_abs=2e-3, rel_l2=2e-2, lse_abs=1e-3),
    "f32": dict(max_abs=1e-4, mean_abs=1e-5, rel_l2=1e-4, lse_abs=1e-4),
}


def errors(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    diff = np.abs(got - ref)
    denom = float(np.sqrt((ref ** 2).sum()))
    return dict(max_abs=float(diff.max()) if diff.size else 0.0,
                mean_abs=float(diff.mean()) if diff.size else 0.0,
                rel_l2=float(np.sqrt((diff ** 2).sum()) / denom) if denom > 0 else 0.0)


def check(got_out, got_lse, ref_out, ref_lse, kind: str, what: str = ""):
    """Raise AssertionError unless out and lse are inside the gates for ``kind``.

    The absolute gates are the stated ones (bf16: 2e-2 max, 2e-3 mean; fp32: 1e-4); the relative-L2 gate is added
    because with near-uniform softmax the outputs themselves are smaller than the
    absolute gate (an all-zero output would pass it).
    """
    g = GATES[kind]
    got_out = np.asarray(got_out, dtype=np.float64)
    if not np.isfinite(got_out).all():
        raise AssertionError(f"{what}: non-finite output")
    e = errors(got_out, ref_out)
    assert e["max_abs"] <= g["max_abs"], f"{what}: max|err| {e['max_abs']:.3e} > {g['max_abs']}"
    assert e["mean_abs"] <= g["mean_abs"], f"{what}: mean|err| {e['mean_abs']:.3e} > {g['mean_abs']}"
    assert e["rel_l2"] <= g["rel_l2"], f"{what}: rel L2 {e['rel_l2']:.3e} > {g['rel_l2']}"
    if got_lse is not None:
        le = float(np.abs(np.asarray(got_lse, dtype=np.float64) - np.asarray(ref_lse, dtype=np.float64)).max())
        assert le <= g["lse_abs"], f"{what}: lse max|err| {le:.3e} > {g['lse_abs']}"
    return e
