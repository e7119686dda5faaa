"""Helpers shared by the GPU parity tests: tolerances, oracle-side copies, device upload.

Tolerances (stated once, used everywhere): hidden states and logits agree with the oracle
within max |diff| <= 2e-2 and max |diff| / max |oracle| <= 1e-2 (bf16 weights, fp32
accumulation against a float64 oracle); token ids and accepted lengths are bit-exact except
where the oracle's two best logits are closer than 1e-2, in which case the oracle adopts the
kernel's token and continues (teacher forcing), so one near tie cannot hide later errors.
"""
import copy

import numpy as np

ABS_TOL = 2e-2
REL_TOL = 1e-2
GAP_TOL = 1e-2


def copy_kv(kv):
    return {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in kv.items()}


def close(got, ref, what=""):
    """Assert the two-part tolerance; returns (max abs diff, relative diff)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.all(np.isfinite(got)), what + ": non-finite values"
    diff = float(np.max(np.abs(got - ref))) if got.size else 0.0
    scale = float(np.max(np.abs(ref))) if ref.size else 1.0
    rel = diff / scale if scale > 0 else diff
    assert diff <= ABS_TOL, f"{what}: max abs diff {diff:.3e} > {ABS_TOL}"
    assert rel <= REL_TOL, f"{what}: relative diff {rel:.3e} > {REL_TOL}"
    return diff, rel


def ids_match(got, ref, gap, what=""):
    """Token ids equal except where the oracle's top-2 gap is below GAP_TOL. Returns the
    number of exempt positions."""
    got = np.asarray(got).ravel()
    ref = np.asarray(ref).ravel()
    gap = np.asarray(gap).ravel()
    bad = (got != ref) & ~(gap < GAP_TOL)
    assert not bad.any(), f"{what}: {int(bad.sum())} token mismatches outside near ties at {np.nonzero(bad)[0][:8]}"
    return int(((got != ref) & (gap < GAP_TOL)).sum())


def deep(x):
    return copy.deepcopy(x)
