"""Acceptance rules for comparing a GPU result with the oracle -- TEST INFRASTRUCTURE.

The paper accepts a kernel on two criteria (section 2.3, "Correctness"): exact
equality on inputs whose sums are exactly representable, and a bounded deviation
from a CPU reference on random inputs.  This module states both in the form this
library is held to:

* exact cases: the fp16 bit patterns must be equal after mapping -0 to +0
  (a sum of signed zeros has no single correct sign; NaN is never accepted);
* random inputs: ``|C - C_ref| <= 2^-10 * |C_ref| + 1e-3 * sqrt(K)`` elementwise,
  C widened to fp64, C_ref the unrounded fp64 oracle value.

The random-input bound is loose when the entries of C are small (an all-zero C
would pass for N(0,1)/sqrt(K) inputs), so two scale-aware checks are asserted
beside it: a relative Frobenius error of at most 2^-11 and an elementwise bound
whose absolute term follows the row norms,
``2^-10 |C_ref| + sqrt(K) 2^-24 ||A_i|| ||B_j|| + 2^-25``
(fp16 output rounding + fp32 accumulation of K products + subnormal output spacing).
"""
from __future__ import annotations

import numpy as np

REL_TERM = 2.0 ** -10
ABS_COEF = 1e-3
FROBENIUS_LIMIT = 2.0 ** -11


def contract_bound(c_ref: np.ndarray, k: int, abs_scale: float = 1.0) -> np.ndarray:
    """``abs_scale`` scales the absolute term: |alpha| for C = alpha A B^T + beta C, whose accumulation
    error is alpha times that of A B^T (the beta C term is exact in fp32 and adds one rounding, which
    the relative term covers).  For the scaled form 2^-24, half the spacing of fp16 subnormals, is added so
    that alpha = 0 leaves a positive bound; the plain product keeps the contract's bound unchanged."""
    if abs_scale == 1.0:
        return REL_TERM * np.abs(c_ref) + ABS_COEF * np.sqrt(float(k))
    return REL_TERM * np.abs(c_ref) + ABS_COEF * np.sqrt(float(k)) * abs(float(abs_scale)) + 2.0 ** -24


def check_contract(c_gpu_f64: np.ndarray, c_ref: np.ndarray, k: int, abs_scale: float = 1.0) -> dict:
    """Elementwise contract check. Returns a report; ``ok`` is the verdict."""
    c_gpu_f64 = np.asarray(c_gpu_f64, dtype=np.float64)
    c_ref = np.asarray(c_ref, dtype=np.float64)
    if c_gpu_f64.shape != c_ref.shape:
        raise ValueError(f"shape mismatch {c_gpu_f64.shape} vs {c_ref.shape}")
    finite = np.isfinite(c_gpu_f64)
    err = np.abs(c_gpu_f64 - c_ref)
    bound = contract_bound(c_ref, k, abs_scale)
    bad = (~finite) | (err > bound)
    ratio = np.where(finite, err / bound, np.inf)
    return {
        "ok": not bool(bad.any()),
        "n": int(c_ref.size),
        "n_bad": int(bad.sum()),
        "max_err": float(err[finite].max()) if finite.any() else float("inf"),
        "max_err_over_bound": float(ratio.max()) if ratio.size else 0.0,
        "first_bad": (tuple(int(v) for v in np.argwhere(bad)[0]) if bad.any() else None),
    }


def check_scale_aware(c_gpu_f64, c_ref, k: int, a_row_norms=None, b_row_norms=None) -> dict:
    """Relative Frobenius error, and (when row norms are given) the norm-scaled elementwise bound.

    ``a_row_norms[i]`` / ``b_row_norms[j]`` are the 2-norms of the A and B rows that
    produced ``c_ref[i, j]`` (for 1-D sampled results: one norm per sample).
    """
    c_gpu_f64 = np.asarray(c_gpu_f64, dtype=np.float64)
    c_ref = np.asarray(c_ref, dtype=np.float64)
    diff = c_gpu_f64 - c_ref
    denom = float(np.sqrt(np.sum(c_ref * c_ref)))
    rel_f = float(np.sqrt(np.sum(diff * diff))) / denom if denom > 0 else float(np.abs(diff).max(initial=0.0))
    rep = {"rel_frobenius": rel_f, "ok": bool(rel_f <= FROBENIUS_LIMIT), "max_err_over_norm_bound": None}
    if a_row_norms is not None and b_row_norms is not None:
        an = np.asarray(a_row_norms, dtype=np.float64)
        bn = np.asarray(b_row_norms, dtype=np.float64)
        scale = np.outer(an, bn) if c_ref.ndim == 2 else an * bn
        bound = REL_TERM * np.abs(c_ref) + np.sqrt(float(k)) * 2.0 ** -24 * scale + 2.0 ** -25
        r = np.abs(diff) / bound
        rep["max_err_over_norm_bound"] = float(r.max()) if r.size else 0.0
        rep["ok"] = rep["ok"] and bool((r <= 1.0).all())
    return rep


def canonical_bits(bits: np.ndarray) -> np.ndarray:
    """fp16 bit patterns with -0 mapped to +0 (the form exact cases are compared in)."""
    b = np.asarray(bits).view(np.uint16).copy()
    b[b == 0x8000] = 0
    return b
