"""ctypes front end of ``hgemm_oracle.c`` -- TEST INFRASTRUCTURE, not product code.

The arithmetic lives in the C file; this module only compiles it with gcc, loads
it, and marshals numpy arrays.  fp16 matrices travel as ``uint16`` bit patterns so
that no half-precision type of numpy, the compiler or CUDA takes part in the
oracle's arithmetic (paper section 2.3, Eq. 1: a CPU reference on widened inputs;
here widened to fp64).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hgemm_oracle.c")
_LIB = os.path.join(_HERE, "libhgemm_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over rows only). Returns the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_f16_bits_to_f64.restype = ctypes.c_double
        lib.oracle_f16_bits_to_f64.argtypes = [ctypes.c_uint16]
        lib.oracle_f64_to_f16_bits_rne.restype = ctypes.c_uint16
        lib.oracle_f64_to_f16_bits_rne.argtypes = [ctypes.c_double]
        lib.oracle_f64_to_f16_bits_rne_array.restype = None
        lib.oracle_f64_to_f16_bits_rne_array.argtypes = [i64, p, p]
        lib.oracle_f16_bits_to_f64_array.restype = None
        lib.oracle_f16_bits_to_f64_array.argtypes = [i64, p, p]
        lib.oracle_hgemm_full.restype = ctypes.c_int
        lib.oracle_hgemm_full.argtypes = [i64, i64, i64, p, i64, p, i64, p]
        lib.oracle_hgemm_sampled.restype = ctypes.c_int
        lib.oracle_hgemm_sampled.argtypes = [i64, p, i64, p, i64, i64, p, p, p]
        lib.oracle_max_threads.restype = ctypes.c_int
        lib.oracle_max_threads.argtypes = []
        _lib = lib
    return _lib


def _bits(x: np.ndarray) -> np.ndarray:
    """Accept uint16 bit patterns (or a float16 array, reinterpreted) as C-contiguous uint16."""
    x = np.asarray(x)
    if x.dtype == np.float16:
        x = x.view(np.uint16)
    if x.dtype != np.uint16:
        raise TypeError(f"fp16 matrices are passed as uint16 bit patterns, got {x.dtype}")
    return np.ascontiguousarray(x)


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def f16_bits_to_f64(bits) -> np.ndarray:
    b = _bits(np.atleast_1d(bits))
    out = np.empty(b.shape, dtype=np.float64)
    _load().oracle_f16_bits_to_f64_array(b.size, b.ctypes.data, out.ctypes.data)
    return out


def f64_to_f16_bits(x) -> np.ndarray:
    v = np.ascontiguousarray(np.atleast_1d(x), dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    _load().oracle_f64_to_f16_bits_rne_array(v.size, v.ctypes.data, out.ctypes.data)
    return out


def hgemm_full(a_bits, b_bits) -> np.ndarray:
    """C_ref (fp64, M x N) for A (M x K) and B (N x K), both as fp16 bit patterns."""
    a, b = _bits(a_bits), _bits(b_bits)
    if a.ndim != 2 or b.ndim != 2 or a.shape[1] != b.shape[1]:
        raise ValueError(f"need A (M,K) and B (N,K); got {a.shape} and {b.shape}")
    m, k = a.shape
    n = b.shape[0]
    c = np.empty((m, n), dtype=np.float64)
    _load().oracle_hgemm_full(m, n, k, a.ctypes.data, k, b.ctypes.data, k, c.ctypes.data)
    return c


def hgemm_sampled(a_bits, b_bits, ii, jj) -> np.ndarray:
    """C_ref[ii[t], jj[t]] (fp64) -- ii indexes rows of ``a_bits``, jj rows of ``b_bits``."""
    a, b = _bits(a_bits), _bits(b_bits)
    if a.ndim != 2 or b.ndim != 2 or a.shape[1] != b.shape[1]:
        raise ValueError(f"need A (*,K) and B (*,K); got {a.shape} and {b.shape}")
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    if ii.shape != jj.shape or ii.ndim != 1:
        raise ValueError("ii and jj must be 1-D and of equal length")
    if ii.size and (ii.min() < 0 or ii.max() >= a.shape[0] or jj.min() < 0 or jj.max() >= b.shape[0]):
        raise IndexError("sample index out of range")
    out = np.empty(ii.shape, dtype=np.float64)
    _load().oracle_hgemm_sampled(a.shape[1], a.ctypes.data, a.shape[1], b.ctypes.data, b.shape[1],
                                 ii.size, ii.ctypes.data, jj.ctypes.data, out.ctypes.data)
    return out


def hgemm_scaled_full(a_bits, b_bits, c_bits, alpha: float, beta: float) -> np.ndarray:
    """alpha * A B^T + beta * C (fp64, M x N): the general form of the operation (paper section 2.1).

    ``alpha`` and ``beta`` are taken as the fp32 values the library receives (both are exact in
    fp64).  With ``beta == 0`` the old C does not enter the result at all, whatever it holds
    (the BLAS convention the library follows).
    """
    ab = hgemm_full(a_bits, b_bits)
    al = float(np.float32(alpha))
    be = float(np.float32(beta))
    if be == 0.0:
        return al * ab
    c = _bits(c_bits)
    if c.shape != ab.shape:
        raise ValueError(f"need C {ab.shape}, got {c.shape}")
    return al * ab + be * f16_bits_to_f64(c)


def hgemm_f16acc_full(a_bits, b_bits, k_step: int = 16) -> np.ndarray:
    """A MODEL of fp16 accumulation, as fp16 bit patterns (M x N) -- a diagnostic, not an acceptance rule.

    The paper names fp16 accumulators as the other valid setting for fp16 inputs (section 1) but
    does not say where such a kernel rounds.  This function writes out one plausible schedule: the K
    dimension is consumed in steps of ``k_step`` = 16 (one MMA instruction); within a step the 16
    products and their sum are exact, and the running sum is rounded to fp16 (round to nearest even)
    once per step:  D <- RN16(D + sum_{k in step} a_k b_k),  D_0 = 0.
    No test passes or fails on it: the GPU tests only REPORT which fraction of a result equals this
    model.  What they assert is what the paper and the arithmetic fix: bit equality where every
    partial sum is representable (section 2.3, "Exact Match"), and ``f16acc_envelope`` below, which
    holds for every schedule that rounds at most once per step.
    """
    a, b = _bits(a_bits), _bits(b_bits)
    if a.ndim != 2 or b.ndim != 2 or a.shape[1] != b.shape[1]:
        raise ValueError(f"need A (M,K) and B (N,K); got {a.shape} and {b.shape}")
    m, k = a.shape
    n = b.shape[0]
    d = np.zeros((m, n), dtype=np.float64)
    for k0 in range(0, k, k_step):
        # 16 products of 11-bit significands and their sum fit fp64 exactly: the plain routine's result is exact
        part = hgemm_full(np.ascontiguousarray(a[:, k0:k0 + k_step]), np.ascontiguousarray(b[:, k0:k0 + k_step]))
        d = f16_bits_to_f64(f64_to_f16_bits((d + part).ravel())).reshape(m, n)
    return f64_to_f16_bits(d.ravel()).reshape(m, n)


def f16_spacing(x) -> np.ndarray:
    """Distance between adjacent fp16 values at magnitude |x|: 2^(floor(log2 |x|) - 10), and 2^-24
    (the subnormal spacing) below the smallest normal 2^-14.  IEEE 754 binary16, 11-bit significand."""
    ax = np.maximum(np.abs(np.asarray(x, dtype=np.float64)), 2.0 ** -14)
    return np.exp2(np.floor(np.log2(ax)) - 10.0)


def f16acc_envelope(a_bits, b_bits, k_step: int = 16):
    """Error envelope of fp16 accumulation that holds for ANY rounding schedule (paper section 1 allows
    fp16 accumulators; section 2.3 bounds the deviation of a kernel from the exact product).

    Returns ``(c_exact, bound)``, both fp64 M x N.  Assumption, and nothing more: the running sum is
    replaced at most once per ``k_step`` columns of K (one MMA instruction consumes 16) by one of the
    two fp16 values that enclose its exact value ("faithful" rounding: to nearest, towards zero, or a
    double rounding all qualify), the products entering a step being summed without further error.
    With P_t the exact prefix sum after step t and E_t a bound on |D_t - P_t|:

        E_0 = 0,    E_t = E_(t-1) + spacing16(|P_t| + E_(t-1))

    because the value being rounded at step t is x = P_t + (D_(t-1) - P_(t-1)), of magnitude at most
    |P_t| + E_(t-1); the two fp16 values that enclose x are one spacing16(|x|) apart, the spacing
    never decreases with the magnitude, so a faithful rounding moves x by less than
    spacing16(|P_t| + E_(t-1)).  A schedule that rounds less often (every 32 columns, or once at the
    end) stays inside the same envelope: every term is non-negative and grows with the running error.
    ``bound`` is E after the last step.  (The prefix sums are fp64 sums of exact step sums: their own
    rounding, below 2^-52 relative, is ten orders of magnitude under one fp16 spacing.)
    """
    a, b = _bits(a_bits), _bits(b_bits)
    if a.ndim != 2 or b.ndim != 2 or a.shape[1] != b.shape[1]:
        raise ValueError(f"need A (M,K) and B (N,K); got {a.shape} and {b.shape}")
    m, k = a.shape
    n = b.shape[0]
    prefix = np.zeros((m, n), dtype=np.float64)
    err = np.zeros((m, n), dtype=np.float64)
    for k0 in range(0, k, k_step):
        prefix = prefix + hgemm_full(np.ascontiguousarray(a[:, k0:k0 + k_step]), np.ascontiguousarray(b[:, k0:k0 + k_step]))
        err = err + f16_spacing(np.abs(prefix) + err)
    return prefix, err
