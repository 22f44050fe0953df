"""CPU oracle for per-example gradient statistics (fp64, one example at a time).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline
leg call this; the product never does.  The arithmetic lives in ``pe_oracle.c`` (plain C,
fp64); this module compiles it with gcc on first use and wraps it with numpy arrays.
It imports nothing from the CUDA package.

Array conventions: ``X`` is ``[B, T, d_in]`` and ``dY`` is ``[B, T, d_out]``, either
``float32`` or ``uint16`` holding bf16 bit patterns; results are ``[d_out, d_in]`` float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pe_oracle.c")
_LIB = os.path.join(_HERE, "libpe_oracle.so")
_lib = None

c_double_p = ctypes.POINTER(ctypes.c_double)
c_int32_p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the C oracle next to its source (gcc -O2 -fopenmp). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_linear_stats.restype = ctypes.c_int
        lib.oracle_linear_stats.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int, ctypes.c_double, c_double_p, c_double_p, c_double_p, c_double_p, c_int32_p,
        ]
        lib.oracle_token_sqstats.restype = ctypes.c_int
        lib.oracle_token_sqstats.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int, c_double_p,
        ]
        lib.oracle_example_sqnorms.restype = ctypes.c_int
        lib.oracle_example_sqnorms.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int, c_double_p,
        ]
        lib.oracle_microadam_step.restype = ctypes.c_int
        lib.oracle_microadam_step.argtypes = [
            c_double_p, c_double_p, c_double_p, c_double_p, c_double_p, ctypes.c_longlong, ctypes.c_int,
            ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double,
            ctypes.c_int, ctypes.c_double, ctypes.c_int,
        ]
        lib.oracle_adam_family_step.restype = ctypes.c_int
        lib.oracle_adam_family_step.argtypes = [
            c_double_p, c_double_p, c_double_p, c_double_p, c_double_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_int,
            ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double,
            ctypes.c_int, ctypes.c_double, ctypes.c_int,
        ]
        lib.oracle_microsignsgd_step.restype = ctypes.c_int
        lib.oracle_microsignsgd_step.argtypes = [
            c_double_p, c_double_p, c_double_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_double,
            ctypes.c_double, ctypes.c_double,
        ]
        lib.oracle_linear_stats_ragged.restype = ctypes.c_int
        lib.oracle_linear_stats_ragged.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_longlong), ctypes.c_int,
            ctypes.c_int, ctypes.c_double, c_double_p, c_double_p, c_double_p, c_double_p, c_int32_p, c_double_p,
        ]
        lib.oracle_clipped_sum.restype = ctypes.c_int
        lib.oracle_clipped_sum.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_double, c_double_p, c_double_p, c_double_p,
        ]
        lib.oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's loops use on this machine."""
    return int(_load().oracle_num_threads())


def _dp(a):
    return None if a is None else a.ctypes.data_as(c_double_p)


def _check_inputs(X: np.ndarray, dY: np.ndarray):
    if X.dtype != dY.dtype or X.dtype not in (np.float32, np.uint16):
        raise TypeError("X and dY must both be float32, or both uint16 (bf16 bit patterns)")
    if X.ndim != 3 or dY.ndim != 3 or X.shape[:2] != dY.shape[:2]:
        raise ValueError("X must be [B,T,d_in] and dY [B,T,d_out] with the same B and T")
    X = np.ascontiguousarray(X)
    dY = np.ascontiguousarray(dY)
    B, T, d_in = X.shape
    d_out = dY.shape[2]
    return X, dY, int(X.dtype == np.uint16), B, T, d_in, d_out


@dataclass
class LinearStats:
    """Outputs of :func:`linear_stats` (all float64 except ``n_small``)."""
    sum_g: np.ndarray      # [d_out, d_in]  sum_b G_b
    sum_g2: np.ndarray     # [d_out, d_in]  sum_b G_b^2
    sum_sign: np.ndarray   # [d_out, d_in]  sum_b sign(G_b)
    max_abs: np.ndarray    # [B]            max |G_b|
    n_small: np.ndarray    # [d_out, d_in]  int32, #b with |G_b[o,i]| <= small_rel * max|G_b|


def linear_stats(X: np.ndarray, dY: np.ndarray, small_rel: float = 1e-3) -> LinearStats:
    """Sequence-level per-example statistics, Section 2.3 / Eq. (2): G_b = dY_b^T X_b per example,
    then sum_b of G_b, G_b^2 and sign(G_b)."""
    X, dY, is_bf16, B, T, d_in, d_out = _check_inputs(X, dY)
    sg = np.empty((d_out, d_in), np.float64)
    sg2 = np.empty((d_out, d_in), np.float64)
    ss = np.empty((d_out, d_in), np.float64)
    mx = np.zeros((max(B, 1),), np.float64)
    ns = np.empty((d_out, d_in), np.int32)
    rc = _load().oracle_linear_stats(
        X.ctypes.data, dY.ctypes.data, is_bf16, B, T, d_in, d_out, float(small_rel),
        _dp(sg), _dp(sg2), _dp(ss), _dp(mx), ns.ctypes.data_as(c_int32_p))
    if rc != 0:
        raise RuntimeError("oracle_linear_stats failed")
    return LinearStats(sg, sg2, ss, mx[:B], ns)


def token_sqstats(X: np.ndarray, dY: np.ndarray) -> np.ndarray:
    """Per-token second moment S' = sum_{b,t} dy^2 x^2 (Section 2.3)."""
    X, dY, is_bf16, B, T, d_in, d_out = _check_inputs(X, dY)
    out = np.empty((d_out, d_in), np.float64)
    rc = _load().oracle_token_sqstats(X.ctypes.data, dY.ctypes.data, is_bf16, B, T, d_in, d_out, _dp(out))
    if rc != 0:
        raise RuntimeError("oracle_token_sqstats failed")
    return out


def example_sqnorms(X: np.ndarray, dY: np.ndarray) -> np.ndarray:
    """Per-example squared gradient norms N_b = ||dY_b^T X_b||_F^2 (Section 2.3), shape [B]."""
    X, dY, is_bf16, B, T, d_in, d_out = _check_inputs(X, dY)
    out = np.zeros((B,), np.float64)
    rc = _load().oracle_example_sqnorms(X.ctypes.data, dY.ctypes.data, is_bf16, B, T, d_in, d_out, _dp(out))
    if rc != 0:
        raise RuntimeError("oracle_example_sqnorms failed")
    return out


@dataclass
class RaggedStats(LinearStats):
    """Outputs of :func:`linear_stats_ragged`: those of :class:`LinearStats` plus ``sq_norms`` [B]."""
    sq_norms: np.ndarray = None


def linear_stats_ragged(X: np.ndarray, dY: np.ndarray, offsets, small_rel: float = 1e-3) -> RaggedStats:
    """Per-example statistics of a packed batch (Section 2.3; Eq. (2)): X [rows, d_in], dY [rows, d_out],
    example b owns rows offsets[b] .. offsets[b+1]-1 and its gradient is contracted over those rows only."""
    if X.dtype != dY.dtype or X.dtype not in (np.float32, np.uint16):
        raise TypeError("X and dY must both be float32, or both uint16 (bf16 bit patterns)")
    if X.ndim != 2 or dY.ndim != 2 or X.shape[0] != dY.shape[0]:
        raise ValueError("X must be [rows, d_in] and dY [rows, d_out] with the same row count")
    offs = np.ascontiguousarray(np.asarray(offsets, np.int64))
    if offs.ndim != 1 or offs.size < 1 or (offs.size > 1 and offs[-1] > X.shape[0]):
        raise ValueError("offsets must be [B+1] and end within the rows")
    B = offs.size - 1
    X = np.ascontiguousarray(X)
    dY = np.ascontiguousarray(dY)
    d_in, d_out = X.shape[1], dY.shape[1]
    sg = np.empty((d_out, d_in), np.float64)
    sg2 = np.empty((d_out, d_in), np.float64)
    ss = np.empty((d_out, d_in), np.float64)
    mx = np.zeros((max(B, 1),), np.float64)
    nr = np.zeros((max(B, 1),), np.float64)
    ns = np.empty((d_out, d_in), np.int32)
    rc = _load().oracle_linear_stats_ragged(
        X.ctypes.data, dY.ctypes.data, int(X.dtype == np.uint16), B, offs.ctypes.data_as(ctypes.POINTER(ctypes.c_longlong)),
        d_in, d_out, float(small_rel), _dp(sg), _dp(sg2), _dp(ss), _dp(mx), ns.ctypes.data_as(c_int32_p), _dp(nr))
    if rc != 0:
        raise RuntimeError("oracle_linear_stats_ragged failed")
    return RaggedStats(sg, sg2, ss, mx[:B], ns, nr[:B])


def clipped_sum(X: np.ndarray, dY: np.ndarray, clip_norm: float, sq_norms=None):
    """Sum over examples of the norm-clipped per-example gradients, c_b = min(1, C / sqrt(N_b)) (Section 2.1's
    clipping statistic with Section 2.3's squared norms N_b).  sq_norms: optional [B] squared norms to clip
    by (default: this layer's own).  Returns (sum [d_out, d_in], coefficients [B])."""
    X, dY, is_bf16, B, T, d_in, d_out = _check_inputs(X, dY)
    out = np.empty((d_out, d_in), np.float64)
    coef = np.zeros((max(B, 1),), np.float64)
    nin = None
    if sq_norms is not None:
        nin = np.ascontiguousarray(np.asarray(sq_norms, np.float64))
        if nin.shape != (B,):
            raise ValueError("sq_norms must be [B]")
    rc = _load().oracle_clipped_sum(X.ctypes.data, dY.ctypes.data, is_bf16, B, T, d_in, d_out, float(clip_norm),
                                    _dp(nin), _dp(out), _dp(coef))
    if rc != 0:
        raise RuntimeError("oracle_clipped_sum failed")
    return out, coef[:B]


def microadam_step(theta, m, v, sum_g, sum_g2, B, *, grad_scale=1.0, lr, beta1, beta2, eps,
                   eps_inside_sqrt=False, weight_decay=0.0, step=1):
    """One MicroAdam step (Algorithm 1, MicroAdam branch) in fp64. Returns new (theta, m, v)."""
    th = np.array(theta, np.float64).ravel().copy()
    mm = np.array(m, np.float64).ravel().copy()
    vv = np.array(v, np.float64).ravel().copy()
    g = np.ascontiguousarray(np.asarray(sum_g, np.float64).ravel())
    g2 = np.ascontiguousarray(np.asarray(sum_g2, np.float64).ravel())
    n = th.size
    if not (mm.size == vv.size == g.size == g2.size == n):
        raise ValueError("size mismatch")
    rc = _load().oracle_microadam_step(_dp(th), _dp(mm), _dp(vv), _dp(g), _dp(g2), n, int(B),
                                       float(grad_scale), float(lr), float(beta1), float(beta2),
                                       float(eps), int(bool(eps_inside_sqrt)), float(weight_decay), int(step))
    if rc != 0:
        raise RuntimeError("oracle_microadam_step failed")
    shp = np.shape(theta)
    return th.reshape(shp), mm.reshape(shp), vv.reshape(shp)


ADAM_VARIANTS = {"adam": 0, "microadam": 1, "microadam_var": 2, "microadam_msq": 3}


def adam_family_step(theta, m, v, sum_g, sum_g2, B, variant, *, grad_scale=1.0, lr, beta1, beta2, eps,
                     eps_inside_sqrt=False, weight_decay=0.0, step=1):
    """One step of a member of the extended Adam family (Section 3.2.3; Algorithm 1 with the estimators of
    Eq. (6)) in fp64.  variant: "adam", "microadam", "microadam_var", "microadam_msq".  Returns new (theta, m, v)."""
    th = np.array(theta, np.float64).ravel().copy()
    mm = np.array(m, np.float64).ravel().copy()
    vv = np.array(v, np.float64).ravel().copy()
    g = np.ascontiguousarray(np.asarray(sum_g, np.float64).ravel())
    g2 = np.ascontiguousarray(np.asarray(sum_g2, np.float64).ravel())
    n = th.size
    if not (mm.size == vv.size == g.size == g2.size == n):
        raise ValueError("size mismatch")
    rc = _load().oracle_adam_family_step(_dp(th), _dp(mm), _dp(vv), _dp(g), _dp(g2), n, int(B), ADAM_VARIANTS[variant],
                                         float(grad_scale), float(lr), float(beta1), float(beta2),
                                         float(eps), int(bool(eps_inside_sqrt)), float(weight_decay), int(step))
    if rc != 0:
        raise RuntimeError("oracle_adam_family_step failed")
    shp = np.shape(theta)
    return th.reshape(shp), mm.reshape(shp), vv.reshape(shp)


def microsignsgd_step(theta, m, sum_sign, B, *, lr, beta, weight_decay=0.0):
    """One MicroSignSGD step (Section 3.1: EMA of the batch mean of per-example signs) in fp64."""
    th = np.array(theta, np.float64).ravel().copy()
    mm = np.array(m, np.float64).ravel().copy()
    s = np.ascontiguousarray(np.asarray(sum_sign, np.float64).ravel())
    n = th.size
    if not (mm.size == s.size == n):
        raise ValueError("size mismatch")
    rc = _load().oracle_microsignsgd_step(_dp(th), _dp(mm), _dp(s), n, int(B), float(lr), float(beta),
                                          float(weight_decay))
    if rc != 0:
        raise RuntimeError("oracle_microsignsgd_step failed")
    shp = np.shape(theta)
    return th.reshape(shp), mm.reshape(shp)
