"""ctypes front-end of the float64 CPU oracle (``gbs_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle restates, by the definition and in double
precision, what the rotate-and-quantize path of arXiv 2504.13989 computes
(Section 2.1 quantizer, Section 3.1 clip ratio, Eq. (1) Sylvester recursion,
Algorithm 2 Paley construction, Section 4.2 zero-pad expansion).  It shares no
code with the CUDA library and must never be imported by the product package;
only the tests, the smoke check and the CPU-baseline / reference leg of the
benchmark use it.

The shared object is compiled on first use with gcc (``build()``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gbs_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libgbs_oracle.so")
_lib = None

F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile gbs_oracle.c into libgbs_oracle.so next to it (gcc, OpenMP)."""
    stale = (not os.path.exists(_LIB_PATH)
             or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC))
    if force or stale:
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared",
                               _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_dp = ctypes.POINTER(ctypes.c_double)
        lib.oracle_legendre.argtypes = [ctypes.c_long, ctypes.c_int]
        lib.oracle_legendre.restype = ctypes.c_int
        lib.oracle_gf27_chi.argtypes = [ctypes.c_int]
        lib.oracle_gf27_chi.restype = ctypes.c_int
        lib.oracle_gf27_mul.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.oracle_gf27_mul.restype = ctypes.c_int
        lib.oracle_gf27_sub.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.oracle_gf27_sub.restype = ctypes.c_int
        lib.oracle_hadamard_m.argtypes = [ctypes.c_int, ctypes.c_void_p]
        lib.oracle_hadamard_m.restype = ctypes.c_int
        lib.oracle_sylvester.argtypes = [ctypes.c_int, ctypes.c_void_p]
        lib.oracle_sylvester.restype = ctypes.c_int
        lib.oracle_rotate_dense.argtypes = [c_dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_int, c_dp]
        lib.oracle_rotate_dense.restype = ctypes.c_int
        lib.oracle_rotate_fast.argtypes = lib.oracle_rotate_dense.argtypes
        lib.oracle_rotate_fast.restype = ctypes.c_int
        lib.oracle_levels.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.oracle_levels.restype = ctypes.c_int
        lib.oracle_quantize.argtypes = [c_dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_double, ctypes.c_int, ctypes.c_void_p, c_dp]
        lib.oracle_quantize.restype = ctypes.c_int
        lib.oracle_clip_error.argtypes = [c_dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_double, ctypes.c_int]
        lib.oracle_clip_error.restype = ctypes.c_double
        lib.oracle_pack.argtypes = [ctypes.c_void_p, ctypes.c_long, ctypes.c_int, ctypes.c_void_p]
        lib.oracle_pack.restype = None
        lib.oracle_unpack.argtypes = [ctypes.c_void_p, ctypes.c_long, ctypes.c_int, ctypes.c_void_p]
        lib.oracle_unpack.restype = None
        lib.oracle_rotate_quantize_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_long, ctypes.c_long,
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
            ctypes.c_int, ctypes.c_int,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        lib.oracle_rotate_quantize_rows.restype = ctypes.c_int
        lib.oracle_clip_error_rows.argtypes = [
            ctypes.c_void_p, ctypes.c_int, ctypes.c_long, ctypes.c_long,
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            c_dp, ctypes.c_int, c_dp, ctypes.c_void_p, ctypes.c_int]
        lib.oracle_clip_error_rows.restype = ctypes.c_int
        lib.oracle_dequantize_rows.argtypes = [
            ctypes.c_void_p, c_dp, ctypes.c_long,
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            c_dp, ctypes.c_int]
        lib.oracle_dequantize_rows.restype = ctypes.c_int
        lib.oracle_max_threads.argtypes = []
        lib.oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _dp(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError("oracle: %s failed (rc=%d: %s)" %
                         (what, rc, "bad arguments" if rc == -1 else "out of memory"))


def max_threads() -> int:
    return _load().oracle_max_threads()


def legendre(a: int, p: int) -> int:
    """Legendre symbol (a/p) by exhaustive squaring (Section 2.3.3)."""
    return _load().oracle_legendre(a, p)


def gf27_chi(e: int) -> int:
    return _load().oracle_gf27_chi(e)


def gf27_mul(e: int, f: int) -> int:
    return _load().oracle_gf27_mul(e, f)


def gf27_sub(e: int, f: int) -> int:
    return _load().oracle_gf27_sub(e, f)


def hadamard_m(m: int) -> np.ndarray:
    """H_m (int8, m x m): [1], Algorithm 2 for prime m-1 = 3 (mod 4), GF(27) for m = 28."""
    H = np.zeros((m, m), dtype=np.int8)
    _check(_load().oracle_hadamard_m(m, H.ctypes.data), "hadamard_m(%d)" % m)
    return H


def sylvester(n: int) -> np.ndarray:
    """H_n by the recursion of Eq. (1)."""
    H = np.zeros((n, n), dtype=np.int8)
    _check(_load().oracle_sylvester(n, H.ctypes.data), "sylvester(%d)" % n)
    return H


def hadamard_full(m: int, k: int) -> np.ndarray:
    """Dense H_m (x) H_{2^k} as int8 (small sizes only)."""
    return np.kron(hadamard_m(m).astype(np.int64), sylvester(1 << k).astype(np.int64)).astype(np.int8)


def levels(bits: int, literal: bool = False) -> int:
    return _load().oracle_levels(bits, int(literal))


def rotate(x, d_pad: int, m: int = 1, dense: bool = True, transpose: bool = False) -> np.ndarray:
    """y = H_{d'} pad(x) / sqrt(d') for one row (x: 1-D float64 of length d <= d')."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty(d_pad, dtype=np.float64)
    fn = _load().oracle_rotate_dense if dense else _load().oracle_rotate_fast
    _check(fn(_dp(x), x.shape[0], d_pad, m, int(transpose), _dp(y)), "rotate")
    return y


def quantize(y, bits: int, group: int = 0, alpha: float = 1.0, literal: bool = False):
    """Codes (int32) and scaling factors Delta (float64) of one rotated row."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    n = y.shape[0]
    q = np.empty(n, dtype=np.int32)
    delta = np.empty(n // group if group else 1, dtype=np.float64)
    _check(_load().oracle_quantize(_dp(y), n, bits, group, float(alpha), int(literal),
                                   q.ctypes.data, _dp(delta)), "quantize")
    return q, delta


def clip_error(y, bits: int, group: int = 0, alpha: float = 1.0, literal: bool = False) -> float:
    y = np.ascontiguousarray(y, dtype=np.float64)
    return float(_load().oracle_clip_error(_dp(y), y.shape[0], bits, group, float(alpha), int(literal)))


def pack(q, bits: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int32).ravel()
    out = np.zeros((q.shape[0] * bits + 7) // 8, dtype=np.uint8)
    _load().oracle_pack(q.ctypes.data, q.shape[0], bits, out.ctypes.data)
    return out


def unpack(buf, n: int, bits: int) -> np.ndarray:
    buf = np.ascontiguousarray(buf, dtype=np.uint8).ravel()
    q = np.empty(n, dtype=np.int32)
    _load().oracle_unpack(buf.ctypes.data, n, bits, q.ctypes.data)
    return q


def _as_input(x):
    """Accept a 2-D float32 array, or a 2-D uint16 array holding bf16 bit patterns."""
    x = np.asarray(x)
    if x.ndim != 2:
        raise ValueError("oracle: x must be 2-D [rows, >=d]")
    if x.dtype == np.float32:
        return np.ascontiguousarray(x), F32
    if x.dtype == np.uint16:
        return np.ascontiguousarray(x), BF16
    raise ValueError("oracle: x must be float32 or uint16 (bf16 bits), got %s" % x.dtype)


def rotate_quantize_rows(x, d: int, d_pad: int, m: int, bits: int, group: int, alpha: float,
                         literal: bool = False, dense: bool = False, want_y: bool = True,
                         want_q: bool = True, want_packed: bool = True, nthreads: int = 0):
    """Batched pad -> rotate -> quantize -> pack.

    Returns dict(y=[n,d'] f64, q=[n,d'] i32, packed=[n,d'*bits/8] u8, delta=[n,spr] f64).
    """
    x, dtype = _as_input(x)
    n, stride = x.shape
    spr = d_pad // group if group else 1
    y = np.empty((n, d_pad), dtype=np.float64) if want_y else None
    q = np.empty((n, d_pad), dtype=np.int32) if want_q else None
    packed = np.empty((n, d_pad * bits // 8), dtype=np.uint8) if want_packed else None
    delta = np.empty((n, spr), dtype=np.float64)
    rc = _load().oracle_rotate_quantize_rows(
        x.ctypes.data, dtype, n, stride, d, d_pad, m, bits, group, float(alpha),
        int(literal), int(dense),
        y.ctypes.data if want_y else None, q.ctypes.data if want_q else None,
        packed.ctypes.data if want_packed else None, delta.ctypes.data, nthreads)
    _check(rc, "rotate_quantize_rows")
    return dict(y=y, q=q, packed=packed, delta=delta)


def clip_error_rows(x, d: int, d_pad: int, m: int, bits: int, group: int, alphas,
                    literal: bool = False, want_rows: bool = False, nthreads: int = 0):
    """E_k = sum over rows and coordinates of (y - yhat_k)^2 for each alpha_k."""
    x, dtype = _as_input(x)
    n, stride = x.shape
    alphas = np.ascontiguousarray(alphas, dtype=np.float64)
    K = alphas.shape[0]
    err = np.empty(K, dtype=np.float64)
    rows = np.empty((n, K), dtype=np.float64) if want_rows else None
    rc = _load().oracle_clip_error_rows(
        x.ctypes.data, dtype, n, stride, d, d_pad, m, bits, group, int(literal),
        _dp(alphas), K, _dp(err), rows.ctypes.data if want_rows else None, nthreads)
    _check(rc, "clip_error_rows")
    return (err, rows) if want_rows else err


def dequantize_rows(packed, delta, d: int, d_pad: int, m: int, bits: int, group: int,
                    inverse: bool = False, nthreads: int = 0) -> np.ndarray:
    """yhat = q * Delta (width d'), or with inverse: xhat = (H^T yhat / sqrt(d'))[:d]."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    delta = np.ascontiguousarray(delta, dtype=np.float64)
    n = packed.shape[0]
    out = np.empty((n, d if inverse else d_pad), dtype=np.float64)
    rc = _load().oracle_dequantize_rows(packed.ctypes.data, _dp(delta), n, d, d_pad, m, bits, group,
                                        int(inverse), _dp(out), nthreads)
    _check(rc, "dequantize_rows")
    return out


def gradual_binary_search(evaluate, eps: float, trace: list | None = None):
    """Algorithm 1 (Gradual Binary Search), the loop for ONE projection, in the paper's order and notation:
    a, b, m, f_m, the probe x on the left of m on even iterations and on the right on odd ones, the four
    bracket updates, until b - a <= eps.  `evaluate(x)` is the objective (the paper uses perplexity).
    Returns (m, f_m, iterations); `trace` (optional list) receives (iteration, x, f_x, a, b, m) per pass.
    PARITY UNPINNED by the paper (it prints no trace): pinned by a hand-worked trace, by the bracket
    invariants and by convergence on convex objectives."""
    a, b = 0.0, 1.0
    m = (a + b) / 2
    f_m = evaluate(m)
    iteration = 0
    while b - a > eps:
        if iteration % 2 == 0:
            x = (a + m) / 2
        else:
            x = (b + m) / 2
        f_x = evaluate(x)
        if f_x < f_m:
            if x < m:
                b = m
            else:
                a = m
            m, f_m = x, f_x
        else:
            if x < m:
                a = x
            else:
                b = x
        iteration += 1
        if trace is not None:
            trace.append((iteration, x, f_x, a, b, m))
    return m, f_m, iteration


def search_clip_ratio_rows(x, d: int, d_pad: int, m: int, bits: int, group: int, eps: float,
                           trace: list | None = None):
    """Algorithm 1's loop with the quantization error of the rows in x as the objective (clip ratios
    are evaluated at their float32 value, the type the library's entry point takes)."""
    def evaluate(alpha):
        return float(clip_error_rows(x, d, d_pad, m, bits, group, np.array([np.float32(alpha)], dtype=np.float64))[0])
    return gradual_binary_search(evaluate, eps, trace)


# ----------------------------------------------------------------------------------------------
# Asymmetric uniform quantizer (the KV-cache setting of Section 5.1: "asymmetric quantization with a
# group size of 128"; the paper gives no formula, so this is the textbook definition with the clip
# ratio of Section 3.1 shrinking both ends of the range).  PARITY UNPINNED by the paper; pinned by a
# hand-worked example, the code range, the reproduction of both range ends at alpha = 1 and the
# half-step error bound.
# ----------------------------------------------------------------------------------------------
def quantize_asym(y, bits: int, group: int = 0, alpha: float = 1.0):
    """Per group of `group` consecutive values (0 = the whole row): lo = alpha*min(y), hi = alpha*max(y),
    Delta = (hi - lo) / (2^bits - 1), q = clamp(rint((y - lo) / Delta), 0, 2^bits - 1) (round half to even),
    yhat = q * Delta + lo.  A constant group (hi == lo) gives codes 0 and Delta 0.
    Returns (q int32 [n], delta float64 [groups], zero float64 [groups])."""
    y = np.ascontiguousarray(y, dtype=np.float64)
    n = y.shape[0]
    g = group if group else n
    L = (1 << bits) - 1
    q = np.zeros(n, dtype=np.int32)
    delta = np.zeros(n // g, dtype=np.float64)
    zero = np.zeros(n // g, dtype=np.float64)
    for i in range(n // g):
        seg = y[i * g:(i + 1) * g]
        lo, hi = alpha * seg.min(), alpha * seg.max()
        zero[i] = lo
        if hi > lo:
            delta[i] = (hi - lo) / L
            q[i * g:(i + 1) * g] = np.clip(np.rint((seg - lo) / delta[i]), 0, L).astype(np.int32)
    return q, delta, zero


def rotate_quantize_asym_rows(x, d: int, d_pad: int, m: int, bits: int, group: int, alpha: float):
    """Pad -> rotate (the symmetric path's rotation) -> asymmetric quantizer -> pack, row by row.
    Returns dict(y, q (0 .. 2^bits-1), packed, delta [n,spr], zero [n,spr])."""
    y = rotate_quantize_rows(x, d, d_pad, m, bits, 0, 1.0, want_q=False, want_packed=False)["y"]
    n = y.shape[0]
    spr = d_pad // group if group else 1
    q = np.empty((n, d_pad), dtype=np.int32)
    delta = np.empty((n, spr), dtype=np.float64)
    zero = np.empty((n, spr), dtype=np.float64)
    for r in range(n):
        q[r], delta[r], zero[r] = quantize_asym(y[r], bits, group, alpha)
    packed = np.stack([pack(q[r], bits) for r in range(n)]) if n else np.empty((0, d_pad * bits // 8), np.uint8)
    return dict(y=y, q=q, packed=packed, delta=delta, zero=zero)


def dequantize_asym_rows(packed, delta, zero, d_pad: int, bits: int, group: int) -> np.ndarray:
    """yhat = q * Delta + zero in the rotated domain (fields are unsigned)."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    g = group if group else d_pad
    out = np.empty((n, d_pad), dtype=np.float64)
    for r in range(n):
        q = unpack(packed[r], d_pad, bits) & ((1 << bits) - 1)
        out[r] = q * np.repeat(np.asarray(delta[r], dtype=np.float64), g) + np.repeat(np.asarray(zero[r], np.float64), g)
    return out
