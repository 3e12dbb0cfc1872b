"""Thin ctypes binding of libgbs.so (the C ABI declared in include/gbs.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch is used for device memory and streams.  There is no CPU fallback: if the shared
library is missing or a call fails, a GbsError is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libgbs.so")

GBS_OK = 0
GBS_ERR_INVALID_ARG = -1
GBS_ERR_UNSUPPORTED = -2
GBS_ERR_ALIGNMENT = -3
GBS_ERR_CUDA = -4
GBS_ERR_ALLOC = -5
GBS_DTYPE_F32 = 0
GBS_DTYPE_BF16 = 1
GBS_INVERSE_ROTATE = 1
GBS_MAX_D_PAD = 32768
GBS_MAX_CANDIDATES = 64

GBS_PLAN_ASYMMETRIC = 1
EXPORTS = ("gbs_plan_create", "gbs_plan_create_ex", "gbs_plan_destroy", "gbs_plan_info", "gbs_plan_device_status", "gbs_rotate_quantize",
           "gbs_rotate_quantize_static", "gbs_static_device_status", "gbs_dequantize", "gbs_clip_error",
           "gbs_search_clip_ratio", "gbs_search_state_init", "gbs_search_clip_ratio_fn", "gbs_search_clip_ratio_batch",
           "gbs_hadamard_m", "gbs_status_string", "gbs_selftest_wait_expiry", "gbs_weight_rotate_quantize",
           "gbs_quantized_matmul")
GBS_STATIC_MAX_D_PAD = 4096


class GbsError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__("%s failed: %s" % (what, status_string(status)))


class PlanInfo(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int), ("d_pad", ctypes.c_int), ("m", ctypes.c_int), ("k", ctypes.c_int),
                ("bits", ctypes.c_int), ("group", ctypes.c_int), ("alpha", ctypes.c_float),
                ("levels", ctypes.c_int), ("q_lo", ctypes.c_int), ("q_hi", ctypes.c_int),
                ("code_bytes_per_row", ctypes.c_int64), ("scales_per_row", ctypes.c_int),
                ("asymmetric", ctypes.c_int), ("scale_floats_per_row", ctypes.c_int),
                ("variant", ctypes.c_int)]


class SearchResult(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_float), ("a", ctypes.c_float), ("b", ctypes.c_float), ("err", ctypes.c_double),
                ("iterations", ctypes.c_int), ("evaluations", ctypes.c_int), ("rounds", ctypes.c_int)]


class SearchState(ctypes.Structure):
    """gbs_search_state_t: the resumable state of one projection's search (plain data; bytes(state) stores it)."""
    _fields_ = [("a", ctypes.c_double), ("b", ctypes.c_double), ("m", ctypes.c_double), ("f_m", ctypes.c_double),
                ("iteration", ctypes.c_int), ("evaluations", ctypes.c_int), ("have_fm", ctypes.c_int),
                ("done", ctypes.c_int)]


class SearchTask(ctypes.Structure):
    _fields_ = [("plan", ctypes.c_void_p), ("x", ctypes.c_void_p), ("x_dtype", ctypes.c_int),
                ("n_rows", ctypes.c_int64), ("x_row_stride", ctypes.c_int64)]


OBJECTIVE_FN = ctypes.CFUNCTYPE(ctypes.c_double, ctypes.c_float, ctypes.c_void_p)
GBS_MAX_SEARCH_TASKS = 4096

_lib = None


def lib() -> ctypes.CDLL:
    """Load libgbs.so (built in-tree by paper_2504_13989_b200.build); fail loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise GbsErrorMissing("libgbs.so not found at %s -- run `python -m paper_2504_13989_b200.build` "
                                  "(or __graft_entry__.build()); there is no CPU fallback" % _LIB_PATH)
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
        L.gbs_plan_create.argtypes = [ctypes.POINTER(vp), i32, i32, i32, i32, i32, ctypes.c_float]
        L.gbs_plan_create.restype = i32
        L.gbs_plan_create_ex.argtypes = [ctypes.POINTER(vp), i32, i32, i32, i32, i32, ctypes.c_float, i32]
        L.gbs_plan_create_ex.restype = i32
        L.gbs_plan_destroy.argtypes = [vp]
        L.gbs_plan_destroy.restype = i32
        L.gbs_plan_info.argtypes = [vp, ctypes.POINTER(PlanInfo)]
        L.gbs_plan_info.restype = i32
        L.gbs_plan_device_status.argtypes = [vp, ctypes.POINTER(i32)]
        L.gbs_plan_device_status.restype = i32
        L.gbs_rotate_quantize.argtypes = [vp, vp, i32, i64, i64, vp, vp, vp, vp]
        L.gbs_rotate_quantize.restype = i32
        L.gbs_rotate_quantize_static.argtypes = [i32, i32, i32, i32, i32, ctypes.c_float, vp, i64, i64, vp, vp, vp]
        L.gbs_rotate_quantize_static.restype = i32
        L.gbs_selftest_wait_expiry.argtypes = [i32, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.gbs_selftest_wait_expiry.restype = i32
        L.gbs_static_device_status.argtypes = [ctypes.POINTER(i32)]
        L.gbs_static_device_status.restype = i32
        L.gbs_dequantize.argtypes = [vp, vp, vp, i64, vp, i32, i32, vp]
        L.gbs_dequantize.restype = i32
        L.gbs_clip_error.argtypes = [vp, vp, i32, i64, i64, ctypes.POINTER(ctypes.c_float), i32, vp, vp, vp]
        L.gbs_clip_error.restype = i32
        L.gbs_search_clip_ratio.argtypes = [vp, vp, i32, i64, i64, ctypes.c_float, vp, ctypes.POINTER(SearchResult), vp]
        L.gbs_search_clip_ratio.restype = i32
        L.gbs_search_state_init.argtypes = [ctypes.POINTER(SearchState)]
        L.gbs_search_state_init.restype = i32
        L.gbs_search_clip_ratio_fn.argtypes = [OBJECTIVE_FN, vp, ctypes.c_float, ctypes.POINTER(SearchState), i32]
        L.gbs_search_clip_ratio_fn.restype = i32
        L.gbs_search_clip_ratio_batch.argtypes = [ctypes.POINTER(SearchTask), i32, ctypes.c_float,
                                                  ctypes.POINTER(SearchState), i32, vp, ctypes.POINTER(ctypes.c_float),
                                                  ctypes.POINTER(i32), vp]
        L.gbs_search_clip_ratio_batch.restype = i32
        L.gbs_weight_rotate_quantize.argtypes = [vp, vp, i32, i64, i64, vp, vp, vp]
        L.gbs_weight_rotate_quantize.restype = i32
        L.gbs_quantized_matmul.argtypes = [vp, vp, vp, i64, vp, vp, vp, i64, vp, i32, i64, vp]
        L.gbs_quantized_matmul.restype = i32
        L.gbs_hadamard_m.argtypes = [i32, vp]
        L.gbs_hadamard_m.restype = i32
        L.gbs_status_string.argtypes = [i32]
        L.gbs_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


class GbsErrorMissing(RuntimeError):
    pass


def status_string(status: int) -> str:
    return lib().gbs_status_string(int(status)).decode()


def _check(status: int, what: str):
    if status != GBS_OK:
        raise GbsError(status, what)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GBS_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return GBS_DTYPE_BF16
    raise TypeError("gbs: tensors must be float32 or bfloat16, got %s" % t.dtype)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _rows_view(x: torch.Tensor, d: int):
    """(pointer, n_rows, row stride in elements) of a [..., d] tensor whose leading dims are contiguous rows."""
    if not x.is_cuda:
        raise ValueError("gbs: x must be a CUDA tensor (device pointer); there is no CPU path")
    if x.dim() < 1 or x.shape[-1] != d:
        raise ValueError("gbs: last dimension of x must be d=%d, got shape %s" % (d, tuple(x.shape)))
    if x.dim() == 1:
        x = x.unsqueeze(0)
    if x.stride(-1) != 1:
        raise ValueError("gbs: the last dimension of x must be contiguous")
    if x.dim() > 2:
        x = x.reshape(-1, d) if x.is_contiguous() else x.flatten(0, -2)
    return x, x.shape[0], (x.stride(0) if x.shape[0] > 1 else max(x.stride(0), d))


def _check_buffer(what: str, t: torch.Tensor, like: torch.Tensor, dtype, min_numel: int):
    """The C ABI cannot validate pointers; the binding knows the tensors behind them.  An undersized, CPU or
    strided buffer would make a kernel write out of bounds on the device, so it is refused here."""
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise ValueError("gbs: %s must be a CUDA tensor" % what)
    if t.device != like.device:
        raise ValueError("gbs: %s is on %s but the rows are on %s" % (what, t.device, like.device))
    if dtype is not None and t.dtype != dtype:
        raise TypeError("gbs: %s must be %s, got %s" % (what, dtype, t.dtype))
    if not t.is_contiguous():
        raise ValueError("gbs: %s must be contiguous" % what)
    if t.numel() < min_numel:
        raise ValueError("gbs: %s holds %d elements, the call writes %d" % (what, t.numel(), min_numel))


# ----------------------------------------------------------------------------------------------
# functions named after the C entry points
# ----------------------------------------------------------------------------------------------
def gbs_plan_create(d: int, d_pad: int, m: int, bits: int, group: int, alpha: float) -> int:
    """Returns an opaque plan handle (int).  See include/gbs.h for the argument ranges."""
    h = ctypes.c_void_p()
    _check(lib().gbs_plan_create(ctypes.byref(h), d, d_pad, m, bits, group, alpha), "gbs_plan_create")
    return h.value


def gbs_plan_create_ex(d: int, d_pad: int, m: int, bits: int, group: int, alpha: float, flags: int) -> int:
    """gbs_plan_create with flags (GBS_PLAN_ASYMMETRIC: the asymmetric quantizer for d' = 128 KV rows)."""
    h = ctypes.c_void_p()
    _check(lib().gbs_plan_create_ex(ctypes.byref(h), d, d_pad, m, bits, group, alpha, flags), "gbs_plan_create_ex")
    return h.value


def gbs_plan_destroy(plan: int) -> None:
    _check(lib().gbs_plan_destroy(ctypes.c_void_p(plan)), "gbs_plan_destroy")


def gbs_plan_info(plan: int) -> PlanInfo:
    info = PlanInfo()
    _check(lib().gbs_plan_info(ctypes.c_void_p(plan), ctypes.byref(info)), "gbs_plan_info")
    return info


def gbs_plan_device_status(plan: int) -> int:
    """Read and clear the plan's device status word (0 = no bounded wait ever expired).  Synchronises."""
    v = ctypes.c_int(0)
    _check(lib().gbs_plan_device_status(ctypes.c_void_p(plan), ctypes.byref(v)), "gbs_plan_device_status")
    return v.value


def gbs_hadamard_m(m: int) -> torch.Tensor:
    """The m x m sign matrix H_m the plans use (host computation, int8)."""
    out = torch.zeros((m, m), dtype=torch.int8)
    _check(lib().gbs_hadamard_m(m, out.data_ptr()), "gbs_hadamard_m")
    return out


def gbs_rotate_quantize(plan: int, x: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor,
                        y_opt: torch.Tensor | None = None, stream=None) -> None:
    info = gbs_plan_info(plan)
    xv, n_rows, stride = _rows_view(x, info.d)
    _check_buffer("codes", codes, xv, torch.uint8, n_rows * info.code_bytes_per_row)
    _check_buffer("scales", scales, xv, torch.float32, n_rows * info.scale_floats_per_row)
    if y_opt is not None:
        _check_buffer("y_opt", y_opt, xv, torch.float32, n_rows * info.d_pad)
    _check(lib().gbs_rotate_quantize(ctypes.c_void_p(plan), xv.data_ptr(), _dtype_code(xv), n_rows, stride,
                                     codes.data_ptr(), scales.data_ptr(),
                                     y_opt.data_ptr() if y_opt is not None else None, _stream_ptr(stream)),
           "gbs_rotate_quantize")


def gbs_rotate_quantize_static(d: int, d_pad: int, m: int, bits: int, group: int, alpha: float, x: torch.Tensor,
                               codes: torch.Tensor, scales: torch.Tensor, stream=None) -> None:
    """gbs_rotate_quantize without a plan and without any device allocation inside the library: for
    processes that may not call cudaMalloc (all memory already claimed by a pool, or no tolerance for
    the device-wide synchronisation an allocation implies).  bf16 rows, d_pad <= GBS_STATIC_MAX_D_PAD;
    see include/gbs.h for the limits and for how calls share the library's fixed device array."""
    xv, n_rows, stride = _rows_view(x, d)
    if xv.dtype != torch.bfloat16:
        raise TypeError("gbs_rotate_quantize_static: x must be bfloat16")
    if d_pad > 0 and bits in (3, 4):
        _check_buffer("codes", codes, xv, torch.uint8, n_rows * (d_pad * bits // 8))
        _check_buffer("scales", scales, xv, torch.float32, n_rows * (d_pad // group if group > 0 else 1))
    _check(lib().gbs_rotate_quantize_static(d, d_pad, m, bits, group, alpha, xv.data_ptr(), n_rows, stride,
                                            codes.data_ptr(), scales.data_ptr(), _stream_ptr(stream)),
           "gbs_rotate_quantize_static")


def gbs_selftest_wait_expiry(limit_us: int = 1000):
    """Run one bounded wait that is certain to run out; returns (code, abort flag, microseconds waited)."""
    code, ab, us = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    _check(lib().gbs_selftest_wait_expiry(int(limit_us), ctypes.byref(code), ctypes.byref(ab), ctypes.byref(us)),
           "gbs_selftest_wait_expiry")
    return code.value, ab.value, us.value


def gbs_static_device_status() -> int:
    """Read and clear the status word of gbs_rotate_quantize_static on the current device.  Synchronises."""
    v = ctypes.c_int(0)
    _check(lib().gbs_static_device_status(ctypes.byref(v)), "gbs_static_device_status")
    return v.value


def gbs_dequantize(plan: int, codes: torch.Tensor, scales: torch.Tensor, n_rows: int, out: torch.Tensor,
                   flags: int = 0, stream=None) -> None:
    info = gbs_plan_info(plan)
    width = info.d if (flags & GBS_INVERSE_ROTATE) else info.d_pad
    _check_buffer("codes", codes, codes, torch.uint8, n_rows * info.code_bytes_per_row)
    _check_buffer("scales", scales, codes, torch.float32, n_rows * info.scale_floats_per_row)
    _check_buffer("out", out, codes, None, n_rows * width)
    _check(lib().gbs_dequantize(ctypes.c_void_p(plan), codes.data_ptr(), scales.data_ptr(), n_rows,
                                out.data_ptr(), _dtype_code(out), flags, _stream_ptr(stream)),
           "gbs_dequantize")


def gbs_clip_error(plan: int, x: torch.Tensor, alphas, err_sum: torch.Tensor,
                   err_rows_opt: torch.Tensor | None = None, stream=None) -> None:
    info = gbs_plan_info(plan)
    xv, n_rows, stride = _rows_view(x, info.d)
    alphas = [float(a) for a in alphas]
    arr = (ctypes.c_float * len(alphas))(*alphas)
    _check_buffer("err_sum", err_sum, xv, torch.float64, len(alphas))
    if err_rows_opt is not None:
        _check_buffer("err_rows_opt", err_rows_opt, xv, torch.float32, n_rows * len(alphas))
    _check(lib().gbs_clip_error(ctypes.c_void_p(plan), xv.data_ptr(), _dtype_code(xv), n_rows, stride,
                                arr, len(alphas), err_sum.data_ptr(),
                                err_rows_opt.data_ptr() if err_rows_opt is not None else None,
                                _stream_ptr(stream)),
           "gbs_clip_error")


def gbs_search_clip_ratio(plan: int, x: torch.Tensor, eps: float, work: torch.Tensor | None = None,
                          stream=None) -> SearchResult:
    """Algorithm 1's bracket search for the clip ratio of the rows in x (objective: quantization error).
    Blocks on the stream after every round of up to 31 probes."""
    info = gbs_plan_info(plan)
    xv, n_rows, stride = _rows_view(x, info.d)
    if work is None:
        work = torch.empty(GBS_MAX_CANDIDATES, dtype=torch.float64, device=x.device)
    _check_buffer("work", work, xv, torch.float64, GBS_MAX_CANDIDATES)
    res = SearchResult()
    _check(lib().gbs_search_clip_ratio(ctypes.c_void_p(plan), xv.data_ptr(), _dtype_code(xv), n_rows, stride,
                                       float(eps), work.data_ptr(), ctypes.byref(res), _stream_ptr(stream)),
           "gbs_search_clip_ratio")
    return res


def gbs_weight_rotate_quantize(plan: int, w: torch.Tensor, codes: torch.Tensor, scales: torch.Tensor, stream=None) -> None:
    """Rows of the weight matrix [n_out, d] through the activation path's rotation and quantizer (Eq. (2))."""
    info = gbs_plan_info(plan)
    wv, n_out, stride = _rows_view(w, info.d)
    _check_buffer("codes", codes, wv, torch.uint8, n_out * info.code_bytes_per_row)
    _check_buffer("scales", scales, wv, torch.float32, n_out * info.scale_floats_per_row)
    _check(lib().gbs_weight_rotate_quantize(ctypes.c_void_p(plan), wv.data_ptr(), _dtype_code(wv), n_out, stride,
                                            codes.data_ptr(), scales.data_ptr(), _stream_ptr(stream)),
           "gbs_weight_rotate_quantize")


def gbs_quantized_matmul(plan_x: int, codes_x: torch.Tensor, scales_x: torch.Tensor, plan_w: int, codes_w: torch.Tensor,
                         scales_w: torch.Tensor, out: torch.Tensor, stream=None) -> None:
    """out[t, o] = Delta_x[t] * Delta_w[o] * sum_j q_x[t, j] * q_w[o, j] from the packed codes of both sides."""
    ix, iw = gbs_plan_info(plan_x), gbs_plan_info(plan_w)
    n_tok, n_out = codes_x.shape[0], codes_w.shape[0]
    _check_buffer("codes_x", codes_x, codes_x, torch.uint8, n_tok * ix.code_bytes_per_row)
    _check_buffer("scales_x", scales_x, codes_x, torch.float32, n_tok * ix.scale_floats_per_row)
    _check_buffer("codes_w", codes_w, codes_x, torch.uint8, n_out * iw.code_bytes_per_row)
    _check_buffer("scales_w", scales_w, codes_x, torch.float32, n_out * iw.scale_floats_per_row)
    if out.dim() != 2 or out.shape[0] != n_tok or out.shape[1] != n_out or out.stride(1) != 1 or not out.is_cuda \
            or out.device != codes_x.device:
        raise ValueError("gbs_quantized_matmul: out must be a CUDA [n_tokens, n_out] tensor with contiguous rows")
    _check(lib().gbs_quantized_matmul(ctypes.c_void_p(plan_x), codes_x.data_ptr(), scales_x.data_ptr(), n_tok,
                                      ctypes.c_void_p(plan_w), codes_w.data_ptr(), scales_w.data_ptr(), n_out,
                                      out.data_ptr(), _dtype_code(out), out.stride(0), _stream_ptr(stream)),
           "gbs_quantized_matmul")


def gbs_search_state_init() -> SearchState:
    st = SearchState()
    _check(lib().gbs_search_state_init(ctypes.byref(st)), "gbs_search_state_init")
    return st


def gbs_search_clip_ratio_fn(objective, eps: float, state: SearchState | None = None,
                             max_iterations: int = 0) -> SearchState:
    """Algorithm 1's loop for one projection with a Python objective `objective(alpha) -> float` (e.g. a model's
    perplexity).  Host only.  Returns the state (done = 1 when b - a <= eps); pass it back to resume."""
    st = state if state is not None else gbs_search_state_init()
    cb = OBJECTIVE_FN(lambda alpha, _ctx: float(objective(float(alpha))))
    _check(lib().gbs_search_clip_ratio_fn(cb, None, float(eps), ctypes.byref(st), int(max_iterations)),
           "gbs_search_clip_ratio_fn")
    return st


def gbs_search_clip_ratio_batch(plans, xs, eps: float, states=None, max_rounds: int = 0, work: torch.Tensor | None = None,
                                stream=None):
    """Algorithm 1's loop for several projections at once (plan i scores rows xs[i]); one wait per round.
    Returns (alphas: the list L, states, rounds).  `plans` are plan handles (ints)."""
    n = len(plans)
    if n < 1 or n != len(xs):
        raise ValueError("gbs_search_clip_ratio_batch: one tensor per plan")
    tasks = (SearchTask * n)()
    keep = []
    for i, (pl, x) in enumerate(zip(plans, xs)):
        info = gbs_plan_info(pl)
        xv, n_rows, stride = _rows_view(x, info.d)
        keep.append(xv)
        tasks[i] = SearchTask(pl, xv.data_ptr(), _dtype_code(xv), n_rows, stride)
    sts = (SearchState * n)()
    for i in range(n):
        sts[i] = states[i] if states is not None else gbs_search_state_init()
    if work is None:
        work = torch.empty(n * GBS_MAX_CANDIDATES, dtype=torch.float64, device=keep[0].device)
    _check_buffer("work", work, keep[0], torch.float64, n * GBS_MAX_CANDIDATES)
    alphas = (ctypes.c_float * n)()
    rounds = ctypes.c_int(0)
    _check(lib().gbs_search_clip_ratio_batch(tasks, n, float(eps), sts, int(max_rounds), work.data_ptr(), alphas,
                                             ctypes.byref(rounds), _stream_ptr(stream)),
           "gbs_search_clip_ratio_batch")
    return [float(a) for a in alphas], [sts[i] for i in range(n)], rounds.value


# ----------------------------------------------------------------------------------------------
# convenience object: owns a plan handle and allocates outputs with torch
# ----------------------------------------------------------------------------------------------
class Plan:
    """RAII wrapper of a gbs plan; allocates output tensors with torch and forwards to the C ABI."""

    def __init__(self, d: int, d_pad: int | None = None, m: int = 1, bits: int = 4, group: int = 0,
                 alpha: float = 1.0, asymmetric: bool = False):
        d_pad = d if d_pad is None else d_pad
        self.handle = gbs_plan_create_ex(d, d_pad, m, bits, group, alpha, GBS_PLAN_ASYMMETRIC if asymmetric else 0)
        self.info = gbs_plan_info(self.handle)

    def close(self):
        if getattr(self, "handle", None):
            gbs_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def device_status(self) -> int:
        return gbs_plan_device_status(self.handle)

    def alloc_outputs(self, n_rows: int, device, want_y: bool = False):
        codes = torch.empty((n_rows, self.info.code_bytes_per_row), dtype=torch.uint8, device=device)
        scales = torch.empty((n_rows, self.info.scale_floats_per_row), dtype=torch.float32, device=device)
        y = torch.empty((n_rows, self.info.d_pad), dtype=torch.float32, device=device) if want_y else None
        return codes, scales, y

    def rotate_quantize(self, x: torch.Tensor, want_y: bool = False, out=None, stream=None):
        n_rows = x.numel() // self.info.d
        codes, scales, y = out if out is not None else self.alloc_outputs(n_rows, x.device, want_y)
        gbs_rotate_quantize(self.handle, x, codes, scales, y, stream)
        return codes, scales, y

    def dequantize(self, codes: torch.Tensor, scales: torch.Tensor, inverse: bool = False,
                   dtype=torch.float32, out=None, stream=None) -> torch.Tensor:
        n_rows = codes.shape[0]
        width = self.info.d if inverse else self.info.d_pad
        if out is None:
            out = torch.empty((n_rows, width), dtype=dtype, device=codes.device)
        gbs_dequantize(self.handle, codes, scales, n_rows, out, GBS_INVERSE_ROTATE if inverse else 0, stream)
        return out

    def clip_error(self, x: torch.Tensor, alphas, want_rows: bool = False, err_sum=None, stream=None):
        n_rows = x.numel() // self.info.d
        K = len(alphas)
        if err_sum is None:
            err_sum = torch.zeros(K, dtype=torch.float64, device=x.device)
        rows = torch.empty((n_rows, K), dtype=torch.float32, device=x.device) if want_rows else None
        gbs_clip_error(self.handle, x, alphas, err_sum, rows, stream)
        return (err_sum, rows) if want_rows else err_sum

    def weight_rotate_quantize(self, w: torch.Tensor, out=None, stream=None):
        """Quantize the rows of a weight matrix [n_out, d] (Eq. (2)); returns (codes, scales)."""
        n_out = w.numel() // self.info.d
        codes, scales, _ = out if out is not None else self.alloc_outputs(n_out, w.device)
        gbs_weight_rotate_quantize(self.handle, w, codes, scales, stream)
        return codes, scales

    def quantized_matmul(self, codes_x, scales_x, plan_w: "Plan", codes_w, scales_w, dtype=torch.float32, out=None,
                         stream=None) -> torch.Tensor:
        """The layer's output from the packed codes of activations (this plan) and weights (plan_w)."""
        if out is None:
            out = torch.empty((codes_x.shape[0], codes_w.shape[0]), dtype=dtype, device=codes_x.device)
        gbs_quantized_matmul(self.handle, codes_x, scales_x, plan_w.handle, codes_w, scales_w, out, stream)
        return out

    def search_clip_ratio(self, x: torch.Tensor, eps: float = 1.0 / 64, stream=None) -> SearchResult:
        return gbs_search_clip_ratio(self.handle, x, eps, stream=stream)

    def rotate_quantize_host(self, x_host: torch.Tensor, codes_host: torch.Tensor, scales_host: torch.Tensor,
                             device="cuda:0", stream=None):
        """End-to-end call for host-resident data: pinned host -> device, rotate_quantize, device -> host.

        x_host / codes_host / scales_host are (ideally pinned) CPU tensors; the copies are enqueued on
        the same stream as the kernel.  Returns after the stream has been synchronised.
        """
        s = stream or torch.cuda.current_stream()
        with torch.cuda.stream(s):
            x = x_host.to(device, non_blocking=True)
            codes, scales, _ = self.rotate_quantize(x, stream=s)
            codes_host.copy_(codes, non_blocking=True)
            scales_host.copy_(scales, non_blocking=True)
        s.synchronize()
        return codes_host, scales_host


class HostPipeline:
    """Host-resident rows through one or more plans: pinned host -> device -> kernels -> pinned host.

    The rows are cut into `chunks` row ranges.  Chunk i+1 is copied to the device on a copy stream
    while chunk i is quantized and its codes and scales travel back on the compute stream, so the
    two PCIe directions work at the same time.  Only copies, events and the plans' launches happen
    here; staging buffers on the device are allocated once.
    """

    def __init__(self, plans, n_rows: int, device="cuda:0", chunks: int = 4, dtype=torch.bfloat16):
        self.plans = list(plans)
        d = self.plans[0].info.d
        assert all(p.info.d == d for p in self.plans)
        self.n_rows, self.d = n_rows, d
        chunks = max(1, min(chunks, n_rows)) if n_rows else 1
        step = (n_rows + chunks - 1) // chunks if n_rows else 0
        self.ranges = [(r, min(n_rows, r + step)) for r in range(0, n_rows, step)] if n_rows else []
        self.x_dev = torch.empty((n_rows, d), dtype=dtype, device=device)
        self.outs = [p.alloc_outputs(n_rows, device) for p in self.plans]
        self.copy_stream = torch.cuda.Stream(device=device)
        self.ev_in = [torch.cuda.Event() for _ in self.ranges]
        self.ev_start = torch.cuda.Event()
        # views of the staging buffers and the marshalled arguments of every launch, made once: the per-call host
        # work is what bounds a pipeline of short launches
        self.x_views = [self.x_dev[r0:r1] for r0, r1 in self.ranges]
        self.calls = []
        dt = _dtype_code(self.x_dev)
        for (r0, r1), xv in zip(self.ranges, self.x_views):
            per_plan = []
            for p, (codes, scales, _) in zip(self.plans, self.outs):
                cv, sv = codes[r0:r1], scales[r0:r1]
                per_plan.append((ctypes.c_void_p(p.handle), xv.data_ptr(), dt, r1 - r0, xv.stride(0) if r1 - r0 > 1 else d,
                                 cv.data_ptr(), sv.data_ptr(), cv, sv))
            self.calls.append(per_plan)

    def run(self, x_host: torch.Tensor, outs_host, stream=None):
        """outs_host: one (codes_host, scales_host) pair per plan.  Work is enqueued on `stream` (and the
        internal copy stream, joined to it); the caller synchronises `stream`."""
        s = stream or torch.cuda.current_stream()
        sp = int(s.cuda_stream)
        rq = lib().gbs_rotate_quantize
        self.ev_start.record(s)
        self.copy_stream.wait_event(self.ev_start)          # staging buffers of the previous call are free
        for i, (r0, r1) in enumerate(self.ranges):
            with torch.cuda.stream(self.copy_stream):
                self.x_views[i].copy_(x_host[r0:r1], non_blocking=True)
                self.ev_in[i].record(self.copy_stream)
            with torch.cuda.stream(s):
                s.wait_event(self.ev_in[i])
                for (h, xp, dt, n, stride, cp, scp, cv, sv), (ch, sh) in zip(self.calls[i], outs_host):
                    _check(rq(h, xp, dt, n, stride, cp, scp, None, sp), "gbs_rotate_quantize")
                    ch[r0:r1].copy_(cv, non_blocking=True)
                    sh[r0:r1].copy_(sv, non_blocking=True)
        return outs_host
