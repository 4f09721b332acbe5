"""Thin Python binding of the C ABI in ``include/tsenor.h``: argument
marshalling only.  Every step of the method runs in the CUDA kernels of
``libtsenor.so``; there is no CPU fallback, and a missing library is an error.

PyTorch is used for device memory and streams only.  Masks are returned as
``torch.int32`` tensors holding the ``uint32`` words of the C ABI (bit
``c % 32`` of word ``c // 32`` of row ``r`` is ``S[r, c]``).
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# The library beside this file; TSENOR_LIBRARY selects another build of the same ABI (for instance
# the checked flavour libtsenor_bounds.so, to run a whole test suite with every index tested).
LIB_PATH = os.environ.get("TSENOR_LIBRARY") or os.path.join(_HERE, "libtsenor.so")

OK, ERR_NULL, ERR_SHAPE, ERR_NM, ERR_ARG, ERR_CUDA = 0, -1, -2, -3, -4, -5
DEV_NONFINITE_SCORE, DEV_UNDERFILLED, DEV_INTERNAL = 1, 2, 4

EXPORTS = (
    "tsenor_solve", "tsenor_dykstra", "tsenor_round", "tsenor_objective", "tsenor_check",
    "tsenor_max_abs", "tsenor_mask_words_per_row", "tsenor_strerror", "tsenor_last_cuda_error",
    "tsenor_launch_count", "tsenor_solve_scores", "tsenor_scores_max", "tsenor_scores_materialize",
    "tsenor_keep_better", "tsenor_simple_round", "tsenor_dykstra_scores", "tsenor_set_layout",
)
LAYOUT_AUTO, LAYOUT_THROUGHPUT, LAYOUT_LATENCY = 0, 1, 2

SCORES_ABS, SCORES_ADMM, SCORES_COLDIV, SCORES_COLMUL = 0, 1, 2, 3


class ScoresDesc(C.Structure):
    """ctypes image of ``tsenor_scores_t`` (a host struct holding device pointers)."""
    _fields_ = [("kind", C.c_int), ("w_is_bf16", C.c_int), ("w", C.c_void_p), ("ld", C.c_int64),
                ("v", C.c_void_p), ("ld_v", C.c_int64), ("scalar", C.c_float), ("colvec", C.c_void_p),
                ("per_block_tau", C.c_int), ("early_exit_eps", C.c_float), ("dev_iters_out", C.c_void_p)]

_lib = None


class TsenorError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        msg = lib().tsenor_strerror(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {lib().tsenor_last_cuda_error()})"
        super().__init__(f"{what}: {msg}")


def lib():
    """The loaded C-ABI library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2505_23949_b200.build` "
                "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32, f32 = C.c_void_p, C.c_int64, C.c_int, C.c_float
        L.tsenor_solve.argtypes = [vp, i64, i64, i64, i32, i32, f32, i32, i32, vp, vp, vp]
        L.tsenor_dykstra.argtypes = [vp, i64, i64, i64, i32, i32, f32, i32, vp, i64, i32, vp, vp]
        L.tsenor_round.argtypes = [vp, i64, vp, i64, i64, i64, i32, i32, i32, vp, vp, vp]
        L.tsenor_objective.argtypes = [vp, i64, vp, i64, i64, vp, vp]
        L.tsenor_check.argtypes = [vp, i64, i64, i32, i32, vp, vp]
        L.tsenor_max_abs.argtypes = [vp, i64, i64, i64, vp, vp]
        for name in ("tsenor_solve", "tsenor_dykstra", "tsenor_round", "tsenor_objective",
                     "tsenor_check", "tsenor_max_abs", "tsenor_last_cuda_error"):
            getattr(L, name).restype = i32
        sp = C.POINTER(ScoresDesc)
        L.tsenor_solve_scores.argtypes = [sp, i64, i64, i32, i32, f32, i32, i32, vp, vp, vp]
        L.tsenor_dykstra_scores.argtypes = [sp, i64, i64, i32, i32, f32, i32, vp, i64, i32, vp, vp]
        L.tsenor_dykstra_scores.restype = i32
        L.tsenor_scores_max.argtypes = [sp, i64, i64, vp, vp]
        L.tsenor_scores_materialize.argtypes = [sp, i64, i64, vp, i64, vp]
        L.tsenor_keep_better.argtypes = [sp, i64, i64, vp, vp, vp, vp]
        L.tsenor_simple_round.argtypes = [vp, i64, i64, i64, i32, i32, vp, vp]
        for name in ("tsenor_solve_scores", "tsenor_scores_max", "tsenor_scores_materialize",
                     "tsenor_keep_better", "tsenor_simple_round"):
            getattr(L, name).restype = i32
        L.tsenor_mask_words_per_row.argtypes = [i64]
        L.tsenor_mask_words_per_row.restype = i64
        L.tsenor_strerror.argtypes = [i32]
        L.tsenor_strerror.restype = C.c_char_p
        L.tsenor_launch_count.argtypes = []
        L.tsenor_launch_count.restype = i64
        L.tsenor_set_layout.argtypes = [i32]
        L.tsenor_set_layout.restype = i32
        _lib = L
    return _lib


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _mat(t, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.float32 and t.dim() == 2):
        raise TypeError(f"{name} must be a 2-D float32 CUDA tensor")
    if t.stride(1) != 1:
        raise ValueError(f"{name} must be row-major (unit column stride)")
    ld = t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])
    return t.data_ptr(), t.shape[0], t.shape[1], ld


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _out(t, name, dtype, device, shape=None, min_numel=None):
    """Checks a caller-supplied output (or status / scratch) tensor before its pointer goes to
    the library: a wrong dtype, shape, layout or device would become an out-of-bounds write
    on the GPU.  None passes through (the argument is optional or allocated by the caller)."""
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda):
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, not {t.dtype}")
    if t.device != torch.device(device):
        raise ValueError(f"{name} is on {t.device}, the input on {torch.device(device)}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, not {tuple(t.shape)}")
    if min_numel is not None and t.numel() < min_numel:
        raise ValueError(f"{name} needs at least {min_numel} element(s)")
    return t


def _mask_out(t, rows, cols, device, name="mask_out"):
    return _out(t, name, torch.int32, device, shape=(rows, mask_words_per_row(cols)))


def _on(device):
    """Makes the tensors' device current around a call: the library launches on the current device."""
    return torch.cuda.device(torch.device(device))


def mask_words_per_row(cols):
    return int(lib().tsenor_mask_words_per_row(int(cols)))


def new_mask(rows, cols, device):
    return torch.empty((rows, mask_words_per_row(cols)), dtype=torch.int32, device=device)


def new_status(device):
    return torch.zeros(1, dtype=torch.int32, device=device)


def launch_count():
    return int(lib().tsenor_launch_count())


def set_layout(layout):
    """tsenor_set_layout: LAYOUT_AUTO / LAYOUT_THROUGHPUT / LAYOUT_LATENCY; returns the previous one."""
    rc = lib().tsenor_set_layout(int(layout))
    if rc < 0:
        raise TsenorError(rc, "tsenor_set_layout")
    return rc


def solve(scores, N, M, tau, iters=300, ls_steps=-1, mask_out=None, status=None, stream=None):
    """tsenor_solve: Algorithm 1 + Algorithm 2 on every M x M block.  Asynchronous."""
    p, rows, cols, ld = _mat(scores, "scores")
    if mask_out is None:
        mask_out = new_mask(rows, cols, scores.device)
    _mask_out(mask_out, rows, cols, scores.device)
    _out(status, "status", torch.int32, scores.device, min_numel=1)
    with _on(scores.device):
        rc = lib().tsenor_solve(p, rows, cols, ld, int(N), int(M), float(tau), int(iters), int(ls_steps),
                                _ptr(mask_out), _ptr(status), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_solve")
    return mask_out


def dykstra(scores, N, M, tau, iters=300, plan_is_log=False, plan_out=None, status=None, stream=None):
    """tsenor_dykstra: Algorithm 1 only; returns the fp32 plan (or log-plan)."""
    p, rows, cols, ld = _mat(scores, "scores")
    if plan_out is None:
        plan_out = torch.empty((rows, cols), dtype=torch.float32, device=scores.device)
    pp, pr, pc, ldp = _mat(plan_out, "plan_out")
    if (pr, pc) != (rows, cols) or plan_out.device != scores.device:
        raise ValueError("plan_out must have the shape and device of scores")
    _out(status, "status", torch.int32, scores.device, min_numel=1)
    with _on(scores.device):
        rc = lib().tsenor_dykstra(p, rows, cols, ld, int(N), int(M), float(tau), int(iters), pp, ldp,
                                  int(bool(plan_is_log)), _ptr(status), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_dykstra")
    return plan_out


def round_plan(plan_key, scores, N, M, ls_steps=-1, mask_out=None, status=None, stream=None):
    """tsenor_round: Algorithm 2 only, from fp32 keys and fp32 scores."""
    pk, rows, cols, ldk = _mat(plan_key, "plan_key")
    ps, r2, c2, ld = _mat(scores, "scores")
    if (rows, cols) != (r2, c2):
        raise ValueError("plan_key and scores differ in shape")
    if plan_key.device != scores.device:
        raise ValueError("plan_key and scores are on different devices")
    if mask_out is None:
        mask_out = new_mask(rows, cols, scores.device)
    _mask_out(mask_out, rows, cols, scores.device)
    _out(status, "status", torch.int32, scores.device, min_numel=1)
    with _on(scores.device):
        rc = lib().tsenor_round(pk, ldk, ps, ld, rows, cols, int(N), int(M), int(ls_steps),
                                _ptr(mask_out), _ptr(status), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_round")
    return mask_out


def objective(scores, mask, out=None, stream=None):
    """tsenor_objective: 1-element float64 device tensor with the retained score."""
    p, rows, cols, ld = _mat(scores, "scores")
    if out is None:
        out = torch.empty(1, dtype=torch.float64, device=scores.device)
    _mask_out(mask, rows, cols, scores.device, "mask")
    _out(out, "out", torch.float64, scores.device, min_numel=1)
    with _on(scores.device):
        rc = lib().tsenor_objective(p, ld, _ptr(mask), rows, cols, _ptr(out), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_objective")
    return out


def check(mask, rows, cols, N, M, out=None, stream=None):
    """tsenor_check: 1-element int64 device tensor with the number of infeasible blocks."""
    if not (isinstance(mask, torch.Tensor) and mask.is_cuda):
        raise TypeError("mask must be a CUDA tensor")
    if out is None:
        out = torch.empty(1, dtype=torch.int64, device=mask.device)
    _mask_out(mask, int(rows), int(cols), mask.device, "mask")
    _out(out, "out", torch.int64, mask.device, min_numel=1)
    with _on(mask.device):
        rc = lib().tsenor_check(_ptr(mask), int(rows), int(cols), int(N), int(M), _ptr(out), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_check")
    return out


def max_abs(scores, out=None, stream=None):
    """tsenor_max_abs: 1-element float32 device tensor with max |score|."""
    p, rows, cols, ld = _mat(scores, "scores")
    if out is None:
        out = torch.empty(1, dtype=torch.float32, device=scores.device)
    _out(out, "out", torch.float32, scores.device, min_numel=1)
    with _on(scores.device):
        rc = lib().tsenor_max_abs(p, rows, cols, ld, _ptr(out), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_max_abs")
    return out


class Scores:
    """A described score matrix (``tsenor_scores_t``): keeps the tensors alive and builds
    the descriptor.  kind: SCORES_ABS |W|, SCORES_ADMM (W + V*scalar)^2, SCORES_COLDIV
    |W / colvec_j|, SCORES_COLMUL |W| * colvec_j.  W may be float32 or bfloat16.
    ``early_exit_eps`` > 0 switches the stopping test of Algorithm 1 on (non-parity mode);
    ``iters_out`` (1-element int64 device tensor, zeroed by the caller) accumulates the
    iterations run over all blocks."""

    def __init__(self, kind, w, v=None, scalar=0.0, colvec=None, per_block_tau=False, early_exit_eps=0.0,
                 iters_out=None):
        if not (isinstance(w, torch.Tensor) and w.is_cuda and w.dim() == 2 and w.stride(1) == 1):
            raise TypeError("w must be a 2-D row-major CUDA tensor")
        if w.dtype not in (torch.float32, torch.bfloat16):
            raise TypeError("w must be float32 or bfloat16")
        self.kind, self.w, self.v, self.colvec = int(kind), w, v, colvec
        self.rows, self.cols = w.shape
        d = ScoresDesc()
        d.kind = self.kind
        d.w_is_bf16 = int(w.dtype == torch.bfloat16)
        d.w = w.data_ptr()
        d.ld = w.stride(0) if self.rows > 1 else max(w.stride(0), self.cols)
        if v is not None:
            _, r2, c2, ldv = _mat(v, "v")
            if (r2, c2) != (self.rows, self.cols) or v.device != w.device:
                raise ValueError("v and w differ in shape or device")
            d.v, d.ld_v = v.data_ptr(), ldv
        d.scalar = float(scalar)
        if colvec is not None:
            if not (colvec.is_cuda and colvec.dtype == torch.float32 and colvec.is_contiguous()
                    and colvec.numel() == self.cols and colvec.device == w.device):
                raise TypeError("colvec must be a contiguous float32 CUDA vector of length cols on w's device")
            d.colvec = colvec.data_ptr()
        d.per_block_tau = int(bool(per_block_tau))
        d.early_exit_eps = float(early_exit_eps)
        self.iters_out = _out(iters_out, "iters_out", torch.int64, w.device, min_numel=1)
        if iters_out is not None:
            d.dev_iters_out = iters_out.data_ptr()
        self.desc = d

    @property
    def device(self):
        return self.w.device


def solve_scores(src, N, M, tau, iters=300, ls_steps=-1, mask_out=None, status=None, stream=None):
    """tsenor_solve_scores: the whole method on a described score matrix."""
    if mask_out is None:
        mask_out = new_mask(src.rows, src.cols, src.device)
    _mask_out(mask_out, src.rows, src.cols, src.device)
    _out(status, "status", torch.int32, src.device, min_numel=1)
    with _on(src.device):
        rc = lib().tsenor_solve_scores(C.byref(src.desc), src.rows, src.cols, int(N), int(M), float(tau), int(iters),
                                       int(ls_steps), _ptr(mask_out), _ptr(status), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_solve_scores")
    return mask_out


def dykstra_scores(src, N, M, tau, iters=300, plan_is_log=False, plan_out=None, status=None, stream=None):
    """tsenor_dykstra_scores: Algorithm 1 only on a described score matrix."""
    if plan_out is None:
        plan_out = torch.empty((src.rows, src.cols), dtype=torch.float32, device=src.device)
    pp, pr, pc, ldp = _mat(plan_out, "plan_out")
    if (pr, pc) != (src.rows, src.cols) or plan_out.device != src.device:
        raise ValueError("plan_out must have the shape and device of the score source")
    _out(status, "status", torch.int32, src.device, min_numel=1)
    with _on(src.device):
        rc = lib().tsenor_dykstra_scores(C.byref(src.desc), src.rows, src.cols, int(N), int(M), float(tau),
                                         int(iters), pp, ldp, int(bool(plan_is_log)), _ptr(status), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_dykstra_scores")
    return plan_out


def scores_max(src, out=None, stream=None):
    """tsenor_scores_max: 1-element float32 device tensor with the largest score."""
    if out is None:
        out = torch.empty(1, dtype=torch.float32, device=src.device)
    _out(out, "out", torch.float32, src.device, min_numel=1)
    with _on(src.device):
        rc = lib().tsenor_scores_max(C.byref(src.desc), src.rows, src.cols, _ptr(out), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_scores_max")
    return out


def scores_materialize(src, out=None, stream=None):
    """tsenor_scores_materialize: the described scores as a float32 matrix."""
    if out is None:
        out = torch.empty((src.rows, src.cols), dtype=torch.float32, device=src.device)
    p, orows, ocols, ld = _mat(out, "out")
    if (orows, ocols) != (src.rows, src.cols) or out.device != src.device:
        raise ValueError("out must have the shape and device of the score source")
    with _on(src.device):
        rc = lib().tsenor_scores_materialize(C.byref(src.desc), src.rows, src.cols, p, ld, _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_scores_materialize")
    return out


def keep_better(src, prev_mask, mask_inout, obj2_out=None, stream=None):
    """tsenor_keep_better: keeps ``prev_mask`` in ``mask_inout`` if it retains more score.
    Returns the 2-element float64 device tensor {objective(new), objective(previous)}."""
    if obj2_out is None:
        obj2_out = torch.empty(2, dtype=torch.float64, device=src.device)
    _mask_out(prev_mask, src.rows, src.cols, src.device, "prev_mask")
    _mask_out(mask_inout, src.rows, src.cols, src.device, "mask_inout")
    _out(obj2_out, "obj2_out", torch.float64, src.device, min_numel=2)
    with _on(src.device):
        rc = lib().tsenor_keep_better(C.byref(src.desc), src.rows, src.cols, _ptr(prev_mask), _ptr(mask_inout),
                                      _ptr(obj2_out), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_keep_better")
    return obj2_out


def simple_round(plan_key, N, M, mask_out=None, stream=None):
    """tsenor_simple_round: row-wise then column-wise N:M rounding of the plan."""
    pk, rows, cols, ldk = _mat(plan_key, "plan_key")
    if mask_out is None:
        mask_out = new_mask(rows, cols, plan_key.device)
    _mask_out(mask_out, rows, cols, plan_key.device)
    with _on(plan_key.device):
        rc = lib().tsenor_simple_round(pk, ldk, rows, cols, int(N), int(M), _ptr(mask_out), _stream(stream))
    if rc:
        raise TsenorError(rc, "tsenor_simple_round")
    return mask_out
