"""CPU oracle for the TSENOR mask solver -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes wrappers around ``tsenor_oracle.c`` (plain fp64 C written
from Algorithm 1, Algorithm 2, Eq. 2 and Eq. 6 of the paper).  Only the tests,
the smoke check and the benchmark's ``cpu_baseline`` / ``--impl reference``
legs may import this package; the CUDA library and its Python binding never
do, and nothing here imports them.

Mask layout everywhere: ``uint32[rows, ceil(cols/32)]``, bit ``c % 32`` of
word ``c // 32`` of row ``r`` is ``S[r, c]``.
"""
import ctypes as C

import numpy as np

from .build import build as _build

_lib = None

_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(np.uint32, flags="C_CONTIGUOUS")
_i32p = np.ctypeslib.ndpointer(np.int32, flags="C_CONTIGUOUS")


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build())
        i64, i32, f32, f64, vp = C.c_int64, C.c_int, C.c_float, C.c_double, C.c_void_p
        L.oracle_dykstra_block.argtypes = [_f64p, i32, i32, f64, i32, i32, _f64p, _f64p]
        L.oracle_dykstra_block.restype = None
        L.oracle_greedy_block.argtypes = [_f64p, i32, i32, _u8p, _i32p, _i32p]
        L.oracle_greedy_block.restype = i32
        L.oracle_swap_scores_block.argtypes = [_f32p, i32, _u8p, i32, i32, _f32p]
        L.oracle_swap_scores_block.restype = None
        L.oracle_repair_block.argtypes = [_f32p, i32, i32, i32, _u8p, _i32p, _i32p,
                                          C.POINTER(i32), C.POINTER(i32)]
        L.oracle_repair_block.restype = i32
        L.oracle_bruteforce_block.argtypes = [_f64p, i32, i32, C.POINTER(f64), vp]
        L.oracle_bruteforce_block.restype = i64
        L.oracle_dykstra.argtypes = [_f32p, i64, i64, i64, i32, i32, f32, i32, _f64p,
                                     i64, i32]
        L.oracle_dykstra.restype = i32
        L.oracle_round.argtypes = [_f32p, i64, _f32p, i64, i64, i64, i32, i32, i32,
                                   _u32p, vp, vp, vp, C.POINTER(i64)]
        L.oracle_round.restype = i32
        L.oracle_solve.argtypes = [_f32p, i64, i64, i64, i32, i32, f32, i32, i32,
                                   _u32p, vp, vp, vp, C.POINTER(i64)]
        L.oracle_solve.restype = i32
        L.oracle_dykstra_blocktau.argtypes = L.oracle_dykstra.argtypes
        L.oracle_dykstra_blocktau.restype = i32
        L.oracle_solve_blocktau.argtypes = L.oracle_solve.argtypes
        L.oracle_solve_blocktau.restype = i32
        L.oracle_objective.argtypes = [_f32p, i64, _u32p, i64, i64]
        L.oracle_objective.restype = f64
        L.oracle_count_infeasible.argtypes = [_u32p, i64, i64, i32, i32]
        L.oracle_count_infeasible.restype = i64
        L.oracle_bruteforce.argtypes = [_f32p, i64, i64, i64, i32, i32, _f64p]
        L.oracle_bruteforce.restype = i32
        L.oracle_block_objectives.argtypes = [_f32p, i64, _u32p, i64, i64, i32, _f64p]
        L.oracle_block_objectives.restype = i32
        L.oracle_max_abs.argtypes = [_f32p, i64, i64, i64]
        L.oracle_max_abs.restype = f32
        L.oracle_scores.argtypes = [i32, _f32p, i64, vp, i64, f32, vp, i64, i64, _f32p, i64]
        L.oracle_scores.restype = i32
        L.oracle_keep_better.argtypes = [_f32p, i64, i64, i64, _u32p, _u32p, _f64p]
        L.oracle_keep_better.restype = i32
        L.oracle_simple_round.argtypes = [_f32p, i64, i64, i64, i32, i32, _u32p]
        L.oracle_simple_round.restype = i32
        L.oracle_dykstra_block_earlyexit.argtypes = [_f64p, i32, i32, f64, i32, f64, i32, _f64p, _f64p]
        L.oracle_dykstra_block_earlyexit.restype = i32
        L.oracle_solve_earlyexit.argtypes = [_f32p, i64, i64, i64, i32, i32, f32, i32, i32, f64, i32, _u32p, _i32p]
        L.oracle_solve_earlyexit.restype = i32
        L.oracle_dykstra_earlyexit.argtypes = [_f32p, i64, i64, i64, i32, i32, f32, i32, f64, i32, _f64p, i64, i32,
                                               _i32p]
        L.oracle_dykstra_earlyexit.restype = i32
        L.oracle_num_threads.argtypes = []
        L.oracle_num_threads.restype = i32
        _lib = L
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what}: bad arguments (status {rc})")


# ---------------------------------------------------------------- per block

def dykstra_block(w, N, tau, iters, extra_steps=0):
    """Algorithm 1 (log domain) on one block.  Returns ``(x, q) = (log S, log Q)``
    after ``iters`` iterations plus ``extra_steps`` (0..2) projections of the
    next one (1: rows, 2: rows and columns)."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    M = w.shape[0]
    assert w.shape == (M, M)
    x = np.empty((M, M), np.float64)
    q = np.empty((M, M), np.float64)
    lib().oracle_dykstra_block(w, M, int(N), float(tau), int(iters), int(extra_steps), x, q)
    return x, q


def greedy_block(key, N):
    """Algorithm 2 lines 1-6.  Returns ``(S uint8[M,M], R int32[M], C int32[M])``."""
    key = np.ascontiguousarray(key, dtype=np.float64)
    M = key.shape[0]
    S = np.zeros((M, M), np.uint8)
    R = np.zeros(M, np.int32)
    Cc = np.zeros(M, np.int32)
    lib().oracle_greedy_block(key, M, int(N), S, R, Cc)
    return S, R, Cc


def swap_scores_block(w, S, i, j):
    """Eq. 6 for unsaturated row ``i`` / column ``j`` (0-based): fp32 ``[M,M]``
    with ``-inf`` where the penalty applies."""
    w = _f32(w)
    M = w.shape[0]
    S = np.ascontiguousarray(S, dtype=np.uint8)
    out = np.empty((M, M), np.float32)
    lib().oracle_swap_scores_block(w, M, S, int(i), int(j), out)
    return out


def repair_block(w, S, R, Cc, N, ls_steps=-1):
    """Algorithm 2 lines 7-13 on a greedy result.  Returns
    ``(S, R, C, feasible, steps, nonpositive_swaps)`` (copies)."""
    w = _f32(w)
    M = w.shape[0]
    S = np.array(S, dtype=np.uint8, order="C", copy=True)
    R = np.array(R, dtype=np.int32, copy=True)
    Cc = np.array(Cc, dtype=np.int32, copy=True)
    steps, nonpos = C.c_int(0), C.c_int(0)
    ok = lib().oracle_repair_block(w, M, int(N), int(ls_steps), S, R, Cc,
                                   C.byref(steps), C.byref(nonpos))
    return S, R, Cc, bool(ok), steps.value, nonpos.value


def bruteforce_block(w, N, want_mask=False):
    """Maximum of Eq. 2 over every feasible 0/1 block by enumeration.
    Returns ``(optimum, count_of_feasible_masks[, mask])``."""
    w = np.ascontiguousarray(np.abs(w), dtype=np.float64)
    M = w.shape[0]
    best = C.c_double(0.0)
    mask = np.zeros((M, M), np.uint8)
    cnt = lib().oracle_bruteforce_block(w, M, int(N), C.byref(best),
                                        mask.ctypes.data_as(C.c_void_p))
    if cnt < 0:
        raise ValueError("bruteforce_block: bad arguments")
    return (best.value, cnt, mask) if want_mask else (best.value, cnt)


# ------------------------------------------------------------ whole matrix

def mask_words_per_row(cols):
    return (int(cols) + 31) // 32


def dykstra(scores, N, M, tau, iters, plan_is_log=False, per_block_tau=False):
    """Algorithm 1 on every aligned M x M tile; fp64 plan in matrix layout.  With
    ``per_block_tau`` every block runs with tau / (its own largest score)."""
    s = _f32(scores)
    rows, cols = s.shape
    plan = np.empty((rows, cols), np.float64)
    fn = lib().oracle_dykstra_blocktau if per_block_tau else lib().oracle_dykstra
    _check(fn(s, rows, cols, cols, int(N), int(M), float(tau),
                                int(iters), plan, cols, int(bool(plan_is_log))), "dykstra")
    return plan


def dykstra_block_earlyexit(w, N, tau, max_iters, eps, check_every=1):
    """Algorithm 1 on one block with the stopping test (marginal violation below ``eps`` at an
    iteration t = 1 + k * ``check_every``, k >= 1).  Returns ``(x, q, iterations run)``."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    M = w.shape[0]
    x = np.empty((M, M), np.float64)
    q = np.empty((M, M), np.float64)
    ran = lib().oracle_dykstra_block_earlyexit(w, M, int(N), float(tau), int(max_iters), float(eps),
                                               int(check_every), x, q)
    return x, q, int(ran)


def solve_earlyexit(scores, N, M, tau, max_iters, eps, check_every=1, ls_steps=-1):
    """The whole method with the stopping test in Algorithm 1.  Returns ``(mask bits, iterations
    run by every block)``."""
    s = _f32(scores)
    rows, cols = s.shape
    bits = np.zeros((rows, mask_words_per_row(cols)), np.uint32)
    iters = np.zeros((rows // M) * (cols // M), np.int32)
    _check(lib().oracle_solve_earlyexit(s, rows, cols, cols, int(N), int(M), float(tau), int(max_iters),
                                        int(ls_steps), float(eps), int(check_every), bits, iters), "solve_earlyexit")
    return bits, iters


def dykstra_earlyexit(scores, N, M, tau, max_iters, eps, check_every=1, plan_is_log=False):
    """Algorithm 1 with the stopping test on every tile: ``(fp64 plan, iterations per block)``."""
    s = _f32(scores)
    rows, cols = s.shape
    plan = np.empty((rows, cols), np.float64)
    iters = np.zeros((rows // M) * (cols // M), np.int32)
    _check(lib().oracle_dykstra_earlyexit(s, rows, cols, cols, int(N), int(M), float(tau), int(max_iters),
                                          float(eps), int(check_every), plan, cols, int(bool(plan_is_log)), iters),
           "dykstra_earlyexit")
    return plan, iters


def _stats_arrays(nblk, want):
    if not want:
        return None, None, None, (None, None, None)
    st = np.zeros(nblk, np.int32)
    npz = np.zeros(nblk, np.int32)
    ob = np.zeros(nblk, np.float64)
    ptrs = tuple(a.ctypes.data_as(C.c_void_p) for a in (st, npz, ob))
    return st, npz, ob, ptrs


def round_plan(plan_key, scores, N, M, ls_steps=-1, stats=False):
    """Algorithm 2 on every tile from fp32 keys and fp32 scores.  Returns the
    packed mask, or ``(mask, info)`` with per-block statistics."""
    k = _f32(plan_key)
    s = _f32(scores)
    rows, cols = s.shape
    assert k.shape == s.shape
    bits = np.zeros((rows, mask_words_per_row(cols)), np.uint32)
    nblk = (rows // M) * (cols // M)
    st, npz, ob, ptrs = _stats_arrays(nblk, stats)
    bad = C.c_int64(0)
    _check(lib().oracle_round(k, cols, s, cols, rows, cols, int(N), int(M),
                              int(ls_steps), bits, *ptrs, C.byref(bad)), "round")
    if stats:
        return bits, dict(steps=st, nonpos=npz, obj=ob, underfilled=bad.value)
    return bits


def solve(scores, N, M, tau, iters, ls_steps=-1, stats=False, per_block_tau=False):
    """Algorithm 1 (fp64) + Algorithm 2 on every tile.  Returns the packed
    mask, or ``(mask, info)`` with per-block statistics.  With ``per_block_tau``
    every block runs with tau / (its own largest score)."""
    s = _f32(scores)
    rows, cols = s.shape
    bits = np.zeros((rows, mask_words_per_row(cols)), np.uint32)
    nblk = (rows // M) * (cols // M)
    st, npz, ob, ptrs = _stats_arrays(nblk, stats)
    bad = C.c_int64(0)
    fn = lib().oracle_solve_blocktau if per_block_tau else lib().oracle_solve
    _check(fn(s, rows, cols, cols, int(N), int(M), float(tau),
                              int(iters), int(ls_steps), bits, *ptrs, C.byref(bad)), "solve")
    if stats:
        return bits, dict(steps=st, nonpos=npz, obj=ob, underfilled=bad.value)
    return bits


def objective(scores, bits):
    s = _f32(scores)
    b = np.ascontiguousarray(bits, dtype=np.uint32)
    return float(lib().oracle_objective(s, s.shape[1], b, s.shape[0], s.shape[1]))


def count_infeasible(bits, rows, cols, N, M):
    b = np.ascontiguousarray(bits, dtype=np.uint32)
    r = lib().oracle_count_infeasible(b, int(rows), int(cols), int(N), int(M))
    if r < 0:
        raise ValueError("count_infeasible: bad shape")
    return int(r)


def bruteforce(scores, N, M):
    """Per-tile optimum of Eq. 2 by enumeration (tiny M only)."""
    s = _f32(scores)
    rows, cols = s.shape
    out = np.empty((rows // M) * (cols // M), np.float64)
    _check(lib().oracle_bruteforce(s, rows, cols, cols, int(N), int(M), out), "bruteforce")
    return out


def block_objectives(scores, bits, M):
    s = _f32(scores)
    rows, cols = s.shape
    b = np.ascontiguousarray(bits, dtype=np.uint32)
    out = np.empty((rows // M) * (cols // M), np.float64)
    _check(lib().oracle_block_objectives(s, cols, b, rows, cols, int(M), out), "block_objectives")
    return out


def max_abs(scores):
    s = _f32(scores)
    return float(lib().oracle_max_abs(s, s.shape[0], s.shape[1], s.shape[1]))


SCORES_ABS, SCORES_ADMM, SCORES_COLDIV, SCORES_COLMUL = 0, 1, 2, 3


def scores(kind, w, v=None, scalar=0.0, colvec=None):
    """Score matrix of a pruning framework (Section 4): |W|, the ADMM D-update score
    (W + V*scalar)^2 with scalar = 1/rho, the SparseGPT group score |W_ij / d_j|, or the
    Wanda score |W_ij| a_j.  fp32 in, fp32 out, one rounding per operation."""
    w = _f32(w)
    rows, cols = w.shape
    out = np.empty((rows, cols), np.float32)
    vv = None if v is None else _f32(v)
    cv = None if colvec is None else _f32(colvec)
    rc = lib().oracle_scores(int(kind), w, cols,
                             None if vv is None else vv.ctypes.data_as(C.c_void_p), cols,
                             float(scalar), None if cv is None else cv.ctypes.data_as(C.c_void_p),
                             rows, cols, out, cols)
    _check(rc, "scores")
    return out


def keep_better(score_matrix, prev_mask, new_mask):
    """Safeguard of the ADMM integration (Appendix A.1.3): the new mask unless it retains
    less score than the previous one.  Returns ``(kept_mask, obj_new, obj_prev)``."""
    s = _f32(score_matrix)
    prev = np.ascontiguousarray(prev_mask, dtype=np.uint32)
    kept = np.array(new_mask, dtype=np.uint32, order="C", copy=True)
    obj2 = np.zeros(2, np.float64)
    _check(lib().oracle_keep_better(s, s.shape[1], s.shape[0], s.shape[1], prev, kept, obj2), "keep_better")
    return kept, float(obj2[0]), float(obj2[1])


def simple_round(plan_key, N, M):
    """"Simple" rounding of the ablation study: row-wise then column-wise N:M rounding."""
    k = _f32(plan_key)
    rows, cols = k.shape
    bits = np.zeros((rows, mask_words_per_row(cols)), np.uint32)
    _check(lib().oracle_simple_round(k, cols, rows, cols, int(N), int(M), bits), "simple_round")
    return bits


def num_threads():
    return int(lib().oracle_num_threads())


def unpack_mask(bits, cols):
    """Packed mask -> uint8[rows, cols] (host helper for tests)."""
    b = np.ascontiguousarray(bits, dtype=np.uint32)
    u8 = b.view(np.uint8).reshape(b.shape[0], -1)
    return np.unpackbits(u8, axis=1, bitorder="little")[:, :cols]
