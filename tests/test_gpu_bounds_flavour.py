"""The checked build flavour of the library (``libtsenor_bounds.so``: the same sources compiled with
-DTSENOR_BOUNDS, every computed index of the loaders, the rounding tables, the local search and the
writers tested before use, a bad one reported as TSENOR_DEV_INTERNAL and skipped).  It stands in for
a memory checker: on every block size, both register layouts, wide matrices with a ragged last
panel and slabs, no index check may fire, and the results must equal the normal library's."""
import numpy as np
import pytest
import torch

from paper_2505_23949_b200 import binding as ts
from paper_2505_23949_b200 import build as ts_build
from paper_2505_23949_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

SHAPES = [(4, 2, 8, 516), (8, 3, 16, 520), (16, 8, 32, 272), (32, 16, 64, 160), (32, 7, 32, 32),
          (4, 2, 4 * 259, 4), (8, 4, 8 * 131, 8), (16, 8, 16 * 35, 16), (32, 16, 32 * 11, 32)]


@pytest.fixture()
def checked_library():
    """Swaps the binding's library for the checked flavour for the duration of a test."""
    path = ts_build.build(bounds=True)
    normal_path, normal_lib = ts.LIB_PATH, ts.lib()
    ts._lib, ts.LIB_PATH = None, path
    try:
        assert ts.lib() is not normal_lib
        yield
    finally:
        ts._lib, ts.LIB_PATH = normal_lib, normal_path


def _run_all(M, N, rows, cols, layout):
    ts.set_layout(layout)
    W = synth.student_t_abs(rows, cols, 0.02, seed=31 * M + N)
    Wd = torch.from_numpy(W).to(DEV)
    tau = synth.default_tau(float(W.max()))
    st = ts.new_status(DEV)
    mask = ts.solve(Wd, N, M, tau, 60, -1, status=st)
    plan = ts.dykstra(Wd, N, M, tau, 60, plan_is_log=True, status=st)
    strict = ts.round_plan(plan, Wd, N, M, ls_steps=1, status=st)
    ee = ts.solve_scores(ts.Scores(ts.SCORES_ABS, Wd, early_exit_eps=1e-2), N, M, tau, 60, -1, status=st)
    torch.cuda.synchronize()
    ts.set_layout(ts.LAYOUT_AUTO)
    return int(st.item()), [t.cpu().numpy() for t in (mask, plan, strict, ee)]


@pytest.mark.parametrize("layout", [ts.LAYOUT_THROUGHPUT, ts.LAYOUT_LATENCY])
@pytest.mark.parametrize("M,N,rows,cols", SHAPES)
def test_no_index_check_fires_and_results_equal_the_normal_build(checked_library, M, N, rows, cols, layout):
    flags, got = _run_all(M, N, rows, cols, layout)
    assert (flags & ts.DEV_INTERNAL) == 0, "an index check fired"
    checked, checked_path = ts._lib, ts.LIB_PATH
    ts._lib, ts.LIB_PATH = None, ts_build.LIB
    try:
        flags_n, want = _run_all(M, N, rows, cols, layout)
    finally:
        ts._lib, ts.LIB_PATH = checked, checked_path
    assert flags == flags_n
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
