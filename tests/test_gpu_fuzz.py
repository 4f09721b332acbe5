"""Randomised GPU-vs-oracle cases: shapes, N:M, tau, iteration counts, repair modes, key
distributions and leading dimensions drawn from a seeded generator."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_23949_b200 import binding as ts

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["throughput", "latency"])
def _both_register_layouts(request):
    """Every case runs under both register layouts of the Dykstra stage (these matrices are
    small, so the automatic choice alone would never exercise the throughput layout)."""
    ts.set_layout(ts.LAYOUT_THROUGHPUT if request.param == "throughput" else ts.LAYOUT_LATENCY)
    yield
    ts.set_layout(ts.LAYOUT_AUTO)
DEV = "cuda:0"


def _bits(t):
    return t.cpu().numpy().view(np.uint32)


def _case(rng):
    M = int(rng.choice([4, 8, 16, 32]))
    N = int(rng.integers(1, M))
    rows = M * int(rng.integers(1, 6))
    cols = M * int(rng.integers(1, 40)) if rng.random() < 0.85 else M
    kind = rng.integers(0, 4)
    if kind == 0:
        W = np.abs(rng.standard_normal((rows, cols)))
    elif kind == 1:
        W = np.abs(rng.standard_t(2.5, (rows, cols)))
    elif kind == 2:
        W = np.round(np.abs(rng.standard_normal((rows, cols))) * 4) / 4      # many equal scores
    else:
        W = np.abs(rng.standard_normal((rows, cols))) * np.where(rng.random(cols) < 0.05, 30.0, 1.0)[None, :]
    W = (W * 10.0 ** rng.uniform(-3, 1)).astype(np.float32)
    return M, N, rows, cols, W


@pytest.mark.parametrize("seed", range(6))
def test_random_rounding_cases_are_bit_exact(seed):
    rng = np.random.default_rng(9000 + seed)
    for _ in range(25):
        M, N, rows, cols, W = _case(rng)
        mode = rng.integers(0, 3)
        if mode == 0:
            key = rng.standard_normal((rows, cols)).astype(np.float32)
        elif mode == 1:
            key = np.minimum(rng.standard_normal((rows, cols)) * 3, 0).astype(np.float32)
        else:
            key = (np.round(rng.standard_normal((rows, cols)) * 2) / 2).astype(np.float32)
        ls = int(rng.choice([-1, -1, 0, 1, 3, 10]))
        pad = int(rng.integers(0, 3))
        kd = torch.zeros((rows, cols + pad), device=DEV)[:, :cols]
        kd.copy_(torch.from_numpy(key))
        wd = torch.zeros((rows, cols + 2 * pad), device=DEV)[:, pad:pad + cols]
        wd.copy_(torch.from_numpy(W))
        st = ts.new_status(DEV)
        got = _bits(ts.round_plan(kd, wd, N, M, ls_steps=ls, status=st))
        want, info = oracle.round_plan(key, W, N, M, ls_steps=ls, stats=True)
        assert np.array_equal(got, want), (seed, M, N, rows, cols, ls)
        assert (int(st.item()) & ts.DEV_INTERNAL) == 0
        assert bool(int(st.item()) & ts.DEV_UNDERFILLED) == (info["underfilled"] > 0)


@pytest.mark.parametrize("seed", range(6))
def test_random_solve_cases_match_the_oracle(seed):
    rng = np.random.default_rng(7000 + seed)
    for _ in range(12):
        M, N, rows, cols, W = _case(rng)
        tau = float(rng.choice([20.0, 60.0, 200.0]) / W.max())
        iters = int(rng.choice([1, 2, 5, 30, 100, 300]))
        Wd = torch.from_numpy(W).to(DEV)
        st = ts.new_status(DEV)
        plan = ts.dykstra(Wd, N, M, tau, iters, status=st).cpu().numpy()
        ref = oracle.dykstra(W, N, M, tau, iters)
        assert np.abs(plan - ref).max() <= 1e-4, (seed, M, N, rows, cols, iters)
        got = _bits(ts.solve(Wd, N, M, tau, iters, status=st))
        assert int(st.item()) == 0
        assert oracle.count_infeasible(got, rows, cols, N, M) == 0
        if iters >= 100:
            # After a handful of iterations hundreds of plan entries sit within rounding of the cap,
            # the greedy order among them is decided by noise (exact ties in fp64, 1e-7 apart in
            # fp32) and masks legitimately differ; the objective is compared once the plan has
            # separated, as at the method's operating point T = 300.
            # These matrices hold a few dozen blocks, so one block that legitimately differs moves
            # the total by more than 1e-4: 2e-3 here; the stated 1e-4 per matrix is held on the
            # matrices of >= 1024 blocks below.
            want = oracle.solve(W, N, M, tau, iters)
            o_gpu, o_ref = oracle.objective(W, got), oracle.objective(W, want)
            assert abs(o_gpu - o_ref) <= 2e-3 * o_ref, ("bound 2e-3 (small matrix)", seed, M, N, rows, cols, iters)


@pytest.mark.parametrize("seed", range(8))
def test_random_matrices_of_1024_blocks_or_more_hold_the_stated_bounds(seed):
    """At the operating point (T = 300) and with at least 1024 blocks per matrix the stated bounds
    apply as they are: plan within 1e-4, per-matrix objective within 1e-4 relative."""
    rng = np.random.default_rng(7100 + seed)
    M = [4, 8, 16, 32][seed % 4]
    N = M // 2 if seed < 4 else int(rng.integers(1, M))
    nbr, nbc = int(rng.integers(16, 40)), int(rng.integers(64, 80))
    rows, cols = M * nbr, M * nbc
    assert nbr * nbc >= 1024
    kind = int(rng.integers(0, 3))
    if kind == 0:
        W = np.abs(rng.standard_normal((rows, cols))) * 0.02
    elif kind == 1:
        W = np.abs(rng.standard_t(3.0, (rows, cols))) * 0.0115
    else:
        W = np.abs(rng.standard_normal((rows, cols))) * 0.02 * np.where(rng.random(cols) < 0.01, 20.0, 1.0)[None, :]
    W = W.astype(np.float32)
    tau = float(rng.choice([50.0, 200.0]) / W.max())
    Wd = torch.from_numpy(W).to(DEV)
    st = ts.new_status(DEV)
    plan = ts.dykstra(Wd, N, M, tau, 300, status=st).cpu().numpy()
    assert np.abs(plan - oracle.dykstra(W, N, M, tau, 300)).max() <= 1e-4, ("bound 1e-4 (plan)", seed, M, N)
    got = _bits(ts.solve(Wd, N, M, tau, 300, status=st))
    assert int(st.item()) == 0
    assert oracle.count_infeasible(got, rows, cols, N, M) == 0
    o_gpu, o_ref = oracle.objective(W, got), oracle.objective(W, oracle.solve(W, N, M, tau, 300))
    assert abs(o_gpu - o_ref) <= 1e-4 * o_ref, ("bound 1e-4 (objective)", seed, M, N, rows, cols, kind)
