"""Pins for the CPU oracle: everything here checks ``oracle/`` against facts the
paper prints or the mathematics fixes, never against the oracle itself and never
against the CUDA path."""
import itertools
import os

import numpy as np
import pytest
from scipy.optimize import linear_sum_assignment, linprog, minimize

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "fig2_worked_example.txt")


def _read_fig2():
    out, cur = {}, None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0][0].isalpha() and tok[0] != "ninf":
            if len(tok) == 1:
                cur = tok[0]
                out[cur] = []
            else:
                out[tok[0]] = [float(t) for t in tok[1:]]
                cur = None
        else:
            out[cur].append([-np.inf if t == "ninf" else float(t) for t in tok])
    return {k: np.array(v) for k, v in out.items()}


def _lp_optimum(w, N):
    """Optimum of the relaxed problem (Eq. 3) with a generic LP solver."""
    M = w.shape[0]
    A = np.zeros((2 * M, M * M))
    for i in range(M):
        A[i, i * M:(i + 1) * M] = 1
        A[M + i, i::M] = 1
    r = linprog(-w.ravel(), A_eq=A, b_eq=np.full(2 * M, N), bounds=(0, 1), method="highs")
    assert r.status == 0
    return -r.fun


# ------------------------------------------------------------------ Fig. 2

def test_fig2_greedy_swap_scores_and_final_mask():
    g = _read_fig2()
    w = g["scores"]
    S, R, C = oracle.greedy_block(w, 2)
    assert np.array_equal(S, g["greedy_mask"].astype(np.uint8))
    assert round(float((S * w).sum()), 2) == g["greedy_objective"][0]
    i, j = int(g["deficit_row"][0]) - 1, int(g["deficit_col"][0]) - 1
    assert list(np.flatnonzero(R < 2)) == [i] and list(np.flatnonzero(C < 2)) == [j]
    sc = oracle.swap_scores_block(w, S, i, j)
    want = g["swap_scores"]
    assert np.array_equal(np.isinf(sc), np.isinf(want))
    fin = np.isfinite(want)
    assert np.allclose(sc[fin], want[fin], atol=5e-3)  # figure prints two decimals
    bi, bj = (int(v) - 1 for v in g["best_swap"])
    assert np.unravel_index(np.argmax(sc), sc.shape) == (bi, bj)
    S2, R2, C2, ok, steps, nonpos = oracle.repair_block(w, S, R, C, 2)
    assert ok and steps == 1 and nonpos == 0
    assert np.array_equal(S2, g["final_mask"].astype(np.uint8))
    assert round(float((S2 * w).sum()), 2) == g["final_objective"][0]
    # the paper-strict loop (L = 10, improving swaps only) gives the same here
    S3, *_ = oracle.repair_block(w, S, R, C, 2, ls_steps=10)
    assert np.array_equal(S3, S2)
    # and the figure's final mask is the true optimum of Eq. 2 for this block
    opt, cnt = oracle.bruteforce_block(w, 2)
    assert cnt == 90 and abs(opt - 6.05) < 1e-12


# ------------------------------------------------------------- brute force

def _count_feasible_by_bit_patterns(M, N):
    cnt = 0
    for code in range(1 << (M * M)):
        rows = [(code >> (i * M)) & ((1 << M) - 1) for i in range(M)]
        if any(bin(r).count("1") != N for r in rows):
            continue
        if all(sum((r >> j) & 1 for r in rows) == N for j in range(M)):
            cnt += 1
    return cnt


def test_bruteforce_counts_match_direct_enumeration():
    w = np.ones((4, 4))
    assert oracle.bruteforce_block(w, 2)[1] == _count_feasible_by_bit_patterns(4, 2) == 90
    assert oracle.bruteforce_block(w, 1)[1] == 24
    assert oracle.bruteforce_block(w, 3)[1] == 24
    assert oracle.bruteforce_block(np.ones((3, 3)), 1)[1] == _count_feasible_by_bit_patterns(3, 1) == 6
    # number of 5x5 0/1 matrices with all line sums 2 (known sequence: 1, 6, 90, 2040)
    assert oracle.bruteforce_block(np.ones((5, 5)), 2)[1] == 2040


def test_bruteforce_equals_lp_and_assignment():
    rng = np.random.default_rng(11)
    for _ in range(25):
        w = np.abs(rng.standard_normal((4, 4)))
        opt, _, mask = oracle.bruteforce_block(w, 2, want_mask=True)
        assert mask.sum(0).tolist() == [2] * 4 and mask.sum(1).tolist() == [2] * 4
        assert abs((mask * w).sum() - opt) < 1e-12
        assert abs(opt - _lp_optimum(w, 2)) < 1e-9       # integrality of Eq. 3
    for M in (4, 5, 6):
        w = np.abs(rng.standard_normal((M, M)))
        r, c = linear_sum_assignment(w, maximize=True)    # N = 1: perfect matching
        assert abs(oracle.bruteforce_block(w, 1)[0] - w[r, c].sum()) < 1e-12
        r, c = linear_sum_assignment(w)                   # N = M-1: drop a min matching
        assert abs(oracle.bruteforce_block(w, M - 1)[0] - (w.sum() - w[r, c].sum())) < 1e-12


# ---------------------------------------------------------------- Dykstra

def test_dykstra_tau_zero_gives_uniform_plan():
    w = np.abs(np.random.default_rng(0).standard_normal((8, 8)))
    x, q = oracle.dykstra_block(w, 4, 0.0, 1)
    assert np.allclose(np.exp(x), 4 / 8, atol=1e-15) and np.all(q == 0)


def test_dykstra_is_sinkhorn_while_cap_is_slack():
    """With small tau no entry reaches the cap, the dual stays 0 and Algorithm 1
    is plain matrix scaling of exp(tau w): cross-ratios of exp(tau w) survive."""
    rng = np.random.default_rng(1)
    w = np.abs(rng.standard_normal((8, 8)))
    tau = 0.05
    for iters in (1, 2, 7):
        x, q = oracle.dykstra_block(w, 4, tau, iters)
        assert np.all(q == 0) and x.max() < 0
        for (i, k, j, l) in [(0, 1, 2, 3), (5, 2, 7, 0), (3, 4, 4, 6)]:
            lhs = x[i, j] + x[k, l] - x[i, l] - x[k, j]
            rhs = tau * (w[i, j] + w[k, l] - w[i, l] - w[k, j])
            assert abs(lhs - rhs) < 1e-13
    # against an independently written linear-domain scaling of exp(tau w)
    S = np.exp(tau * w)
    for _ in range(7):
        S = S * (4 / S.sum(1, keepdims=True))
        S = S * (4 / S.sum(0, keepdims=True))
    assert np.allclose(np.exp(x), S, rtol=1e-12)


@pytest.mark.parametrize("M,N", [(4, 2), (8, 4), (16, 8), (32, 16), (8, 3)])
def test_dykstra_invariants_every_iteration(M, N):
    rng = np.random.default_rng(100 + M + N)
    w = np.abs(rng.standard_normal((M, M)))
    tau = 200.0 / w.max()
    for iters in (1, 2, 5, 40):
        x, q = oracle.dykstra_block(w, N, tau, iters)
        assert np.all(x <= 0) and np.all(q >= 0) and np.all(x[q > 0] == 0)
        # x + q - tau w is a sum of a row term and a column term at every iterate
        # (each projection only rescales rows or columns of S .* Q)
        D = x + q - tau * w
        assert np.allclose(D - D[:, :1] - D[:1, :] + D[0, 0], 0, atol=1e-9)
        xa, _ = oracle.dykstra_block(w, N, tau, iters, extra_steps=1)
        assert np.allclose(np.exp(xa).sum(1), N, rtol=1e-12)
        xb, _ = oracle.dykstra_block(w, N, tau, iters, extra_steps=2)
        assert np.allclose(np.exp(xb).sum(0), N, rtol=1e-12)
        # the row step only shifts rows, the column step only shifts columns
        d = xa - x
        assert np.allclose(d, d[:, :1], atol=1e-9)
        d = xb - xa
        assert np.allclose(d, d[:1, :], atol=1e-9)


def test_dykstra_row_first_order_and_symmetries():
    rng = np.random.default_rng(5)
    M, N = 8, 4
    w = np.abs(rng.standard_normal((M, M)))
    tau = 30.0 / w.max()
    x, _ = oracle.dykstra_block(w, N, tau, 25)
    # after ONE iteration and no clip activity the column sums (last projection) are exact
    x1, q1 = oracle.dykstra_block(w, N, 0.01, 1)
    assert np.allclose(np.exp(x1).sum(0), N, rtol=1e-13)
    assert not np.allclose(np.exp(x1).sum(1), N, rtol=1e-9)   # rows came first
    # permuting rows / columns of w permutes the plan
    pr, pc = rng.permutation(M), rng.permutation(M)
    xp, _ = oracle.dykstra_block(w[pr][:, pc], N, tau, 25)
    assert np.allclose(xp, x[pr][:, pc], atol=1e-10)
    # a constant added to a whole row of w is removed by the first row projection
    w2 = w.copy()
    w2[3] += 0.7
    x2, _ = oracle.dykstra_block(w2, N, tau, 25)
    assert np.allclose(x2, x, atol=1e-9)


def test_dykstra_converges_to_the_entropy_regularised_optimum():
    """Fixed point of Algorithm 1 = maximiser of Eq. 4.  The problem is strictly
    concave, so a feasible S with multipliers f_i, g_j, mu_ij >= 0 such that
    log S = tau w + f_i + g_j - mu, mu > 0 only where S = 1, IS the optimum.  The
    certificate is rebuilt here from the plan alone (the oracle's dual is not used),
    and a generic constrained optimiser must not find anything better."""
    rng = np.random.default_rng(7)
    M, N = 4, 2
    w = np.abs(rng.standard_normal((M, M)))
    tau = 6.0
    x, _ = oracle.dykstra_block(w, N, tau, 20000)
    S = np.exp(x)
    assert np.allclose(S.sum(0), N, atol=1e-9) and np.allclose(S.sum(1), N, atol=1e-9)
    assert S.max() <= 1.0
    capped = S > 1 - 1e-12
    assert capped.any() and (~capped).sum() >= 2 * M    # the capacity constraint binds
    # fit f, g on the uncapped entries
    rows, cols = np.nonzero(~capped)
    A = np.zeros((len(rows), 2 * M))
    A[np.arange(len(rows)), rows] = 1
    A[np.arange(len(rows)), M + cols] = 1
    rhs = (x - tau * w)[~capped]
    fg, *_ = np.linalg.lstsq(A, rhs, rcond=None)
    assert np.abs(A @ fg - rhs).max() < 1e-8             # stationarity off the cap
    mu = tau * w + fg[:M, None] + fg[None, M:] - x       # multiplier of S <= 1
    assert np.all(mu[capped] >= -1e-8)                   # dual feasibility on the cap

    def neg(s):
        s = np.clip(s, 1e-300, None)
        return -(s @ w.ravel()) + (s * np.log(s)).sum() / tau

    Aeq = np.zeros((2 * M, M * M))
    for i in range(M):
        Aeq[i, i * M:(i + 1) * M] = 1
        Aeq[M + i, i::M] = 1
    cons = {"type": "eq", "fun": lambda s: Aeq @ s - N, "jac": lambda s: Aeq}
    for start in (np.full(M * M, N / M), S.ravel() * 0.9 + 0.05):
        r = minimize(neg, start, bounds=[(1e-9, 1)] * (M * M), constraints=cons,
                     method="SLSQP", options={"maxiter": 1000, "ftol": 1e-14})
        if np.abs(Aeq @ r.x - N).max() < 1e-7:
            assert neg(S.ravel()) <= r.fun + 1e-8


def test_plan_objective_approaches_lp_optimum_as_entropy_weight_shrinks():
    rng = np.random.default_rng(8)
    M, N = 4, 2
    gaps = {tau: [] for tau in (2.0, 10.0, 50.0)}
    for _ in range(20):
        w = np.abs(rng.standard_normal((M, M)))
        opt = oracle.bruteforce_block(w, N)[0]
        for tau in gaps:
            x, _ = oracle.dykstra_block(w, N, tau / w.max(), 20000)
            gaps[tau].append((opt - (np.exp(x) * w).sum()) / opt)
    m = {t: float(np.mean(g)) for t, g in gaps.items()}
    assert all(min(g) > -1e-9 for g in gaps.values())   # a fractional plan never beats the LP
    assert m[2.0] > m[10.0] > m[50.0] and m[50.0] < 0.02


# --------------------------------------------------------------- rounding

def _order_positions(key):
    M = key.shape[0]
    flat = key.ravel()
    order = sorted(range(M * M), key=lambda e: (-flat[e], e))
    pos = np.empty(M * M, int)
    pos[order] = np.arange(M * M)
    return pos.reshape(M, M)


@pytest.mark.parametrize("M,N", [(4, 2), (8, 4), (8, 2), (16, 8), (32, 16), (6, 5)])
def test_greedy_is_the_unique_fixed_point_of_its_definition(M, N):
    """An entry is taken iff fewer than N taken entries precede it in its row AND in
    its column (strict order: key descending, flat index ascending).  That property
    has exactly one solution, so checking it pins the greedy scan."""
    rng = np.random.default_rng(1000 * M + N)
    for trial in range(12):
        key = rng.standard_normal((M, M))
        if trial % 3 == 1:
            key = np.round(key * 2) / 2          # heavy ties
        if trial % 3 == 2:
            key = np.minimum(key, 0.0)           # many entries exactly at the cap
        S, R, C = oracle.greedy_block(key, N)
        assert np.array_equal(R, S.sum(1)) and np.array_equal(C, S.sum(0))
        assert R.max() <= N and C.max() <= N
        pos = _order_positions(key)
        for i in range(M):
            for j in range(M):
                before_r = int((S[i] * (pos[i] < pos[i, j])).sum())
                before_c = int((S[:, j] * (pos[:, j] < pos[i, j])).sum())
                assert bool(S[i, j]) == (before_r < N and before_c < N)
        # every (unsaturated row, unsaturated column) cell is already taken
        for i in np.flatnonzero(R < N):
            for j in np.flatnonzero(C < N):
                assert S[i, j] == 1


@pytest.mark.parametrize("M,N", [(4, 2), (8, 4), (16, 8), (32, 16), (8, 7), (8, 1)])
def test_repair_reaches_feasibility_in_exactly_deficit_steps(M, N):
    rng = np.random.default_rng(77 * M + N)
    for trial in range(10):
        w = np.abs(rng.standard_normal((M, M))).astype(np.float32)
        key = w if trial % 2 == 0 else np.round(w * 3) / 3
        S, R, C = oracle.greedy_block(key, N)
        deficit = M * N - int(S.sum())
        S2, R2, C2, ok, steps, nonpos = oracle.repair_block(w, S, R, C, N)
        assert ok and steps == deficit
        assert np.all(S2.sum(0) == N) and np.all(S2.sum(1) == N)
        # strict mode never lowers the objective and equals greedy for L = 0
        S0, *_ = oracle.repair_block(w, S, R, C, N, ls_steps=0)
        assert np.array_equal(S0, S)
        SL, _, _, okL, stepsL, nonposL = oracle.repair_block(w, S, R, C, N, ls_steps=10)
        assert nonposL == 0 and (SL * w).sum() >= (S * w).sum() - 1e-6
        if nonpos == 0 and steps <= 10:
            assert np.array_equal(SL, S2)


def test_one_repair_step_applies_the_argmax_of_eq6():
    rng = np.random.default_rng(4)
    M, N = 8, 4
    found = 0
    for _ in range(200):
        w = np.abs(rng.standard_normal((M, M))).astype(np.float32)
        S, R, C = oracle.greedy_block(w, N)
        if S.sum() == M * N:
            continue
        found += 1
        i, j = int(np.flatnonzero(R < N)[0]), int(np.flatnonzero(C < N)[0])
        best, arg = -np.inf, None
        for ip, jp in itertools.product(range(M), range(M)):     # Eq. 6, fp32
            if S[ip, jp] and not S[i, jp] and not S[ip, j]:
                v = np.float32(np.float32(w[i, jp] + w[ip, j]) - w[ip, jp])
                if v > best:
                    best, arg = v, (ip, jp)
        S1, *_ = oracle.repair_block(w, S, R, C, N, ls_steps=1)
        exp = S.copy()
        if best > 0:
            exp[arg] = 0
            exp[arg[0], j] = 1
            exp[i, arg[1]] = 1
        assert np.array_equal(S1, exp)
    assert found > 10


# ------------------------------------------------------------ whole method

def test_solve_never_beats_and_mostly_reaches_the_optimum_2_4():
    rng = np.random.default_rng(21)
    W = np.abs(rng.standard_normal((128, 128)) * 0.02).astype(np.float32)
    tau = 200.0 / W.max()
    bits, info = oracle.solve(W, 2, 4, tau, 300, stats=True)
    assert oracle.count_infeasible(bits, 128, 128, 2, 4) == 0 and info["underfilled"] == 0
    opt = oracle.bruteforce(W, 2, 4)
    obj = info["obj"]
    assert np.all(obj <= opt + 1e-9)
    assert np.mean(obj >= opt - 1e-9) > 0.98
    assert np.mean((opt - obj) / opt) < 1e-3
    assert abs(oracle.objective(W, bits) - obj.sum()) < 1e-6 * obj.sum()
    assert np.allclose(oracle.block_objectives(W, bits, 4), obj, rtol=1e-12)


def test_solve_against_assignment_optimum_n1_and_complement():
    rng = np.random.default_rng(22)
    M = 8
    W = np.abs(rng.standard_normal((M * 6, M * 6))).astype(np.float32)
    tau = 200.0 / W.max()
    for N in (1, M - 1):
        bits, info = oracle.solve(W, N, M, tau, 300, stats=True)
        assert info["underfilled"] == 0
        gaps = []
        for b in range(36):
            r0, c0 = (b // 6) * M, (b % 6) * M
            blk = W[r0:r0 + M, c0:c0 + M].astype(np.float64)
            if N == 1:
                r, c = linear_sum_assignment(blk, maximize=True)
                opt = blk[r, c].sum()
            else:
                r, c = linear_sum_assignment(blk)
                opt = blk.sum() - blk[r, c].sum()
            assert info["obj"][b] <= opt + 1e-9
            gaps.append((opt - info["obj"][b]) / opt)
        assert np.mean(gaps) < 0.01


def test_rounding_the_plan_beats_rounding_the_scores_8_16():
    rng = np.random.default_rng(23)
    M, N, nb = 16, 8, 6
    W = np.abs(rng.standard_normal((M * nb, M * nb)) * 0.02).astype(np.float32)
    tau = 200.0 / W.max()
    _, a = oracle.solve(W, N, M, tau, 300, stats=True)
    _, b = oracle.round_plan(W, W, N, M, stats=True)       # Algorithm 2 straight on |W|
    opts = np.array([_lp_optimum(W[(k // nb) * M:(k // nb + 1) * M,
                                   (k % nb) * M:(k % nb + 1) * M].astype(np.float64), N)
                     for k in range(nb * nb)])
    assert np.all(a["obj"] <= opts + 1e-7) and np.all(b["obj"] <= opts + 1e-7)
    ga, gb = np.mean((opts - a["obj"]) / opts), np.mean((opts - b["obj"]) / opts)
    assert ga < gb and ga < 2e-3


def test_solve_with_zero_iterations_is_greedy_on_scores():
    rng = np.random.default_rng(24)
    W = np.abs(rng.standard_normal((32, 64))).astype(np.float32)
    a = oracle.solve(W, 4, 8, 3.0, 0)
    b = oracle.round_plan(W, W, 4, 8)
    assert np.array_equal(a, b)


def test_mask_bit_layout_and_helpers():
    W = np.zeros((4, 40), np.float32)
    W[0, 0] = W[0, 1] = W[1, 2] = W[1, 3] = 5   # block (0,0): force a known 2:4 pattern
    W[2, 0] = W[2, 2] = W[3, 1] = W[3, 3] = 5
    W[0, 36] = W[0, 37] = W[1, 38] = W[1, 39] = 7   # last block: columns 36..39 -> word 1
    W[2, 36] = W[2, 38] = W[3, 37] = W[3, 39] = 7
    bits = oracle.round_plan(W, W, 2, 4)
    assert bits.shape == (4, 2) and bits.dtype == np.uint32
    assert bits[0, 0] & 0xF == 0b0011 and bits[1, 0] & 0xF == 0b1100
    assert bits[2, 0] & 0xF == 0b0101 and bits[3, 0] & 0xF == 0b1010
    assert bits[0, 1] >> 4 == 0b0011 and bits[3, 1] >> 4 == 0b1010
    assert bits[0, 1] >> 8 == 0                     # nothing beyond column 39
    dense = oracle.unpack_mask(bits, 40)
    assert dense.shape == (4, 40) and dense[0, 36] == 1 and dense[0, 38] == 0
    assert oracle.count_infeasible(bits, 4, 40, 2, 4) == 0
    bad = bits.copy()
    bad[0, 0] ^= 1
    assert oracle.count_infeasible(bad, 4, 40, 2, 4) == 1
    assert oracle.max_abs(-W) == 7.0
    with pytest.raises(ValueError):
        oracle.solve(np.zeros((6, 8), np.float32), 2, 4, 1.0, 1)


# ------------------------------------- framework scores, safeguard, simple rounding

def test_framework_score_formulas():
    rng = np.random.default_rng(31)
    W = rng.standard_normal((24, 40)).astype(np.float32)
    V = rng.standard_normal((24, 40)).astype(np.float32)
    rho = 3.0
    s = oracle.scores(oracle.SCORES_ADMM, W, V, 1.0 / rho)
    ref = (W.astype(np.float64) + V.astype(np.float64) / rho) ** 2
    assert np.allclose(s, ref, rtol=1e-5, atol=1e-6)          # three fp32 roundings, cancellation in the sum
    # D-update of Proposition 1: with D = (W + V/rho) .* S the distance to W + V/rho is the
    # score mass left outside the mask, so maximising the retained score minimises it
    S = (rng.random((24, 40)) < 0.5)
    Z = W.astype(np.float64) + V.astype(np.float64) / rho
    assert np.isclose(((Z * S - Z) ** 2).sum(), (ref * (~S)).sum(), rtol=1e-12)
    X = rng.standard_normal((64, 40))
    a = np.linalg.norm(X, axis=0).astype(np.float32)          # input-feature norms (Wanda)
    assert np.allclose(oracle.scores(oracle.SCORES_COLMUL, W, colvec=a), np.abs(W) * a, rtol=1e-7)
    d = (np.abs(rng.standard_normal(40)) + 0.1).astype(np.float32)
    assert np.allclose(oracle.scores(oracle.SCORES_COLDIV, W, colvec=d), np.abs(-W / d), rtol=1e-7)
    assert np.array_equal(oracle.scores(oracle.SCORES_ABS, W), np.abs(W))


def test_keep_better_never_lowers_the_objective():
    rng = np.random.default_rng(32)
    M, N = 8, 4
    W = rng.standard_normal((32, 64)).astype(np.float32)
    prev = None
    for t in range(6):                                    # a drifting score matrix, as in ADMM
        V = (0.3 * t) * rng.standard_normal(W.shape).astype(np.float32)
        sc = oracle.scores(oracle.SCORES_ADMM, W, V, 0.5)
        new = oracle.solve(sc, N, M, 200.0 / sc.max(), 60)
        if prev is None:
            prev = new
            continue
        if t == 3:                                        # force the other branch once
            new = oracle.round_plan(-sc, sc, N, M)        # a deliberately poor mask
        kept, o_new, o_prev = oracle.keep_better(sc, prev, new)
        assert o_new == oracle.objective(sc, new) and o_prev == oracle.objective(sc, prev)
        assert oracle.objective(sc, kept) == max(o_new, o_prev)
        assert np.array_equal(kept, new if o_new >= o_prev else prev)
        if t == 3:
            assert o_new < o_prev
        prev = kept


def test_simple_rounding_properties_and_ablation_order():
    rng = np.random.default_rng(33)
    M, N, nb = 8, 4, 8
    W = np.abs(rng.standard_normal((M * nb, M * nb)) * 0.02).astype(np.float32)
    tau = 200.0 / W.max()
    x = oracle.dykstra(W, N, M, tau, 300, plan_is_log=True).astype(np.float32)
    simple = oracle.unpack_mask(oracle.simple_round(x, N, M), M * nb)
    for b in range(nb * nb):
        r0, c0 = (b // nb) * M, (b % nb) * M
        S = simple[r0:r0 + M, c0:c0 + M]
        k = x[r0:r0 + M, c0:c0 + M]
        assert S.sum(0).max() <= N and S.sum(1).max() <= N
        for i in range(M):                                # survivors come from the row's top N
            top = sorted(range(M), key=lambda j: (-k[i, j], j))[:N]
            assert set(np.flatnonzero(S[i])) <= set(top)
    # a plan that already is a feasible mask is returned unchanged
    feas = oracle.unpack_mask(oracle.solve(W, N, M, tau, 300), M * nb).astype(np.float32)
    assert np.array_equal(oracle.unpack_mask(oracle.simple_round(feas, N, M), M * nb), feas.astype(np.uint8))
    # ablation order of Appendix B.2 on the same plan: simple <= greedy only <= greedy + local search
    o_simple = (simple * W.astype(np.float64)).sum()
    o_greedy = oracle.objective(W, oracle.round_plan(x, W, N, M, ls_steps=0))
    o_full = oracle.objective(W, oracle.round_plan(x, W, N, M))
    assert o_simple < o_greedy <= o_full


def _simple_round_by_definition(k, N):
    """Appendix B.2 "Simple", written out: keep the N best keys of every row, then the N best
    of the survivors of every column; "best" = key descending, position ascending."""
    M = k.shape[0]
    S = np.zeros((M, M), np.uint8)
    for i in range(M):
        for j in sorted(range(M), key=lambda j: (-k[i, j], j))[:N]:
            S[i, j] = 1
    for j in range(M):
        surv = [i for i in range(M) if S[i, j]]
        for i in sorted(surv, key=lambda i: (-k[i, j], i))[N:]:
            S[i, j] = 0
    return S


def test_simple_rounding_worked_examples_and_definition():
    """Pins both passes of the "Simple" rounding.  Two blocks worked by hand (the dropped
    entries are named), then the definition written out above on random, heavy-tie and
    at-cap keys for every block size, N = M/2 and N != M/2."""
    # 2:4, column 0 is the best entry of every row: rows keep {0, their second best}; column 0
    # then has 4 survivors and keeps the two largest, 0.9 (row 2) and 0.8 (row 0): (1,0), (3,0) go.
    k = np.array([[0.8, 0.1, 0.3, 0.2],
                  [0.7, 0.2, 0.1, 0.6],
                  [0.9, 0.5, 0.4, 0.3],
                  [0.6, 0.1, 0.2, 0.5]], np.float32)
    want = np.array([[1, 0, 1, 0],
                     [0, 0, 0, 1],
                     [1, 1, 0, 0],
                     [0, 0, 0, 1]], np.uint8)
    got = oracle.unpack_mask(oracle.simple_round(k, 2, 4), 4)
    assert np.array_equal(got, want)
    assert got[1, 0] == 0 and got[3, 0] == 0 and got[0, 0] == 1 and got[2, 0] == 1
    # all keys equal (every comparison is a tie): rows keep columns 0 and 1, columns 0 and 1
    # then keep rows 0 and 1 -- ties go to the smaller position in both passes
    flat = oracle.unpack_mask(oracle.simple_round(np.zeros((4, 4), np.float32), 2, 4), 4)
    assert np.array_equal(flat, np.array([[1, 1, 0, 0], [1, 1, 0, 0], [0, 0, 0, 0], [0, 0, 0, 0]], np.uint8))
    # 1:4 with a tie inside a column: rows 0 and 2 both send their best entry to column 1 with
    # the same key; the smaller row index survives
    k1 = np.array([[0.1, 0.5, 0.2, 0.3],
                   [0.9, 0.1, 0.2, 0.3],
                   [0.2, 0.5, 0.1, 0.4],
                   [0.1, 0.2, 0.3, 0.8]], np.float32)
    got1 = oracle.unpack_mask(oracle.simple_round(k1, 1, 4), 4)
    assert np.array_equal(got1, np.array([[0, 1, 0, 0], [1, 0, 0, 0], [0, 0, 0, 0], [0, 0, 0, 1]], np.uint8))

    rng = np.random.default_rng(34)
    seen_overfull = 0
    for M, N in [(4, 2), (4, 1), (4, 3), (8, 4), (8, 3), (16, 8), (16, 5), (32, 16), (32, 7), (32, 25)]:
        nb = 3
        for kind in ("random", "ties", "cap"):
            if kind == "random":
                K = rng.standard_normal((M * nb, M * nb))
            elif kind == "ties":
                K = rng.integers(0, 4, (M * nb, M * nb)).astype(np.float64)
            else:   # like a log-plan: many entries exactly at the cap (0), the rest negative
                K = np.minimum(rng.standard_normal((M * nb, M * nb)) * 3 - 1, 0.0)
            K = K.astype(np.float32)
            dense = oracle.unpack_mask(oracle.simple_round(K, N, M), M * nb)
            for b in range(nb * nb):
                r0, c0 = (b // nb) * M, (b % nb) * M
                k = K[r0:r0 + M, c0:c0 + M]
                assert np.array_equal(dense[r0:r0 + M, c0:c0 + M], _simple_round_by_definition(k, N)), (M, N, kind)
                rows_top = np.zeros((M, M), np.uint8)
                for i in range(M):
                    rows_top[i, sorted(range(M), key=lambda j: (-k[i, j], j))[:N]] = 1
                seen_overfull += int((rows_top.sum(0) > N).any())
    assert seen_overfull > 50          # the column pass had survivors to drop in most blocks


def test_log_domain_oracle_equals_algorithm1_in_its_printed_linear_form():
    """Algorithm 1 as printed works on S and Q themselves (no logarithms).  Written out here
    in numpy fp64 it must give the oracle's exp(x) and exp(q) at every iteration count, cap
    active or not -- up to the operating point tau max(w) = 200 and T = 300, where exp(tau w)
    reaches 7e86 (far outside fp32, which is why the method needs its log-domain form, but
    inside fp64, so the printed form can still serve as the reference)."""
    rng = np.random.default_rng(41)
    cases = [(4, 2, 8.0, (1, 2, 3, 10, 60)), (8, 4, 25.0, (1, 2, 3, 10, 60)), (16, 8, 40.0, (1, 2, 3, 10, 60)),
             (8, 3, 25.0, (1, 2, 3, 10, 60)), (32, 16, 60.0, (1, 2, 3, 10, 60)),
             (4, 2, 200.0, (1, 5, 300)), (8, 4, 200.0, (1, 5, 300)), (16, 8, 200.0, (1, 5, 300)),
             (32, 16, 200.0, (1, 2, 3, 10, 60, 300)), (32, 9, 200.0, (1, 300))]
    for M, N, tau, counts in cases:
        w = np.abs(rng.standard_normal((M, M)))
        w /= w.max()
        S = np.exp(tau * w)
        Q = np.ones((M, M))
        done = 0
        for iters in counts:
            for _ in range(iters - done):
                S = S * (N / S.sum(1, keepdims=True))          # line 3: Diag(N / (S 1)) S
                S = S * (N / S.sum(0, keepdims=True))          # line 4: S Diag(N / (S^T 1))
                Snew = np.minimum(S * Q, 1.0)                  # line 5
                Q = Q * (S / Snew)                             # line 6
                S = Snew
            done = iters
            x, q = oracle.dykstra_block(w, N, tau, iters)
            assert np.allclose(np.exp(x), S, rtol=1e-8, atol=1e-300), (M, N, tau, iters)
            assert np.allclose(np.exp(q), Q, rtol=1e-8), (M, N, tau, iters)
            if tau == 200.0:   # at the operating point also as an absolute bound on the plan
                assert np.abs(np.exp(x) - S).max() < 1e-11
        assert (S == 1.0).any()                                # the cap was active on the way


def test_per_block_tau_is_the_plain_method_block_by_block():
    """The per-block variant must equal running the method on each block alone with
    tau = tau_rel / max of that block, and must help when one column dwarfs the rest."""
    M, N, nb = 8, 4, 5
    W = np.abs(np.random.default_rng(51).standard_normal((M * nb, M * nb)) * 0.02).astype(np.float32)
    W[:, 3] *= 20
    bits = oracle.solve(W, N, M, 200.0, 300, per_block_tau=True)
    plan = oracle.dykstra(W, N, M, 200.0, 40, per_block_tau=True)
    dense = oracle.unpack_mask(bits, M * nb)
    for b in range(nb * nb):
        r0, c0 = (b // nb) * M, (b % nb) * M
        blk = np.ascontiguousarray(W[r0:r0 + M, c0:c0 + M])
        one = oracle.unpack_mask(oracle.solve(blk, N, M, 200.0 / blk.max(), 300), M)
        assert np.array_equal(dense[r0:r0 + M, c0:c0 + M], one)
        # (the stand-alone call rounds its tau to fp32, the per-block one divides in fp64)
        assert np.allclose(plan[r0:r0 + M, c0:c0 + M], oracle.dykstra(blk, N, M, 200.0 / blk.max(), 40), rtol=1e-4)
    opt = sum(_lp_optimum(W[(b // nb) * M:(b // nb + 1) * M, (b % nb) * M:(b % nb + 1) * M].astype(np.float64), N)
              for b in range(nb * nb))
    gap_pb = opt - oracle.objective(W, bits)
    gap_gl = opt - oracle.objective(W, oracle.solve(W, N, M, 200.0 / W.max(), 300))
    assert 0 <= gap_pb <= gap_gl
    zero = np.zeros((M, M), np.float32)                    # an all-zero block gets tau = 0
    assert oracle.count_infeasible(oracle.solve(zero, N, M, 200.0, 10, per_block_tau=True), M, M, N, M) == 0


def test_stopping_test_variant_of_algorithm1():
    """The variant of Algorithm 1 with a stopping test: identical to the fixed count when the test
    is off; the count it returns is the first tested iteration t = 1 + 4k whose marginal violation,
    recomputed here from the fixed-count oracle's iterates, is below eps; counts fall as eps grows."""
    rng = np.random.default_rng(61)
    for M, N, tau in [(4, 2, 30.0), (8, 4, 40.0), (16, 8, 25.0), (32, 16, 12.0), (8, 3, 60.0)]:
        w = np.abs(rng.standard_normal((M, M)))
        w /= w.max()
        x0, q0 = oracle.dykstra_block(w, N, tau, 80)
        x1, q1, ran = oracle.dykstra_block_earlyexit(w, N, tau, 80, 0.0, 4)
        assert ran == 80 and np.array_equal(x0, x1) and np.array_equal(q0, q1)
        prev = 10 ** 9
        for eps in (1e-6, 1e-4, 1e-2, 0.3):
            x, q, ran = oracle.dykstra_block_earlyexit(w, N, tau, 400, eps, 4)
            assert ran <= prev
            prev = ran
            first = None
            for t in range(5, 401, 4):                     # iterations at which the test is made
                s_in = np.exp(oracle.dykstra_block(w, N, tau, t - 1)[0])              # iterate entering t
                s_row = np.exp(oracle.dykstra_block(w, N, tau, t - 1, extra_steps=1)[0])  # after its row step
                delta = max(np.abs(s_in.sum(1) - N).max(), np.abs(s_row.sum(0) - N).max())
                if delta < eps:
                    first = t
                    break
            assert ran == (first if first is not None else 400), (M, N, eps)
            xr, qr = oracle.dykstra_block(w, N, tau, ran)      # and it returns that iteration's iterate
            assert np.array_equal(x, xr) and np.array_equal(q, qr)
    W = np.abs(rng.standard_normal((32, 48)) * 0.02).astype(np.float32)
    tau = 15.0 / W.max()
    bits, iters = oracle.solve_earlyexit(W, 4, 8, tau, 300, 0.0, 4)
    assert np.array_equal(bits, oracle.solve(W, 4, 8, tau, 300)) and (iters == 300).all()
    bits, iters = oracle.solve_earlyexit(W, 4, 8, tau, 300, 1e-3, 4)
    assert iters.max() < 300 and ((iters - 1) % 4 == 0).all()
    assert oracle.count_infeasible(bits, 32, 48, 4, 8) == 0
    plan, iters2 = oracle.dykstra_earlyexit(W, 4, 8, tau, 300, 1e-3, 4)
    assert np.array_equal(iters, iters2)
    assert np.abs(plan - oracle.dykstra(W, 4, 8, tau, 300)).max() < 5e-3   # stopped close to the fixed point
