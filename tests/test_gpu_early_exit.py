"""The stopping-test mode of Algorithm 1 (a performance mode outside the parity contract, which
is the fixed iteration count): the CUDA path against the oracle's twin of the same test, and
against its own fixed-count result."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_23949_b200 import binding as ts
from paper_2505_23949_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bits(t):
    return t.cpu().numpy().view(np.uint32)


def _block_diff(a, b, rows, cols, M):
    return oracle.unpack_mask(a ^ b, cols).reshape(rows // M, M, cols // M, M).any(axis=(1, 3))


@pytest.mark.parametrize("M,N,rows,cols,tau_rel", [(32, 16, 256, 1024, 12.0), (32, 16, 128, 1024, 40.0),
                                                   (16, 8, 128, 1024, 25.0), (8, 4, 64, 1024, 15.0),
                                                   (4, 2, 32, 1024, 10.0)])
def test_early_exit_against_the_oracle_twin(M, N, rows, cols, tau_rel):
    W = synth.gaussian_abs(rows, cols, 0.02, 600 + M)
    tau = tau_rel / float(W.max())
    eps = 1e-3
    Wd = torch.from_numpy(W).to(DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    src = ts.Scores(ts.SCORES_ABS, Wd, early_exit_eps=eps, iters_out=cnt)
    st = ts.new_status(DEV)
    got = _bits(ts.solve_scores(src, N, M, tau, 300, -1, status=st))
    total = int(cnt.item())
    assert int(st.item()) == 0 and oracle.count_infeasible(got, rows, cols, N, M) == 0
    want, iters = oracle.solve_earlyexit(W, N, M, tau, 300, eps, 4)
    nblk = len(iters)
    assert iters.max() < 300                                      # the test fires on these inputs
    if M == 32:     # one block per warp: the same stopping rule, up to fp32 at the threshold
        assert abs(total - int(iters.sum())) <= 0.02 * iters.sum()
    else:           # a warp stops when the last of its blocks has converged
        assert iters.sum() <= total <= 300 * nblk
        assert total < 0.9 * 300 * nblk
    assert _block_diff(got, want, rows, cols, M).mean() <= 0.01
    o_gpu, o_ref = oracle.objective(W, got), oracle.objective(W, want)
    assert abs(o_gpu - o_ref) <= 1e-4 * o_ref
    # plan: every block stopped within eps of its fixed point, wherever exactly it stopped
    cnt.zero_()
    plan = ts.dykstra_scores(src, N, M, tau, 300).cpu().numpy()
    ref, _ = oracle.dykstra_earlyexit(W, N, M, tau, 300, eps, 4)
    err = np.abs(plan - ref)
    assert err.max() <= 20 * eps
    if M == 32:     # same stopping iteration for (nearly) every block: the usual plan bound holds there
        assert np.mean(err <= 1e-4) >= 0.97


def test_early_exit_off_is_the_fixed_count_and_counts_iterations():
    W = synth.gaussian_abs(64, 256, 0.02, 77)
    tau = synth.default_tau(float(W.max()))
    Wd = torch.from_numpy(W).to(DEV)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    src = ts.Scores(ts.SCORES_ABS, Wd, iters_out=cnt)
    a = ts.solve_scores(src, 8, 16, tau, 37, -1)
    b = ts.solve(Wd, 8, 16, tau, 37, -1)
    assert torch.equal(a, b) and int(cnt.item()) == 37 * (64 // 16) * (256 // 16)
    with pytest.raises(ts.TsenorError):
        ts.solve_scores(ts.Scores(ts.SCORES_ABS, Wd, early_exit_eps=-1.0), 8, 16, tau, 10, -1)


def test_early_exit_on_the_headline_matrix_keeps_the_masks():
    """Config 4 (up-projection): under the whole-matrix tau rule most blocks are far softer than
    tau max|w| = 200 and converge in a dozen iterations; the masks of at least 99.9 % of the blocks
    equal those of the full 300 iterations and the objective moves by far less than 1e-4."""
    wl = synth.config(4, part="up")
    W, N, M = wl.scores, wl.N, wl.M
    rows, cols = W.shape
    tau = synth.default_tau(float(W.max()))
    Wd = torch.from_numpy(W).to(DEV)
    full = ts.solve(Wd, N, M, tau, 300, -1)
    cnt = torch.zeros(1, dtype=torch.int64, device=DEV)
    fast = ts.solve_scores(ts.Scores(ts.SCORES_ABS, Wd, early_exit_eps=1e-3, iters_out=cnt), N, M, tau, 300, -1)
    assert int(ts.check(fast, rows, cols, N, M).item()) == 0
    nblk = (rows // M) * (cols // M)
    assert int(cnt.item()) / nblk < 40
    assert _block_diff(_bits(fast), _bits(full), rows, cols, M).mean() <= 1e-3
    o_fast, o_full = float(ts.objective(Wd, fast).item()), float(ts.objective(Wd, full).item())
    assert abs(o_fast - o_full) <= 1e-4 * o_full
