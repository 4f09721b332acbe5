"""GPU parity of the framework score sources (magnitude, ADMM D-update, SparseGPT group,
Wanda), the mask safeguard and the simple rounding, against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_23949_b200 import binding as ts
from paper_2505_23949_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["throughput", "latency"])
def _both_register_layouts(request):
    """Every case runs under both register layouts of the Dykstra stage (these matrices are
    small, so the automatic choice alone would never exercise the throughput layout)."""
    ts.set_layout(ts.LAYOUT_THROUGHPUT if request.param == "throughput" else ts.LAYOUT_LATENCY)
    yield
    ts.set_layout(ts.LAYOUT_AUTO)
DEV = "cuda:0"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def _bits(t):
    return t.cpu().numpy().view(np.uint32)


def _sources(rows, cols, seed):
    """(name, binding Scores, oracle fp32 score matrix) for every kind."""
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    V = (rng.standard_normal((rows, cols)) * 0.01).astype(np.float32)
    d = (np.abs(rng.standard_normal(cols)) + 0.05).astype(np.float32)
    a = rng.lognormal(0.0, 1.0, cols).astype(np.float32)
    Wb = torch.from_numpy(W).to(torch.bfloat16)
    Wb32 = Wb.to(torch.float32).numpy()
    Wd, Vd, dd, ad = _dev(W), _dev(V), _dev(d), _dev(a)
    return [
        ("abs", ts.Scores(ts.SCORES_ABS, Wd), oracle.scores(oracle.SCORES_ABS, W)),
        ("admm", ts.Scores(ts.SCORES_ADMM, Wd, v=Vd, scalar=1 / 3.0), oracle.scores(oracle.SCORES_ADMM, W, V, np.float32(1 / 3.0))),
        ("coldiv", ts.Scores(ts.SCORES_COLDIV, Wd, colvec=dd), oracle.scores(oracle.SCORES_COLDIV, W, colvec=d)),
        ("colmul", ts.Scores(ts.SCORES_COLMUL, Wd, colvec=ad), oracle.scores(oracle.SCORES_COLMUL, W, colvec=a)),
        ("colmul_bf16", ts.Scores(ts.SCORES_COLMUL, Wb.to(DEV), colvec=ad), oracle.scores(oracle.SCORES_COLMUL, Wb32, colvec=a)),
        ("abs_bf16", ts.Scores(ts.SCORES_ABS, Wb.to(DEV)), oracle.scores(oracle.SCORES_ABS, Wb32)),
        ("admm_bf16", ts.Scores(ts.SCORES_ADMM, Wb.to(DEV), v=Vd, scalar=0.5), oracle.scores(oracle.SCORES_ADMM, Wb32, V, np.float32(0.5))),
    ]


@pytest.mark.parametrize("M,N,rows,cols", [(32, 16, 64, 352), (16, 8, 32, 592), (8, 4, 24, 1096), (4, 2, 16, 1060)])
def test_described_scores_are_bit_exact_and_solve_like_materialised_ones(M, N, rows, cols):
    for name, src, ref in _sources(rows, cols, 7 * M + N):
        got = ts.scores_materialize(src).cpu().numpy()
        assert np.array_equal(got, ref), name                       # same fp32 bits as the oracle
        assert float(ts.scores_max(src).item()) == float(ref.max()), name
        tau = synth.default_tau(ref.max())
        st = ts.new_status(DEV)
        mask = _bits(ts.solve_scores(src, N, M, tau, 300, status=st))
        assert int(st.item()) == 0
        assert np.array_equal(mask, _bits(ts.solve(_dev(ref), N, M, tau, 300))), name
        assert oracle.count_infeasible(mask, rows, cols, N, M) == 0
        want = oracle.solve(ref, N, M, tau, 300)
        o_gpu, o_ref = oracle.objective(ref, mask), oracle.objective(ref, want)
        assert abs(o_gpu - o_ref) <= 1e-4 * o_ref, name


def test_unaligned_and_strided_sources():
    rng = np.random.default_rng(5)
    big = (rng.standard_normal((40, 300)) * 0.02).astype(np.float32)
    bigd = _dev(big)
    a = rng.lognormal(0, 1, 264).astype(np.float32)
    buf = torch.zeros(265, device=DEV)
    buf[1:] = _dev(a)
    wv = bigd[1:33, 3:267]                                          # ld 300, odd offset
    src = ts.Scores(ts.SCORES_COLMUL, wv, colvec=buf[1:])
    ref = oracle.scores(oracle.SCORES_COLMUL, big[1:33, 3:267], colvec=a)
    assert np.array_equal(ts.scores_materialize(src).cpu().numpy(), ref)
    wb = torch.from_numpy(big).to(torch.bfloat16).to(DEV)[1:33, 3:267]
    srcb = ts.Scores(ts.SCORES_COLMUL, wb, colvec=buf[1:])
    refb = oracle.scores(oracle.SCORES_COLMUL, wb.to(torch.float32).cpu().numpy(), colvec=a)
    assert np.array_equal(ts.scores_materialize(srcb).cpu().numpy(), refb)
    m = _bits(ts.solve_scores(srcb, 4, 8, synth.default_tau(refb.max()), 100))
    assert oracle.count_infeasible(m, 32, 264, 4, 8) == 0


@pytest.mark.parametrize("M,N", [(4, 2), (8, 4), (16, 8), (32, 16)])
def test_sparsegpt_column_groups(M, N):
    """SparseGPT walks a weight matrix in groups of M columns and prunes each rows x M slab with
    the score |W_ij / d_j|: every group is a strided view into the wide matrix."""
    rng = np.random.default_rng(100 + M)
    rows, cols = M * 37, M * 5
    W = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    d = (np.abs(rng.standard_normal(cols)) + 0.05).astype(np.float32)
    Wd, dd = _dev(W), _dev(d)
    full = np.zeros((rows, (cols + 31) // 32), np.uint32)
    for g in range(cols // M):
        c0 = g * M
        src = ts.Scores(ts.SCORES_COLDIV, Wd[:, c0:c0 + M], colvec=dd[c0:c0 + M].contiguous())
        ref = oracle.scores(oracle.SCORES_COLDIV, W[:, c0:c0 + M], colvec=d[c0:c0 + M])
        assert np.array_equal(ts.scores_materialize(src).cpu().numpy(), ref)
        assert float(ts.scores_max(src).item()) == float(ref.max())
        tau = float(200.0 / ref.max())
        st = ts.new_status(DEV)
        m = _bits(ts.solve_scores(src, N, M, tau, 300, status=st))
        assert int(st.item()) == 0 and m.shape == (rows, 1)
        assert oracle.count_infeasible(m, rows, M, N, M) == 0
        want = oracle.solve(ref, N, M, tau, 300)
        assert abs(oracle.objective(ref, m) - oracle.objective(ref, want)) <= 1e-4 * oracle.objective(ref, want)
        # the slab path and the wide path of the same kernel agree block for block
        wide = np.ascontiguousarray(ref.reshape(rows // M, M, M).transpose(1, 0, 2).reshape(M, rows))
        mw = oracle.unpack_mask(_bits(ts.solve(_dev(wide), N, M, tau, 300)), rows)
        assert np.array_equal(mw.reshape(M, rows // M, M).transpose(1, 0, 2).reshape(rows, M),
                              oracle.unpack_mask(m, M))
        full[:, c0 // 32] |= m[:, 0] << np.uint32(c0 % 32)
    assert oracle.count_infeasible(full, rows, cols, N, M) == 0


def test_admm_sequence_with_safeguard_matches_oracle():
    """A short ADMM-like sequence: the score matrix drifts, every iteration proposes a mask and the
    safeguard keeps the previous one if the new one retains less (Appendix A.1.3).  Both sides are
    given the same candidate masks (made by the oracle) and the same previous mask."""
    rng = np.random.default_rng(9)
    M, N, rows, cols = 16, 8, 64, 512
    W = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    Wd = _dev(W)
    prev = None
    kept_prev = kept_new = 0
    for t in range(6):
        V = ((0.2 * t) * rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
        rho = np.float32(1.0 / (0.5 + 0.3 * t))
        src = ts.Scores(ts.SCORES_ADMM, Wd, v=_dev(V), scalar=float(rho))
        sc = oracle.scores(oracle.SCORES_ADMM, W, V, rho)
        if t % 3 == 2:                                              # a deliberately poor candidate
            cand = oracle.round_plan(-sc, sc, N, M)
        else:
            cand = oracle.solve(sc, N, M, 200.0 / sc.max(), 60)
        if prev is None:
            prev = cand
            continue
        mask_d = _dev(cand.view(np.int32))
        obj2 = ts.keep_better(src, _dev(prev.view(np.int32)), mask_d).cpu().numpy()
        kept_ref, o_new, o_prev = oracle.keep_better(sc, prev, cand)
        assert np.array_equal(_bits(mask_d), kept_ref)
        assert abs(obj2[0] - o_new) <= 1e-12 * o_new and abs(obj2[1] - o_prev) <= 1e-12 * o_prev
        kept_prev += int(o_new < o_prev)
        kept_new += int(o_new >= o_prev)
        prev = kept_ref
    assert kept_prev >= 1 and kept_new >= 1                         # both branches were taken
    # the GPU's own solve on the described scores is a candidate the safeguard accepts or rejects
    # consistently with the objectives it reports
    new_gpu = ts.solve_scores(src, N, M, float(200.0 / ts.scores_max(src).item()), 120)
    before = _bits(new_gpu).copy()
    obj2 = ts.keep_better(src, _dev(prev.view(np.int32)), new_gpu).cpu().numpy()
    assert np.array_equal(_bits(new_gpu), before if obj2[0] >= obj2[1] else prev)


@pytest.mark.parametrize("M,N", [(4, 2), (8, 4), (16, 8), (32, 16), (8, 3), (32, 5)])
def test_simple_rounding_is_bit_exact(M, N):
    rng = np.random.default_rng(M * 10 + N)
    rows, cols = 2 * M, 10 * M + (32 if M < 32 else 0)
    W = synth.gaussian_abs(rows, cols, 0.02, M + N)
    tau = synth.default_tau(W.max())
    x = oracle.dykstra(W, N, M, tau, 300, plan_is_log=True).astype(np.float32)
    for key in (x, np.round(rng.standard_normal((rows, cols)) * 2).astype(np.float32)):
        got = _bits(ts.simple_round(_dev(key), N, M))
        assert np.array_equal(got, oracle.simple_round(key, N, M))


def test_descriptor_errors():
    W = _dev(np.zeros((8, 16), np.float32))
    src = ts.Scores(ts.SCORES_ADMM, W, v=W, scalar=float("nan"))
    with pytest.raises(ts.TsenorError) as e:
        ts.solve_scores(src, 2, 4, 1.0)
    assert e.value.status == ts.ERR_ARG
    bad = ts.Scores(ts.SCORES_COLDIV, W)                            # colvec missing
    with pytest.raises(ts.TsenorError) as e:
        ts.scores_max(bad)
    assert e.value.status == ts.ERR_NULL
    src = ts.Scores(ts.SCORES_ABS, W)
    src.desc.kind = 7                                               # unknown kind
    with pytest.raises(ts.TsenorError) as e:
        ts.scores_materialize(src)
    assert e.value.status == ts.ERR_ARG


@pytest.mark.parametrize("M,N,rows,cols", [(32, 16, 64, 352), (16, 8, 32, 592), (8, 4, 24, 1096), (4, 2, 16, 1060)])
def test_per_block_tau_matches_oracle(M, N, rows, cols):
    """tau divided by each block's own largest score (Appendix B.1 rule applied per block)."""
    W = synth.gaussian_outlier_columns_abs(rows, cols, 0.02, 77 + M, frac=0.01)
    W[0:M, 0:M] = 0.0                                               # an all-zero block: tau = 0 there
    src = ts.Scores(ts.SCORES_ABS, _dev(W), per_block_tau=True)
    st = ts.new_status(DEV)
    plan = ts.dykstra_scores(src, N, M, 200.0, 300, status=st).cpu().numpy()
    ref = oracle.dykstra(W, N, M, 200.0, 300, per_block_tau=True)
    assert np.abs(plan - ref).max() <= 1e-4
    mask = _bits(ts.solve_scores(src, N, M, 200.0, 300, status=st))
    assert int(st.item()) == 0
    assert oracle.count_infeasible(mask, rows, cols, N, M) == 0
    want = oracle.solve(W, N, M, 200.0, 300, per_block_tau=True)
    o_gpu, o_ref = oracle.objective(W, mask), oracle.objective(W, want)
    assert abs(o_gpu - o_ref) <= 1e-4 * o_ref
    # and it retains more than the whole-matrix rule when a few columns dominate
    glob = _bits(ts.solve(_dev(W), N, M, synth.default_tau(W.max()), 300))
    assert o_gpu >= oracle.objective(W, glob)
    # iters = 0 uses the same per-block scaling (key = tau_b |w|: same order as |w| inside a block)
    assert np.array_equal(_bits(ts.solve_scores(src, N, M, 200.0, 0)), oracle.round_plan(W, W, N, M))
