"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times
(one tsenor_solve per matrix): every block feasible, and sampled blocks against the oracle,
which solves them one by one."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_23949_b200 import binding as ts
from paper_2505_23949_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PLAN_TOL = 1e-4
OBJ_RTOL = 1e-4


def _bits(t):
    return t.cpu().numpy().view(np.uint32)


def _sample_strip(W, M, block_ids):
    """Stack the sampled M x M blocks of W into one (len*M) x M matrix (one block per block row)."""
    nbc = W.shape[1] // M
    return np.concatenate([W[(b // nbc) * M:(b // nbc + 1) * M, (b % nbc) * M:(b % nbc + 1) * M]
                           for b in block_ids], axis=0)


def _check_full(W, N, M, nsample, seed, extra_blocks=()):
    rows, cols = W.shape
    tau = synth.default_tau(float(W.max()))
    Wd = torch.from_numpy(W).to(DEV)
    st = ts.new_status(DEV)
    mask = ts.solve(Wd, N, M, tau, 300, -1, status=st)
    assert int(ts.check(mask, rows, cols, N, M).item()) == 0          # every block, on the device
    assert int(st.item()) == 0
    got = _bits(mask)
    nblk = (rows // M) * (cols // M)
    rng = np.random.default_rng(seed)
    ids = np.unique(np.concatenate([rng.choice(nblk, size=min(nsample, nblk), replace=False),
                                    np.asarray(extra_blocks, dtype=np.int64)]))
    strip = _sample_strip(W, M, ids)
    # masks of the sampled blocks, cut out of the packed output
    dense = oracle.unpack_mask(got, cols)
    got_strip = _sample_strip(dense, M, ids)
    assert np.all(got_strip.reshape(len(ids), M, M).sum(1) == N)
    assert np.all(got_strip.reshape(len(ids), M, M).sum(2) == N)
    want, info = oracle.solve(strip, N, M, tau, 300, stats=True)
    obj_gpu = (got_strip * strip.astype(np.float64)).reshape(len(ids), -1).sum(1)
    assert abs(obj_gpu.sum() - info["obj"].sum()) <= OBJ_RTOL * info["obj"].sum()
    same = np.mean([np.array_equal(g, w) for g, w in zip(
        got_strip.reshape(len(ids), M, M), oracle.unpack_mask(want, M).reshape(len(ids), M, M))])
    assert same >= 0.98                                                # fp32 plan vs fp64 plan
    # fractional plan of the same blocks
    plan = ts.dykstra(Wd, N, M, tau, 300)
    plan_strip = _sample_strip(plan.cpu().numpy(), M, ids)
    ref = oracle.dykstra(strip, N, M, tau, 300)
    assert np.abs(plan_strip - ref).max() <= PLAN_TOL
    return got, ids


@pytest.mark.parametrize("part", ["up", "down"])
def test_config4_llama_mlp_16_32(part):
    wl = synth.config(4, part=part)
    _check_full(wl.scores, wl.N, wl.M, 192, seed=4)


def test_config3_wanda_8_16():
    wl = synth.config(3)
    _check_full(wl.scores, wl.N, wl.M, 512, seed=3)


def test_config2_every_block_against_brute_force_2_4():
    wl = synth.config(2)
    W = wl.scores
    got, _ = _check_full(W, 2, 4, 2048, seed=2)
    opt = oracle.bruteforce(W, 2, 4)                                   # all 1,048,576 blocks
    obj = oracle.block_objectives(W, got, 4)
    assert np.all(obj <= opt * (1 + 1e-12) + 1e-12)
    assert np.mean(obj >= opt * (1 - 1e-9)) > 0.99
    assert np.mean((opt - obj) / opt) < 1e-4


def test_config0_paper_table_shape_8_16():
    wl = synth.config(0, scale_rows=2048)                              # 2048 x 8192 of the 8192^2 shape
    _check_full(wl.scores, wl.N, wl.M, 256, seed=0)


def _outlier_blocks_first_block_row(W, M):
    """Blocks of the first block row that contain an outlier column (config 5)."""
    colmax = W[: 4 * M].max(0)
    out_cols = np.flatnonzero(colmax > 8 * np.median(colmax))
    assert len(out_cols) > 0
    return sorted({int(c // M) for c in out_cols})


@pytest.mark.parametrize("N,M", synth.NM_SWEEP)
@pytest.mark.parametrize("name", list(synth.LLAMA3_8B_LAYER_SHAPES))
def test_config5_every_shape_every_pattern_full_size(name, N, M):
    """Config 5, layer 0: each of the seven linear shapes at its full size under each of the four
    patterns.  Every block is checked for feasibility on the device; 128 random blocks plus every
    block of the first block row that holds an outlier column go through the oracle."""
    wl = synth.llama_layer(name, N, M)
    W = wl.scores
    assert W.shape == synth.LLAMA3_8B_LAYER_SHAPES[name]
    _check_full(W, N, M, 128, seed=5, extra_blocks=_outlier_blocks_first_block_row(W, M))


@pytest.mark.parametrize("layer", [1, 31])
def test_config5_other_layers_q_proj_16_32(layer):
    """The layer index only changes the seed: two more layers of the sweep for one shape."""
    wl = synth.llama_layer("q_proj", 16, 32, layer=layer)
    assert not np.array_equal(wl.scores[:64], synth.llama_layer("q_proj", 16, 32).scores[:64])
    _check_full(wl.scores, 16, 32, 128, seed=50 + layer,
                extra_blocks=_outlier_blocks_first_block_row(wl.scores, 32))


@pytest.mark.parametrize("cfg,part", [(4, "up"), (3, "up"), (1, "up")])
def test_whole_matrix_objective_against_the_oracle(cfg, part):
    """The retained-score objective of the whole matrix (every block solved by the oracle, not
    a sample): within 1e-4 relative, and the masks of at least 98 % of the blocks identical."""
    wl = synth.config(cfg, part=part)
    W, N, M = wl.scores, wl.N, wl.M
    rows, cols = W.shape
    tau = synth.default_tau(float(W.max()))
    got = _bits(ts.solve(torch.from_numpy(W).to(DEV), N, M, tau, 300, -1))
    want = oracle.solve(W, N, M, tau, 300)
    o_gpu, o_ref = oracle.objective(W, got), oracle.objective(W, want)
    assert abs(o_gpu - o_ref) <= OBJ_RTOL * o_ref, (o_gpu, o_ref)
    differ = oracle.unpack_mask(got ^ want, cols).reshape(rows // M, M, cols // M, M).any(axis=(1, 3))
    assert differ.mean() <= 0.02
