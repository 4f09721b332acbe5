"""Seeded synthetic score matrices for the TSENOR hot path.

Input generation only: nothing here performs any step of the method.  Both
the CUDA path (through its binding) and the CPU oracle are fed the arrays
made here, so that they read identical bytes.  The paper measured on LLaMA-3
weight matrices; those are not available, so these generators stand in for
them with the same shapes and rough value distributions (Section 5 and the
appendix on experimental details describe the originals).

Every generator is host-side numpy, ``numpy.random.Generator(PCG64(seed))``,
seed = 1000 * config + index unless the caller passes one.
"""
from dataclasses import dataclass

import numpy as np

# Linear layers of one Llama-3-8B-shaped decoder layer, (out_features, in_features).
LLAMA3_8B_LAYER_SHAPES = {
    "q_proj": (4096, 4096),
    "k_proj": (1024, 4096),
    "v_proj": (1024, 4096),
    "o_proj": (4096, 4096),
    "gate_proj": (14336, 4096),
    "up_proj": (14336, 4096),
    "down_proj": (4096, 14336),
}
LLAMA3_8B_NUM_LAYERS = 32
NM_SWEEP = ((2, 4), (4, 8), (8, 16), (16, 32))


@dataclass
class Workload:
    name: str
    scores: np.ndarray  # float32 [rows, cols], non-negative
    N: int
    M: int

    @property
    def blocks(self) -> int:
        r, c = self.scores.shape
        return (r // self.M) * (c // self.M)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def _round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 to the nearest bf16 (ties to even), returned as fp32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def gaussian_abs(rows: int, cols: int, std: float, seed: int) -> np.ndarray:
    """|W| with W i.i.d. N(0, std^2)."""
    w = _rng(seed).standard_normal((rows, cols), dtype=np.float32)
    w *= np.float32(std)
    return np.abs(w, out=w)


def student_t_abs(rows: int, cols: int, std: float, seed: int, df: float = 3.0) -> np.ndarray:
    """|W| with W Student-t(df) scaled to standard deviation ``std`` (heavy tails)."""
    rng = _rng(seed)
    out = np.empty((rows, cols), np.float32)
    scale = std / np.sqrt(df / (df - 2.0))
    step = max(1, (1 << 24) // max(cols, 1))
    for r0 in range(0, rows, step):  # chunked to bound the fp64 temporary
        r1 = min(rows, r0 + step)
        out[r0:r1] = np.abs(rng.standard_t(df, size=(r1 - r0, cols)) * scale)
    return out


def wanda_scores(rows: int, cols: int, std: float, seed: int) -> np.ndarray:
    """Wanda-style importance |W_ij| * a_j: W ~ N(0, std^2) rounded to bf16,
    a_j ~ lognormal(0, 1) one per input feature (column)."""
    rng = _rng(seed)
    w = rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)
    w = np.abs(_round_to_bf16(w))
    a = rng.lognormal(0.0, 1.0, size=cols).astype(np.float32)
    return (w * a[None, :]).astype(np.float32)


def gaussian_outlier_columns_abs(rows: int, cols: int, std: float, seed: int,
                                 frac: float = 1e-3, gain: float = 20.0) -> np.ndarray:
    """|W| with W ~ N(0, std^2) and a random ``frac`` of columns scaled by ``gain``."""
    rng = _rng(seed)
    w = rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(std)
    k = max(1, int(round(frac * cols)))
    idx = rng.choice(cols, size=k, replace=False)
    w[:, idx] *= np.float32(gain)
    return np.abs(w, out=w)


def config(n: int, index: int = 0, part: str = "up", scale_rows: int = 0) -> Workload:
    """The benchmark configurations.

    0: 8192x8192 N(0,0.02^2), 8:16 (the shape of the paper's runtime tables)
    1: 512x512 N(0,1), 4:8
    2: 4096x4096 N(0,0.02^2), 2:4
    3: 4096x4096 Wanda-style, 8:16
    4: Llama-3-8B MLP, Student-t(3) std 0.02, 16:32; part = "up" (14336x4096)
       or "down" (4096x14336)
    ``scale_rows`` > 0 keeps only that many rows (reduced copies for tests).
    """
    seed = 1000 * n + index
    if n == 0:
        r, c, N, M = 8192, 8192, 8, 16
        s = gaussian_abs(scale_rows or r, c, 0.02, seed)
    elif n == 1:
        r, c, N, M = 512, 512, 4, 8
        s = gaussian_abs(scale_rows or r, c, 1.0, seed)
    elif n == 2:
        r, c, N, M = 4096, 4096, 2, 4
        s = gaussian_abs(scale_rows or r, c, 0.02, seed)
    elif n == 3:
        r, c, N, M = 4096, 4096, 8, 16
        s = wanda_scores(scale_rows or r, c, 0.02, seed)
    elif n == 4:
        r, c = (14336, 4096) if part == "up" else (4096, 14336)
        N, M = 16, 32
        s = student_t_abs(scale_rows or r, c, 0.02, seed + (0 if part == "up" else 1))
    else:
        raise ValueError("config 5 is a sweep: use llama_layer()")
    return Workload(f"config{n}" + (f"-{part}" if n == 4 else ""), s, N, M)


def llama_layer(name: str, N: int, M: int, layer: int = 0, scale_rows: int = 0) -> Workload:
    """Config 5: one linear layer of a Llama-3-8B-shaped model, N(0,0.02^2) with
    0.1 % outlier columns scaled x20."""
    r, c = LLAMA3_8B_LAYER_SHAPES[name]
    order = list(LLAMA3_8B_LAYER_SHAPES).index(name)
    seed = 1000 * 5 + 7 * layer + order
    s = gaussian_outlier_columns_abs(scale_rows or r, c, 0.02, seed)
    return Workload(f"config5-L{layer}-{name}-{N}:{M}", s, N, M)


def default_tau(max_abs_score: float) -> float:
    """Regularisation parameter used throughout: the paper's setting
    "0.005 max|W|" read as the entropy weight 1/tau, i.e. tau = 200 / max|W|
    (argument only; the maximum itself is computed by the caller)."""
    return 200.0 / float(max_abs_score)
