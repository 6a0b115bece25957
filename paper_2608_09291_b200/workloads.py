"""Seeded synthetic inputs (weights, activations, scales) shared by the tests, the bench and
the oracle checks. Holds none of the method's arithmetic: it only draws random numbers.

The shapes stand in for the LLaMA-2-7B/13B/70B projection matrices the paper's kernel corpus is
built from (paper Sec. VII-A); masks are Bernoulli, either uniform or with a per-row keep rate.
"""
from __future__ import annotations

import numpy as np

ROW_CHUNK = 1024
_X_STREAM = 10 ** 6


def make_weight(M: int, K: int, sparsity: float, seed: int, row_varying: bool = False) -> np.ndarray:
    """Dense int8 matrix, values uniform on [-8,7] without 0 where kept, 0 where pruned.

    Rows are drawn in chunks of 1024 from ``default_rng([seed, chunk])``: (row-varying only)
    per-row keep rates ~U(0.3, 0.7), then the keep draws, then the values.
    """
    W = np.zeros((M, K), dtype=np.int8)
    for c, r0 in enumerate(range(0, M, ROW_CHUNK)):
        rows = min(ROW_CHUNK, M - r0)
        rng = np.random.default_rng([seed, c])
        if row_varying:
            p = rng.uniform(0.3, 0.7, rows)
        U = rng.random((rows, K))
        keep = U < (p[:, None] if row_varying else (1.0 - sparsity))
        v = rng.integers(0, 15, (rows, K))
        v = np.where(v < 8, v - 8, v - 7).astype(np.int8)
        W[r0:r0 + rows] = np.where(keep, v, 0)
    return W


def make_weight_w2(M: int, K: int, sparsity: float, seed: int) -> np.ndarray:
    """INT2 weights for the W2A4 rows: the mask of make_weight(seed), kept values uniform on
    {-2, -1, 1} (the nonzero values of [-2, 1])."""
    W4 = make_weight(M, K, sparsity, seed)
    out = np.zeros_like(W4)
    for c, r0 in enumerate(range(0, M, ROW_CHUNK)):
        rows = min(ROW_CHUNK, M - r0)
        rng = np.random.default_rng([seed, c, 2])
        v = np.array([-2, -1, 1], dtype=np.int8)[rng.integers(0, 3, (rows, K))]
        out[r0:r0 + rows] = np.where(W4[r0:r0 + rows] != 0, v, 0)
    return out


def make_x(K: int, N_max: int, seed: int) -> np.ndarray:
    """Activations, int8 values uniform on [-8,7], token-major (N_max, K)."""
    rng = np.random.default_rng([seed, _X_STREAM])
    return rng.integers(-8, 8, (N_max, K)).astype(np.int8)


def make_x_f16(K: int, N_max: int, seed: int, outliers: bool = True) -> np.ndarray:
    """fp16 activations for the chained calls, token-major (N_max, K): normal draws with a
    per-token spread ~U(0.2, 3) and (optionally) a few channels 8x larger, the usual shape of LLM
    hidden states."""
    rng = np.random.default_rng([seed, _X_STREAM + 2])
    x = rng.standard_normal((N_max, K)) * rng.uniform(0.2, 3.0, (N_max, 1))
    if outliers and K >= 64:
        ch = rng.choice(K, size=max(1, K // 256), replace=False)
        x[:, ch] *= 8.0
    return x.astype(np.float16)


def make_scales(M: int, N_max: int, seed: int):
    """fp16 per-output-channel weight scales ~U(0.005,0.02) and per-token activation scales
    ~U(0.01,0.05)."""
    rng = np.random.default_rng([seed, _X_STREAM + 1])
    s_w = rng.uniform(0.005, 0.02, M).astype(np.float16)
    s_x = rng.uniform(0.01, 0.05, N_max).astype(np.float16)
    return s_w, s_x


def make_chain_weight_scales(M: int, K: int, seed: int) -> np.ndarray:
    """Weight scales for a chain of projections: those of make_scales times 16 / sqrt(K), which
    keeps the magnitude of the activations about level from one projection to the next (the job
    the normalisation layers do in a real decoder), so that a chain stays inside the fp16 range."""
    s_w, _ = make_scales(M, 1, seed)
    return (s_w.astype(np.float64) * 16.0 / np.sqrt(K)).astype(np.float16)


# The synthetic configurations of the build's target (name -> list of cases).
def config_cases(name: str):
    if name == "single":
        return [dict(M=1024, K=1024, s=0.5, N=[8], seed=0, row_varying=False)]
    if name == "attn7b":
        return [dict(M=4096, K=4096, s=s, N=[1, 8, 16, 32], seed=200 + i, row_varying=False)
                for i, s in enumerate((0.3, 0.5, 0.7))]
    if name == "ffn7b":
        return [dict(M=11008, K=4096, s=0.5, N=[1, 8, 32], seed=300, row_varying=True),
                dict(M=11008, K=4096, s=0.5, N=[1, 8, 32], seed=301, row_varying=True),
                dict(M=4096, K=11008, s=0.5, N=[1, 8, 32], seed=302, row_varying=True)]
    if name == "layer13b":
        shapes = [(5120, 5120)] * 4 + [(13824, 5120)] * 2 + [(5120, 13824)]
        return [dict(M=m, K=k, s=s, N=[16], seed=400 + 10 * j + i, row_varying=False)
                for j, s in enumerate((0.3, 0.5, 0.7)) for i, (m, k) in enumerate(shapes)]
    if name == "ffn70b":
        return [dict(M=28672, K=8192, s=0.6, N=[1, 4, 8, 16, 32, 64], seed=500, row_varying=False),
                dict(M=8192, K=28672, s=0.6, N=[1, 4, 8, 16, 32, 64], seed=501, row_varying=False)]
    raise KeyError(name)
