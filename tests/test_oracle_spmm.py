"""Pins of the oracle's SpMM and dequantisation (the product of paper Alg. 2 and the fused
per-channel x per-token fp16 epilogue). CPU only."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2608_09291_b200 import workloads


def _brute(W, X):
    M, K = W.shape
    N = X.shape[0]
    Y = [[0] * M for _ in range(N)]
    for n in range(N):
        for m in range(M):
            acc = 0
            for k in range(K):
                acc += int(W[m, k]) * int(X[n, k])
            Y[n][m] = acc
    return np.array(Y, dtype=np.int64)


def test_brute_force_tiny():
    W = workloads.make_weight(19, 70, 0.5, seed=2)       # M != K, ragged
    X = workloads.make_x(70, 3, seed=2)
    ref = _brute(W, X)
    assert (oracle.spmm_dense(W, X) == ref).all()
    for fmt in [(16, 64, 2, 2), (16, 64, 1, 1), (16, 64, 2, 1)]:
        assert (oracle.spmm_encoded(oracle.encode(W, *fmt), X) == ref).all()


@pytest.mark.parametrize("M,K,N", [(256, 512, 8), (144, 1088, 5), (1024, 1024, 8)])
def test_against_library_matmul(M, K, N):
    W = workloads.make_weight(M, K, 0.5, seed=M + K)
    X = workloads.make_x(K, N, seed=M)
    ref = X.astype(np.int64) @ W.astype(np.int64).T       # numpy's own integer matmul
    got = oracle.spmm_dense(W, X)
    assert got.dtype == np.int32 and (got == ref).all()
    for fmt in [(16, 64, 2, 2), (16, 64, 1, 1), (16, 256, 2, 1)]:
        assert (oracle.spmm_encoded(oracle.encode(W, *fmt), X) == ref).all()


def test_special_cases():
    M, K, N = 64, 192, 4
    X = workloads.make_x(K, N, seed=9)
    # s = 1: empty payload, Y = 0
    Z = np.zeros((M, K), np.int8)
    assert not oracle.spmm_dense(Z, X).any()
    assert not oracle.spmm_encoded(oracle.encode(Z), X).any()
    # s = 0: dense GEMM, extreme values (no overflow: |acc| <= 64 K)
    D = np.full((M, K), -8, np.int8)
    Xm = np.full((N, K), -8, np.int8)
    assert (oracle.spmm_dense(D, Xm) == 64 * K).all()
    # X = ones -> row sums
    W = workloads.make_weight(M, K, 0.5, seed=4)
    ones = np.ones((N, K), np.int8)
    assert (oracle.spmm_dense(W, ones) == W.astype(np.int64).sum(1)[None, :]).all()
    # one nonzero per row -> a gather of X columns
    G = np.zeros((M, K), np.int8)
    cols = (np.arange(M) * 7) % K
    G[np.arange(M), cols] = 1
    assert (oracle.spmm_dense(G, X) == X[:, cols]).all()
    assert (oracle.spmm_encoded(oracle.encode(G, 16, 64, 2, 1), X) == X[:, cols]).all()
    # linearity in X
    X2 = workloads.make_x(K, N, seed=10) // 2
    X1 = X // 2
    assert (oracle.spmm_dense(W, (X1 + X2).astype(np.int8))
            == oracle.spmm_dense(W, X1.astype(np.int8)) + oracle.spmm_dense(W, X2.astype(np.int8))).all()


def _rn_fp16_exact(fr: Fraction) -> np.float16:
    """Round an exact rational to nearest-even fp16 by search over the fp16 grid."""
    approx = np.float16(float(fr))
    cands = {approx, np.nextafter(approx, np.float16(np.inf)), np.nextafter(approx, np.float16(-np.inf))}
    best = None
    for c in cands:
        if not np.isfinite(c):
            continue
        d = abs(Fraction(float(c)) - fr)
        even = (int(np.array(c).view(np.uint16)) & 1) == 0
        key = (d, 0 if even else 1)
        if best is None or key < best[0]:
            best = (key, c)
    return best[1]


def test_dequant_exact_rational():
    rng = np.random.default_rng(0)
    acc = rng.integers(-200000, 200000, (4, 32)).astype(np.int32)
    acc[0, 0], acc[0, 1] = 0, 1
    s_w, s_x = workloads.make_scales(32, 4, seed=1)
    got = oracle.dequant(acc, s_w, s_x)
    assert got.dtype == np.float16
    for n in range(4):
        for m in range(32):
            fr = Fraction(int(acc[n, m])) * Fraction(float(s_w[m])) * Fraction(float(s_x[n]))
            assert got[n, m] == _rn_fp16_exact(fr)


def test_dequant_closed_form_and_tolerance_rule():
    W = workloads.make_weight(1024, 1024, 0.5, seed=0)
    X = workloads.make_x(1024, 8, seed=0)
    s_w, s_x = workloads.make_scales(1024, 8, seed=0)
    acc = oracle.spmm_dense(W, X)
    y = oracle.dequant(acc, s_w, s_x)
    exact = acc.astype(np.float64) * s_w.astype(np.float64)[None, :] * s_x.astype(np.float64)[:, None]
    # correctly rounded: within half an fp16 ulp of the exact product everywhere
    assert (np.abs(y.astype(np.float64) - exact) <= 0.5 * np.abs(np.spacing(y)).astype(np.float64)).all()
    # the stated bar accepts the reference itself and a 1-ulp neighbour, rejects a 2% error
    ok = oracle.fp16_within_tolerance
    assert ok(y, acc, s_w, s_x).all()
    assert ok(np.nextafter(y, np.float16(np.inf)), acc, s_w, s_x).all()
    big = np.abs(exact) > 1.0
    assert not ok((y.astype(np.float32) * 1.02).astype(np.float16), acc, s_w, s_x)[big].any()
    # power-of-two scales: exact scaling
    acc2 = np.array([[3, -5, 1024]], np.int32)
    assert (oracle.dequant(acc2, np.full(3, 0.5, np.float16), np.array([0.25], np.float16))
            == np.array([[0.375, -0.625, 128.0]], np.float16)).all()


def test_generator_statistics():
    W = workloads.make_weight(2048, 512, 0.7, seed=42)
    assert abs((W == 0).mean() - 0.7) < 5e-3
    assert W.min() == -8 and W.max() == 7
    Wr = workloads.make_weight(2048, 512, 0.5, seed=42, row_varying=True)
    dens = (Wr != 0).mean(1)
    assert 0.25 < dens.min() < 0.36 and 0.64 < dens.max() < 0.75
    assert (workloads.make_weight(2048, 512, 0.7, seed=42) == W).all()       # seeded
    X = workloads.make_x(512, 64, seed=1)
    assert X.min() == -8 and X.max() == 7 and X.shape == (64, 512)
