"""Seeded random sweep over shapes, formats, encoder flags and N: every case bit-exact in INT32 against
the oracle's plain product, fp16 within the stated bar. Catches interactions the hand-picked parity
cases do not (ragged edges with folded tiles, sorted rows with INT2 weights, tiny matrices, ...)."""
import numpy as np
import pytest

import oracle
from paper_2608_09291_b200 import workloads

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def b():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2608_09291_b200 import binding
    torch.cuda.set_device(0)
    return binding


def _case(rng):
    kind = rng.choice(["q2", "q2", "q4", "w2"])
    M = int(rng.choice([1, 15, 16, 17, 100, 333, 1024, 2500]))
    K = int(rng.choice([1, 7, 31, 64, 129, 1000, 2048, 4100]))
    s = float(rng.choice([0.0, 0.3, 0.5, 0.7, 0.95, 1.0]))
    if kind == "q2":
        K_L = int(rng.choice([128, 256, 512, 1024, 2048]))
        fmt, flags = (16, K_L, 2, 1), int(rng.choice([0, 2, 4, 6]))
    else:
        K_L = int(rng.choice([256, 512, 1024, 2048]))
        fmt, flags = (16, K_L, 2, 2), int(rng.choice([0, 2]))
    N = int(rng.choice([1, 2, 7, 8, 9, 16, 23, 32, 40, 64]))
    return kind, M, K, s, fmt, flags, N


@pytest.mark.parametrize("i", range(48))
def test_random_case(b, i):
    rng = np.random.default_rng([2024, i])
    kind, M, K, s, fmt, flags, N = _case(rng)
    seed = 9000 + i
    if kind == "w2":
        W = workloads.make_weight_w2(M, K, s, seed=seed)
        flags |= b.US_ENCODE_W2
    else:
        W = workloads.make_weight(M, K, s, seed=seed, row_varying=bool(flags & 2))
    X = workloads.make_x(K, N, seed=seed)
    s_w, s_x = workloads.make_scales(M, N, seed=seed)
    sw = b.SparseWeight(W, s_w, fmt=fmt, max_N=N, flags=flags)
    try:
        assert (b.us_decode(sw.handle) == W).all()
        Xd = torch.from_numpy(b.pack_int4(X)).cuda()
        xs = torch.from_numpy(s_x.copy()).cuda()
        ref = oracle.spmm_dense(W, X)
        for n in sorted({N, max(1, N // 2), 1}):
            for rep in range(2):
                y32 = sw.spmm(Xd[:n].contiguous(), n)
                torch.cuda.synchronize()
                sw.check()
                assert (y32.cpu().numpy() == ref[:n]).all(), (kind, M, K, s, fmt, flags, n, rep)
            y16 = sw.spmm(Xd[:n].contiguous(), n, xs[:n].contiguous())
            torch.cuda.synchronize()
            sw.check()
            assert oracle.fp16_within_tolerance(y16.cpu().numpy(), ref[:n], s_w, s_x[:n]).all(), (kind, M, K, s, fmt, flags, n)
    finally:
        sw.close()
