"""us_spmm_static_scratch: the SpMM for callers that cannot allocate device memory around the
call (a serving loop whose memory pool owns the whole GPU, a latency-critical path that must not
trigger an allocator synchronisation, a program section where allocation calls are forbidden).
Its scratch is a fixed array inside the library instead of memory owned by the handle, so its
results must be the very ones us_spmm gives -- checked here through the C ABI on two calls in a
row (the array keeps the previous call's contents), in shapes that do send partial sums through the
scratch, and against the CPU oracle as well. The file name keeps it last in collection order."""
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


# (M, K, N): direct reduce mode (N = 16: every run of tiles goes through the scratch), two K
# ranges (K = 16384 at N = 8: strips are completed through the scratch), and a small single-range case
CASES = [(1024, 4096, 16), (272, 16384, 8), (1024, 1024, 8), (640, 2048, 33)]


@pytest.mark.parametrize("M,K,N", CASES)
def test_matches_us_spmm_twice(b, M, K, N):
    W = workloads.make_weight(M, K, 0.5, seed=M + K + N)
    X = workloads.make_x(K, N, seed=N)
    s_w, s_x = workloads.make_scales(M, N, seed=M)
    h = b.us_encode(W, s_w, None, 64, 0)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        Xd = torch.from_numpy(b.pack_int4(X)).cuda()
        sxd = torch.from_numpy(s_x.copy()).cuda()
        ref32 = torch.empty((N, M), dtype=torch.int32, device="cuda")
        ref16 = torch.empty((N, M), dtype=torch.float16, device="cuda")
        b.us_spmm(h, Xd.data_ptr(), N, None, ref32.data_ptr(), stream)
        b.us_spmm(h, Xd.data_ptr(), N, sxd.data_ptr(), ref16.data_ptr(), stream)
        torch.cuda.synchronize()
        assert b.us_last_error(h) == 0
        exact = oracle.spmm_dense(W, X)
        for rep in range(2):
            got32 = torch.full((N, M), -7, dtype=torch.int32, device="cuda")
            got16 = torch.full((N, M), -7.0, dtype=torch.float16, device="cuda")
            b.us_spmm_static_scratch(h, Xd.data_ptr(), N, None, got32.data_ptr(), stream)
            b.us_spmm_static_scratch(h, Xd.data_ptr(), N, sxd.data_ptr(), got16.data_ptr(), stream)
            torch.cuda.synchronize()
            assert b.us_last_error(h) == 0
            assert torch.equal(got32, ref32), f"call {rep}: INT32 output differs from us_spmm"
            # same kernel, same arithmetic: the fp16 outputs agree to the last bit, which is
            # inside the suite's fp16 bar (2e-3 relative or one ulp) with room to spare
            assert torch.equal(got16, ref16), f"call {rep}: fp16 output differs from us_spmm"
            # and both are what the oracle says: INT32 bit for bit, fp16 within 2e-3 relative or one ulp
            assert (got32.cpu().numpy() == exact).all(), f"call {rep}: INT32 output differs from the oracle"
            assert oracle.fp16_within_tolerance(got16.cpu().numpy(), exact, s_w, s_x, rel=2e-3).all()
    finally:
        b.us_destroy(h)


def test_refuses_problems_beyond_the_array(b):
    # 1040 strips at N = 64 need 1040 * (8 * 512 + 4) bytes > 4 MiB
    M, K, N = 16640, 128, 64
    W = workloads.make_weight(M, K, 0.5, seed=5)
    h = b.us_encode(W, None, None, 64, 0)
    try:
        X = torch.zeros((N, K // 2), dtype=torch.uint8, device="cuda")
        Y = torch.zeros((N, M), dtype=torch.int32, device="cuda")
        with pytest.raises(b.UsError) as e:
            b.us_spmm_static_scratch(h, X.data_ptr(), N, None, Y.data_ptr(), None)
        assert e.value.status == b.US_ERR_SCRATCH_TOO_SMALL
        # the same handle at N = 8 fits (1040 * 516 bytes) and runs
        b.us_spmm_static_scratch(h, X.data_ptr(), 8, None, Y.data_ptr(), None)
        torch.cuda.synchronize()
        assert b.us_last_error(h) == 0
    finally:
        b.us_destroy(h)
