"""Parity of the CUDA library (through the C ABI) against the CPU oracle, element by element on
the same seeded inputs. INT32 outputs must be bit-exact; fp16 outputs within max(2e-3 relative,
1 fp16 ulp) of the exactly rounded reference."""
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


def _run(b, sw, X, N, scales=None):
    Xd = torch.from_numpy(b.pack_int4(X[:N])).cuda()
    xs = torch.from_numpy(scales[:N].copy()).cuda() if scales is not None else None
    Y = sw.spmm(Xd, N, xs)
    torch.cuda.synchronize()
    sw.check()
    return Y.cpu().numpy()


def _check_case(b, W, X, Ns, s_w=None, s_x=None, fmt=None, flags=0, max_N=64):
    sw = b.SparseWeight(W, s_w, fmt=fmt, max_N=max_N, flags=flags)
    try:
        for N in Ns:
            ref = oracle.spmm_dense(W, X[:N])
            for rep in range(2):     # second call checks the self-cleaning split-K workspace
                got = _run(b, sw, X, N)
                assert got.dtype == np.int32 and got.shape == ref.shape
                bad = int((got != ref).sum())
                assert bad == 0, f"N={N} rep={rep}: {bad} INT32 mismatches"
            if s_w is not None:
                got16 = _run(b, sw, X, N, s_x)
                assert got16.dtype == np.float16
                ok = oracle.fp16_within_tolerance(got16, ref, s_w, s_x[:N], rel=2e-3)
                assert ok.all(), f"N={N}: {int((~ok).sum())} fp16 outputs outside tolerance"
    finally:
        sw.close()


def test_single_1024(b):
    """1024x1024, 50 % uniform sparsity, N = 8, INT32, seed 0."""
    W = workloads.make_weight(1024, 1024, 0.5, seed=0)
    X = workloads.make_x(1024, 8, seed=0)
    _check_case(b, W, X, [8])
    enc = oracle.encode(W, 16, 64, 2, 2)           # the two oracle paths agree on this case too
    assert (oracle.spmm_encoded(enc, X) == oracle.spmm_dense(W, X)).all()


@pytest.mark.parametrize("i,s", [(0, 0.3), (1, 0.5), (2, 0.7)])
def test_attention_4096(b, i, s):
    """LLaMA-2-7B-shaped attention projection, fused fp16 dequant, N in {1, 8, 16, 32}."""
    W = workloads.make_weight(4096, 4096, s, seed=200 + i)
    X = workloads.make_x(4096, 32, seed=200 + i)
    s_w, s_x = workloads.make_scales(4096, 32, seed=200 + i)
    _check_case(b, W, X, [1, 8, 16, 32], s_w, s_x, max_N=32)


@pytest.mark.parametrize("M,K,seed", [(11008, 4096, 300), (4096, 11008, 302)])
@pytest.mark.parametrize("flags", [0, 2, 4, 6])
def test_ffn_7b_row_varying(b, M, K, seed, flags):
    """Row-varying density (keep rate ~U(0.3, 0.7) per row); flags: rows sorted by density (2),
    rows paired inside each strip as Alg. 1 says (4), both (6)."""
    W = workloads.make_weight(M, K, 0.5, seed=seed, row_varying=True)
    X = workloads.make_x(K, 32, seed=seed)
    s_w, s_x = workloads.make_scales(M, 32, seed=seed)
    _check_case(b, W, X, [1, 8, 32], s_w, s_x, flags=flags, max_N=32)


def test_ffn_7b_gate_matrix(b):
    """The second 11008 x 4096 matrix of the 7B-shaped FFN (gate, seed 301): INT32 and fp16."""
    W = workloads.make_weight(11008, 4096, 0.5, seed=301, row_varying=True)
    X = workloads.make_x(4096, 32, seed=301)
    s_w, s_x = workloads.make_scales(11008, 32, seed=301)
    _check_case(b, W, X, [1, 8, 32], s_w, s_x, flags=2, max_N=32)


LAYER13B = [(5120, 5120)] * 4 + [(13824, 5120)] * 2 + [(5120, 13824)]   # Q, K, V, O, gate, up, down


@pytest.mark.parametrize("M,K", [(5120, 5120), (13824, 5120), (5120, 13824)])
@pytest.mark.parametrize("j,s", [(0, 0.3), (1, 0.5), (2, 0.7)])
def test_layer_13b_shapes(b, M, K, j, s):
    """Every shape x sparsity combination of the 13B-shaped layer at full size, N = 16, fp16 output
    (tile sizes, ring depth, warps, K ranges and the reduce mode all depend on the sparsity)."""
    i = LAYER13B.index((M, K))
    W = workloads.make_weight(M, K, s, seed=400 + 10 * j + i)
    X = workloads.make_x(K, 16, seed=400 + 10 * j + i)
    s_w, s_x = workloads.make_scales(M, 16, seed=400 + 10 * j + i)
    _check_case(b, W, X, [16], s_w, s_x, max_N=16)


@pytest.mark.parametrize("j,s", [(0, 0.3), (1, 0.5), (2, 0.7)])
def test_layer_13b_projections_back_to_back(b, j, s):
    """All seven projections of one 13B-shaped decoder layer enqueued back to back on one stream
    (no synchronisation in between, programmatic dependent launch on), three rounds; every output
    is then compared with the oracle: bit-exact INT32 in the first two rounds, fp16 within the bar
    in the third."""
    N = 16
    mats = []
    try:
        for i, (M, K) in enumerate(LAYER13B):
            seed = 400 + 10 * j + i
            W = workloads.make_weight(M, K, s, seed=seed)
            X = workloads.make_x(K, N, seed=seed)
            s_w, s_x = workloads.make_scales(M, N, seed=seed)
            sw = b.SparseWeight(W, s_w, max_N=N)
            mats.append(dict(sw=sw, ref=oracle.spmm_dense(W, X), s_w=s_w, s_x=s_x,
                             Xd=torch.from_numpy(b.pack_int4(X)).cuda(), sxd=torch.from_numpy(s_x.copy()).cuda(),
                             y32=torch.zeros((N, M), dtype=torch.int32, device="cuda"),
                             y16=torch.zeros((N, M), dtype=torch.float16, device="cuda")))
            del W
        for rnd in range(3):
            for m in mats:
                if rnd < 2:
                    m["sw"].spmm(m["Xd"], N, out=m["y32"])
                else:
                    m["sw"].spmm(m["Xd"], N, m["sxd"], out=m["y16"])
        torch.cuda.synchronize()
        for i, m in enumerate(mats):
            m["sw"].check()
            assert (m["y32"].cpu().numpy() == m["ref"]).all(), f"projection {i}: INT32 mismatch"
            ok = oracle.fp16_within_tolerance(m["y16"].cpu().numpy(), m["ref"], m["s_w"], m["s_x"], rel=2e-3)
            assert ok.all(), f"projection {i}: {int((~ok).sum())} fp16 outputs outside tolerance"
    finally:
        for m in mats:
            m["sw"].close()


def test_long_k_single_range_with_packed_activations(b):
    """5120 x 13824 at 50 %: at N <= 8 the whole K extent fits one K range only with the
    activations staged packed (the launch plan picks that); N = 16 needs two ranges."""
    W = workloads.make_weight(5120, 13824, 0.5, seed=411)
    X = workloads.make_x(13824, 16, seed=411)
    s_w, s_x = workloads.make_scales(5120, 16, seed=411)
    _check_case(b, W, X, [3, 8, 16], s_w, s_x, max_N=16)
    _check_case(b, W, X, [8], max_N=8)


@pytest.mark.parametrize("M,K,seed", [(28672, 8192, 500), (8192, 28672, 501)])
def test_ffn_70b_full_size(b, M, K, seed):
    """Full-size 70B FFN shapes in the launch configuration the bench times: every output, bit
    for bit, at every N of the sweep."""
    W = workloads.make_weight(M, K, 0.6, seed=seed)
    X = workloads.make_x(K, 64, seed=seed)
    sw = b.SparseWeight(W, None, max_N=64)
    try:
        for N in (1, 4, 8, 16, 32, 64):
            got = _run(b, sw, X, N)
            ref = oracle.spmm_dense(W, X[:N])
            assert got.shape == ref.shape and (got == ref).all(), N
    finally:
        sw.close()


@pytest.mark.parametrize("M,K", [(16, 128), (1, 1), (17, 130), (100, 999), (250, 1031), (33, 4096 + 8)])
def test_ragged_shapes(b, M, K):
    """M not a multiple of 16, K not a multiple of 8 / 2 / the tile; several tiles plus a tail."""
    W = workloads.make_weight(M, K, 0.5, seed=M * 7 + K)
    X = workloads.make_x(K, 64, seed=K)
    s_w, s_x = workloads.make_scales(M, 64, seed=K)
    _check_case(b, W, X, [1, 3, 8, 13, 24, 33, 64], s_w, s_x)


@pytest.mark.parametrize("K_L", [128, 256, 512, 1024, 2048])
def test_tile_widths(b, K_L):
    W = workloads.make_weight(272, 4096, 0.6, seed=K_L)
    X = workloads.make_x(4096, 16, seed=K_L)
    _check_case(b, W, X, [5, 16], fmt=(16, K_L, 2, 1), max_N=16)


def test_degenerate_matrices(b):
    K, M = 2048, 96
    X = workloads.make_x(K, 16, seed=5)
    Xmin = np.full((16, K), -8, np.int8)
    _check_case(b, np.zeros((M, K), np.int8), X, [1, 16])                # s = 1: empty payload
    _check_case(b, np.full((M, K), -8, np.int8), Xmin, [1, 16])          # dense, extreme product
    _check_case(b, np.full((M, K), 7, np.int8), Xmin, [16])
    W = workloads.make_weight(M, K, 0.0, seed=6)                         # s = 0: dense GEMM
    _check_case(b, W, X, [8])
    G = np.zeros((M, K), np.int8)                                        # one nonzero per row
    G[np.arange(M), (np.arange(M) * 37) % K] = -8
    _check_case(b, G, X, [8])
    H = np.zeros((M, K), np.int8)                                        # only upper-half rows of
    H[8:16] = workloads.make_weight(8, K, 0.5, seed=7)                   # a strip are populated
    _check_case(b, H, X, [8])


def test_invalid_calls(b):
    W = workloads.make_weight(64, 256, 0.5, seed=1)
    sw = b.SparseWeight(W, None, max_N=8)
    X = torch.zeros((8, 128), dtype=torch.uint8, device="cuda")
    Y = torch.zeros((8, 64), dtype=torch.int32, device="cuda")
    s = torch.ones(8, dtype=torch.float16, device="cuda")
    for args in [(X.data_ptr(), 9, None, Y.data_ptr()), (X.data_ptr(), 0, None, Y.data_ptr()),
                 (0, 8, None, Y.data_ptr()), (X.data_ptr(), 8, None, 0),
                 (X.data_ptr(), 8, s.data_ptr(), Y.data_ptr()),      # no weight scales in handle
                 (X.data_ptr() + 4, 4, None, Y.data_ptr())]:         # X not 16-byte aligned
        with pytest.raises(b.UsError) as e:
            b.us_spmm(sw.handle, args[0], args[1], args[2], args[3], None)
        assert e.value.status == 1
    sw.check()
    sw.close()


def test_other_stream(b):
    W = workloads.make_weight(512, 2048, 0.5, seed=3)
    X = workloads.make_x(2048, 8, seed=3)
    sw = b.SparseWeight(W, None, max_N=8)
    st = torch.cuda.Stream()
    Xd = torch.from_numpy(b.pack_int4(X)).cuda()
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        outs = [sw.spmm(Xd, 8) for _ in range(5)]
    st.synchronize()
    sw.check()
    ref = oracle.spmm_dense(W, X)
    for o in outs:
        assert (o.cpu().numpy() == ref).all()
    sw.close()


@pytest.mark.parametrize("M,K,N", [(1024, 4096, 16), (272, 16384, 8), (2048, 2048, 8)])
def test_back_to_back_launches_share_a_handle(b, M, K, N):
    """Consecutive launches may overlap their prologues (programmatic dependent launch). Calls on
    one handle reuse its split-K workspace and counters, and a call's X may be the output of the
    kernel just before it: results must be those of strictly serial execution."""
    W = workloads.make_weight(M, K, 0.5, seed=M + K)
    X1 = workloads.make_x(K, N, seed=1)
    X2 = workloads.make_x(K, N, seed=2)
    sw = b.SparseWeight(W, None, max_N=N)
    try:
        X1d = torch.from_numpy(b.pack_int4(X1)).cuda()
        X2d = torch.from_numpy(b.pack_int4(X2)).cuda()
        Xbuf = torch.empty_like(X1d)
        outs = []
        for i in range(12):
            Xbuf.copy_(X1d if i % 2 == 0 else X2d)        # X written by the kernel right before
            outs.append(sw.spmm(Xbuf, N).clone())
            outs.append(sw.spmm(X2d if i % 2 == 0 else X1d, N))   # two SpMMs back to back
        torch.cuda.synchronize()
        sw.check()
        ref1, ref2 = oracle.spmm_dense(W, X1), oracle.spmm_dense(W, X2)
        for i in range(12):
            a, c = outs[2 * i].cpu().numpy(), outs[2 * i + 1].cpu().numpy()
            assert (a == (ref1 if i % 2 == 0 else ref2)).all(), i
            assert (c == (ref2 if i % 2 == 0 else ref1)).all(), i
    finally:
        sw.close()


def test_chain_of_different_matrices_without_synchronisation(b):
    """Several encoded matrices of different shapes and launch plans (half-SM and full-SM CTAs,
    one and several K ranges, int8 and packed activations) enqueued back to back on one stream,
    many rounds, no synchronisation in between: consecutive launches of different kernels overlap
    their prologues, and each must still see exactly its own inputs, workspace and output."""
    shapes = [(1024, 1024, 8), (4096, 2048, 8), (2048, 4096, 16), (5120, 1024, 8), (768, 8192, 16),
              (3072, 3072, 32), (2048, 12288, 8)]
    cases = []
    try:
        for i, (M, K, N) in enumerate(shapes):
            W = workloads.make_weight(M, K, (0.5, 0.3, 0.7)[i % 3], seed=900 + i)
            X = workloads.make_x(K, N, seed=900 + i)
            sw = b.SparseWeight(W, None, max_N=N)
            cases.append((sw, W, X, N, torch.from_numpy(b.pack_int4(X)).cuda(),
                          torch.zeros((N, M), dtype=torch.int32, device="cuda")))
        for rnd in range(15):
            for sw, W, X, N, Xd, Y in (cases if rnd % 2 == 0 else cases[::-1]):
                sw.spmm(Xd, N, out=Y)
        torch.cuda.synchronize()
        for sw, W, X, N, Xd, Y in cases:
            sw.check()
            assert (Y.cpu().numpy() == oracle.spmm_dense(W, X)).all(), (W.shape, N)
    finally:
        for c in cases:
            c[0].close()


def test_seeded_random_shapes(b):
    """Forty seeded random problems -- shape, sparsity, N, tile width, row-order flags -- each
    checked element by element (INT32 exact, fp16 within the bar), twice per handle."""
    rng = np.random.default_rng(20240917)
    for case in range(40):
        M = int(rng.integers(1, 700))
        K = int(rng.integers(1, 6000))
        s = float(rng.choice([0.0, 0.3, 0.5, 0.7, 0.9, 1.0]))
        N = int(rng.integers(1, 65))
        K_L = int(rng.choice([128, 256, 512, 1024]))
        flags = int(rng.choice([0, 2, 4, 6]))
        W = workloads.make_weight(M, K, s, seed=7000 + case, row_varying=bool(flags & 2))
        X = workloads.make_x(K, N, seed=7000 + case)
        s_w, s_x = workloads.make_scales(M, N, seed=7000 + case)
        try:
            _check_case(b, W, X, [N], s_w, s_x, fmt=(16, K_L, 2, 1), flags=flags, max_N=N)
        except AssertionError as e:
            raise AssertionError(f"case {case}: M={M} K={K} s={s} N={N} K_L={K_L} flags={flags}: {e}")


def test_bounded_wait_gives_up_and_the_handle_recovers(b):
    """A tile copy that never happens (test hook; nothing is left in flight, nothing traps): the
    warp that waits for it gives up after the shortened limit, the call is reported as
    US_ERR_DEVICE_TIMEOUT, the workspace is cleared, and the next call on the handle is correct."""
    M, K, N = 1024, 4096, 8
    W = workloads.make_weight(M, K, 0.5, seed=77)
    X = workloads.make_x(K, N, seed=77)
    ref = oracle.spmm_dense(W, X)
    sw = b.SparseWeight(W, None, max_N=N)
    try:
        Xd = torch.from_numpy(b.pack_int4(X)).cuda()
        n_tiles = sw.stats["n_tiles"]
        for position in (0, n_tiles // 2 + 3, n_tiles - 1):
            b.us_debug_withhold_copy(sw.handle, position, wait_us=2000)
            Y = sw.spmm(Xd, N)
            torch.cuda.synchronize()                       # the kernel returns by itself
            assert b.us_last_error(sw.handle) == 7         # US_ERR_DEVICE_TIMEOUT
            assert b.us_last_error(sw.handle) == 0         # the record was cleared
            b.us_debug_withhold_copy(sw.handle, -1)
            for _ in range(2):
                Y = sw.spmm(Xd, N)
                torch.cuda.synchronize()
                sw.check()
                assert (Y.cpu().numpy() == ref).all(), position
        with pytest.raises(b.UsError) as e:
            b.us_debug_withhold_copy(sw.handle, n_tiles, wait_us=1000)
        assert e.value.status == 1
    finally:
        sw.close()


@pytest.mark.skipif(not torch.cuda.is_available() or torch.cuda.device_count() < 2, reason="needs two GPUs")
def test_call_with_another_device_current_is_refused(b):
    W = workloads.make_weight(64, 256, 0.5, seed=1)
    sw = b.SparseWeight(W, None, max_N=8)
    X = torch.zeros((8, 128), dtype=torch.uint8, device="cuda:0")
    Y = torch.zeros((8, 64), dtype=torch.int32, device="cuda:0")
    try:
        torch.cuda.set_device(1)
        for fn in (b.us_spmm, b.us_spmm_static_scratch):
            with pytest.raises(b.UsError) as e:
                fn(sw.handle, X.data_ptr(), 8, None, Y.data_ptr(), None)
            assert e.value.status == 1
    finally:
        torch.cuda.set_device(0)
        sw.close()


# ---- folded tiles: format (16, K_L, 2, 2), one mask bit per 2 x 2 weights (the paper's Q = 4 union), N <= 8 ----
@pytest.mark.parametrize("M,K,s,K_L,flags", [
    (1024, 1024, 0.5, 256, 0), (1024, 1024, 0.5, 512, 0), (1024, 1024, 0.5, 1024, 0),
    (2000, 1000, 0.5, 512, 0),            # ragged rows and columns
    (1030, 2056, 0.6, 1024, 2),           # ragged, rows sorted by density
    (4096, 4096, 0.3, 512, 0), (4096, 4096, 0.7, 512, 0),
    (512, 8192, 0.5, 2048, 0),            # long tiles
    (4096, 11008, 0.5, 1024, 0),          # several K ranges
    (16, 256, 0.0, 256, 0), (48, 512, 1.0, 512, 0),
])
def test_folded_format(b, M, K, s, K_L, flags):
    seed = 600 + M % 91 + K % 83
    W = workloads.make_weight(M, K, s, seed=seed, row_varying=bool(flags & 2))
    X = workloads.make_x(K, 8, seed=seed)
    s_w, s_x = workloads.make_scales(M, 8, seed=seed)
    _check_case(b, W, X, [1, 3, 8], s_w, s_x, fmt=(16, K_L, 2, 2), flags=flags, max_N=8)


def test_folded_format_70b_full_size(b):
    """28672 x 8192 at 60 % sparsity in the folded format: every row, N = 8 and 1."""
    W = workloads.make_weight(28672, 8192, 0.6, seed=500)
    X = workloads.make_x(8192, 8, seed=500)
    _check_case(b, W, X, [8, 1], fmt=(16, 1024, 2, 2), max_N=8)


@pytest.mark.parametrize("M,K,s,K_L,Ns", [
    (1024, 1024, 0.5, 512, [9, 16, 17, 32, 33, 64]),
    (2000, 1000, 0.5, 256, [12, 24, 48]),
    (5120, 5120, 0.5, 1024, [16, 32]),
    (4096, 11008, 0.5, 1024, [16, 32, 64]),      # several K ranges / global split-K
    (13824, 5120, 0.7, 1024, [16]),
])
def test_folded_format_wider_N(b, M, K, s, K_L, Ns):
    seed = 650 + M % 91 + K % 83
    W = workloads.make_weight(M, K, s, seed=seed)
    X = workloads.make_x(K, max(Ns), seed=seed)
    s_w, s_x = workloads.make_scales(M, max(Ns), seed=seed)
    _check_case(b, W, X, Ns, s_w, s_x, fmt=(16, K_L, 2, 2), max_N=max(Ns))


def test_folded_format_limits(b):
    """Chained calls that leave an absmax have no folded-tile kernel: refused, not silently wrong."""
    W = workloads.make_weight(256, 512, 0.5, seed=3)
    s_w, _ = workloads.make_scales(256, 8, seed=3)
    sw = b.SparseWeight(W, s_w, fmt=(16, 256, 2, 2), max_N=8)
    try:
        X = torch.zeros((8, 512), dtype=torch.float16, device="cuda")
        a, a2 = b.new_amax(), b.new_amax()
        Y = torch.zeros((8, 256), dtype=torch.float16, device="cuda")
        assert b._lib.us_spmm_requant(sw.handle, X.data_ptr(), 512, a.data_ptr(), 8, Y.data_ptr(), a2.data_ptr(), 0, 256, None) == 4
        y = sw.spmm_requant(X, 8, b.absmax_f16(X))      # without an absmax output the plain kernels serve
        torch.cuda.synchronize()
        sw.check()
        assert float(y.abs().max()) == 0.0
    finally:
        sw.close()


# ---- W2A4: INT2 weights in the folded format, one payload byte per union-mask bit ----
@pytest.mark.parametrize("M,K,s,K_L,Ns", [
    (1024, 1024, 0.5, 256, [1, 8]), (1024, 1024, 0.5, 1024, [3, 8, 16]),
    (2000, 1000, 0.5, 512, [5, 8, 24]),           # ragged rows and columns
    (4096, 4096, 0.3, 512, [8]), (4096, 4096, 0.7, 512, [8, 32]),
    (4096, 11008, 0.5, 1024, [8, 32, 64]),        # several K ranges / global split-K
    (48, 512, 1.0, 512, [8]), (16, 256, 0.0, 256, [8]),
])
def test_w2a4(b, M, K, s, K_L, Ns):
    seed = 680 + M % 91 + K % 83
    W = workloads.make_weight_w2(M, K, s, seed=seed)
    X = workloads.make_x(K, max(Ns), seed=seed)
    s_w, s_x = workloads.make_scales(M, max(Ns), seed=seed)
    _check_case(b, W, X, Ns, s_w, s_x, fmt=(16, K_L, 2, 2), flags=b.US_ENCODE_W2, max_N=max(Ns))


def test_w2a4_70b_full_size(b):
    W = workloads.make_weight_w2(28672, 8192, 0.6, seed=500)
    X = workloads.make_x(8192, 8, seed=500)
    _check_case(b, W, X, [8, 1], fmt=(16, 1024, 2, 2), flags=b.US_ENCODE_W2, max_N=8)


def test_stage_timers_on_every_plan_variant(b):
    """Switching the stage timers on must never launch a kernel variant the plan was not laid out for: plans
    without a timer build (folded tiles with packed activations, INT2 weights, N > 8 on folded tiles) simply
    run untimed. Values are checked with the timers on."""
    cases = [((16, 1024, 2, 2), 0, 4096, 4096, 0.5, 8),      # folded, packed X (half-SM plan)
             ((16, 1024, 2, 2), 0, 1024, 2048, 0.5, 16),     # folded, N > 8
             ((16, 512, 2, 2), b.US_ENCODE_W2, 1024, 1024, 0.5, 8),
             ((16, 1024, 2, 1), 0, 4096, 4096, 0.3, 8),      # default format, packed X (half-SM plan)
             (None, 0, 1024, 1024, 0.5, 8)]
    for fmt, flags, M, K, s, N in cases:
        W = workloads.make_weight_w2(M, K, s, seed=77) if flags & b.US_ENCODE_W2 else workloads.make_weight(M, K, s, seed=77)
        X = workloads.make_x(K, N, seed=77)
        sw = b.SparseWeight(W, None, fmt=fmt, max_N=N, flags=flags)
        try:
            b.us_stage_timers(sw.handle, 1)
            Xd = torch.from_numpy(b.pack_int4(X)).cuda()
            for _ in range(2):
                y = sw.spmm(Xd, N)
                torch.cuda.synchronize()
                sw.check()
                assert (y.cpu().numpy() == oracle.spmm_dense(W, X)).all(), (fmt, flags, M, K, N)
            d = b.us_stage_timers(sw.handle, 0, read=True)
            assert d["warps"] >= 0
        finally:
            sw.close()
