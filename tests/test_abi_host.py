"""Host side of the C-ABI library: exported symbols, encoder / decoder / statistics against the
oracle, error behaviour, schedule geometry. No GPU needed (US_ENCODE_HOST_ONLY)."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2608_09291_b200 import workloads

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def b():
    from paper_2608_09291_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(b):
    header = (ROOT / "include" / "unionsparse.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(us_[a-z_0-9]+)\s*\(", header))
    assert declared == set(b.EXPORTS)
    lib = ctypes.CDLL(str(ROOT / "paper_2608_09291_b200" / "libunionsparse.so"))
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("M,K,s,K_L", [(64, 1024, 0.5, 1024), (37, 300, 0.5, 128), (160, 2176, 0.7, 256),
                                       (16, 128, 0.0, 128), (48, 512, 1.0, 512), (1024, 1024, 0.3, 256)])
@pytest.mark.parametrize("flags", [0, 2, 4, 6])
def test_round_trip_and_stats_match_oracle(b, M, K, s, K_L, flags):
    W = workloads.make_weight(M, K, s, seed=M + K, row_varying=bool(flags & 2))
    h = b.us_encode(W, fmt=(16, K_L, 2, 1), flags=b.US_ENCODE_HOST_ONLY | flags)
    try:
        assert (b.us_decode(h) == W).all()
        st = b.us_get_stats(h)
        order = b.us_get_row_order(h)
        assert sorted(order[order >= 0]) == list(range(M)) and (order < 0).sum() == st["Mp"] - M
        Wp = np.zeros((st["Mp"], K), np.int8)
        Wp[order >= 0] = W[order[order >= 0]]
        ref = oracle.encode(Wp, 16, K_L, 2, 1)["stats"]
        assert st["nnz"] == ref["nnz"] == int((W != 0).sum())
        assert st["sum_P"] == ref["sum_P"]
        assert st["n_tiles"] == ref["n_lt"]
        assert st["bytes_payload"] == ref["bytes_payload"]
        assert st["bytes_bitmap"] == ref["bytes_bitmap"]
        assert st["bytes_offsets"] == ref["bytes_offsets"]
        assert st["pmr"] == pytest.approx(ref["pmr"], rel=1e-12)
        assert st["fill"] == pytest.approx(2 * ref["sum_P"] / (M * K), rel=1e-12)
        assert st["bytes_payload_padded"] >= st["bytes_payload"]
        assert st["bytes_payload_padded"] % 128 == 0
        assert st["bytes_total"] == st["bytes_payload_padded"] + st["bytes_bitmap"] + st["bytes_offsets"]
        if flags == 2:   # rows ordered by nonzero count
            cnt = (Wp != 0).sum(1)[: M]
            assert (np.diff(cnt) >= 0).all()
        if flags & 4:    # rows paired inside each strip (Alg. 1 on the 16 x K strip, R_A = 2, C_A = 1)
            plain = b.us_encode(W, fmt=(16, K_L, 2, 1), flags=b.US_ENCODE_HOST_ONLY | (flags & 2))
            base = b.us_get_row_order(plain)
            plain_P = b.us_get_stats(plain)["sum_P"]
            b.us_destroy(plain)
            best = 0
            for rb in range(st["Mp"] // 16):
                # the same 16 rows as without the flag, in some other order
                assert sorted(order[16 * rb: 16 * rb + 16]) == sorted(base[16 * rb: 16 * rb + 16])
                rows = base[16 * rb: 16 * rb + 16]
                strip = np.zeros((16, K), np.int8)
                strip[rows >= 0] = W[rows[rows >= 0]]
                best += oracle.reorder_tile(strip != 0, 2, 1)[1]
            assert st["sum_P"] == best <= plain_P
    finally:
        b.us_destroy(h)


def test_default_format_and_padding_overhead(b):
    W = workloads.make_weight(1024, 2048, 0.5, seed=1)
    h = b.us_encode(W, flags=b.US_ENCODE_HOST_ONLY)
    st = b.us_get_stats(h)
    assert st["fmt"][0] == 16 and st["fmt"][2:] == (2, 1) and st["fmt"][1] in (256, 512, 1024)
    assert st["bytes_payload_padded"] < 1.35 * st["bytes_payload"]
    info = b.us_launch_info(h, 8)
    assert info["block"] % 32 == 0 and 64 <= info["block"] <= 512
    assert info["smem_bytes"] <= 227 * 1024
    assert b.us_spmm_bytes(h, 8, True) == st["bytes_total"] + 8 * 1024 + 8 * 1024 * 2 + 2 * (1024 + 8)
    b.us_destroy(h)


def test_error_behaviour(b):
    W = np.zeros((16, 128), np.int8)
    W[3, 5] = 9
    with pytest.raises(b.UsError) as e:
        b.us_encode(W, flags=b.US_ENCODE_HOST_ONLY)
    assert e.value.status == 2                                    # value range
    W[3, 5] = -8
    for fmt, status in [((16, 64, 3, 1), 3), ((16, 100, 2, 1), 3), ((16, 24, 2, 2), 3), ((0, 64, 1, 1), 3)]:
        with pytest.raises(b.UsError) as e:
            b.us_encode(W, fmt=fmt, flags=b.US_ENCODE_HOST_ONLY)
        assert e.value.status == status, fmt
    with pytest.raises(b.UsError) as e:                           # row reordering: kernel layout only
        b.us_encode(W, fmt=(16, 64, 2, 2), flags=b.US_ENCODE_HOST_ONLY | b.US_ENCODE_PAIR_ROWS)
    assert e.value.status == 4
    with pytest.raises(b.UsError) as e:
        b.us_encode(W, max_N=65, flags=b.US_ENCODE_HOST_ONLY)
    assert e.value.status == 1
    h = b.us_encode(W, fmt=(16, 128, 2, 1), flags=b.US_ENCODE_HOST_ONLY)
    with pytest.raises(b.UsError) as e:                           # host-only handle cannot multiply
        b.us_spmm(h, 16, 1, None, 16, None)
    assert e.value.status == 4
    assert b.us_last_error(h) == 0
    b.us_destroy(h)
    assert b.us_status_string(0) == "ok" and "outside" in b.us_status_string(2)


# Formats without a kernel (the paper's 2 x 2 areas, a per-element bitmap, column pairs, a taller
# tile) are encoded in the paper's own array layout: same arrays, bit for bit, as the oracle's.
@pytest.mark.parametrize("fmt", [(16, 64, 2, 2), (16, 64, 1, 1), (16, 64, 1, 2), (16, 64, 2, 1), (32, 128, 4, 2)])
@pytest.mark.parametrize("M,K,s", [(64, 256, 0.5), (37, 300, 0.7), (16, 64, 0.0), (48, 128, 1.0)])
def test_paper_layout_formats_round_trip_and_stats(b, fmt, M, K, s):
    W = workloads.make_weight(M, K, s, seed=M * K + fmt[2] * 10 + fmt[3])
    h = b.us_encode(W, fmt=fmt, flags=b.US_ENCODE_HOST_ONLY)
    try:
        assert (b.us_decode(h) == W).all()
        st = b.us_get_stats(h)
        ref = oracle.encode(W, *fmt)["stats"]
        assert st["fmt"] == fmt
        for lib_key, ref_key in [("nnz", "nnz"), ("sum_P", "sum_P"), ("n_tiles", "n_lt"), ("Mp", "Mp"), ("Kp", "Kp"),
                                 ("bytes_payload", "bytes_payload"), ("bytes_bitmap", "bytes_bitmap"),
                                 ("bytes_offsets", "bytes_offsets")]:
            assert st[lib_key] == ref[ref_key], lib_key
        assert st["bytes_payload_padded"] == st["bytes_payload"]
        assert st["pmr"] == pytest.approx(ref["pmr"], rel=1e-12)
        assert st["fill"] == pytest.approx(ref["fill"], rel=1e-12)
        order = b.us_get_row_order(h)
        assert list(order[:M]) == list(range(M)) and (order[M:] == -1).all()
        with pytest.raises(b.UsError) as e:      # no kernel reads this layout
            b.us_spmm(h, 16, 1, None, 16, None)
        assert e.value.status == 4
        with pytest.raises(b.UsError) as e:
            b.us_launch_info(h, 8)
        assert e.value.status == 4
    finally:
        b.us_destroy(h)


# The folded kernel layout (two column areas: one mask bit covers rows i, i + 8 and columns j, j + K_L/2):
# the library's own tile layout, the oracle's union rule and counts.
@pytest.mark.parametrize("M,K,s,K_L", [(64, 1024, 0.5, 1024), (37, 300, 0.5, 256), (160, 2176, 0.7, 256),
                                       (16, 256, 0.0, 256), (48, 512, 1.0, 512), (512, 2048, 0.6, 512)])
@pytest.mark.parametrize("flags", [0, 2])
def test_folded_kernel_layout_round_trip_and_stats(b, M, K, s, K_L, flags):
    W = workloads.make_weight(M, K, s, seed=M + K + 7, row_varying=bool(flags & 2))
    h = b.us_encode(W, fmt=(16, K_L, 2, 2), max_N=8, flags=b.US_ENCODE_HOST_ONLY | flags)
    try:
        assert (b.us_decode(h) == W).all()
        st = b.us_get_stats(h)
        assert st["fmt"] == (16, K_L, 2, 2)
        order = b.us_get_row_order(h)
        Wp = np.zeros((st["Mp"], K), np.int8)
        Wp[order >= 0] = W[order[order >= 0]]
        ref = oracle.encode(Wp, 16, K_L, 2, 2)["stats"]
        for lib_key, ref_key in [("nnz", "nnz"), ("sum_P", "sum_P"), ("n_tiles", "n_lt"), ("Kp", "Kp"),
                                 ("bytes_payload", "bytes_payload"), ("bytes_bitmap", "bytes_bitmap"),
                                 ("bytes_offsets", "bytes_offsets")]:
            assert st[lib_key] == ref[ref_key], lib_key
        assert st["pmr"] == pytest.approx(ref["pmr"], rel=1e-12)
        assert st["fill"] == pytest.approx(4 * ref["sum_P"] / (M * K), rel=1e-12)
        assert st["bytes_payload_padded"] >= st["bytes_payload"] and st["bytes_payload_padded"] % 256 == 0
    finally:
        b.us_destroy(h)
    with pytest.raises(b.UsError) as e:      # the pairing cost is defined for one column area
        b.us_encode(W, fmt=(16, K_L, 2, 2), max_N=8, flags=b.US_ENCODE_HOST_ONLY | b.US_ENCODE_PAIR_ROWS)
    assert e.value.status == 4


# W2A4: INT2 weights in the folded layout, one payload byte per union-mask bit.
@pytest.mark.parametrize("M,K,s,K_L", [(64, 1024, 0.5, 1024), (37, 300, 0.5, 256), (160, 2176, 0.7, 256), (48, 512, 1.0, 512)])
def test_w2_round_trip_and_stats(b, M, K, s, K_L):
    W = workloads.make_weight_w2(M, K, s, seed=M + K + 11)
    assert W.min() >= -2 and W.max() <= 1
    h = b.us_encode(W, fmt=(16, K_L, 2, 2), max_N=8, flags=b.US_ENCODE_HOST_ONLY | b.US_ENCODE_W2)
    try:
        assert (b.us_decode(h) == W).all()
        st = b.us_get_stats(h)
        ref = oracle.encode(W, 16, K_L, 2, 2)["stats"]     # same union mask; the oracle packs INT4 values
        assert st["weight_bits"] == 2
        assert st["nnz"] == ref["nnz"] and st["sum_P"] == ref["sum_P"] and st["n_tiles"] == ref["n_lt"]
        assert st["bytes_payload"] == ref["sum_P"]         # Q * P_t values of 2 bits = P_t bytes
        assert 2 * st["bytes_payload"] == ref["bytes_payload"]
        assert st["bytes_bitmap"] == ref["bytes_bitmap"] and st["bytes_offsets"] == ref["bytes_offsets"]
        # Eq. 1 with B_w = 0.25 bytes per weight
        assert st["pmr"] == pytest.approx(0.25 * ref["nnz"] / (ref["bytes_bitmap"] + ref["bytes_offsets"]), rel=1e-12)
        assert st["pmr"] == pytest.approx(0.5 * ref["pmr"], rel=1e-12)
    finally:
        b.us_destroy(h)


def test_w2_errors(b):
    W = np.zeros((16, 256), np.int8)
    W[2, 3] = 2                                            # outside [-2, 1]
    with pytest.raises(b.UsError) as e:
        b.us_encode(W, fmt=(16, 256, 2, 2), flags=b.US_ENCODE_HOST_ONLY | b.US_ENCODE_W2)
    assert e.value.status == 2
    W[2, 3] = -2
    for fmt in [(16, 256, 2, 1), (16, 64, 2, 2), None]:    # only the folded kernel layout holds INT2 weights
        with pytest.raises(b.UsError) as e:
            b.us_encode(W, fmt=fmt, flags=b.US_ENCODE_HOST_ONLY | b.US_ENCODE_W2)
        assert e.value.status == 4, fmt
    with pytest.raises(b.UsError) as e:
        b.us_encode(W, fmt=(16, 256, 2, 2), flags=b.US_ENCODE_HOST_ONLY | b.US_ENCODE_W2 | b.US_ENCODE_PAIR_ROWS)
    assert e.value.status == 4


def test_pack_int4(b):
    X = np.array([[1, -2, 7, -8, 0]], np.int8)
    assert list(b.pack_int4(X)[0]) == [0x1 | (0xE << 4), 0x7 | (0x8 << 4), 0x0]
