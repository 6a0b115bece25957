"""Pins of the oracle's IE-BME encoder / decoder / PMR against what the paper and the
mathematics fix (paper Sec. V-A, Sec. VI-B, Eq. 1). CPU only."""
import itertools
import math

import numpy as np
import pytest

import oracle
from paper_2608_09291_b200 import workloads

FORMATS = [(16, 64, 2, 2), (16, 64, 1, 1), (16, 64, 2, 1), (16, 64, 1, 2),
           (8, 32, 2, 2), (16, 256, 2, 1), (16, 128, 4, 2)]


def _read_golden(path):
    out = {}
    for line in path.read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        k, *v = line.split()
        out.setdefault(k, []).append(v)
    return out


# ---- values the paper prints -------------------------------------------------------------

def test_paper_packing_example(golden_dir):
    g = _read_golden(golden_dir / "union_bitmap_packing.txt")
    words = [int(x, 16) for x in g["row_words"][0]]
    rows = [r[0] for r in g["mask_row"]]
    Q = int(g["Q"][0][0])
    # the fixture is self-consistent: rows written out LSB-first equal the printed words
    for w, r in zip(words, rows):
        assert sum(int(b) << i for i, b in enumerate(r)) == w
        assert r.count("1") == int(g["active_per_row"][0][0])
    # build an 8x32 tile (2x2 areas -> 4x16 union mask) whose union mask is the printed one;
    # put the nonzero in a different area for every active position
    mask = np.array([[int(b) for b in r] for r in rows], dtype=np.uint8)
    W = np.zeros((8, 32), dtype=np.int8)
    area = 0
    for i in range(4):
        for j in range(16):
            if mask[i, j]:
                a, c = divmod(area % 4, 2)
                W[a * 4 + i, c * 16 + j] = 3
                area += 1
    # two tiles side by side so that a "next offset" exists
    enc = oracle.encode(np.hstack([W, W]), H_L=8, K_L=32, R_A=2, C_A=2)
    expect_word = sum(w << (16 * i) for i, w in enumerate(words))
    assert int(enc["bitmaps"][0]) == expect_word
    assert int(enc["bitmaps"][1]) == expect_word
    assert list(enc["offsets"]) == [0, int(g["next_offset"][0][0]), 2 * int(g["next_offset"][0][0])]
    assert enc["stats"]["sum_P"] == 2 * int(g["P_t"][0][0])
    assert enc["stats"]["n_values"] == 2 * Q * int(g["P_t"][0][0])


def test_paper_union_group_example(golden_dir):
    g = _read_golden(golden_dir / "union_group.txt")
    active = [int(x) for x in g["group_active"][0]]
    W = np.zeros((16, 64), dtype=np.int8)
    i, j = 5, 17  # one grouped position; areas are contiguous halves of the tile
    for q, v in enumerate(active):
        a, c = divmod(q, 2)
        W[a * 8 + i, c * 32 + j] = v
    enc = oracle.encode(W, 16, 64, 2, 2)
    assert enc["stats"]["sum_P"] == 1                      # one union bit
    beta = i * 32 + j
    bm = enc["bitmaps"]
    assert int(bm[beta // 64]) == 1 << (beta % 64) and int(np.bitwise_count(bm).sum()) == 1
    assert list(oracle.cv_values(enc)) == active           # all four values, the zero included
    assert enc["stats"]["n_values"] - enc["stats"]["nnz"] == 1   # exactly one stored zero
    # the all-zero group emits nothing
    enc0 = oracle.encode(np.zeros((16, 64), np.int8), 16, 64, 2, 2)
    assert enc0["stats"]["n_values"] == 0 and not enc0["bitmaps"].any()
    assert list(enc0["offsets"]) == [0, 0]


def test_paper_lspd_segment_example(golden_dir):
    g = _read_golden(golden_dir / "lspd_segment.txt")
    seg = [int(b) for b in g["segment"][0][0]]
    pos = [int(x) for x in g["active_positions"][0]]
    rel = [int(x) for x in g["payload_index_minus_base"][0]]
    assert [p for p, b in enumerate(seg) if b] == pos
    # place the segment as segment g=2 of row r=3 of an 8x32 mask with other bits around it
    rng = np.random.default_rng(7)
    mask = (rng.random((8, 32)) < 0.4).astype(np.uint8)
    r, gseg, G = 3, 2, 8
    mask[r, gseg * G:(gseg + 1) * G] = seg
    W = np.zeros((16, 64), dtype=np.int8)
    vals = rng.integers(1, 8, (8, 32)).astype(np.int8)
    W[:8, :32] = mask * vals                               # area 0 carries the values
    enc = oracle.encode(W, 16, 64, 2, 2)
    base = oracle.lspd_idx_base(mask, r, gseg, G)
    cv = oracle.cv_values(enc)
    for p, d in zip(pos, rel):                             # stream 0 at idx_base + seg_rank
        assert cv[base + d] == W[r, gseg * G + p]
    P = int(mask.sum())
    assert (cv[P:] == 0).all() and len(cv) == 4 * P       # streams 1..3 hold aligned zeros


# ---- closed forms and invariants ---------------------------------------------------------

@pytest.mark.parametrize("fmt", FORMATS)
@pytest.mark.parametrize("s", [0.0, 0.3, 0.5, 0.7, 1.0])
def test_round_trip_and_invariants(fmt, s):
    H_L, K_L, R_A, C_A = fmt
    Q = R_A * C_A
    M, K = 3 * H_L + 5, 2 * K_L + 7                        # ragged: exercises zero padding
    W = workloads.make_weight(M, K, s, seed=11)
    enc = oracle.encode(W, *fmt)
    st = enc["stats"]
    assert (oracle.decode(enc) == W).all()
    off = enc["offsets"].astype(np.int64)
    wpl = st["words_per_lt"]
    P = np.bitwise_count(enc["bitmaps"]).reshape(-1, wpl).sum(1).astype(np.int64)
    assert off[0] == 0 and (np.diff(off) == Q * P).all()   # o_t = sum_{tau<t} Q P_tau
    assert off[-1] == Q * P.sum() == st["n_values"]
    assert st["nnz"] == int((W != 0).sum())
    cv = oracle.cv_values(enc)
    assert int((cv == 0).sum()) == st["n_values"] - st["nnz"]   # stored zeros = Q sum P - nnz
    if Q == 1:
        assert st["sum_P"] == st["nnz"]                    # degenerates to bitmap + nonzeros
    assert st["bytes_bitmap"] == st["n_lt"] * H_L * K_L // (8 * Q)
    assert st["bytes_offsets"] == 4 * (st["n_lt"] + 1)
    assert st["bytes_payload"] == (st["n_values"] + 1) // 2
    meta = st["n_lt"] * (H_L * K_L // (8 * Q) + 4) + 4
    assert st["pmr"] == pytest.approx(0.5 * st["nnz"] / meta, rel=1e-12)


def test_address_formula_brute_force():
    """CV[o_t + q P_t + rho_t(i,j)] = W_t^(q)(i,j), rho counted by brute force, tiny tiles."""
    for fmt in [(8, 32, 2, 2), (16, 64, 2, 1), (16, 64, 1, 2), (16, 64, 1, 1)]:
        H_L, K_L, R_A, C_A = fmt
        H_B, K_B = H_L // R_A, K_L // C_A
        W = workloads.make_weight(2 * H_L, 3 * K_L, 0.6, seed=5)
        enc = oracle.encode(W, *fmt)
        cv, off = oracle.cv_values(enc), enc["offsets"]
        for t, (rb, kb) in enumerate(itertools.product(range(2), range(3))):
            tile = W[rb * H_L:(rb + 1) * H_L, kb * K_L:(kb + 1) * K_L]
            areas = [tile[a * H_B:(a + 1) * H_B, c * K_B:(c + 1) * K_B]
                     for a in range(R_A) for c in range(C_A)]
            B = np.zeros((H_B, K_B), bool)
            for A in areas:
                B |= A != 0
            P, flat = int(B.sum()), B.ravel()
            for beta in np.flatnonzero(flat):
                rho = int(flat[:beta].sum())
                i, j = divmod(int(beta), K_B)
                for q, A in enumerate(areas):
                    assert cv[off[t] + q * P + rho] == A[i, j]


def test_pmr_closed_form_bernoulli():
    """Eq. 1 on a Bernoulli mask at 16x64 tiles: 14.22*(1-s) for Q=4, 3.88*(1-s) for Q=1
    (up to sampling error and the one trailing offset), E[P_t] = (H_L K_L / Q)(1 - s^Q)."""
    M = K = 1024
    for s in (0.3, 0.5, 0.7):
        W = workloads.make_weight(M, K, s, seed=3)
        for (R_A, C_A) in ((2, 2), (1, 1), (2, 1)):
            Q = R_A * C_A
            st = oracle.encode(W, 16, 64, R_A, C_A)["stats"]
            expect = 0.5 * (1 - s) * 1024 / (1024 / (8 * Q) + 4)
            assert st["pmr"] == pytest.approx(expect, rel=5e-3)
            assert st["sum_P"] / st["n_lt"] == pytest.approx(1024 / Q * (1 - s ** Q), rel=5e-3)
    assert 0.5 * 0.5 * 1024 / (32 + 4) == pytest.approx(7.11, abs=5e-3)


def test_bit_order_is_lsb_first_row_major():
    """A single nonzero at mask position (i, j) sets bit i*K_B + j and nothing else."""
    for (i, j) in [(0, 0), (0, 1), (0, 31), (1, 0), (7, 31), (3, 20)]:
        W = np.zeros((16, 64), np.int8)
        W[i + 8, j + 32] = -8                              # area 3 of the 2x2 partition
        enc = oracle.encode(W, 16, 64, 2, 2)
        beta = i * 32 + j
        expect = np.zeros(4, np.uint64)
        expect[beta // 64] = np.uint64(1) << np.uint64(beta % 64)
        assert (enc["bitmaps"] == expect).all()
        assert list(oracle.cv_values(enc)) == [0, 0, 0, -8]   # q-major, q = a*C_A + c


def test_tile_order_is_row_block_major():
    W = np.zeros((32, 192), np.int8)
    W[16, 64] = 5          # tile (rb=1, kb=1) -> t = 1*3 + 1 = 4
    enc = oracle.encode(W, 16, 64, 1, 1)
    P = np.bitwise_count(enc["bitmaps"]).reshape(-1, 16).sum(1)
    assert list(np.flatnonzero(P)) == [4]
    assert list(enc["offsets"]) == [0, 0, 0, 0, 0, 1, 1]


def test_value_range_and_format_errors():
    W = np.zeros((16, 64), np.int8)
    W[0, 0] = 8
    with pytest.raises(ValueError):
        oracle.encode(W, 16, 64, 2, 2)
    W[0, 0] = -8
    oracle.encode(W, 16, 64, 2, 2)                         # -8 is a legal INT4 value
    assert oracle.check_format(16, 64, 3, 2) != 0          # R_A does not divide H_L
    assert oracle.check_format(8, 8, 2, 2) != 0            # mask not a whole 64-bit word
    assert oracle.check_format(16, 64, 2, 2) == 0


def test_idx_base_equals_running_rank():
    """idx_base(r, g) + seg_rank (Sec. VI-B) is the row-major rank rho of Sec. V-A."""
    rng = np.random.default_rng(1)
    mask = (rng.random((8, 32)) < 0.5).astype(np.uint8)
    flat = mask.ravel()
    G = 8
    for r in range(8):
        for g in range(4):
            base = oracle.lspd_idx_base(mask, r, g, G)
            assert base == int(flat[: r * 32 + g * G].sum())
            seg = mask[r, g * G:(g + 1) * G]
            for rank, p in enumerate(np.flatnonzero(seg)):
                assert base + rank == int(flat[: r * 32 + g * G + p].sum())


def test_nibble_packing_low_first():
    W = np.zeros((16, 64), np.int8)
    W[0, 0], W[0, 1], W[0, 2] = 1, -2, 7
    enc = oracle.encode(W, 16, 64, 1, 1)
    assert list(enc["cv"][:2]) == [0x1 | (0xE << 4), 0x7]
