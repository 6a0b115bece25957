"""CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Thin ctypes/numpy front end of ``iebme_oracle.c`` (plain C, fp64/int32 arithmetic) plus the
fp16 dequantisation written out in numpy float64. Only ``tests/``, the smoke check and the
bench's cpu-baseline leg may import this package; the CUDA library never does, and this
package never imports the CUDA library.

What each function follows:
  encode / decode      paper Sec. V-A (area partition, union mask, the three IE-BME arrays)
  stats["pmr"]         paper Eq. 1 with Stor_meta = bitmaps + offsets, B_w = 0.5
  spmm_dense           the plain definition of the product the kernel of Alg. 2 reaches
  spmm_encoded         the same product taken straight from the IE-BME arrays
  lspd_idx_base        paper Sec. VI-B, idx_base(r, g)
  dequant              per-channel x per-token scaling to fp16; not in the paper -- defined by
                       the build's target: RN_fp16(double(acc) * double(s_w) * double(s_x))
  absmax_f16           max |y| per token over a column range, exact in fp16
  requant_int4         per-token symmetric INT4 re-quantisation of an fp16 activation. The paper
                       takes INT4 activations as given (W4A4, Sec. VII-A) and defines no
                       quantiser; the reading used here is the plain symmetric absmax one with
                       a reciprocal step: s = RN_fp16(fp32(amax) / 7) is the dequantisation
                       scale, inv = min(RN_fp16(7 / fp32(amax)), 65504) (65504 when amax = 0),
                       code = clamp(RNE(y * inv), -8, 7) with the product of the two fp16
                       numbers taken exactly (it fits fp32). Floating point decides an integer
                       here, so this precision is part of the definition on both sides.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "iebme_oracle.c"
_LIB_PATH = _HERE / "libiebme_oracle.so"
_lib = None


class _Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "M", "K", "Mp", "Kp", "n_lt", "words_per_lt", "nnz", "sum_P", "n_values",
        "bytes_payload", "bytes_bitmap", "bytes_offsets")] + [
        ("pmr", ctypes.c_double), ("fill", ctypes.c_double)]


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2, OpenMP for the naive GEMM's row loop)."""
    if force or not _LIB_PATH.exists() or _LIB_PATH.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB_PATH.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-Wextra",
                        str(_SRC), "-o", str(tmp)], check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB_PATH))
        lib.orc_lspd_idx_base.restype = ctypes.c_int64
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i64(v):
    return ctypes.c_int64(int(v))


def check_format(H_L: int, K_L: int, R_A: int, C_A: int) -> int:
    return int(_load().orc_check_format(int(H_L), int(K_L), int(R_A), int(C_A)))


def encode(W: np.ndarray, H_L: int = 16, K_L: int = 64, R_A: int = 2, C_A: int = 2) -> dict:
    """IE-BME encode of an int8 matrix with values in [-8,7] (0 = pruned)."""
    lib = _load()
    W = np.ascontiguousarray(W, dtype=np.int8)
    M, K = W.shape
    if check_format(H_L, K_L, R_A, C_A):
        raise ValueError("unusable IE-BME format parameters")
    n_lt, wpl, cap = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
    lib.orc_sizes(_i64(M), _i64(K), H_L, K_L, R_A, C_A,
                  ctypes.byref(n_lt), ctypes.byref(wpl), ctypes.byref(cap))
    bitmaps = np.zeros(n_lt.value * wpl.value, dtype=np.uint64)
    offsets = np.zeros(n_lt.value + 1, dtype=np.uint32)
    cv = np.zeros(cap.value, dtype=np.uint8)
    st = _Stats()
    rc = lib.orc_encode(_p(W), _i64(M), _i64(K), H_L, K_L, R_A, C_A,
                        _p(bitmaps), _p(offsets), _p(cv), ctypes.byref(st))
    if rc:
        raise ValueError("weight value outside [-8, 7]")
    stats = {n: getattr(st, n) for n, _ in _Stats._fields_}
    return {"bitmaps": bitmaps, "offsets": offsets, "cv": cv[: stats["bytes_payload"] + 1],
            "stats": stats, "fmt": (H_L, K_L, R_A, C_A), "shape": (M, K)}


def decode(enc: dict) -> np.ndarray:
    lib = _load()
    M, K = enc["shape"]
    H_L, K_L, R_A, C_A = enc["fmt"]
    out = np.zeros((M, K), dtype=np.int8)
    lib.orc_decode(_p(enc["bitmaps"]), _p(enc["offsets"]), _p(enc["cv"]),
                   _i64(M), _i64(K), H_L, K_L, R_A, C_A, _p(out))
    return out


def cv_values(enc: dict) -> np.ndarray:
    """The Compressed Values array unpacked to one int8 per INT4 value."""
    n = enc["stats"]["n_values"]
    b = enc["cv"]
    nib = np.empty(2 * len(b), dtype=np.int16)
    nib[0::2] = b & 0xF
    nib[1::2] = b >> 4
    nib = nib[:n]
    return np.where(nib >= 8, nib - 16, nib).astype(np.int8)


def spmm_dense(W: np.ndarray, X: np.ndarray) -> np.ndarray:
    """Y[n, m] = sum_k W[m, k] * X[n, k] in INT32. W: (M, K) int8; X: (N, K) int8."""
    lib = _load()
    W = np.ascontiguousarray(W, dtype=np.int8)
    X = np.ascontiguousarray(X, dtype=np.int8)
    M, K = W.shape
    N = X.shape[0]
    assert X.shape[1] == K
    Y = np.zeros((N, M), dtype=np.int32)
    lib.orc_spmm_dense(_p(W), _p(X), _i64(M), _i64(K), _i64(N), _p(Y))
    return Y


def spmm_encoded(enc: dict, X: np.ndarray) -> np.ndarray:
    lib = _load()
    X = np.ascontiguousarray(X, dtype=np.int8)
    M, K = enc["shape"]
    H_L, K_L, R_A, C_A = enc["fmt"]
    N = X.shape[0]
    assert X.shape[1] == K
    Y = np.zeros((N, M), dtype=np.int32)
    lib.orc_spmm_encoded(_p(enc["bitmaps"]), _p(enc["offsets"]), _p(enc["cv"]),
                         _i64(M), _i64(K), H_L, K_L, R_A, C_A, _p(X), _i64(N), _p(Y))
    return Y


def lspd_idx_base(mask: np.ndarray, r: int, g: int, G: int) -> int:
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    return int(_load().orc_lspd_idx_base(_p(mask), int(mask.shape[1]), int(r), int(g), int(G)))


def reorder_tile(mask: np.ndarray, R_A: int, C_A: int):
    """Alg. 1 on one local tile. mask: (H_L, K_L) array, nonzero = surviving weight.
    Returns (perm, cost): perm[p * (H_L // R_A) + g] = the p-th row of the g-th group; cost = the
    least number of active union-mask entries (Eq. 5 at the full row set)."""
    lib = _load()
    m = np.ascontiguousarray(mask != 0, dtype=np.uint8)
    H_L, K_L = m.shape
    perm = np.full(H_L, -1, dtype=np.int32)
    lib.orc_reorder_tile.restype = ctypes.c_int64
    cost = lib.orc_reorder_tile(_p(m), int(H_L), int(K_L), int(R_A), int(C_A), _p(perm))
    if cost < 0:
        raise ValueError("unusable reordering parameters")
    return perm, int(cost)


def dequant(acc: np.ndarray, s_w: np.ndarray, s_x: np.ndarray) -> np.ndarray:
    """fp16(acc[n, m] * s_w[m] * s_x[n]); the scales are fp16 inputs, the product is taken in
    float64 and rounded once to nearest-even fp16."""
    sw = np.asarray(s_w, dtype=np.float16).astype(np.float64)
    sx = np.asarray(s_x, dtype=np.float16).astype(np.float64)
    y = acc.astype(np.float64) * sw[None, :] * sx[:, None]
    return y.astype(np.float16)


def fp16_within_tolerance(got: np.ndarray, ref_acc: np.ndarray, s_w: np.ndarray,
                          s_x: np.ndarray, rel: float = 2e-3) -> np.ndarray:
    """Element-wise check against the stated bar: |got - exact| <= max(rel*|exact|, 1 fp16 ulp of
    the correctly rounded reference)."""
    sw = np.asarray(s_w, dtype=np.float16).astype(np.float64)
    sx = np.asarray(s_x, dtype=np.float16).astype(np.float64)
    exact = ref_acc.astype(np.float64) * sw[None, :] * sx[:, None]
    ref16 = exact.astype(np.float16)
    ulp = np.abs(np.spacing(ref16)).astype(np.float64)
    err = np.abs(got.astype(np.float64) - ref16.astype(np.float64))
    return err <= np.maximum(rel * np.abs(exact), ulp)


def absmax_f16(y16: np.ndarray, m0: int = 0, m1: int | None = None) -> np.ndarray:
    """amax[n] = max over m in [m0, m1) of |y16[n, m]| as fp16 (0 for an empty range)."""
    y = np.asarray(y16, dtype=np.float16)[:, m0:m1]
    if y.shape[1] == 0:
        return np.zeros(y.shape[0], dtype=np.float16)
    return np.abs(y).max(axis=1).astype(np.float16)


FP16_MAX = np.float16(65504.0)


def requant_scale(amax16: np.ndarray) -> np.ndarray:
    """s[n] = RN_fp16(fp32(amax[n]) / fp32(7)): the dequantisation scale per token."""
    a = np.asarray(amax16, dtype=np.float16).astype(np.float32)
    return (a / np.float32(7.0)).astype(np.float16)


def requant_inverse(amax16: np.ndarray) -> np.ndarray:
    """inv[n] = min(RN_fp16(fp32(7) / fp32(amax[n])), 65504); 65504 for amax = 0."""
    a = np.asarray(amax16, dtype=np.float16).astype(np.float32)
    with np.errstate(divide="ignore", over="ignore"):
        inv = np.float32(7.0) / a                       # +inf for amax = 0
        inv16 = inv.astype(np.float16)                  # overflows to +inf above 65504 (+ half an ulp)
    return np.minimum(inv16, FP16_MAX)


def requant_int4(y16: np.ndarray, amax16: np.ndarray | None = None):
    """(codes int8 (N, M) in [-8, 7], scales fp16 (N,)) of a finite fp16 activation y16 (N, M).
    amax16 defaults to the per-token absmax over all of y16's columns."""
    y = np.asarray(y16, dtype=np.float16)
    if amax16 is None:
        amax16 = absmax_f16(y)
    inv = requant_inverse(amax16)
    r = y.astype(np.float32) * inv.astype(np.float32)[:, None]     # exact: 11-bit x 11-bit significands
    q = np.clip(np.rint(r), -8, 7).astype(np.int8)                  # rint: ties to even
    return q, requant_scale(amax16)


def num_threads() -> int:
    return int(_load().orc_num_threads())
