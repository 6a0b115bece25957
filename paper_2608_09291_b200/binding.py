"""ctypes front end of the C-ABI library (``include/unionsparse.h``): argument marshalling only.

Every step of the SpMM runs in the CUDA library; there is no CPU fallback. Importing this module
fails loudly when the compiled library is missing (build it with ``python -m
paper_2608_09291_b200.build`` or ``__graft_entry__.build()``).
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

_LIB_PATH = Path(__file__).resolve().parent / "libunionsparse.so"
if not _LIB_PATH.exists():
    raise ImportError(f"{_LIB_PATH} is missing: build the CUDA library first "
                      "(python -m paper_2608_09291_b200.build)")
_lib = ctypes.CDLL(str(_LIB_PATH))

US_OK = 0
US_ENCODE_HOST_ONLY = 1
US_ENCODE_SORT_ROWS = 2
US_ENCODE_PAIR_ROWS = 4
US_ENCODE_W2 = 8

EXPORTS = ["us_encode", "us_get_stats", "us_decode", "us_get_row_order", "us_spmm", "us_spmm_static_scratch",
           "us_spmm_requant", "us_absmax_f16", "us_quantize_f16",
           "us_last_error", "us_debug_withhold_copy", "us_stage_timers", "us_destroy", "us_spmm_bytes", "us_launch_info", "us_status_string"]


class us_format(ctypes.Structure):
    _fields_ = [("H_L", ctypes.c_int32), ("K_L", ctypes.c_int32),
                ("R_A", ctypes.c_int32), ("C_A", ctypes.c_int32)]


class us_stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "M", "K", "Mp", "Kp", "nnz", "n_tiles", "sum_P", "bytes_payload", "bytes_payload_padded",
        "bytes_bitmap", "bytes_offsets", "bytes_total")] + [
        ("pmr", ctypes.c_double), ("fill", ctypes.c_double), ("fmt", us_format),
        ("weight_bits", ctypes.c_int32), ("reserved", ctypes.c_int32)]


_vp = ctypes.c_void_p
_lib.us_encode.argtypes = [_vp, ctypes.c_int64, ctypes.c_int64, _vp, ctypes.POINTER(us_format),
                           ctypes.c_int32, ctypes.c_uint32, ctypes.POINTER(_vp)]
_lib.us_get_stats.argtypes = [_vp, ctypes.POINTER(us_stats)]
_lib.us_decode.argtypes = [_vp, _vp]
_lib.us_get_row_order.argtypes = [_vp, _vp]
_lib.us_spmm.argtypes = [_vp, _vp, ctypes.c_int32, _vp, _vp, _vp]
_lib.us_last_error.argtypes = [_vp]
_lib.us_spmm_static_scratch.argtypes = [_vp, _vp, ctypes.c_int32, _vp, _vp, _vp]
_lib.us_spmm_requant.argtypes = [_vp, _vp, ctypes.c_int64, _vp, ctypes.c_int32, _vp, _vp, ctypes.c_int64,
                                 ctypes.c_int64, _vp]
_lib.us_absmax_f16.argtypes = [_vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, _vp, _vp]
_lib.us_quantize_f16.argtypes = [_vp, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, _vp, _vp, _vp, _vp]
_lib.us_destroy.argtypes = [_vp]
_lib.us_stage_timers.argtypes = [_vp, ctypes.c_int32, _vp, ctypes.c_int32]
_lib.us_debug_withhold_copy.argtypes = [_vp, ctypes.c_int64, ctypes.c_int64]
_lib.us_spmm_bytes.argtypes = [_vp, ctypes.c_int32, ctypes.c_int32]
_lib.us_spmm_bytes.restype = ctypes.c_int64
_lib.us_launch_info.argtypes = [_vp, ctypes.c_int32] + [ctypes.POINTER(ctypes.c_int32)] * 3
_lib.us_status_string.argtypes = [ctypes.c_int]
_lib.us_status_string.restype = ctypes.c_char_p


class UsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_lib.us_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != US_OK:
        raise UsError(status, where)


def us_status_string(status: int) -> str:
    return _lib.us_status_string(int(status)).decode()


def us_encode(W: np.ndarray, w_scale: np.ndarray | None = None, fmt: tuple | None = None,
              max_N: int = 64, flags: int = 0) -> int:
    """W: host int8 (M, K); w_scale: host float16 (M,) or None. Returns the handle."""
    W = np.ascontiguousarray(W, dtype=np.int8)
    M, K = W.shape
    ws = None
    if w_scale is not None:
        ws = np.ascontiguousarray(w_scale, dtype=np.float16)
        assert ws.shape == (M,)
    f = us_format(*fmt) if fmt is not None else None
    h = _vp()
    st = _lib.us_encode(W.ctypes.data, M, K, ws.ctypes.data if ws is not None else None,
                        ctypes.byref(f) if f is not None else None, int(max_N), int(flags),
                        ctypes.byref(h))
    _check(st, "us_encode")
    return h.value


def us_get_stats(h: int) -> dict:
    st = us_stats()
    _check(_lib.us_get_stats(h, ctypes.byref(st)), "us_get_stats")
    d = {n: getattr(st, n) for n, _ in us_stats._fields_ if n != "fmt"}
    d["fmt"] = (st.fmt.H_L, st.fmt.K_L, st.fmt.R_A, st.fmt.C_A)
    return d


def us_decode(h: int) -> np.ndarray:
    st = us_get_stats(h)
    out = np.zeros((st["M"], st["K"]), dtype=np.int8)
    _check(_lib.us_decode(h, out.ctypes.data), "us_decode")
    return out


def us_get_row_order(h: int) -> np.ndarray:
    st = us_get_stats(h)
    out = np.zeros(st["Mp"], dtype=np.int32)
    _check(_lib.us_get_row_order(h, out.ctypes.data), "us_get_row_order")
    return out


def us_spmm(h: int, X_ptr: int, N: int, x_scale_ptr: int | None, Y_ptr: int, stream: int | None = None):
    """Raw call: device pointers as integers, stream as a cudaStream_t integer (None = default)."""
    _check(_lib.us_spmm(h, X_ptr, int(N), x_scale_ptr, Y_ptr, stream), "us_spmm")


US_STATIC_SCRATCH_BYTES = 4 << 20
US_ERR_SCRATCH_TOO_SMALL = 8


def us_spmm_static_scratch(h: int, X_ptr: int, N: int, x_scale_ptr: int | None, Y_ptr: int,
                           stream: int | None = None):
    """us_spmm for callers that may not allocate device memory around the call: the kernel's
    scratch (strip sums and arrival counters) is a fixed 4 MiB array inside the library image,
    shared by all calls on the GPU -- overlapping calls race, and a problem that does not fit
    is refused with status US_ERR_SCRATCH_TOO_SMALL. Same arguments as us_spmm."""
    _check(_lib.us_spmm_static_scratch(h, X_ptr, int(N), x_scale_ptr, Y_ptr, stream),
           "us_spmm_static_scratch")


def us_spmm_requant(h: int, X16_ptr: int, ldx: int, x_amax_ptr: int, N: int, Y16_ptr: int,
                    y_amax_ptr: int | None = None, amax_m0: int = 0, amax_m1: int = 0,
                    stream: int | None = None):
    """Chained call: fp16 activations (row stride ldx elements) quantised per token to INT4 with
    the step max|x| / 7 while they are staged, fp16 output, and optionally the per-token absmax
    of output columns [amax_m0, amax_m1) for the next call. Device pointers as integers."""
    _check(_lib.us_spmm_requant(h, X16_ptr, int(ldx), x_amax_ptr, int(N), Y16_ptr, y_amax_ptr,
                                int(amax_m0), int(amax_m1), stream), "us_spmm_requant")


def us_absmax_f16(X16_ptr: int, ldx: int, N: int, K: int, amax_ptr: int, stream: int | None = None):
    """Fills the absmax buffer at amax_ptr with max_k |X16[n][k]| per token."""
    _check(_lib.us_absmax_f16(X16_ptr, int(ldx), int(N), int(K), amax_ptr, stream), "us_absmax_f16")


def us_quantize_f16(X16_ptr: int, ldx: int, N: int, K: int, amax_ptr: int, Xq_ptr: int,
                    x_scale_ptr: int | None = None, stream: int | None = None):
    """The INT4 codes of the chained call's quantiser, packed as us_spmm expects X, and the steps."""
    _check(_lib.us_quantize_f16(X16_ptr, int(ldx), int(N), int(K), amax_ptr, Xq_ptr, x_scale_ptr, stream),
           "us_quantize_f16")


def us_last_error(h: int) -> int:
    return int(_lib.us_last_error(h))


def us_debug_withhold_copy(h: int, position: int, wait_us: int = 1000):
    """Test hook: later us_spmm calls on the handle never copy the tile at `position` and bound
    their waits to wait_us microseconds (position < 0: back to normal)."""
    _check(_lib.us_debug_withhold_copy(h, int(position), int(wait_us)), "us_debug_withhold_copy")


def us_stage_timers(h: int, enable: int = -1, read: bool = False, per_cta: int = 0):
    """Switch the kernel's stage timers on/off; with read=True return (and clear) the sums
    {wait, decode, epilogue, lifetime, prologue} in SM cycles, the number of warps, the
    longest warp lifetime and the first-start-to-last-end span in ns; with per_cta = n also the
    prologue checkpoints and, for the first n CTAs, the time stamps (start, first warp end,
    activations staged, end, past the dependency wait) in ns."""
    n = 8 + (4 + 5 * per_cta if per_cta else 0)
    out = (ctypes.c_uint64 * n)() if read else None
    _check(_lib.us_stage_timers(h, int(enable), out, n if read else 0), "us_stage_timers")
    if read:
        d = dict(zip(("wait", "decode", "epilogue", "lifetime", "warps", "prologue", "max_lifetime", "span_ns"),
                     [int(v) for v in out[:8]]))
        if per_cta:
            d["checkpoints"] = [int(v) for v in out[8:12]]
            d["ctas"] = [tuple(int(v) for v in out[12 + 5 * c: 17 + 5 * c]) for c in range(per_cta)]
        return d
    return None


def us_destroy(h: int):
    _check(_lib.us_destroy(h), "us_destroy")


def us_spmm_bytes(h: int, N: int, fp16_out: bool) -> int:
    return int(_lib.us_spmm_bytes(h, int(N), int(bool(fp16_out))))


def us_launch_info(h: int, N: int) -> dict:
    g, b, s = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(_lib.us_launch_info(h, int(N), ctypes.byref(g), ctypes.byref(b), ctypes.byref(s)),
           "us_launch_info")
    return {"grid": g.value, "block": b.value, "smem_bytes": s.value}


def pack_int4(X: np.ndarray) -> np.ndarray:
    """(N, K) int8 values in [-8, 7] -> (N, ceil(K/2)) bytes, k even in the low nibble."""
    X = np.ascontiguousarray(X, dtype=np.int8)
    N, K = X.shape
    if K % 2:
        X = np.concatenate([X, np.zeros((N, 1), np.int8)], axis=1)
    u = X.view(np.uint8) & 0xF
    return np.ascontiguousarray(u[:, 0::2] | (u[:, 1::2] << 4))


US_AMAX_BYTES = 4 * 64 * (1 + 192)


def new_amax(device="cuda"):
    """An absmax buffer (device int32 tensor) for the chained calls."""
    import torch
    return torch.zeros(US_AMAX_BYTES // 4, device=device, dtype=torch.int32)


def amax_values(buf, N: int):
    """The per-token absmax an absmax buffer holds, as a host uint16 array of fp16 bit patterns."""
    w = buf.cpu().numpy()
    parts = int(w[0])
    return w[64:64 + 64 * parts].reshape(parts, 64)[:, :N].max(axis=0).astype(np.uint16)


def absmax_f16(X16, out=None, stream=None):
    """Per-token absmax of a device float16 (N, K) tensor or view (unit column stride), as the
    absmax buffer the chained call takes."""
    import torch
    assert X16.dtype == torch.float16 and X16.stride(1) == 1
    N, K = X16.shape
    if out is None:
        out = new_amax(X16.device)
    if stream is None:
        stream = torch.cuda.current_stream(X16.device).cuda_stream
    us_absmax_f16(X16.data_ptr(), X16.stride(0), N, K, out.data_ptr(), stream)
    return out


def quantize_f16(X16, amax, stream=None):
    """(packed INT4 codes uint8 (N, ceil(K/2)), steps float16 (N,)) of a device float16 (N, K)."""
    import torch
    assert X16.dtype == torch.float16 and X16.stride(1) == 1
    N, K = X16.shape
    Xq = torch.empty((N, (K + 1) // 2), device=X16.device, dtype=torch.uint8)
    sc = torch.empty(N, device=X16.device, dtype=torch.float16)
    if stream is None:
        stream = torch.cuda.current_stream(X16.device).cuda_stream
    us_quantize_f16(X16.data_ptr(), X16.stride(0), N, K, amax.data_ptr(), Xq.data_ptr(), sc.data_ptr(), stream)
    return Xq, sc


class SparseWeight:
    """An encoded weight on the current CUDA device. Torch tensors are used only as device memory."""

    def __init__(self, W: np.ndarray, w_scale: np.ndarray | None = None, fmt: tuple | None = None,
                 max_N: int = 64, flags: int = 0):
        self.handle = us_encode(W, w_scale, fmt, max_N, flags)
        self.stats = us_get_stats(self.handle)
        self.M, self.K = self.stats["M"], self.stats["K"]
        self.has_scale = w_scale is not None

    def spmm(self, X, N: int, x_scale=None, out=None, stream=None):
        """X: device uint8 tensor (N, ceil(K/2)); x_scale: device float16 (N,) or None.
        Returns a device tensor (N, M): int32, or float16 when x_scale is given."""
        import torch
        if out is None:
            out = torch.empty((N, self.M), device=X.device,
                              dtype=torch.float16 if x_scale is not None else torch.int32)
        if stream is None:
            stream = torch.cuda.current_stream(X.device).cuda_stream
        us_spmm(self.handle, X.data_ptr(), N, x_scale.data_ptr() if x_scale is not None else None,
                out.data_ptr(), stream)
        return out

    def spmm_requant(self, X16, N: int, x_amax, out=None, y_amax=None, amax_range=None, stream=None):
        """X16: device float16 tensor or view, (N, K) with unit column stride; x_amax: absmax buffer
        from absmax_f16 or an earlier call's y_amax. Returns the (N, M) float16 output; if y_amax
        (an absmax buffer) is given it receives the absmax of columns amax_range of the output."""
        import torch
        assert X16.dtype == torch.float16 and X16.stride(1) == 1 and X16.shape[1] == self.K
        if out is None:
            out = torch.empty((N, self.M), device=X16.device, dtype=torch.float16)
        if stream is None:
            stream = torch.cuda.current_stream(X16.device).cuda_stream
        m0, m1 = amax_range if amax_range is not None else (0, self.M)
        us_spmm_requant(self.handle, X16.data_ptr(), X16.stride(0), x_amax.data_ptr(), N, out.data_ptr(),
                        y_amax.data_ptr() if y_amax is not None else None, m0, m1, stream)
        return out

    def check(self):
        st = us_last_error(self.handle)
        _check(st, "us_last_error")

    def close(self):
        if self.handle:
            us_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
