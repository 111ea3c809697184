"""CPU oracle for the ZCCL hot path -- TEST INFRASTRUCTURE, not the product.

Thin ctypes access to ``zccl_oracle.c`` and ``zccl_oracle_f64.c`` (plain C, single thread).  Only tests, the smoke check and the
benchmark's CPU-baseline legs may import this package; the CUDA path never does and shares no code with it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "zccl_oracle.c"
_SRC_F64 = _HERE / "zccl_oracle_f64.c"
_LIB = _HERE / "libzccl_oracle.so"

OK, E_ARG, E_CAPACITY, E_RANGE, E_BAD_STREAM, E_DEGENERATE, W_PRECISION = 0, -1, -3, -4, -5, -7, 1
EB_ABS, EB_REL = 0, 1
FLAG_CONSISTENT_OWNER = 1
OP_SUM, OP_MAX, OP_MIN, OP_AVG = 0, 2, 4, 6   # reduce operation, or-ed into flags
DEFAULT_TILE = 4096
HEADER_BYTES = 32


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (IEEE arithmetic, no contraction)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < max(_SRC.stat().st_mtime, _SRC_F64.stat().st_mtime):
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c99", "-fPIC", "-shared",
                               "-o", str(tmp), str(_SRC), str(_SRC_F64), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(str(_LIB))
        fp, u8p, i32p, szp = C.POINTER(C.c_float), C.POINTER(C.c_uint8), C.POINTER(C.c_int32), C.POINTER(C.c_size_t)
        L.zo_compress_bound.restype = C.c_size_t
        L.zo_compress_bound.argtypes = [C.c_size_t, C.c_uint32]
        L.zo_resolve_range.argtypes = [C.c_int, C.c_float, C.c_float, C.c_float, fp, fp, fp]
        L.zo_resolve.argtypes = [C.c_int, C.c_float, C.c_void_p, C.c_size_t, fp, fp, fp]
        L.zo_quantise.argtypes = [C.c_void_p, C.c_size_t, C.c_float, C.c_void_p]
        L.zo_compress_core.argtypes = [C.c_void_p, C.c_size_t, C.c_float, C.c_float, C.c_float, C.c_uint32,
                                       C.c_void_p, C.c_size_t, szp]
        L.zo_compress.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_float, C.c_uint32, C.c_void_p, C.c_size_t, szp]
        L.zo_decompress_codes.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_size_t, szp]
        L.zo_drc.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_size_t, C.c_size_t,
                             C.c_void_p, C.c_size_t, szp, C.c_void_p, C.c_uint]
        L.zo_sim_allreduce.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_int, C.c_float, C.c_uint,
                                       C.c_uint32, C.c_void_p]
        L.zo_sim_allgather.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_int, C.c_float, C.c_uint32,
                                       C.c_void_p]
        L.zo_sim_bcast.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_int, C.c_float, C.c_uint32, szp]
        L.zo_sim_reduce_scatter.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_int, C.c_float, C.c_uint32,
                                            C.c_void_p]
        L.zo_quality.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.zo_stream_stats.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
        L.zo_sim_scatter.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_size_t, C.c_int, C.c_float, C.c_uint32,
                                     C.c_void_p, C.c_void_p]
        dp = C.POINTER(C.c_double)
        L.zo_resolve_f64.argtypes = [C.c_int, C.c_double, C.c_double, C.c_double, dp, dp, dp]
        L.zo_quantise_f64.argtypes = [C.c_void_p, C.c_size_t, C.c_double, C.c_void_p]
        L.zo_compress_f64.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_double, C.c_uint32, C.c_void_p, C.c_size_t, szp]
        L.zo_decompress_f64.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_size_t, szp]
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: oracle status {code}")
        self.code = code


def _f32(x) -> np.ndarray:
    a = np.ascontiguousarray(x, dtype=np.float32)
    return a


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def compress_bound(n: int, T: int = DEFAULT_TILE) -> int:
    return int(lib().zo_compress_bound(n, T))


def resolve(eb_mode: int, eb: float, x=None, *, mn: float | None = None, mx: float | None = None):
    """(eb_abs, s, r) as float32 scalars."""
    ea, s, r = C.c_float(), C.c_float(), C.c_float()
    if mn is not None:
        rc = lib().zo_resolve_range(eb_mode, eb, mn, mx, C.byref(ea), C.byref(s), C.byref(r))
    else:
        x = _f32(x if x is not None else np.zeros(0, np.float32))
        rc = lib().zo_resolve(eb_mode, eb, _ptr(x), x.size, C.byref(ea), C.byref(s), C.byref(r))
    if rc != OK:
        raise OracleError(rc, "resolve")
    return np.float32(ea.value), np.float32(s.value), np.float32(r.value)


def quantise(x, r) -> tuple[np.ndarray, int]:
    x = _f32(x)
    q = np.empty(x.size, np.int32)
    rc = lib().zo_quantise(_ptr(x), x.size, float(r), _ptr(q))
    if rc < 0:
        raise OracleError(rc, "quantise")
    return q, rc


def compress_core(x, eb_abs, s, r, T: int = DEFAULT_TILE, cap: int | None = None) -> tuple[np.ndarray, int]:
    """Stream bytes (uint8 array) and status (OK or W_PRECISION) for a pre-resolved bound."""
    x = _f32(x)
    cap = compress_bound(x.size, T) if cap is None else cap
    out = np.zeros(max(cap, 1), np.uint8)
    nb = C.c_size_t(0)
    rc = lib().zo_compress_core(_ptr(x), x.size, float(eb_abs), float(s), float(r), T, _ptr(out), cap, C.byref(nb))
    if rc < 0:
        raise OracleError(rc, "compress_core")
    return out[: nb.value].copy(), rc


def compress(x, eb_mode: int, eb: float, T: int = DEFAULT_TILE) -> tuple[np.ndarray, int]:
    x = _f32(x)
    cap = compress_bound(x.size, T)
    out = np.zeros(max(cap, 1), np.uint8)
    nb = C.c_size_t(0)
    rc = lib().zo_compress(_ptr(x), x.size, eb_mode, eb, T, _ptr(out), cap, C.byref(nb))
    if rc < 0:
        raise OracleError(rc, "compress")
    return out[: nb.value].copy(), rc


def stream_n(stream: np.ndarray) -> int:
    return int(np.frombuffer(stream[8:16].tobytes(), np.uint64)[0])


def decompress(stream, want_codes: bool = False):
    st = np.ascontiguousarray(stream, dtype=np.uint8)
    if st.size < HEADER_BYTES:
        raise OracleError(E_BAD_STREAM, "decompress")
    n = stream_n(st)
    if n > (1 << 40):
        raise OracleError(E_BAD_STREAM, "decompress")
    y = np.empty(n, np.float32)
    q = np.empty(n, np.int32) if want_codes else None
    no = C.c_size_t(0)
    rc = lib().zo_decompress_codes(_ptr(st), st.size, _ptr(y), _ptr(q) if want_codes else None, n, C.byref(no))
    if rc != OK:
        raise OracleError(rc, "decompress")
    return (y, q) if want_codes else y


def drc(in_c, local=None, local_c=None, flags: int = 0, want_raw: bool = False, cap: int | None = None):
    """Reduce-scatter hop: compress(decompress(in_c) + local).  Returns (stream, status[, raw])."""
    in_c = np.ascontiguousarray(in_c, dtype=np.uint8)
    n = stream_n(in_c)
    T = int(np.frombuffer(in_c[24:28].tobytes(), np.uint32)[0])
    cap = compress_bound(n, T) if cap is None else cap
    out = np.zeros(max(cap, 1), np.uint8)
    nb = C.c_size_t(0)
    raw = np.empty(n, np.float32) if want_raw else None
    loc = _f32(local) if local is not None else None
    lc = np.ascontiguousarray(local_c, dtype=np.uint8) if local_c is not None else None
    rc = lib().zo_drc(_ptr(in_c), in_c.size, _ptr(loc) if loc is not None else None,
                      _ptr(lc) if lc is not None else None, lc.size if lc is not None else 0, n,
                      _ptr(out), cap, C.byref(nb), _ptr(raw) if want_raw else None, flags)
    if rc < 0:
        raise OracleError(rc, "drc")
    res = (out[: nb.value].copy(), rc)
    return res + (raw,) if want_raw else res


def _ptr_array(arrs):
    return (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])


def sim_allreduce(send, eb_mode: int, eb: float, flags: int = 0, T: int = DEFAULT_TILE, want_hop_bytes: bool = False):
    send = [_f32(a) for a in send]
    N, n = len(send), send[0].size
    recv = [np.zeros(n, np.float32) for _ in range(N)]
    hop = np.zeros(N * N, dtype=np.uintp)
    rc = lib().zo_sim_allreduce(_ptr_array(send), _ptr_array(recv), N, n, eb_mode, eb, flags, T, _ptr(hop))
    if rc < 0:
        raise OracleError(rc, "sim_allreduce")
    return (recv, rc, hop.reshape(N, N)) if want_hop_bytes else (recv, rc)


def sim_allgather(send, eb_mode: int, eb: float, T: int = DEFAULT_TILE):
    send = [_f32(a) for a in send]
    N, n = len(send), send[0].size
    recv = [np.zeros(N * n, np.float32) for _ in range(N)]
    sizes = np.zeros(N, dtype=np.uintp)
    rc = lib().zo_sim_allgather(_ptr_array(send), _ptr_array(recv), N, n, eb_mode, eb, T, _ptr(sizes))
    if rc < 0:
        raise OracleError(rc, "sim_allgather")
    return recv, rc, sizes


def sim_bcast(root, nsinks: int, eb_mode: int, eb: float, T: int = DEFAULT_TILE):
    root = _f32(root)
    recv = [np.zeros(root.size, np.float32) for _ in range(nsinks)]
    sb = C.c_size_t(0)
    rc = lib().zo_sim_bcast(_ptr(root), _ptr_array(recv), nsinks, root.size, eb_mode, eb, T, C.byref(sb))
    if rc < 0:
        raise OracleError(rc, "sim_bcast")
    return recv, rc, sb.value


def chunk_span(n: int, N: int, c: int):
    """Offset and length of chunk c when n elements are split into N chunks of ceil(n / N) (the last ones shorter)."""
    m = (n + N - 1) // N
    off = min(c * m, n)
    return off, min(m, n - off)


def sim_reduce_scatter(send, eb_mode: int, eb: float, T: int = DEFAULT_TILE):
    """Ring Reduce-scatter: recv[r] = chunk r of the sum.  Returns (recv, rc, hop_bytes[(N-1) x N])."""
    send = [_f32(a) for a in send]
    N, n = len(send), send[0].size
    recv = [np.zeros(chunk_span(n, N, r)[1], np.float32) for r in range(N)]
    hop = np.zeros(max(N - 1, 1) * N, dtype=np.uintp)
    rc = lib().zo_sim_reduce_scatter(_ptr_array(send), _ptr_array(recv), N, n, eb_mode, eb, T, _ptr(hop))
    if rc < 0:
        raise OracleError(rc, "sim_reduce_scatter")
    return recv, rc, hop.reshape(max(N - 1, 1), N)


def sim_scatter(root, N: int, eb_mode: int, eb: float, T: int = DEFAULT_TILE):
    """Binomial-tree Scatter of N chunks held by rank 0.  Returns (recv, rc, sizes[N], round_bytes)."""
    root = _f32(root)
    assert root.size % N == 0
    n = root.size // N
    recv = [np.zeros(n, np.float32) for _ in range(N)]
    sizes = np.zeros(N, dtype=np.uintp)
    rounds = np.zeros(32, dtype=np.uintp)
    rc = lib().zo_sim_scatter(_ptr(root), _ptr_array(recv), N, n, eb_mode, eb, T, _ptr(sizes), _ptr(rounds))
    if rc < 0:
        raise OracleError(rc, "sim_scatter")
    nrounds = max(N - 1, 0).bit_length()
    return recv, rc, sizes, rounds[:nrounds]


def quality(x, y):
    """Quality of the reconstruction y of x: dict with max_abs_err, mse, nrmse, psnr, min, max (fp64)."""
    x, y = _f32(x), _f32(y)
    assert x.size == y.size
    out = np.zeros(6, dtype=np.float64)
    rc = lib().zo_quality(_ptr(x), _ptr(y), x.size, _ptr(out))
    if rc < 0:
        raise OracleError(rc, "quality")
    return dict(max_abs_err=out[0], mse=out[1], nrmse=out[2], psnr=out[3], min=out[4], max=out[5])


def stream_stats(stream):
    """Code-length histogram of a stream: uint64[33], entry L = blocks stored with code length L, entry 32 = blocks."""
    st = np.ascontiguousarray(stream, dtype=np.uint8)
    hist = np.zeros(33, dtype=np.uint64)
    rc = lib().zo_stream_stats(_ptr(st), st.size, _ptr(hist))
    if rc != OK:
        raise OracleError(rc, "stream_stats")
    return hist


# ------------------------------------------------------------------------------------------------ binary64 input

def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(x, dtype=np.float64)


def resolve_f64(eb_mode: int, eb: float, mn: float = 0.0, mx: float = 0.0):
    ea, s, r = C.c_double(0.0), C.c_double(0.0), C.c_double(0.0)
    rc = lib().zo_resolve_f64(eb_mode, eb, mn, mx, C.byref(ea), C.byref(s), C.byref(r))
    if rc != OK:
        raise OracleError(rc, "resolve_f64")
    return ea.value, s.value, r.value


def quantise_f64(x, r: float) -> np.ndarray:
    x = _f64(x)
    q = np.empty(x.size, np.int32)
    rc = lib().zo_quantise_f64(_ptr(x), x.size, r, _ptr(q))
    if rc < 0:
        raise OracleError(rc, "quantise_f64")
    return q


def compress_f64(x, eb_mode: int, eb: float, T: int = DEFAULT_TILE, cap: int | None = None) -> np.ndarray:
    """Stream bytes (uint8 array) of a binary64 array."""
    x = _f64(x)
    cap = compress_bound(x.size, T) if cap is None else cap
    out = np.zeros(max(cap, 1), np.uint8)
    nb = C.c_size_t(0)
    rc = lib().zo_compress_f64(_ptr(x), x.size, eb_mode, eb, T, _ptr(out), cap, C.byref(nb))
    if rc < 0:
        raise OracleError(rc, "compress_f64")
    return out[: nb.value].copy()


def decompress_f64(stream, want_codes: bool = False):
    st = np.ascontiguousarray(stream, dtype=np.uint8)
    if st.size < HEADER_BYTES:
        raise OracleError(E_BAD_STREAM, "decompress_f64")
    n = stream_n(st)
    if n > (1 << 40):
        raise OracleError(E_BAD_STREAM, "decompress_f64")
    y = np.empty(n, np.float64)
    q = np.empty(n, np.int32) if want_codes else None
    no = C.c_size_t(0)
    rc = lib().zo_decompress_f64(_ptr(st), st.size, _ptr(y), _ptr(q) if want_codes else None, n, C.byref(no))
    if rc != OK:
        raise OracleError(rc, "decompress_f64")
    return (y, q) if want_codes else y
