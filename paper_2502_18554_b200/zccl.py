"""Thin binding over the C-ABI library ``libzccl.so`` (declared in ``include/zccl.h``): argument marshalling only.
PyTorch supplies device memory and streams; every step of the path runs in the library's CUDA kernels.  There is
no CPU fallback: if the library is missing or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libzccl.so"

OK, E_ARG, E_CUDA, E_CAPACITY, E_RANGE, E_BAD_STREAM, E_TIMEOUT, E_DEGENERATE, W_PRECISION = 0, -1, -2, -3, -4, -5, -6, -7, 1
E_TOO_LARGE = -8
NOALLOC_MAX_ELEMS = 1 << 26
EB_ABS, EB_REL, EB_RESOLVED = 0, 1, 2
CONSISTENT_OWNER = 1
OP_SUM, OP_MAX, OP_MIN, OP_AVG = 0, 2, 4, 6   # reduce operation, or-ed into flags
TILE, BLOCK, HEADER_BYTES = 4096, 32, 32

EXPORTS = [
    "zccl_ctx_create", "zccl_ctx_destroy", "zccl_compress_bound", "zccl_launch_count", "zccl_status", "zccl_strerror",
    "zccl_compress", "zccl_decompress", "zccl_decompress_reduce_compress",
    "zccl_sim_allreduce", "zccl_sim_allgather", "zccl_sim_bcast", "zccl_sim_reduce_scatter", "zccl_sim_scatter",
    "zccl_sim_sizes", "zccl_quality", "zccl_compress_f64", "zccl_decompress_f64", "zccl_range", "zccl_resolve_range", "zccl_resolve_range_host", "zccl_scale", "zccl_stream_stats",
    "zccl_compress_bound_tiled", "zccl_compress_tiled", "zccl_decompress_tiled",
    "zccl_compress_host", "zccl_decompress_host", "zccl_compress_noalloc", "zccl_debug_skip_publish",
    "zccl_debug_set_launch_counter",
]

_lib = None


class ZcclError(RuntimeError):
    def __init__(self, code: int, what: str):
        msg = lib().zccl_strerror(code).decode() if _lib is not None else str(code)
        super().__init__(f"{what}: {msg} ({code})")
        self.code = code


def lib():
    """Loads the shared library (no compute happens here; a GPU is not needed to load it)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2502_18554_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(str(LIB_PATH))
        vp, sz = C.c_void_p, C.c_size_t
        L.zccl_ctx_create.argtypes = [C.POINTER(vp), sz, C.c_int]
        L.zccl_ctx_destroy.argtypes = [vp]
        L.zccl_ctx_destroy.restype = None
        L.zccl_compress_bound.argtypes = [sz]
        L.zccl_compress_bound.restype = sz
        L.zccl_launch_count.argtypes = []
        L.zccl_launch_count.restype = C.c_ulonglong
        L.zccl_status.argtypes = [vp, vp]
        L.zccl_strerror.argtypes = [C.c_int]
        L.zccl_strerror.restype = C.c_char_p
        L.zccl_compress.argtypes = [vp, vp, sz, C.c_int, C.c_float, vp, sz, vp, vp]
        L.zccl_decompress.argtypes = [vp, vp, sz, vp, sz, vp]
        L.zccl_decompress_reduce_compress.argtypes = [vp, vp, sz, vp, vp, sz, sz, vp, sz, vp, vp, C.c_uint, vp]
        L.zccl_sim_allreduce.argtypes = [vp, vp, vp, C.c_int, sz, C.c_int, C.c_float, C.c_uint, vp]
        L.zccl_sim_allgather.argtypes = [vp, vp, vp, C.c_int, sz, C.c_int, C.c_float, vp]
        L.zccl_sim_reduce_scatter.argtypes = [vp, vp, vp, C.c_int, sz, C.c_int, C.c_float, vp]
        L.zccl_sim_scatter.argtypes = [vp, vp, vp, C.c_int, sz, C.c_int, C.c_float, vp]
        L.zccl_quality.argtypes = [vp, vp, vp, sz, vp, vp]
        L.zccl_range.argtypes = [vp, vp, sz, vp, vp]
        L.zccl_compress_f64.argtypes = [vp, vp, sz, C.c_int, C.c_double, vp, sz, vp, vp]
        L.zccl_decompress_f64.argtypes = [vp, vp, sz, vp, sz, vp]
        L.zccl_resolve_range.argtypes = [vp, vp, C.c_float, vp, vp]
        L.zccl_resolve_range_host.argtypes = [C.c_float, C.c_float, C.c_float, vp, vp, vp]
        L.zccl_stream_stats.argtypes = [vp, vp, sz, vp, vp]
        L.zccl_compress_bound_tiled.argtypes = [sz, C.c_uint]
        L.zccl_compress_bound_tiled.restype = sz
        L.zccl_compress_tiled.argtypes = [vp, vp, sz, C.c_int, C.c_float, C.c_uint, vp, sz, vp, vp]
        L.zccl_decompress_tiled.argtypes = [vp, vp, sz, C.c_uint, vp, sz, vp]
        L.zccl_scale.argtypes = [vp, vp, sz, C.c_float, vp]
        L.zccl_sim_bcast.argtypes = [vp, vp, vp, C.c_int, sz, C.c_int, C.c_float, vp]
        L.zccl_sim_sizes.argtypes = [vp, vp, C.c_int, vp]
        L.zccl_compress_host.argtypes = [vp, vp, sz, C.c_int, C.c_float, vp, sz, vp, vp]
        L.zccl_decompress_host.argtypes = [vp, vp, sz, vp, sz, vp]
        L.zccl_compress_noalloc.argtypes = [vp, sz, C.c_float, vp, sz, vp, vp]
        L.zccl_debug_skip_publish.argtypes = [vp, C.c_longlong]
        L.zccl_debug_set_launch_counter.argtypes = [vp, C.c_uint, vp]
        _lib = L
    return _lib


def compress_bound(n: int) -> int:
    return int(lib().zccl_compress_bound(n))


def resolve_range_host(mn: float, mx: float, eb_rel: float) -> tuple[int, float, float, float]:
    """zccl_resolve_range_host: (status, eb_abs, step, reciprocal) of a relative bound over [mn, mx]; a pure host
    function (no GPU needed)."""
    ea, s, r = C.c_float(0.0), C.c_float(0.0), C.c_float(0.0)
    rc = int(lib().zccl_resolve_range_host(mn, mx, eb_rel, C.byref(ea), C.byref(s), C.byref(r)))
    return rc, float(ea.value), float(s.value), float(r.value)


def compress_bound_tiled(n: int, tile: int) -> int:
    return int(lib().zccl_compress_bound_tiled(n, tile))


def launch_count() -> int:
    return int(lib().zccl_launch_count())


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_ptr(t: torch.Tensor | None, dtype=None) -> int | None:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _check(rc: int, what: str):
    if rc != OK:
        raise ZcclError(rc, what)


def compress_noalloc(x: torch.Tensor, eb_abs: float, out: torch.Tensor, out_bytes: torch.Tensor, stream=None,
                     n: int | None = None) -> int:
    """zccl_compress_noalloc: compression without a context, for callers that must not allocate device memory (its
    scan workspace is a fixed array inside the library).  Returns the host-side status code instead of raising,
    so that callers can tell ZCCL_E_TOO_LARGE from other errors."""
    n = x.numel() if n is None else n
    return int(lib().zccl_compress_noalloc(_dev_ptr(x, torch.float32) if x.numel() else None, n, eb_abs,
                                           _dev_ptr(out, torch.uint8), out.numel(), _dev_ptr(out_bytes, torch.int64),
                                           _stream_ptr(stream)))


class Context:
    """Owns the library context (scan workspace, status word, slots of the emulated ranks)."""

    def __init__(self, max_elems: int, max_ranks: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("zccl needs a CUDA device (sm_100a); there is no CPU fallback")
        torch.cuda.init()
        torch.cuda.current_stream()   # make sure a CUDA context exists on the current device
        h = C.c_void_p()
        _check(lib().zccl_ctx_create(C.byref(h), max_elems, max_ranks), "zccl_ctx_create")
        self._h = h
        self.max_elems, self.max_ranks = max_elems, max_ranks

    def close(self):
        if getattr(self, "_h", None):
            lib().zccl_ctx_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- status
    def status(self, stream=None) -> int:
        return int(lib().zccl_status(self._h, _stream_ptr(stream)))

    def check(self, stream=None, allow_warning: bool = True) -> int:
        rc = self.status(stream)
        if rc < 0 or (rc > 0 and not allow_warning):
            raise ZcclError(rc, "device status")
        return rc

    def debug_skip_publish(self, tile: int):
        """Test hook: tile number whose size is never published to the placement scan (negative = off)."""
        _check(lib().zccl_debug_skip_publish(self._h, tile), "zccl_debug_skip_publish")

    def debug_set_launch_counter(self, value: int, stream=None):
        """Test hook: sets the launch counter that validates the placement scan's states."""
        _check(lib().zccl_debug_set_launch_counter(self._h, value, _stream_ptr(stream)), "zccl_debug_set_launch_counter")

    # ---- codec
    def compress(self, x: torch.Tensor, eb_mode: int, eb: float, out: torch.Tensor, out_bytes: torch.Tensor,
                 stream=None, n: int | None = None):
        """zccl_compress: x float32 [n] -> stream bytes in `out` (uint8), length in `out_bytes` (int64[1], device)."""
        n = x.numel() if n is None else n
        _check(lib().zccl_compress(self._h, _dev_ptr(x, torch.float32) if n else None, n, eb_mode, eb,
                                   _dev_ptr(out, torch.uint8), out.numel(), _dev_ptr(out_bytes, torch.int64),
                                   _stream_ptr(stream)), "zccl_compress")

    def decompress(self, stream_bytes: torch.Tensor, y: torch.Tensor, in_bytes_max: int | None = None, stream=None):
        """zccl_decompress: stream bytes (uint8) -> y float32; element count comes from the stream's header."""
        cap = stream_bytes.numel() if in_bytes_max is None else in_bytes_max
        _check(lib().zccl_decompress(self._h, _dev_ptr(stream_bytes, torch.uint8), cap,
                                     _dev_ptr(y, torch.float32) if y.numel() else None, y.numel(),
                                     _stream_ptr(stream)), "zccl_decompress")

    def decompress_reduce_compress(self, in_c: torch.Tensor, n: int, out_c: torch.Tensor, out_bytes: torch.Tensor,
                                   local: torch.Tensor | None = None, local_c: torch.Tensor | None = None,
                                   raw_out: torch.Tensor | None = None, flags: int = 0, stream=None):
        """zccl_decompress_reduce_compress: out_c = compress(decompress(in_c) + local) in one kernel."""
        _check(lib().zccl_decompress_reduce_compress(
            self._h, _dev_ptr(in_c, torch.uint8), in_c.numel(),
            _dev_ptr(local, torch.float32), _dev_ptr(local_c, torch.uint8),
            local_c.numel() if local_c is not None else 0, n,
            _dev_ptr(out_c, torch.uint8), out_c.numel(), _dev_ptr(out_bytes, torch.int64),
            _dev_ptr(raw_out, torch.float32), flags, _stream_ptr(stream)), "zccl_decompress_reduce_compress")

    # ---- emulated collectives
    @staticmethod
    def _ptrs(tensors):
        return (C.c_void_p * len(tensors))(*[_dev_ptr(t, torch.float32) for t in tensors])

    def sim_allreduce(self, send, recv, eb_mode: int, eb: float, flags: int = 0, stream=None):
        n = send[0].numel()
        _check(lib().zccl_sim_allreduce(self._h, self._ptrs(send), self._ptrs(recv), len(send), n, eb_mode, eb, flags,
                                        _stream_ptr(stream)), "zccl_sim_allreduce")

    def sim_allgather(self, send, recv, eb_mode: int, eb: float, stream=None):
        n = send[0].numel()
        _check(lib().zccl_sim_allgather(self._h, self._ptrs(send), self._ptrs(recv), len(send), n, eb_mode, eb,
                                        _stream_ptr(stream)), "zccl_sim_allgather")

    def sim_bcast(self, root: torch.Tensor, recv, eb_mode: int, eb: float, stream=None):
        _check(lib().zccl_sim_bcast(self._h, _dev_ptr(root, torch.float32), self._ptrs(recv), len(recv), root.numel(),
                                    eb_mode, eb, _stream_ptr(stream)), "zccl_sim_bcast")

    def sim_reduce_scatter(self, send, recv, eb_mode: int, eb: float, stream=None):
        """zccl_sim_reduce_scatter: recv[r] receives chunk r of the sum of the send buffers."""
        n = send[0].numel()
        _check(lib().zccl_sim_reduce_scatter(self._h, self._ptrs(send), self._ptrs(recv), len(send), n, eb_mode, eb,
                                             _stream_ptr(stream)), "zccl_sim_reduce_scatter")

    def sim_scatter(self, root: torch.Tensor, recv, eb_mode: int, eb: float, stream=None):
        """zccl_sim_scatter: root holds len(recv) chunks; recv[r] receives chunk r."""
        N = len(recv)
        _check(lib().zccl_sim_scatter(self._h, _dev_ptr(root, torch.float32), self._ptrs(recv), N, root.numel() // N,
                                      eb_mode, eb, _stream_ptr(stream)), "zccl_sim_scatter")

    def quality(self, x: torch.Tensor, y: torch.Tensor, out: torch.Tensor, stream=None):
        """zccl_quality: out (float64[6], device) <- max |x - y|, MSE, NRMSE, PSNR, min x, max x."""
        _check(lib().zccl_quality(self._h, _dev_ptr(x, torch.float32), _dev_ptr(y, torch.float32), x.numel(),
                                  _dev_ptr(out, torch.float64), _stream_ptr(stream)), "zccl_quality")

    def compress_tiled(self, x: torch.Tensor, eb_mode: int, eb: float, tile: int, out: torch.Tensor, out_bytes: torch.Tensor,
                       stream=None):
        """zccl_compress_tiled: as compress, for a tile size other than 4096 (multiple of 32 in 1024..8192)."""
        n = x.numel()
        _check(lib().zccl_compress_tiled(self._h, _dev_ptr(x, torch.float32) if n else None, n, eb_mode, eb, tile,
                                         _dev_ptr(out, torch.uint8), out.numel(), _dev_ptr(out_bytes, torch.int64),
                                         _stream_ptr(stream)), "zccl_compress_tiled")

    def decompress_tiled(self, stream_bytes: torch.Tensor, tile: int, y: torch.Tensor, stream=None):
        """zccl_decompress_tiled: as decompress, for a stream of tile size `tile`."""
        _check(lib().zccl_decompress_tiled(self._h, _dev_ptr(stream_bytes, torch.uint8), stream_bytes.numel(), tile,
                                           _dev_ptr(y, torch.float32) if y.numel() else None, y.numel(),
                                           _stream_ptr(stream)), "zccl_decompress_tiled")

    def stream_stats(self, stream_bytes: torch.Tensor, hist: torch.Tensor, stream=None):
        """zccl_stream_stats: hist (int64[33], device) <- blocks per code length 0..31, then the number of blocks."""
        _check(lib().zccl_stream_stats(self._h, _dev_ptr(stream_bytes, torch.uint8), stream_bytes.numel(),
                                       _dev_ptr(hist, torch.int64), _stream_ptr(stream)), "zccl_stream_stats")

    def compress_f64(self, x: torch.Tensor, eb_mode: int, eb: float, out: torch.Tensor, out_bytes: torch.Tensor, stream=None):
        """zccl_compress_f64: x float64 [n] -> stream bytes in `out` (uint8), length in `out_bytes` (int64[1], device)."""
        _check(lib().zccl_compress_f64(self._h, _dev_ptr(x, torch.float64) if x.numel() else None, x.numel(), eb_mode, eb,
                                       _dev_ptr(out, torch.uint8), out.numel(), _dev_ptr(out_bytes, torch.int64),
                                       _stream_ptr(stream)), "zccl_compress_f64")

    def decompress_f64(self, in_c: torch.Tensor, y: torch.Tensor, stream=None):
        """zccl_decompress_f64: stream bytes -> y float64 (capacity y.numel())."""
        _check(lib().zccl_decompress_f64(self._h, _dev_ptr(in_c, torch.uint8), in_c.numel(),
                                         _dev_ptr(y, torch.float64) if y.numel() else None, y.numel(), _stream_ptr(stream)),
               "zccl_decompress_f64")

    def range(self, x: torch.Tensor, minmax: torch.Tensor, stream=None):
        """zccl_range: minmax (float32[2], device) <- (min x, max x)."""
        _check(lib().zccl_range(self._h, _dev_ptr(x, torch.float32) if x.numel() else None, x.numel(),
                                _dev_ptr(minmax, torch.float32), _stream_ptr(stream)), "zccl_range")

    def resolve_range(self, minmax: torch.Tensor, eb_rel: float, eb_abs_out: torch.Tensor | None = None, stream=None):
        """zccl_resolve_range: the bound eb_rel * (max - min) from a device (min, max) pair into the context's
        resolved-bound block, for calls with EB_RESOLVED; eb_abs_out (float32[1], device) also receives it."""
        _check(lib().zccl_resolve_range(self._h, _dev_ptr(minmax, torch.float32), eb_rel,
                                        _dev_ptr(eb_abs_out, torch.float32) if eb_abs_out is not None else None,
                                        _stream_ptr(stream)), "zccl_resolve_range")

    def scale(self, y: torch.Tensor, divisor: float, stream=None):
        """zccl_scale: y <- y / divisor in place."""
        _check(lib().zccl_scale(self._h, _dev_ptr(y, torch.float32) if y.numel() else None, y.numel(), divisor,
                                _stream_ptr(stream)), "zccl_scale")

    def sim_sizes(self, stream=None) -> list[int]:
        cap = 2 * max(self.max_ranks, 1) ** 2 + 2
        buf = (C.c_size_t * cap)()
        cnt = lib().zccl_sim_sizes(self._h, buf, cap, _stream_ptr(stream))
        if cnt < 0:
            raise ZcclError(cnt, "zccl_sim_sizes")
        return [int(buf[i]) for i in range(min(cnt, cap))]

    # ---- host-buffer forms (pinned CPU tensors)
    def compress_host(self, x_host: torch.Tensor, eb_mode: int, eb: float, out_host: torch.Tensor, stream=None) -> int:
        nb = C.c_size_t(0)
        _check(lib().zccl_compress_host(self._h, x_host.data_ptr(), x_host.numel(), eb_mode, eb, out_host.data_ptr(),
                                        out_host.numel(), C.byref(nb), _stream_ptr(stream)), "zccl_compress_host")
        return int(nb.value)

    def decompress_host(self, in_host: torch.Tensor, in_bytes: int, y_host: torch.Tensor, stream=None):
        _check(lib().zccl_decompress_host(self._h, in_host.data_ptr(), in_bytes, y_host.data_ptr(), y_host.numel(),
                                          _stream_ptr(stream)), "zccl_decompress_host")


# ---- convenience wrappers used by tests and examples (allocate with torch, call the entry points above)

def compress_to_bytes(ctx: Context, x: torch.Tensor, eb_mode: int, eb: float, capacity: int | None = None):
    """Returns (stream as a CUDA uint8 tensor trimmed to its length, device status)."""
    cap = compress_bound(x.numel()) if capacity is None else capacity
    out = torch.empty(max(cap, 1), dtype=torch.uint8, device=x.device)
    nbytes = torch.zeros(1, dtype=torch.int64, device=x.device)
    ctx.compress(x, eb_mode, eb, out[:cap] if cap else out[:0], nbytes)
    rc = ctx.status()
    return out[: int(nbytes.item())], rc


def decompress_from_bytes(ctx: Context, stream_bytes: torch.Tensor, n: int):
    y = torch.empty(n, dtype=torch.float32, device=stream_bytes.device)
    ctx.decompress(stream_bytes, y)
    rc = ctx.status()
    return y, rc
