"""Host-side checks that need no GPU: the C-ABI library loads and exports every symbol the header declares, its
pure host functions agree with the oracle, and argument errors the host can see are reported without CUDA."""
import ctypes as C
import re
from pathlib import Path

import pytest

import oracle

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2502_18554_b200 import build, zccl
    build.build()
    return zccl.lib()


def declared_symbols():
    text = (ROOT / "include" / "zccl.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zccl_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2502_18554_b200 import zccl
    names = declared_symbols()
    assert "zccl_compress" in names and "zccl_decompress_reduce_compress" in names and "zccl_sim_allreduce" in names
    for name in names:
        assert hasattr(lib, name), f"{name} is declared in zccl.h but not exported"
    assert sorted(zccl.EXPORTS) == [n for n in names]


def test_compress_bound_matches_oracle(lib):
    for n in [0, 1, 31, 32, 33, 4095, 4096, 4097, 8192, 10 ** 6 + 7, 2 ** 24, 2 ** 28 + 5]:
        assert lib.zccl_compress_bound(n) == oracle.compress_bound(n)


def test_strerror(lib):
    from paper_2502_18554_b200 import zccl
    assert lib.zccl_strerror(0) == b"ok"
    for code in (zccl.E_ARG, zccl.E_CUDA, zccl.E_CAPACITY, zccl.E_RANGE, zccl.E_BAD_STREAM, zccl.E_TIMEOUT,
                 zccl.E_DEGENERATE, zccl.W_PRECISION):
        assert lib.zccl_strerror(code) not in (b"ok", b"unknown status")


def test_null_context_is_rejected_without_cuda(lib):
    from paper_2502_18554_b200 import zccl
    assert lib.zccl_status(None, None) == zccl.E_ARG
    assert lib.zccl_compress(None, None, 0, 0, 1.0, None, 0, None, None) == zccl.E_ARG
    assert lib.zccl_decompress(None, None, 0, None, 0, None) == zccl.E_ARG
    assert lib.zccl_ctx_create(None, 1, 0) == zccl.E_ARG
    h = C.c_void_p()
    assert lib.zccl_ctx_create(C.byref(h), 0, 0) == zccl.E_ARG
    assert lib.zccl_ctx_create(C.byref(h), 10, 1000) == zccl.E_ARG
    lib.zccl_ctx_destroy(None)


def test_binding_refuses_to_run_without_gpu():
    import torch
    from paper_2502_18554_b200 import zccl
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        zccl.Context(1 << 20)


def test_compress_bound_for_other_tile_sizes_is_the_oracles():
    """Pure host arithmetic of the library (no GPU involved) against the oracle's worst case: every block at 31 bits
    plus its sign word, per tile an outlier, the padded code-length bytes and an index entry."""
    import oracle
    from paper_2502_18554_b200 import zccl
    for T in (1024, 4096, 5120, 8192):
        for n in (0, 1, 31, 32, 33, T - 1, T, T + 1, 7 * T + 100, 1 << 24):
            assert zccl.compress_bound_tiled(n, T) == oracle.compress_bound(n, T)
    assert zccl.compress_bound_tiled(1000, 5000) == 0 and zccl.compress_bound_tiled(1000, 512) == 0
    assert zccl.compress_bound_tiled(12345, 4096) == zccl.compress_bound(12345)


def test_resolve_range_host_is_the_oracles_arithmetic(lib):
    """The host-side resolution of a relative bound (what a ring rank without a device-side resolver calls) against
    the oracle's, bit for bit, over ranges of many magnitudes, and its refusals."""
    import numpy as np
    from paper_2502_18554_b200 import zccl
    rng = np.random.default_rng(7)
    cases = [(-1.0, 1.0, 1e-3), (0.0, 3.0, 1e-2), (-7.25, -7.0, 1e-4), (1e-30, 2e-30, 1e-3), (-3e38, 3e38, 1e-3)]
    for _ in range(200):
        a, b = np.sort(rng.standard_normal(2).astype(np.float32) * np.float32(10.0 ** rng.integers(-20, 20)))
        cases.append((float(a), float(b), float(10.0 ** rng.uniform(-6, -1))))
    for mn, mx, eb in cases:
        rc, ea, s, r = zccl.resolve_range_host(mn, mx, eb)
        try:
            want = oracle.resolve(oracle.EB_REL, eb, mn=mn, mx=mx)
        except oracle.OracleError as exc:
            assert rc == exc.code, (mn, mx, eb)
            continue
        assert rc == zccl.OK, (mn, mx, eb)
        assert np.float32(ea).tobytes() + np.float32(s).tobytes() + np.float32(r).tobytes() == \
            np.float32(want[0]).tobytes() + np.float32(want[1]).tobytes() + np.float32(want[2]).tobytes(), (mn, mx, eb)
    assert zccl.resolve_range_host(2.0, 2.0, 1e-3)[0] == zccl.E_DEGENERATE
    assert zccl.resolve_range_host(3.0, 2.0, 1e-3)[0] == zccl.E_DEGENERATE
    assert zccl.resolve_range_host(0.0, float("inf"), 1e-3)[0] == zccl.E_DEGENERATE
    assert zccl.resolve_range_host(0.0, 1.0, 0.0)[0] == zccl.E_ARG
    assert zccl.resolve_range_host(0.0, 1.0, float("nan"))[0] == zccl.E_ARG
