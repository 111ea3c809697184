"""Parity of the binary64 entry points (zccl_compress_f64 / zccl_decompress_f64) with the CPU oracle, through the
C-ABI: streams byte for byte, values bit for bit, at the sizes of the small and the 64 MiB-class configurations,
ragged lengths, both bound modes, and the errors."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_18554_b200 import fields

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def z():
    from paper_2502_18554_b200 import build, zccl
    build.build()
    return zccl


@pytest.fixture(scope="module")
def ctx(z):
    c = z.Context(1 << 24, 0)
    yield c
    c.close()


def gpu_round_trip(z, ctx, x, mode, eb):
    dx = torch.from_numpy(x).cuda()
    out = torch.empty(z.compress_bound(x.size), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress_f64(dx, mode, eb, out, nb)
    rc = ctx.status()
    stream = out[: int(nb.item())]
    y = torch.empty(x.size, dtype=torch.float64, device="cuda")
    if rc >= 0 and stream.numel():
        ctx.decompress_f64(stream, y)
        assert ctx.status() == z.OK
    return stream.cpu().numpy(), y.cpu().numpy(), rc


def as_f64(a, seed):
    """A binary64 array with the shape of a binary32 field and low-order bits of its own."""
    rng = np.random.default_rng(seed)
    return a.astype(np.float64) * (1.0 + 1e-9 * rng.standard_normal(a.size))


@pytest.mark.parametrize("n", [1, 31, 32, 33, 4095, 4096, 4097, 70_001, 1 << 20])
@pytest.mark.parametrize("mode,eb", [(0, 1e-6), (1, 1e-3)])
def test_streams_and_values_match_the_oracle(z, ctx, n, mode, eb):
    x = as_f64(fields.smooth_1d(n, seed=n % 89), n)
    if mode == 1 and n == 1:
        pytest.skip("a single value has no range")
    got, y, rc = gpu_round_trip(z, ctx, x, mode, eb)
    want = oracle.compress_f64(x, mode, eb)
    assert rc == z.OK
    assert np.array_equal(got, want)
    assert np.array_equal(y.view(np.uint64), oracle.decompress_f64(want).view(np.uint64))
    bound = eb if mode == 0 else eb * (x.max() - x.min())
    assert float(np.abs(x - y).max()) <= bound


def test_fourier_field_at_full_size(z, ctx):
    x = as_f64(fields.fourier_field_3d(256, seed=1), 5)
    got, y, rc = gpu_round_trip(z, ctx, x, z.EB_REL, 1e-3)
    want = oracle.compress_f64(x, oracle.EB_REL, 1e-3)
    assert rc == z.OK and np.array_equal(got, want)
    assert np.array_equal(y.view(np.uint64), oracle.decompress_f64(want).view(np.uint64))


def test_codes_beyond_binary32_precision(z, ctx):
    """Values whose codes need more than 24 bits: the binary64 route keeps them exact (the bound holds with no warning)."""
    rng = np.random.default_rng(2)
    x = rng.standard_normal(50_000) * 3e3 + 1e4
    got, y, rc = gpu_round_trip(z, ctx, x, z.EB_ABS, 1e-4)      # codes up to about 1e8
    assert rc == z.OK
    assert np.array_equal(got, oracle.compress_f64(x, oracle.EB_ABS, 1e-4))
    assert float(np.abs(x - y).max()) <= 1e-4


def test_errors(z, ctx):
    x = np.array([0.0, 1e9], dtype=np.float64)
    _, _, rc = gpu_round_trip(z, ctx, x, z.EB_ABS, 1e-3)         # |x r| >= 2^30
    assert rc == z.E_RANGE
    c = np.full(1000, 2.5, dtype=np.float64)
    _, _, rc = gpu_round_trip(z, ctx, c, z.EB_REL, 1e-3)
    assert rc == z.E_DEGENERATE
    # a binary32 stream is refused by the binary64 decoder and the other way round
    x32 = fields.smooth_1d(5000, seed=1)
    st32, _ = oracle.compress(x32, oracle.EB_ABS, 1e-3)
    y = torch.empty(5000, dtype=torch.float64, device="cuda")
    ctx.decompress_f64(torch.from_numpy(st32.copy()).cuda(), y)
    assert ctx.status() == z.E_BAD_STREAM
    st64 = oracle.compress_f64(x32.astype(np.float64), oracle.EB_ABS, 1e-3)
    y32 = torch.empty(5000, dtype=torch.float32, device="cuda")
    ctx.decompress(torch.from_numpy(st64.copy()).cuda(), y32)
    assert ctx.status() == z.E_BAD_STREAM
    with pytest.raises(z.ZcclError):
        ctx.compress_f64(torch.zeros(8, dtype=torch.float64, device="cuda"), z.EB_ABS, 0.0,
                         torch.empty(1024, dtype=torch.uint8, device="cuda"), torch.zeros(1, dtype=torch.int64, device="cuda"))
