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


@pytest.mark.parametrize("n", [5000, 3 * 4096 + 1024, 3 * 4096 + 1025, 200_001])
@pytest.mark.parametrize("shift_x,shift_y", [(1, 0), (0, 1), (1, 1)])
def test_arrays_off_the_16_byte_boundary(z, ctx, n, shift_x, shift_y):
    """Input or output that starts 8 bytes past a 16-byte boundary: plain loads and stores take the place of the
    tensor copies; streams and values stay those of the oracle."""
    x = as_f64(fields.smooth_1d(n, seed=7), n + 1)
    want = oracle.compress_f64(x, oracle.EB_ABS, 1e-5)
    buf = torch.empty(n + 2, dtype=torch.float64, device="cuda")
    dx = buf[shift_x: shift_x + n]
    dx.copy_(torch.from_numpy(x))
    assert dx.data_ptr() % 16 == 8 * shift_x
    out = torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress_f64(dx, z.EB_ABS, 1e-5, out, nb)
    assert ctx.status() == z.OK
    assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
    ybuf = torch.full((n + 2,), -7.0, dtype=torch.float64, device="cuda")
    y = ybuf[shift_y: shift_y + n]
    ctx.decompress_f64(torch.from_numpy(want.copy()).cuda(), y)
    assert ctx.status() == z.OK
    assert np.array_equal(y.cpu().numpy().view(np.uint64), oracle.decompress_f64(want).view(np.uint64))
    edge = ybuf.cpu().numpy()
    assert all(edge[k] == -7.0 for k in list(range(shift_y)) + list(range(shift_y + n, n + 2)))   # nothing written outside


@pytest.mark.parametrize("scale,eb", [(1.0, 1e-3), (1.0, 1e-6), (3e3, 1e-4), (5e4, 1e-3)])
def test_noise_of_every_width(z, ctx, scale, eb):
    """Uncorrelated values: code lengths from a few bits up to 31 (the general route), blobs larger than the decoder's
    window, mixed with smooth tiles and constant ones."""
    rng = np.random.default_rng(11)
    n = 40 * 4096 + 777
    x = rng.standard_normal(n) * scale
    x[3 * 4096: 5 * 4096] = fields.smooth_1d(2 * 4096, seed=3).astype(np.float64)
    x[9 * 4096: 10 * 4096] = 0.25
    x[20 * 4096 + 100: 20 * 4096 + 164] = 1e-9          # a constant block inside a wide tile
    got, y, rc = gpu_round_trip(z, ctx, x, z.EB_ABS, eb)
    want = oracle.compress_f64(x, oracle.EB_ABS, eb)
    assert rc == z.OK
    assert np.array_equal(got, want)
    assert np.array_equal(y.view(np.uint64), oracle.decompress_f64(want).view(np.uint64))
    assert float(np.abs(x - y).max()) <= eb


def test_range_error_inside_a_large_array(z, ctx):
    x = fields.smooth_1d(100_000, seed=5).astype(np.float64)
    x[77_777] = 1e12
    _, _, rc = gpu_round_trip(z, ctx, x, z.EB_ABS, 1e-3)
    assert rc == z.E_RANGE
    x[77_777] = np.nan
    _, _, rc = gpu_round_trip(z, ctx, x, z.EB_ABS, 1e-3)
    assert rc == z.E_RANGE


def test_damaged_streams_are_refused(z, ctx):
    x = as_f64(fields.smooth_1d(30_000, seed=9), 4)
    good = oracle.compress_f64(x, oracle.EB_ABS, 1e-5)
    y = torch.empty(x.size, dtype=torch.float64, device="cuda")

    def status_of(stream, cap=None):
        d = torch.from_numpy(stream.copy()).cuda()
        ctx.decompress_f64(d if cap is None else d[:cap], y)
        return ctx.status()

    assert status_of(good) == z.OK
    words = good.view(np.uint32).copy()
    bad = words.copy(); bad[8 + 2] = bad[8 + 1]                       # an index entry that does not grow
    assert status_of(bad.view(np.uint8)) == z.E_BAD_STREAM
    nT = int(words[7])
    bad = words.copy(); bad[8 + nT + 1] |= 0x20                       # a code length of 32 or more in tile 0
    assert status_of(bad.view(np.uint8)) == z.E_BAD_STREAM
    assert status_of(good, cap=len(good) - 64) == z.E_BAD_STREAM     # the last blob reaches past the readable bytes
    small = torch.empty(x.size - 1, dtype=torch.float64, device="cuda")
    ctx.decompress_f64(torch.from_numpy(good.copy()).cuda(), small)
    assert ctx.status() == z.E_CAPACITY


def test_output_capacity_too_small(z, ctx):
    x = np.random.default_rng(3).standard_normal(50_000)
    dx = torch.from_numpy(x).cuda()
    out = torch.empty(40_000, dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress_f64(dx, z.EB_ABS, 1e-6, out, nb)
    assert ctx.status() == z.E_CAPACITY


def _draw_f64_case(seed):
    """Length, values (several kinds, some unkind to the codec), bound and the two arrays' offsets from a 16-byte
    boundary, from one seed."""
    rng = np.random.default_rng(seed)
    pick = rng.random()
    if pick < 0.15:
        n = int(rng.integers(1, 70))
    elif pick < 0.45:
        n = int(rng.integers(1, 9)) * 4096 + int(rng.integers(-40, 41))
    else:
        n = int(rng.integers(100, 300_000))
    kind = int(rng.integers(0, 6))
    if kind == 0:
        x = fields.smooth_1d(n, seed=int(rng.integers(1 << 30))).astype(np.float64) * (1 + 1e-11 * rng.standard_normal(n))
    elif kind == 1:
        x = rng.normal(0.0, 10.0 ** rng.uniform(-3, 3), n)
    elif kind == 2:
        x = np.repeat(rng.normal(0, 1, n // 50 + 1), 50)[:n]
    elif kind == 3:
        x = fields.smooth_1d(n, seed=int(rng.integers(1 << 30))).astype(np.float64)
        for _ in range(int(rng.integers(1, 6))):
            a = int(rng.integers(0, max(n - 1, 1)))
            b = min(n, a + int(rng.integers(1, 3000)))
            x[a:b] += rng.normal(0, 10.0 ** rng.uniform(-2, 1), b - a)
    elif kind == 4:
        x = 10.0 ** rng.uniform(0, 4) + rng.normal(0, 1e-2, n)
    else:
        x = rng.normal(0, 1e-300, n)
        x[rng.random(n) < 0.2] = 0.0
        x[rng.random(n) < 0.1] = -0.0
    x = np.ascontiguousarray(x, dtype=np.float64)
    span = float(x.max() - x.min())
    if span == 0.0 or rng.random() < 0.5:
        # an absolute bound that keeps |x / (2 eb)| below 2^30, from coarse to nearly that fine
        floor = max(float(np.abs(x).max()), 1e-300) / 2.0 ** 29
        mode, eb = oracle.EB_ABS, float(floor * 10.0 ** rng.uniform(0.1, 7))
    else:
        mode, eb = oracle.EB_REL, float(10.0 ** rng.uniform(-8, -1))
    return x, mode, eb, int(rng.integers(0, 2)), int(rng.integers(0, 2))


@pytest.mark.parametrize("seed", range(60))
def test_seeded_random_cases(z, ctx, seed):
    x, mode, eb, shift_x, shift_y = _draw_f64_case(1000 + seed)
    n = x.size
    try:
        want = oracle.compress_f64(x, mode, eb)
    except oracle.OracleError as e:
        want = e
    buf = torch.empty(n + 2, dtype=torch.float64, device="cuda")
    dx = buf[shift_x: shift_x + n]
    dx.copy_(torch.from_numpy(x))
    out = torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress_f64(dx, mode, eb, out, nb)
    rc = ctx.status()
    if isinstance(want, Exception):
        assert rc == want.code          # the oracle's status codes are the library's
        return
    assert rc == z.OK
    assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
    ybuf = torch.zeros(n + 2, dtype=torch.float64, device="cuda")
    y = ybuf[shift_y: shift_y + n]
    ctx.decompress_f64(out[: int(nb.item())], y)
    assert ctx.status() == z.OK
    assert np.array_equal(y.cpu().numpy().view(np.uint64), oracle.decompress_f64(want).view(np.uint64))
