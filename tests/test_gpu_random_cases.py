"""Seeded random cases, CUDA path against the oracle through the C boundary: lengths, value distributions, bounds,
reduce operations and rank counts are drawn at random (fixed seeds), and every byte of every stream and every bit
of every reconstruction must agree.  The hand-made cases elsewhere aim at known edges; these sweep the space in
between them (Section 3.3 for the codec, Eq. 2 for the fused hop, Sections 3.1.1 and 3.1.2 for the collectives)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2502_18554_b200 import fields

pytestmark = pytest.mark.gpu
f32 = np.float32


@pytest.fixture(scope="module")
def z():
    from paper_2502_18554_b200 import build, zccl
    build.build()
    return zccl


@pytest.fixture(scope="module")
def ctx(z):
    c = z.Context(1 << 20, 9)
    yield c
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def same_bits(a, b):
    return a.shape == b.shape and np.array_equal(a.view(np.uint32), b.view(np.uint32))


def draw_field(rng, n):
    """One of several kinds of input, some of them unkind to the codec."""
    kind = int(rng.integers(0, 8))
    if kind == 0:
        x = fields.smooth_1d(n, seed=int(rng.integers(1 << 30)))
    elif kind == 1:
        x = rng.normal(0.0, 10.0 ** rng.uniform(-3, 3), n)
    elif kind == 2:                                     # steps: long constant runs with jumps
        x = np.repeat(rng.normal(0, 1, n // 50 + 1), 50)[:n]
    elif kind == 3:                                     # smooth with bursts of noise
        x = fields.smooth_1d(n, seed=int(rng.integers(1 << 30))).astype(np.float64)
        for _ in range(int(rng.integers(1, 6))):
            a = int(rng.integers(0, max(n - 1, 1)))
            b = min(n, a + int(rng.integers(1, 3000)))
            x[a:b] += rng.normal(0, 10.0 ** rng.uniform(-2, 1), b - a)
    elif kind == 4:                                     # large offset, small variation
        x = 10.0 ** rng.uniform(0, 4) + rng.normal(0, 1e-2, n)
    elif kind == 5:                                     # heavy tails
        x = rng.standard_cauchy(n) * 1e-2
        x = np.clip(x, -1e3, 1e3)
    elif kind == 6:                                     # tiny values, zeros of both signs
        x = rng.normal(0, 1e-30, n)
        x[rng.random(n) < 0.2] = 0.0
        x[rng.random(n) < 0.1] = -0.0
    else:                                               # ramp
        x = np.linspace(rng.normal(), rng.normal() * 100, n)
    return np.asarray(x, dtype=np.float64).astype(f32)


def draw_bound(rng, x):
    if x.size == 0 or float(x.max()) == float(x.min()) or rng.random() < 0.4:
        return oracle.EB_ABS, float(10.0 ** rng.uniform(-6, 0))
    return oracle.EB_REL, float(10.0 ** rng.uniform(-5, -1))


def draw_length(rng):
    pick = rng.random()
    if pick < 0.15:
        return int(rng.integers(1, 70))
    if pick < 0.4:
        return int(rng.integers(1, 9)) * 4096 + int(rng.integers(-40, 41))
    return int(rng.integers(100, 300_000))


@pytest.mark.parametrize("seed", range(96))
def test_random_codec_and_hop(z, ctx, seed):
    rng = np.random.default_rng(1000 + seed)
    n = max(1, draw_length(rng))
    x = draw_field(rng, n)
    mode, eb = draw_bound(rng, x)
    try:
        want, wrc = oracle.compress(x, mode, eb)
    except oracle.OracleError as e:                      # the CUDA path must refuse the same way
        out = torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda")
        nb = torch.zeros(1, dtype=torch.int64, device="cuda")
        try:
            ctx.compress(dev(x), mode, eb, out, nb)
            assert ctx.status() == e.code
        except z.ZcclError as ze:                        # found on the host side of the boundary
            assert ze.code == e.code
        return
    st, rc = z.compress_to_bytes(ctx, dev(x), mode, eb)
    assert rc == wrc
    assert np.array_equal(st.cpu().numpy(), want)
    y, rc2 = z.decompress_from_bytes(ctx, dev(want), n)
    assert rc2 == z.OK
    wy = oracle.decompress(want)
    assert same_bits(y.cpu().numpy(), wy)

    # one hop on top: a second field of the same length, a random operation, raw output on
    b = draw_field(rng, n)
    op = [oracle.OP_SUM, oracle.OP_MAX, oracle.OP_MIN, oracle.OP_AVG][int(rng.integers(0, 4))]
    flags = op | (oracle.FLAG_CONSISTENT_OWNER if rng.random() < 0.3 else 0)
    try:
        fw, frc, fraw = oracle.drc(want, local=b, flags=flags, want_raw=True)
    except oracle.OracleError as e:
        fw, frc, fraw = None, e.code, None
    out = torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    raw = torch.empty(n, dtype=torch.float32, device="cuda")
    ctx.decompress_reduce_compress(dev(want), n, out, nb, local=dev(b), raw_out=raw, flags=flags)
    grc = ctx.status()
    assert grc == frc
    if fw is not None:
        assert np.array_equal(out[: int(nb.item())].cpu().numpy(), fw)
        assert same_bits(raw.cpu().numpy(), fraw)


@pytest.mark.parametrize("seed", range(24))
def test_random_collectives(z, ctx, seed):
    rng = np.random.default_rng(2000 + seed)
    N = int(rng.integers(2, 10))
    n = int(rng.integers(200, 60_000))
    base = draw_field(rng, n).astype(np.float64)
    send = [(base * rng.uniform(0.5, 2.0) + rng.normal(0, 1e-3 * (np.abs(base).max() + 1e-6), n)).astype(f32)
            for _ in range(N)]
    mode, eb = draw_bound(rng, np.concatenate(send))
    op = [oracle.OP_SUM, oracle.OP_MAX, oracle.OP_MIN, oracle.OP_AVG][int(rng.integers(0, 4))]
    try:
        want, wrc = oracle.sim_allreduce(send, mode, eb, flags=op)
    except oracle.OracleError as e:                      # e.g. codes beyond the range at a tight bound: refused alike
        recv = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(N)]
        ctx.sim_allreduce([dev(a) for a in send], recv, mode, eb, flags=op)
        assert ctx.status() == e.code
        return
    recv = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(N)]
    ctx.sim_allreduce([dev(a) for a in send], recv, mode, eb, flags=op)
    assert ctx.status() == wrc
    for r in range(N):
        assert same_bits(recv[r].cpu().numpy(), want[r]), f"allreduce rank {r}"

    want, wrc, sizes = oracle.sim_allgather(send, mode, eb)
    recv = [torch.empty(N * n, dtype=torch.float32, device="cuda") for _ in range(N)]
    ctx.sim_allgather([dev(a) for a in send], recv, mode, eb)
    assert ctx.status() == wrc
    assert ctx.sim_sizes()[:N] == [int(v) for v in sizes]
    for r in range(N):
        assert same_bits(recv[r].cpu().numpy(), want[r]), f"allgather rank {r}"

    want, wrc, _ = oracle.sim_reduce_scatter(send, mode, eb)
    recv = [torch.empty(want[r].size, dtype=torch.float32, device="cuda") for r in range(N)]
    ctx.sim_reduce_scatter([dev(a) for a in send], recv, mode, eb)
    assert ctx.status() == wrc
    for r in range(N):
        assert same_bits(recv[r].cpu().numpy(), want[r]), f"reduce-scatter rank {r}"


@pytest.mark.parametrize("seed", range(40))
def test_random_tile_sizes(z, ctx, seed):
    """Any multiple of 32 between 1024 and 8192 as the tile size, random lengths, kinds of data, bounds and offsets of
    both arrays from a 16-byte boundary: stream and values are the oracle's for that tile size."""
    rng = np.random.default_rng(7000 + seed)
    T = int(rng.integers(32, 257)) * 32
    n = draw_length(rng)
    x = draw_field(rng, n)
    mode, eb = draw_bound(rng, x)
    sx, sy = int(rng.integers(0, 4)), int(rng.integers(0, 4))
    try:
        want, wrc = oracle.compress(x, mode, eb, T)
    except oracle.OracleError as e:
        want, wrc = None, e.code
    buf = torch.empty(n + 4, dtype=torch.float32, device="cuda")
    dx = buf[sx: sx + n]
    dx.copy_(torch.from_numpy(x))
    out = torch.empty(z.compress_bound_tiled(n, T), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress_tiled(dx, mode, eb, T, out, nb)
    assert ctx.status() == wrc
    if want is None:
        return
    assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
    ybuf = torch.full((n + 4,), -3.0, dtype=torch.float32, device="cuda")
    ctx.decompress_tiled(out[: int(nb.item())], T, ybuf[sy: sy + n])
    assert ctx.status() == z.OK
    assert same_bits(ybuf[sy: sy + n].cpu().numpy(), oracle.decompress(want))
    assert bool((ybuf[:sy] == -3.0).all()) and bool((ybuf[sy + n:] == -3.0).all())
