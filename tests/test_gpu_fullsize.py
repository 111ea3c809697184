"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times (same
context limits, same entry points).  Where the oracle finishes in seconds the comparison is element by element;
for the 2 GiB case it is on sampled tiles (tiles are independent given the resolved bound) plus properties that
hold at any size (length, error bound against the input in fp64)."""
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


def _same_bits(a, b):
    return a.shape == b.shape and np.array_equal(a.view(np.uint32), b.view(np.uint32))


def _compress(z, ctx, dx, mode, eb):
    out = torch.empty(z.compress_bound(dx.numel()), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress(dx, mode, eb, out, nb)
    rc = ctx.status()
    return out[: int(nb.item())], rc


def test_config1_field_three_bounds(z):
    # 256^3 field, 64 MiB: streams byte for byte, reconstructions bit for bit, fused hop on the full field
    ctx = z.Context(1 << 24, 8)
    x = fields.fourier_field_3d(256, seed=1)
    loc = fields.fourier_field_3d(256, seed=2)
    dx, dl = torch.from_numpy(x).cuda(), torch.from_numpy(loc).cuda()
    for rel in (1e-2, 1e-3, 1e-4):
        want, wrc = oracle.compress(x, oracle.EB_REL, rel)
        st, rc = _compress(z, ctx, dx, z.EB_REL, rel)
        assert rc == wrc
        assert np.array_equal(st.cpu().numpy(), want)
        y = torch.empty_like(dx)
        ctx.decompress(st, y)
        assert ctx.status() == z.OK
        ref = oracle.decompress(want)
        assert _same_bits(y.cpu().numpy(), ref)
        ea, _, _ = oracle.resolve(oracle.EB_REL, rel, x)
        assert float((dx.double() - y.double()).abs().max()) <= float(ea)
    want, wrc = oracle.compress(x, oracle.EB_REL, 1e-3)
    want2, wrc2, wraw = oracle.drc(want, local=loc, want_raw=True)
    out = torch.empty(z.compress_bound(x.size), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    raw = torch.empty_like(dx)
    ctx.decompress_reduce_compress(torch.from_numpy(want).cuda(), x.size, out, nb, local=dl, raw_out=raw)
    assert ctx.status() == wrc2
    assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want2)
    assert _same_bits(raw.cpu().numpy(), wraw)
    ctx.close()


def test_config2_ring_allreduce_8x64MiB(z):
    N = 8
    ctx = z.Context(1 << 24, N)
    send = fields.rank_fields(N, 1 << 24, base_seed=100)
    want, wrc, whop = oracle.sim_allreduce(send, oracle.EB_REL, 1e-3, want_hop_bytes=True)
    d_send = [torch.from_numpy(a).cuda() for a in send]
    d_recv = [torch.zeros_like(t) for t in d_send]
    ctx.sim_allreduce(d_send, d_recv, z.EB_REL, 1e-3)
    assert ctx.status() == wrc
    sizes = np.array(ctx.sim_sizes()).reshape(N, N)
    assert np.array_equal(sizes, whop)
    for r in range(N):
        assert _same_bits(d_recv[r].cpu().numpy(), want[r])
    # accumulated error of the chain (Eq. 2): N compressions at most
    ea, _, _ = oracle.resolve(oracle.EB_REL, 1e-3, np.concatenate(send))
    exact = torch.zeros(1 << 24, dtype=torch.float64, device="cuda")
    mag = torch.zeros_like(exact)
    for t in d_send:
        exact += t.double()
        mag += t.double().abs()
    err = (d_recv[0].double() - exact).abs()
    assert bool((err <= N * float(ea) + N * 2.0 ** -24 * mag).all())
    ctx.close()


def test_config3_gradient_like_1GiB(z):
    n = 1 << 28
    ctx = z.Context(n, 0)
    x = fields.gradient_like(n, seed=3)
    want, wrc = oracle.compress(x, oracle.EB_ABS, 1e-5)
    dx = torch.from_numpy(x).cuda()
    st, rc = _compress(z, ctx, dx, z.EB_ABS, 1e-5)
    assert rc == wrc
    assert st.numel() == want.size
    assert bool((st == torch.from_numpy(want).cuda()).all())
    y = torch.empty_like(dx)
    ctx.decompress(st, y)
    assert ctx.status() == z.OK
    ref = oracle.decompress(want)
    assert bool((y.view(torch.int32) == torch.from_numpy(ref).cuda().view(torch.int32)).all())
    assert float((dx.double() - y.double()).abs().max()) <= 1e-5
    assert 2.5 < 4 * n / want.size < 4.5
    ctx.close()


@pytest.mark.parametrize("log2_bytes", [12, 14, 16, 18, 20, 22, 24, 26, 28])
def test_config4_message_sizes(z, log2_bytes):
    n = (1 << log2_bytes) // 4
    ctx = z.Context(max(n, 4096), 0)
    x = fields.smooth_1d(n, seed=log2_bytes)
    dx = torch.from_numpy(x).cuda()
    for rel in (1e-2, 1e-3, 1e-4):
        want, wrc = oracle.compress(x, oracle.EB_REL, rel)
        st, rc = _compress(z, ctx, dx, z.EB_REL, rel)
        assert rc == wrc and np.array_equal(st.cpu().numpy(), want)
        y = torch.empty_like(dx)
        ctx.decompress(st, y)
        assert ctx.status() == z.OK
        assert _same_bits(y.cpu().numpy(), oracle.decompress(want))
    ctx.close()


def test_config4_largest_message_sampled_tiles(z):
    # 2 GiB: the oracle checks sampled tiles one by one; length and error bound are checked on everything
    n = 1 << 29
    T = 4096
    ctx = z.Context(n, 0)
    x = fields.smooth_1d(n, seed=31)
    eb = 2.5e-3
    ea, s, r = oracle.resolve(oracle.EB_ABS, eb)
    dx = torch.from_numpy(x).cuda()
    st, rc = _compress(z, ctx, dx, z.EB_ABS, eb)
    assert rc == z.OK
    nT = n // T
    head = st[: 32 + 4 * nT].cpu().numpy()
    assert head[:4].tobytes() == b"ZCL1"
    assert int(np.frombuffer(head[8:16].tobytes(), np.uint64)[0]) == n
    idx = np.frombuffer(head[32:].tobytes(), np.uint32).astype(np.int64)
    assert np.all(np.diff(idx) > 0) and st.numel() == 32 + 4 * nT + 4 * int(idx[-1])
    y = torch.empty_like(dx)
    ctx.decompress(st, y)
    assert ctx.status() == z.OK
    assert float((dx.double() - y.double()).abs().max()) <= float(ea)
    rng = np.random.default_rng(0)
    for t in [0, 1, nT // 2, nT - 2, nT - 1] + list(rng.integers(0, nT, 40)):
        t = int(t)
        tile = x[t * T:(t + 1) * T]
        ref_stream, _ = oracle.compress_core(tile, ea, s, r)             # one-tile stream: header, 1 index word, blob
        ref_blob = ref_stream[36:]
        beg = 32 + 4 * nT + 4 * (int(idx[t - 1]) if t else 0)
        end = 32 + 4 * nT + 4 * int(idx[t])
        assert np.array_equal(st[beg:end].cpu().numpy(), ref_blob), t
        assert _same_bits(y[t * T:(t + 1) * T].cpu().numpy(), oracle.decompress(ref_stream))
    ctx.close()


@pytest.mark.parametrize("n", [1 << 10, 1 << 16, 1 << 20])
def test_config4_allgather_and_bcast(z, n):
    N = 8
    ctx = z.Context(N * n, N)
    send = [fields.smooth_1d(n, seed=200 + r) for r in range(N)]
    want, wrc, wsizes = oracle.sim_allgather(send, oracle.EB_REL, 1e-3)
    d_send = [torch.from_numpy(a).cuda() for a in send]
    d_recv = [torch.zeros(N * n, dtype=torch.float32, device="cuda") for _ in range(N)]
    ctx.sim_allgather(d_send, d_recv, z.EB_REL, 1e-3)
    assert ctx.status() == wrc
    for r in range(N):
        assert _same_bits(d_recv[r].cpu().numpy(), want[r])
    assert np.array_equal(np.array(ctx.sim_sizes()), wsizes)
    wantb, wrcb, wbytes = oracle.sim_bcast(send[0], N, oracle.EB_REL, 1e-3)
    b_recv = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(N)]
    ctx.sim_bcast(d_send[0], b_recv, z.EB_REL, 1e-3)
    assert ctx.status() == wrcb
    for k in range(N):
        assert _same_bits(b_recv[k].cpu().numpy(), wantb[k])
    ctx.close()


def test_two_gib_of_binary64_and_one_gib_in_tiles_of_5120(z):
    """2^28 elements and a ragged end through the binary64 kernels (2 GiB in) and through the kernels for other tile
    sizes (1 GiB in, tiles of 5120): tile, round and row numbers of the copy engine's maps at the top of the range."""
    n = (1 << 28) + 12345
    x = np.tile(fields.fourier_field_3d(256, seed=1).astype(np.float64), 17)[:n] * (1 + 1e-9)
    ctx = z.Context(n, 0)
    try:
        nb = torch.zeros(1, dtype=torch.int64, device="cuda")
        out = torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda")
        ctx.compress_f64(torch.from_numpy(x).cuda(), z.EB_REL, 1e-4, out, nb)
        assert ctx.status() == z.OK
        want = oracle.compress_f64(x, oracle.EB_REL, 1e-4)
        assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
        y = torch.empty(n, dtype=torch.float64, device="cuda")
        ctx.decompress_f64(out[: int(nb.item())], y)
        assert ctx.status() == z.OK
        assert np.array_equal(y.cpu().numpy().view(np.uint64), oracle.decompress_f64(want).view(np.uint64))
        del out, y, x, want
        n2 = (1 << 28) + 777
        x2 = np.tile(fields.fourier_field_3d(256, seed=2), 17)[:n2]
        out2 = torch.empty(z.compress_bound_tiled(n2, 5120), dtype=torch.uint8, device="cuda")
        ctx.compress_tiled(torch.from_numpy(x2).cuda(), z.EB_REL, 1e-3, 5120, out2, nb)
        want2, wrc2 = oracle.compress(x2, oracle.EB_REL, 1e-3, 5120)
        assert ctx.status() == wrc2
        assert np.array_equal(out2[: int(nb.item())].cpu().numpy(), want2)
        y2 = torch.empty(n2, dtype=torch.float32, device="cuda")
        ctx.decompress_tiled(out2[: int(nb.item())], 5120, y2)
        assert ctx.status() == z.OK
        assert _same_bits(y2.cpu().numpy(), oracle.decompress(want2))
    finally:
        ctx.close()
