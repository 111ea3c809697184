"""GPU parity: the CUDA path through the C-ABI against the CPU oracle, element by element (streams byte for byte,
reconstructions bit for bit) on the same seeded inputs.  Sizes span several tiles and ragged tails."""
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
    c = z.Context(1 << 22, 8)
    yield c
    c.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_compress(z, ctx, x, mode, eb, capacity=None):
    st, rc = z.compress_to_bytes(ctx, dev(x), mode, eb, capacity)
    return st.cpu().numpy(), rc


def gpu_decompress(z, ctx, stream, n):
    y, rc = z.decompress_from_bytes(ctx, dev(stream), n)
    return y.cpu().numpy(), rc


def assert_same_bits(a, b):
    assert a.shape == b.shape
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


# ----------------------------------------------------------------------------- compress / decompress

def _codec_case(z, ctx, x, mode, eb):
    want, wrc = oracle.compress(x, mode, eb)
    got, rc = gpu_compress(z, ctx, x, mode, eb)
    assert rc == wrc
    assert got.size == want.size
    assert np.array_equal(got, want), f"first differing byte {np.flatnonzero(got != want)[:4]}"
    y, rc2 = gpu_decompress(z, ctx, want, x.size)
    assert rc2 == z.OK
    assert_same_bits(y, oracle.decompress(want))
    ea, s, r = oracle.resolve(mode, eb, x)
    if wrc == oracle.OK and x.size:
        assert np.abs(x.astype(np.float64) - y.astype(np.float64)).max() <= float(ea)
    return want


def test_config0_bit_exact(z, ctx):
    x = fields.smooth_1d(1 << 20, seed=0)
    st = _codec_case(z, ctx, x, z.EB_REL, 1e-3)
    assert 10 < x.nbytes / st.size < 20


@pytest.mark.parametrize("rel", [1e-2, 1e-3, 1e-4])
def test_fourier_field_bit_exact(z, ctx, rel):
    x = fields.fourier_field_3d(96, seed=1)          # 884736 elements = 216 tiles
    _codec_case(z, ctx, x, z.EB_REL, rel)


def test_gradient_like_bit_exact(z, ctx):
    x = fields.gradient_like((1 << 21) + 12345, seed=3)
    _codec_case(z, ctx, x, z.EB_ABS, 1e-5)


@pytest.mark.parametrize("n", [0, 1, 2, 31, 32, 33, 63, 64, 65, 511, 512, 513, 4095, 4096, 4097, 8191, 8192, 8193,
                               12288 + 31, 3 * 4096 + 1000])
def test_ragged_lengths(z, ctx, n):
    rng = np.random.default_rng(1000 + n)
    x = np.cumsum(rng.normal(0, 2e-3, n)).astype(f32)
    _codec_case(z, ctx, x, z.EB_ABS, 1e-3)


def test_every_length_around_tile_edges(z, ctx):
    rng = np.random.default_rng(5)
    base = np.cumsum(rng.normal(0, 1.0, 2 * 4096 + 40)).astype(f32)
    for n in list(range(0, 70)) + list(range(4096 - 34, 4096 + 35)) + list(range(8192 - 3, 8192 + 34)):
        want, _ = oracle.compress(base[:n], oracle.EB_ABS, 0.25)
        got, rc = gpu_compress(z, ctx, base[:n], z.EB_ABS, 0.25)
        assert np.array_equal(got, want), n
        y, _ = gpu_decompress(z, ctx, want, n)
        assert_same_bits(y, oracle.decompress(want))


def test_wide_code_lengths(z, ctx):
    # white noise at a tight bound: code lengths well above 16 bits, precision warning expected
    rng = np.random.default_rng(4)
    x = rng.normal(0, 1.0, 50_000).astype(f32)
    want, wrc = oracle.compress(x, oracle.EB_ABS, 1e-6)
    assert wrc == oracle.W_PRECISION
    got, rc = gpu_compress(z, ctx, x, z.EB_ABS, 1e-6)
    assert rc == z.W_PRECISION
    assert np.array_equal(got, want)
    y, _ = gpu_decompress(z, ctx, want, x.size)
    assert_same_bits(y, oracle.decompress(want))


def test_all_code_lengths_occur(z, ctx):
    # one block per code length 0..31 (deltas of magnitude 2^(L-1)), unit step through a tiny bound
    ea, s, r = oracle.resolve(oracle.EB_ABS, 0.5)
    vals = []
    level = 0.0
    for L in range(0, 30):
        blk = np.full(32, level)
        if L:
            level += float(2 ** (L - 1)) * float(s) * (1 if L % 2 else -1)
            blk[16:] = level
        vals.append(blk)
    x = np.concatenate(vals).astype(f32)
    want, wrc = oracle.compress(x, oracle.EB_ABS, 0.5)
    got, rc = gpu_compress(z, ctx, x, z.EB_ABS, 0.5)
    assert rc == wrc
    assert np.array_equal(got, want)
    y, _ = gpu_decompress(z, ctx, want, x.size)
    assert_same_bits(y, oracle.decompress(want))


def _mixed_length_field(seed, nblocks, lmax):
    """Blocks whose code lengths are drawn independently from 0..lmax (amplitude 2^(L-1) around a common level), so
    that neighbouring blocks of every pair and every group of four differ in length."""
    rng = np.random.default_rng(seed)
    ea, s, r = oracle.resolve(oracle.EB_ABS, 0.5)
    q = np.zeros(nblocks * 32, np.int64)
    for b in range(nblocks):
        L = int(rng.integers(0, lmax + 1))
        if L:
            q[32 * b: 32 * b + 32] = rng.integers(-(2 ** (L - 1)), 2 ** (L - 1) + 1, 32)
        elif b:
            q[32 * b: 32 * b + 32] = q[32 * b - 1]           # a constant block continues the last value
    return (q.astype(np.float64) * float(s)).astype(f32)


@pytest.mark.parametrize("lmax", [7, 9, 15, 17, 22])
def test_neighbouring_blocks_of_different_code_lengths(z, ctx, lmax):
    # the encoder and the decoder handle four, two or one block per bit-matrix transpose depending on the longest
    # code of a group of four; every mixture of lengths inside a group must give the oracle's bytes and values
    x = _mixed_length_field(100 + lmax, 5 * 128 + 37, lmax)
    want, wrc = oracle.compress(x, oracle.EB_ABS, 0.5)
    got, rc = gpu_compress(z, ctx, x, z.EB_ABS, 0.5)
    assert rc == wrc
    assert np.array_equal(got, want)
    y, _ = gpu_decompress(z, ctx, want, x.size)
    assert_same_bits(y, oracle.decompress(want))
    b = _mixed_length_field(200 + lmax, 5 * 128 + 37, max(lmax - 2, 1))
    fw, frc, fraw = oracle.drc(want, local=b, want_raw=True)
    fg, grc, graw = _drc_gpu(z, ctx, want, x.size, local=b, raw=True)
    assert grc == frc
    assert np.array_equal(fg, fw)
    assert_same_bits(graw, fraw)


def test_adversarial_ties_and_denormals(z, ctx):
    ea, s, r = oracle.resolve(oracle.EB_ABS, 1e-3)
    k = np.arange(-3000, 3000, dtype=np.float64)
    half = ((k + 0.5) * float(s)).astype(f32)
    x = np.concatenate([half, np.nextafter(half, f32(np.inf)), np.nextafter(half, f32(-np.inf)),
                        np.array([0.0, -0.0, 1e-45, -1e-45, 1e-38, -1e-38], f32)])
    np.random.default_rng(0).shuffle(x)
    _codec_case(z, ctx, x, z.EB_ABS, 1e-3)


def test_constant_input_and_degenerate_rel(z, ctx):
    x = np.full(3 * 4096 + 5, 2.5, f32)
    _codec_case(z, ctx, x, z.EB_ABS, 1e-2)
    st, rc = gpu_compress(z, ctx, x, z.EB_REL, 1e-3)       # zero range
    assert rc == z.E_DEGENERATE


def test_range_error_is_reported_and_memory_safe(z, ctx):
    x = np.array([0.0, 3e6, -3e6, 1.0] * 2000, f32)
    cap = z.compress_bound(x.size)
    out = torch.full((cap + 64,), 0xAB, dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress(dev(x), z.EB_ABS, 1e-3, out[:cap], nbytes)
    assert ctx.status() == z.E_RANGE
    assert bool((out[cap:] == 0xAB).all())


def test_capacity_overrun_is_reported_not_written(z, ctx):
    x = fields.smooth_1d(40_000, seed=3)
    want, _ = oracle.compress(x, oracle.EB_REL, 1e-3)
    cap = want.size - 40
    out = torch.full((want.size + 64,), 0xCD, dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress(dev(x), z.EB_REL, 1e-3, out[:cap], nbytes)
    assert ctx.status() == z.E_CAPACITY
    assert bool((out[cap:] == 0xCD).all())
    with pytest.raises(z.ZcclError) as e:
        ctx.compress(dev(x), z.EB_REL, 1e-3, out[:40], nbytes)     # below header + index: seen by the host
    assert e.value.code == z.E_CAPACITY
    # exactly enough is fine
    got, rc = gpu_compress(z, ctx, x, z.EB_REL, 1e-3, capacity=want.size)
    assert rc == z.OK and np.array_equal(got, want)


def test_malformed_streams(z, ctx):
    x = fields.smooth_1d(9000, seed=4)
    st, _ = oracle.compress(x, oracle.EB_REL, 1e-3)

    def status_of(b, n=9000, cap=None):
        y = torch.full((n + 16,), 7.0, dtype=torch.float32, device="cuda")
        ctx.decompress(dev(b), y[:n], in_bytes_max=cap)
        rc = ctx.status()
        assert bool((y[n:] == 7.0).all())
        return rc

    assert status_of(st) == z.OK
    for mut in (lambda b: b.__setitem__(0, 0), lambda b: b.__setitem__(4, 2),
                lambda b: b.__setitem__(slice(24, 28), [0, 0, 0, 0]),
                lambda b: b.__setitem__(slice(28, 32), [9, 0, 0, 0]),
                lambda b: b.__setitem__(slice(32, 36), [0xFF, 0xFF, 0xFF, 0x7F]),
                lambda b: b.__setitem__(32 + 12 + 4, 40),
                lambda b: b.__setitem__(32 + 12 + 4, b[32 + 12 + 4] + 1)):
        b = st.copy()
        mut(b)
        assert status_of(b) == z.E_BAD_STREAM
    assert status_of(st, cap=st.size - 4) == z.E_BAD_STREAM      # truncated
    assert status_of(st, n=8000) == z.E_CAPACITY                 # output too small for the header's n


# ----------------------------------------------------------------------------- fused reduce hop

def _drc_gpu(z, ctx, in_c, n, local=None, local_c=None, raw=False, flags=0):
    out = torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    raw_out = torch.empty(n, dtype=torch.float32, device="cuda") if raw else None
    ctx.decompress_reduce_compress(dev(in_c), n, out, nbytes,
                                   local=dev(local) if local is not None else None,
                                   local_c=dev(local_c) if local_c is not None else None,
                                   raw_out=raw_out, flags=flags)
    rc = ctx.status()
    res = out[: int(nbytes.item())].cpu().numpy()
    return res, rc, (raw_out.cpu().numpy() if raw else None)


@pytest.mark.parametrize("n", [1, 33, 4096, 4097, 70_000, 5 * 4096 + 17])
def test_fused_hop_matches_unfused_composition(z, ctx, n):
    a = fields.smooth_1d(n, seed=1)
    b = fields.smooth_1d(n, seed=2)
    ea, s, r = oracle.resolve(oracle.EB_REL, 1e-3, np.concatenate([a, b]))
    sa, _ = oracle.compress_core(a, ea, s, r)
    want, wrc, wraw = oracle.drc(sa, local=b, want_raw=True)
    got, rc, raw = _drc_gpu(z, ctx, sa, n, local=b, raw=True)
    assert rc == wrc
    assert np.array_equal(got, want)
    assert_same_bits(raw, wraw)
    # owner copy as the dequantised value
    want2, _, wraw2 = oracle.drc(sa, local=b, want_raw=True, flags=oracle.FLAG_CONSISTENT_OWNER)
    got2, _, raw2 = _drc_gpu(z, ctx, sa, n, local=b, raw=True, flags=z.CONSISTENT_OWNER)
    assert np.array_equal(got2, want2)
    assert_same_bits(raw2, wraw2)
    # two-compressed form
    sb, _ = oracle.compress_core(b, ea, s, r)
    want3, _, wraw3 = oracle.drc(sa, local_c=sb, want_raw=True)
    got3, rc3, raw3 = _drc_gpu(z, ctx, sa, n, local_c=sb, raw=True)
    assert np.array_equal(got3, want3)
    assert_same_bits(raw3, wraw3)


def test_fused_hop_fourier_and_gradient(z, ctx):
    a = fields.fourier_field_3d(64, seed=11)
    b = fields.fourier_field_3d(64, seed=12)
    for rel in (1e-2, 1e-4):
        ea, s, r = oracle.resolve(oracle.EB_REL, rel, np.concatenate([a, b]))
        sa, _ = oracle.compress_core(a, ea, s, r)
        want, wrc = oracle.drc(sa, local=b)
        got, rc, _ = _drc_gpu(z, ctx, sa, a.size, local=b)
        assert rc == wrc and np.array_equal(got, want)
    g1 = fields.gradient_like(100_000, seed=5)
    g2 = fields.gradient_like(100_000, seed=6)
    sa, _ = oracle.compress(g1, oracle.EB_ABS, 1e-5)
    want, wrc = oracle.drc(sa, local=g2)
    got, rc, _ = _drc_gpu(z, ctx, sa, g1.size, local=g2)
    assert rc == wrc and np.array_equal(got, want)


def test_fused_hop_wide_code_lengths(z, ctx):
    # noisy operands at a tight bound: encoded tiles larger than the shared-memory regions of the encoder, which
    # then encodes them again straight into the stream; mixed with smooth tiles that take the ordinary route
    rng = np.random.default_rng(12)
    n = 9 * 4096 + 100
    a = fields.smooth_1d(n, seed=3)
    b = fields.smooth_1d(n, seed=4)
    b[2 * 4096: 5 * 4096] += rng.normal(0, 0.5, 3 * 4096).astype(f32)
    a[7 * 4096:] += rng.normal(0, 0.5, n - 7 * 4096).astype(f32)
    ea, s, r = oracle.resolve(oracle.EB_ABS, 2e-6)
    sa, _ = oracle.compress_core(a, ea, s, r)
    want, wrc, wraw = oracle.drc(sa, local=b, want_raw=True)
    got, rc, raw = _drc_gpu(z, ctx, sa, n, local=b, raw=True)
    assert rc == wrc
    assert np.array_equal(got, want)
    assert_same_bits(raw, wraw)
    st, rc2 = gpu_compress(z, ctx, a, z.EB_ABS, 2e-6)
    assert np.array_equal(st, sa)


def test_fused_hop_rejects_mismatch(z, ctx):
    a = fields.smooth_1d(9000, seed=1)
    sa, _ = oracle.compress(a, oracle.EB_ABS, 1e-3)
    _, rc, _ = _drc_gpu(z, ctx, sa, 8000, local=a[:8000])          # n differs from the header
    assert rc == z.E_BAD_STREAM
    sb, _ = oracle.compress(a, oracle.EB_ABS, 2e-3)
    _, rc, _ = _drc_gpu(z, ctx, sa, 9000, local_c=sb)              # different steps
    assert rc == z.E_BAD_STREAM
    bad = sa.copy()
    bad[32 + 12 + 4] = 33
    _, rc, _ = _drc_gpu(z, ctx, bad, 9000, local=a)
    assert rc == z.E_BAD_STREAM
    with pytest.raises(z.ZcclError):
        ctx.decompress_reduce_compress(dev(sa), 9000, torch.empty(100000, dtype=torch.uint8, device="cuda"),
                                       torch.zeros(1, dtype=torch.int64, device="cuda"))   # neither operand


# ----------------------------------------------------------------------------- emulated collectives

def _run_allreduce(z, ctx, send, mode, eb, flags=0):
    d_send = [dev(a) for a in send]
    d_recv = [torch.zeros_like(t) for t in d_send]
    ctx.sim_allreduce(d_send, d_recv, mode, eb, flags)
    rc = ctx.status()
    sizes = ctx.sim_sizes()
    return [t.cpu().numpy() for t in d_recv], rc, np.array(sizes)


@pytest.mark.parametrize("N,n", [(2, 1000), (3, 10_001), (8, 8 * 4096 * 3), (8, 8 * 5000 + 3), (8, 5), (5, 4096 * 5 + 1),
                                 (1, 5000)])
def test_allreduce_matches_oracle(z, ctx, N, n):
    send = [fields.smooth_1d(n, seed=40 + r) for r in range(N)]
    want, wrc, whop = oracle.sim_allreduce(send, oracle.EB_REL, 1e-3, want_hop_bytes=True)
    got, rc, sizes = _run_allreduce(z, ctx, send, z.EB_REL, 1e-3)
    assert rc == wrc
    for r in range(N):
        assert_same_bits(got[r], want[r])
    assert np.array_equal(sizes.reshape(N, N), whop)


def test_allreduce_consistent_owner_and_bound(z, ctx):
    N = 8
    send = [fields.fourier_field_3d(64, seed=100 + r) for r in range(N)]
    n = send[0].size
    want, wrc = oracle.sim_allreduce(send, oracle.EB_REL, 1e-3, flags=oracle.FLAG_CONSISTENT_OWNER)
    got, rc, _ = _run_allreduce(z, ctx, send, z.EB_REL, 1e-3, flags=z.CONSISTENT_OWNER)
    for r in range(N):
        assert_same_bits(got[r], want[r])
        assert_same_bits(got[r], got[0])
    ea, s, r_ = oracle.resolve(oracle.EB_REL, 1e-3, np.concatenate(send))
    exact = np.sum(np.stack(send).astype(np.float64), axis=0)
    slack = N * 2.0 ** -24 * np.sum(np.abs(np.stack(send).astype(np.float64)), axis=0)
    assert np.all(np.abs(got[0].astype(np.float64) - exact) <= N * float(ea) + slack)   # error chain of Eq. 2


def test_allreduce_lossless_on_grid(z, ctx):
    from _util import find_power_of_two_step_bound
    eb, s = find_power_of_two_step_bound(-7)
    N, n = 8, 8 * 4096 + 17
    send = fields.on_grid_ranks(N, n, float(s), seed=7)
    exact = np.sum(np.stack(send).astype(np.float64), axis=0)
    got, rc, _ = _run_allreduce(z, ctx, send, z.EB_ABS, eb)
    assert rc == z.OK
    for r in range(N):
        assert np.array_equal(got[r].astype(np.float64), exact)


@pytest.mark.parametrize("N,n", [(2, 4097), (8, 2 * 4096 + 77), (3, 1)])
def test_allgather_matches_oracle(z, ctx, N, n):
    send = [fields.smooth_1d(n, seed=80 + r) for r in range(N)]
    want, wrc, wsizes = oracle.sim_allgather(send, oracle.EB_REL, 1e-3)
    d_send = [dev(a) for a in send]
    d_recv = [torch.zeros(N * n, dtype=torch.float32, device="cuda") for _ in range(N)]
    ctx.sim_allgather(d_send, d_recv, z.EB_REL, 1e-3)
    assert ctx.status() == wrc
    for r in range(N):
        assert_same_bits(d_recv[r].cpu().numpy(), want[r])
    assert np.array_equal(np.array(ctx.sim_sizes()), wsizes)


@pytest.mark.parametrize("nsinks", [1, 3, 8])
def test_bcast_matches_oracle(z, ctx, nsinks):
    x = fields.smooth_1d(20_000, seed=90)
    want, wrc, wbytes = oracle.sim_bcast(x, nsinks, oracle.EB_REL, 1e-4)
    d_recv = [torch.zeros(x.size, dtype=torch.float32, device="cuda") for _ in range(nsinks)]
    ctx.sim_bcast(dev(x), d_recv, z.EB_REL, 1e-4)
    assert ctx.status() == wrc
    for k in range(nsinks):
        assert_same_bits(d_recv[k].cpu().numpy(), want[k])
    assert ctx.sim_sizes() == [wbytes]


def test_repeated_calls_reuse_workspace(z, ctx):
    # the scan workspace is re-armed by each launch: many back-to-back calls on one stream stay exact
    x = fields.smooth_1d(200_000, seed=21)
    want, _ = oracle.compress(x, oracle.EB_REL, 1e-3)
    dx = dev(x)
    out = torch.empty(z.compress_bound(x.size), dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    for _ in range(50):
        ctx.compress(dx, z.EB_REL, 1e-3, out, nbytes)
    assert ctx.status() == z.OK
    assert np.array_equal(out[: int(nbytes.item())].cpu().numpy(), want)


def test_host_buffer_forms(z, ctx):
    x = fields.smooth_1d(100_000, seed=22)
    want, _ = oracle.compress(x, oracle.EB_REL, 1e-3)
    xh = torch.from_numpy(x).pin_memory()
    oh = torch.empty(z.compress_bound(x.size), dtype=torch.uint8).pin_memory()
    nb = ctx.compress_host(xh, z.EB_REL, 1e-3, oh)
    torch.cuda.synchronize()
    assert nb == want.size and np.array_equal(oh[:nb].numpy(), want)
    yh = torch.empty(x.size, dtype=torch.float32).pin_memory()
    ctx.decompress_host(oh, nb, yh)
    torch.cuda.synchronize()
    assert ctx.status() == z.OK
    assert_same_bits(yh.numpy(), oracle.decompress(want))


def test_look_back_wait_is_bounded(z):
    # a tile whose size is never published: the tiles after it give up after their poll limit, report a time-out
    # and write nothing; no hang, and the context works again afterwards
    ctx = z.Context(1 << 20, 0)
    x = fields.smooth_1d(5 * 4096, seed=33)
    dx = dev(x)
    want, _ = oracle.compress(x, oracle.EB_REL, 1e-3)
    out = torch.full((z.compress_bound(x.size) + 64,), 0x5A, dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.debug_skip_publish(1)
    ctx.compress(dx, z.EB_REL, 1e-3, out[: z.compress_bound(x.size)], nbytes)
    assert ctx.status() == z.E_TIMEOUT
    assert bool((out[z.compress_bound(x.size):] == 0x5A).all())
    ctx.debug_skip_publish(-1)
    ctx.compress(dx, z.EB_REL, 1e-3, out[: z.compress_bound(x.size)], nbytes)
    assert ctx.status() == z.OK
    assert np.array_equal(out[: int(nbytes.item())].cpu().numpy(), want)
    ctx.close()


def test_launch_counter_wraps_cleanly(z):
    # the scan states are validated by a launch counter: run compress, fused hop and decompress on both sides of its
    # wrap-around (states of earlier launches must not look current afterwards)
    ctx = z.Context(1 << 20, 0)
    x = fields.smooth_1d(37 * 4096 + 123, seed=35)
    loc = fields.smooth_1d(x.size, seed=36)
    dx, dl = dev(x), dev(loc)
    want, wrc = oracle.compress(x, oracle.EB_REL, 1e-3)
    want2, wrc2 = oracle.drc(want, local=loc)
    cap = z.compress_bound(x.size)
    ctx.debug_set_launch_counter(0x7FFFFFFF - 2)
    for _ in range(3):   # counters 2^31 - 3, 2^31 - 2, 2^31 - 1 for the encoder launches, then 1, 2, ...
        out = torch.zeros(cap, dtype=torch.uint8, device="cuda")
        nb = torch.zeros(1, dtype=torch.int64, device="cuda")
        ctx.compress(dx, z.EB_REL, 1e-3, out, nb)
        assert ctx.status() == wrc
        assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
        out2 = torch.zeros(cap, dtype=torch.uint8, device="cuda")
        nb2 = torch.zeros(1, dtype=torch.int64, device="cuda")
        ctx.decompress_reduce_compress(out[: int(nb.item())], x.size, out2, nb2, local=dl)
        assert ctx.status() == wrc2
        assert np.array_equal(out2[: int(nb2.item())].cpu().numpy(), want2)
    ctx.close()


@pytest.mark.parametrize("N,n", [(2, 1000), (3, 10_001), (8, 8 * 4096 * 3), (8, 8 * 5000 + 3), (8, 11), (5, 4096 * 5 + 1),
                                 (1, 5000)])
def test_reduce_scatter_matches_oracle(z, ctx, N, n):
    send = [fields.smooth_1d(n, seed=60 + r) for r in range(N)]
    want, wrc, whop = oracle.sim_reduce_scatter(send, oracle.EB_REL, 1e-3)
    d_send = [dev(a) for a in send]
    guard = 8   # elements after each receive buffer that must stay untouched
    d_recv = [torch.full((want[r].size + guard,), 7.0, dtype=torch.float32, device="cuda") for r in range(N)]
    ctx.sim_reduce_scatter(d_send, d_recv, z.EB_REL, 1e-3)
    assert ctx.status() == wrc
    for r in range(N):
        got = d_recv[r].cpu().numpy()
        assert_same_bits(got[: want[r].size], want[r])
        assert np.all(got[want[r].size:] == 7.0)
    if N > 1:
        assert np.array_equal(np.array(ctx.sim_sizes()).reshape(N - 1, N), whop)


def test_reduce_scatter_lossless_on_grid(z, ctx):
    from _util import find_power_of_two_step_bound
    eb, s = find_power_of_two_step_bound(-6)
    N, n = 8, 8 * 4096 + 77
    send = fields.on_grid_ranks(N, n, float(s), seed=5)
    exact = np.sum(np.stack(send).astype(np.float64), axis=0)
    d_recv = [torch.zeros(oracle.chunk_span(n, N, r)[1], dtype=torch.float32, device="cuda") for r in range(N)]
    ctx.sim_reduce_scatter([dev(a) for a in send], d_recv, z.EB_ABS, eb)
    assert ctx.status() == z.OK
    for r in range(N):
        off, ln = oracle.chunk_span(n, N, r)
        assert np.array_equal(d_recv[r].cpu().numpy().astype(np.float64), exact[off:off + ln])


@pytest.mark.parametrize("N,n", [(1, 300), (2, 1000), (3, 5000), (5, 4096 + 7), (8, 3 * 4096), (13, 777), (16, 4096)])
def test_scatter_matches_oracle(z, N, n):
    c = z.Context(max(N * n, 4096), max(N, 2))
    root = fields.smooth_1d(N * n, seed=70 + N)
    want, wrc, wsizes, _ = oracle.sim_scatter(root, N, oracle.EB_REL, 1e-3)
    d_recv = [torch.full((n + 8,), 7.0, dtype=torch.float32, device="cuda") for _ in range(N)]
    c.sim_scatter(dev(root), d_recv, z.EB_REL, 1e-3)
    assert c.status() == wrc
    for r in range(N):
        got = d_recv[r].cpu().numpy()
        assert_same_bits(got[:n], want[r])
        assert np.all(got[n:] == 7.0)
    assert np.array_equal(np.array(c.sim_sizes()), wsizes)
    c.close()


def _quality(ctx, x, y):
    out = torch.zeros(6, dtype=torch.float64, device="cuda")
    ctx.quality(x, y, out)
    v = out.cpu().numpy()
    return dict(max_abs_err=v[0], mse=v[1], nrmse=v[2], psnr=v[3], min=v[4], max=v[5])


@pytest.mark.parametrize("n", [1, 5, 4099, 1 << 20, (1 << 22) - 3])
def test_quality_matches_oracle(z, ctx, n):
    # exact for the extrema and the largest error (fp64 differences of fp32 values are exact); the sum of squares is
    # formed in another order than the oracle's, so MSE and what derives from it agree to fp64 summation accuracy:
    # n terms of one sign, relative error at most n * 2^-53 < 1e-9
    import math
    x = fields.smooth_1d(n, seed=50)
    rng = np.random.default_rng(n)
    y = (x + rng.normal(0, 1e-3, n)).astype(f32)
    want = oracle.quality(x, y)
    dx, dy = dev(x), dev(y)
    got = _quality(ctx, dx, dy)
    assert got["max_abs_err"] == want["max_abs_err"] and got["min"] == want["min"] and got["max"] == want["max"]
    assert math.isclose(got["mse"], want["mse"], rel_tol=1e-9)
    if n > 1:
        assert math.isclose(got["nrmse"], want["nrmse"], rel_tol=1e-9) and math.isclose(got["psnr"], want["psnr"], rel_tol=1e-9)
    else:
        assert math.isnan(got["nrmse"]) and math.isnan(want["nrmse"])
    again = _quality(ctx, dx, dy)                              # same bits on a second run
    assert np.array_equal(np.array(list(again.values())), np.array(list(got.values())), equal_nan=True)
    got_u = _quality(ctx, dev(np.concatenate([[0], x]).astype(f32))[1:], dev(np.concatenate([[0], y]).astype(f32))[1:])
    assert got_u["max_abs_err"] == want["max_abs_err"] and math.isclose(got_u["mse"], want["mse"], rel_tol=1e-9)   # unaligned


def test_quality_of_a_compressed_field(z, ctx):
    import math
    x = fields.fourier_field_3d(128, seed=4)
    dx = dev(x)
    out = torch.empty(z.compress_bound(x.size), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress(dx, z.EB_REL, 1e-3, out, nb)
    y = torch.empty_like(dx)
    ctx.decompress(out[: int(nb.item())], y)
    q = _quality(ctx, dx, y)
    ea, s, _ = oracle.resolve(oracle.EB_REL, 1e-3, x)
    assert q["max_abs_err"] <= float(ea)
    assert q["nrmse"] < 1e-3 and q["psnr"] > 60.0
    assert _quality(ctx, dx, dx)["psnr"] == math.inf
    want = oracle.quality(x, y.cpu().numpy())
    assert q["max_abs_err"] == want["max_abs_err"] and math.isclose(q["mse"], want["mse"], rel_tol=1e-9)


@pytest.mark.parametrize("op", ["max", "min"])
@pytest.mark.parametrize("n", [4096 * 3 + 50, 4096 * 40, 777])
def test_fused_hop_max_min_matches_oracle(z, ctx, op, n):
    zop, oop = (z.OP_MAX, oracle.OP_MAX) if op == "max" else (z.OP_MIN, oracle.OP_MIN)
    a, b = fields.smooth_1d(n, seed=11), fields.smooth_1d(n, seed=12)
    st, _ = oracle.compress(a, oracle.EB_REL, 1e-3)
    want, wrc, wraw = oracle.drc(st, local=b, flags=oop, want_raw=True)
    out = torch.empty(z.compress_bound(n), dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    raw = torch.empty(n, dtype=torch.float32, device="cuda")
    ctx.decompress_reduce_compress(dev(st), n, out, nb, local=dev(b), raw_out=raw, flags=zop)
    assert ctx.status() == wrc
    assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
    assert_same_bits(raw.cpu().numpy(), wraw)


@pytest.mark.parametrize("op", ["max", "min", "avg"])
@pytest.mark.parametrize("N,n", [(3, 10_001), (8, 8 * 4096 * 2 + 5)])
def test_allreduce_other_operations_match_oracle(z, ctx, op, N, n):
    zop = dict(max=z.OP_MAX, min=z.OP_MIN, avg=z.OP_AVG)[op]
    oop = dict(max=oracle.OP_MAX, min=oracle.OP_MIN, avg=oracle.OP_AVG)[op]
    send = [fields.smooth_1d(n, seed=210 + r) for r in range(N)]
    want, wrc, whop = oracle.sim_allreduce(send, oracle.EB_REL, 1e-3, flags=oop, want_hop_bytes=True)
    got, rc, sizes = _run_allreduce(z, ctx, send, z.EB_REL, 1e-3, flags=zop)
    assert rc == wrc
    for r in range(N):
        assert_same_bits(got[r], want[r])
    assert np.array_equal(sizes.reshape(N, N), whop)


def test_collectives_with_more_jobs_than_a_launch_holds(z):
    # 12 ranks: 132 decode jobs per collective, more than the 64 chunk-operations one launch takes, so the batches are
    # cut in the middle of a rank's chunks; tile counts per chunk differ (ragged last chunk)
    N, n = 12, 12 * 3000 + 7
    c = z.Context(1 << 20, N)
    send = [fields.smooth_1d(n, seed=400 + r) for r in range(N)]
    want, wrc, whop = oracle.sim_allreduce(send, oracle.EB_REL, 1e-3, want_hop_bytes=True)
    d_send = [dev(a) for a in send]
    d_recv = [torch.zeros_like(t) for t in d_send]
    c.sim_allreduce(d_send, d_recv, z.EB_REL, 1e-3)
    assert c.status() == wrc
    for r in range(N):
        assert_same_bits(d_recv[r].cpu().numpy(), want[r])
    assert np.array_equal(np.array(c.sim_sizes()).reshape(N, N), whop)
    m = 5000
    send = [fields.smooth_1d(m, seed=500 + r) for r in range(N)]
    want, wrc, wsizes = oracle.sim_allgather(send, oracle.EB_REL, 1e-3)
    d_recv = [torch.zeros(N * m, dtype=torch.float32, device="cuda") for _ in range(N)]
    c.sim_allgather([dev(a) for a in send], d_recv, z.EB_REL, 1e-3)
    assert c.status() == wrc
    for r in range(N):
        assert_same_bits(d_recv[r].cpu().numpy(), want[r])
    c.close()


def test_step_replayed_from_a_cuda_graph(z):
    # every entry point only enqueues work on its stream, so a whole step (relative-bound compress with its range
    # pass, decompress, fused hop, ring Allreduce) can be captured once and replayed: same bytes as the oracle
    c = z.Context(1 << 20, 4)
    n, N = 4 * 4096 * 3 + 40, 4
    x, loc = fields.smooth_1d(n, seed=61), fields.smooth_1d(n, seed=62)
    send = [fields.smooth_1d(n, seed=63 + r) for r in range(N)]
    dx, dl = dev(x), dev(loc)
    d_send = [dev(a) for a in send]
    d_recv = [torch.zeros_like(t) for t in d_send]
    cap = z.compress_bound(n)
    out = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    out2 = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    nb2 = torch.zeros(1, dtype=torch.int64, device="cuda")
    y = torch.zeros(n, dtype=torch.float32, device="cuda")

    def step():
        c.compress(dx, z.EB_REL, 1e-3, out, nb)
        c.decompress(out, y)
        c.decompress_reduce_compress(out, n, out2, nb2, local=dl)
        c.sim_allreduce(d_send, d_recv, z.EB_REL, 1e-3)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                   # first calls set kernel attributes: outside the capture
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            step()
    torch.cuda.synchronize()
    want, wrc = oracle.compress(x, oracle.EB_REL, 1e-3)
    want2, _ = oracle.drc(want, local=loc)
    want3, _ = oracle.sim_allreduce(send, oracle.EB_REL, 1e-3)
    for _ in range(3):
        for t in (out, out2, y, nb, nb2, *d_recv):
            t.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert c.status() == wrc
        assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
        assert_same_bits(y.cpu().numpy(), oracle.decompress(want))
        assert np.array_equal(out2[: int(nb2.item())].cpu().numpy(), want2)
        for r in range(N):
            assert_same_bits(d_recv[r].cpu().numpy(), want3[r])
    c.close()


def test_range_and_scale_steps_of_a_real_rank(z, ctx):
    """zccl_range against numpy's min and max (any order of comparisons gives the same two values) and zccl_scale
    against one fp32 division per element."""
    for n in (1, 5, 4097, 1_000_003):
        a = fields.smooth_1d(n, seed=n % 97)
        x = dev(a)
        mm = torch.zeros(2, dtype=torch.float32, device="cuda")
        ctx.range(x, mm)
        got = mm.cpu().numpy()
        assert got[0] == a.min() and got[1] == a.max()
        y = x.clone()
        ctx.scale(y, 7.0)
        np.testing.assert_array_equal(y.cpu().numpy(), a / np.float32(7.0))
    mm = torch.zeros(2, dtype=torch.float32, device="cuda")
    ctx.range(torch.zeros(0, dtype=torch.float32, device="cuda"), mm)
    assert mm.cpu().numpy().tolist() == [np.inf, -np.inf]
    # the keys are re-armed: a second call sees only its own data
    ctx.range(torch.full((10,), 3.0, device="cuda"), mm)
    assert mm.cpu().numpy().tolist() == [3.0, 3.0]
    with pytest.raises(z.ZcclError):
        ctx.scale(torch.ones(4, device="cuda"), 0.0)


@pytest.mark.parametrize("n,eb", [(1, 1e-3), (37, 1e-3), (4096 * 5 + 77, 1e-2), (300_000, 1e-3), (300_000, 1e-5)])
def test_stream_stats_match_oracle(z, ctx, n, eb):
    x = fields.smooth_1d(n, seed=n % 89)
    if n > 1000:
        x[n // 3: n // 3 + 900] += np.random.default_rng(n).normal(0, 0.2, 900).astype(f32)
    st, _ = oracle.compress(x, oracle.EB_ABS, eb)
    hist = torch.full((33,), -1, dtype=torch.int64, device="cuda")
    ctx.stream_stats(dev(st), hist)
    assert ctx.status() == z.OK
    assert np.array_equal(hist.cpu().numpy().astype(np.uint64), oracle.stream_stats(st))


def test_stream_stats_constant_and_damaged(z, ctx):
    x = np.full(10_000, -3.0, f32)
    st, _ = oracle.compress(x, oracle.EB_ABS, 1e-2)
    hist = torch.zeros(33, dtype=torch.int64, device="cuda")
    ctx.stream_stats(dev(st), hist)
    assert ctx.status() == z.OK
    h = hist.cpu().numpy()
    assert h[0] == h[32] == -(-10_000 // 32) and h[1:32].sum() == 0
    bad = st.copy()
    bad[32 + 4 * 3 - 1] = 0xFF                     # last index entry far beyond the stream
    ctx.stream_stats(dev(bad), hist)
    assert ctx.status() == z.E_BAD_STREAM
    y = x.copy()
    y[5000] = 4.0
    st2, _ = oracle.compress(y, oracle.EB_ABS, 1e-2)
    bad2 = st2.copy()
    nT = 3
    first_L = 32 + 4 * nT + 4                      # first tile: outlier word, then the code-length bytes
    bad2[first_L] = 77
    ctx.stream_stats(dev(bad2), hist)
    assert ctx.status() == z.E_BAD_STREAM


# ----------------------------------------------------------------------------- other tile sizes

def _tiled_case(z, ctx, x, mode, eb, T):
    want, wrc = oracle.compress(x, mode, eb, T)
    out = torch.full((z.compress_bound_tiled(x.size, T) + 64,), 0xCD, dtype=torch.uint8, device="cuda")
    cap = out.numel() - 64
    nb = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress_tiled(dev(x), mode, eb, T, out[:cap], nb)
    assert ctx.status() == wrc
    got = out[: int(nb.item())].cpu().numpy()
    assert got.size == want.size and np.array_equal(got, want)
    assert bool((out[cap:] == 0xCD).all())
    y = torch.full((x.size + 16,), 7.0, dtype=torch.float32, device="cuda")
    ctx.decompress_tiled(dev(want), T, y[: x.size])
    assert ctx.status() == z.OK
    assert_same_bits(y[: x.size].cpu().numpy(), oracle.decompress(want))
    assert bool((y[x.size:] == 7.0).all())
    return want


@pytest.mark.parametrize("T", [5120, 1024, 8192, 4096, 4128])
@pytest.mark.parametrize("n", [1, 33, 5119, 5120, 5121, 3 * 5120 + 77, 200_001])
def test_other_tile_sizes_match_oracle(z, ctx, T, n):
    # Section 3.5.2: chunks of 5120 points; the tile size is a header field, the oracle takes any
    x = fields.smooth_1d(n, seed=T % 97 + n % 13)
    if n > 3000:
        x[n // 2: n // 2 + 1500] += np.random.default_rng(n).normal(0, 0.4, 1500).astype(f32)
    _tiled_case(z, ctx, x, z.EB_REL if n > 1 else z.EB_ABS, 1e-3, T)
    _tiled_case(z, ctx, x, z.EB_ABS, 3e-6, T)       # long codes, precision warning on the larger arrays


@pytest.mark.parametrize("T", [5120, 1024, 7168, 4128])
def test_other_tile_sizes_many_groups_and_alignments(z, T):
    """Hundreds of tiles (several groups of 32 in the placement), wide and narrow code lengths side by side, input and
    output on and off a 16-byte boundary; at T = 4128 the first array (5 rounds per tile of 4128 elements) is too large
    for the context's round slots and goes to the plain kernels."""
    c = z.Context(1 << 21, 0)
    try:
        for n, shift in ((1 << 21, 0), ((1 << 20) + 4321, 1), (900_000, 3)):
            x = fields.fourier_field_3d(128, seed=T % 7)[:n].copy()
            x[n // 3: n // 3 + 70_000] += np.random.default_rng(T).normal(0, 0.3, 70_000).astype(f32)
            want, wrc = oracle.compress(x, oracle.EB_REL, 1e-4, T)
            buf = torch.empty(n + 4, dtype=torch.float32, device="cuda")
            dx = buf[shift: shift + n]
            dx.copy_(torch.from_numpy(x))
            out = torch.empty(z.compress_bound_tiled(n, T), dtype=torch.uint8, device="cuda")
            nb = torch.zeros(1, dtype=torch.int64, device="cuda")
            c.compress_tiled(dx, z.EB_REL, 1e-4, T, out, nb)
            assert c.status() == wrc
            assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
            ybuf = torch.full((n + 4,), 7.0, dtype=torch.float32, device="cuda")
            c.decompress_tiled(out[: int(nb.item())], T, ybuf[shift: shift + n])
            assert c.status() == z.OK
            assert_same_bits(ybuf[shift: shift + n].cpu().numpy(), oracle.decompress(want))
            assert bool((ybuf[:shift] == 7.0).all()) and bool((ybuf[shift + n:] == 7.0).all())
    finally:
        c.close()


def test_plain_kernels_forced_by_the_environment():
    """ZCCL_PLAIN=1 keeps other tile sizes and binary64 on the plain kernels (the fallback when a context's round slots
    do not cover an input): the same streams and values, checked in a process of its own because the switch is read
    once."""
    import os
    import subprocess
    import sys
    code = r"""
import numpy as np, torch
import oracle
from paper_2502_18554_b200 import fields, zccl as z
c = z.Context(1 << 20, 0)
nb = torch.zeros(1, dtype=torch.int64, device="cuda")
for T, n in ((5120, 300_001), (1024, 70_000), (8192, 5)):
    x = fields.smooth_1d(n, seed=T % 11)
    want, wrc = oracle.compress(x, oracle.EB_REL if n > 1 else oracle.EB_ABS, 1e-3, T)
    out = torch.empty(z.compress_bound_tiled(n, T), dtype=torch.uint8, device="cuda")
    c.compress_tiled(torch.from_numpy(x).cuda(), z.EB_REL, 1e-3, T, out, nb)
    assert c.status() == wrc and np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
    y = torch.empty(n, dtype=torch.float32, device="cuda")
    c.decompress_tiled(out[: int(nb.item())], T, y)
    assert c.status() == z.OK and np.array_equal(y.cpu().numpy().view(np.uint32), oracle.decompress(want).view(np.uint32))
x = fields.smooth_1d(200_003, seed=3).astype(np.float64) * (1 + 1e-12)
want = oracle.compress_f64(x, oracle.EB_ABS, 1e-7)
out = torch.empty(z.compress_bound(x.size), dtype=torch.uint8, device="cuda")
c.compress_f64(torch.from_numpy(x).cuda(), z.EB_ABS, 1e-7, out, nb)
assert c.status() == z.OK and np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
y = torch.empty(x.size, dtype=torch.float64, device="cuda")
c.decompress_f64(out[: int(nb.item())], y)
assert c.status() == z.OK and np.array_equal(y.cpu().numpy().view(np.uint64), oracle.decompress_f64(want).view(np.uint64))
print("launches", z.launch_count())
"""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, ZCCL_PLAIN="1", PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600, cwd=root)
    assert r.returncode == 0, r.stdout + r.stderr
    # three launches per compression and one per decompression on the plain kernels, plus a range pass per relative bound
    assert "launches 19" in r.stdout, r.stdout


def test_tile_4096_streams_of_both_routes_are_the_same(z, ctx):
    x = fields.fourier_field_3d(64, seed=5)
    a = _tiled_case(z, ctx, x, z.EB_REL, 1e-3, 4096)
    b, _ = gpu_compress(z, ctx, x, z.EB_REL, 1e-3)
    assert np.array_equal(a, b)


def test_other_tile_sizes_errors(z, ctx):
    x = fields.smooth_1d(30_000, seed=8)
    want, _ = oracle.compress(x, oracle.EB_REL, 1e-3, 5120)
    out = torch.full((want.size + 64,), 0xCD, dtype=torch.uint8, device="cuda")
    nb = torch.ones(1, dtype=torch.int64, device="cuda")
    ctx.compress_tiled(dev(x), z.EB_REL, 1e-3, 5120, out[: want.size - 8], nb)      # too small: nothing is written
    assert ctx.status() == z.E_CAPACITY
    assert int(nb.item()) == 0 and bool((out == 0xCD).all())
    with pytest.raises(z.ZcclError):
        ctx.compress_tiled(dev(x), z.EB_REL, 1e-3, 5000, out, nb)                   # not a multiple of 32
    with pytest.raises(z.ZcclError):
        ctx.compress_tiled(dev(x), z.EB_REL, 1e-3, 512, out, nb)                    # below the supported range
    y = torch.zeros(x.size, dtype=torch.float32, device="cuda")
    ctx.decompress_tiled(dev(want), 4096, y)                                        # the header says 5120
    assert ctx.status() == z.E_BAD_STREAM
    ctx.decompress(dev(want), y)                                                    # the tuned decoder is for 4096
    assert ctx.status() == z.E_BAD_STREAM
    ctx.decompress_tiled(dev(want), 5120, y[:100])                                  # output too small
    assert ctx.status() == z.E_CAPACITY
    bad = want.copy()
    bad[32 + 4 * 6 + 4] = 40                                                        # a code length above 31
    ctx.decompress_tiled(dev(bad), 5120, y)
    assert ctx.status() == z.E_BAD_STREAM
    const = np.full(9000, 1.25, f32)
    ctx.compress_tiled(dev(const), z.EB_REL, 1e-3, 5120, out, nb)                   # no range to relate the bound to
    assert ctx.status() == z.E_DEGENERATE and int(nb.item()) == 0


# ----------------------------------------------------------------------------- one-wave launches of the fused hop

def test_fused_hop_launches_that_fit_the_device_at_once(z, ctx):
    """A fused launch of more tiles than the persistent kernel holds at once (3 CTAs per SM) but not more than the
    compact instance does (4 per SM) runs as one tile per CTA; the streams must not depend on which instance ran."""
    props = torch.cuda.get_device_properties(0)
    sms = props.multi_processor_count
    for tiles in (3 * sms + 1, 3 * sms + sms // 2, 4 * sms):
        n = tiles * 4096 - 1000                      # ragged last tile
        if n > ctx.max_elems:
            pytest.skip("context too small for this device")
        a = fields.smooth_1d(n, seed=tiles % 50)
        b = fields.smooth_1d(n, seed=tiles % 50 + 1)
        sa, _ = oracle.compress(a, oracle.EB_REL, 1e-3)
        want, wrc, wraw = oracle.drc(sa, local=b, want_raw=True)
        got, rc, raw = _drc_gpu(z, ctx, sa, n, local=b, raw=True)
        assert rc == wrc
        assert np.array_equal(got, want)
        assert_same_bits(raw, wraw)


def test_allreduce_whose_hops_fit_the_device_at_once(z):
    """8 ranks x 8 MiB: every reduce-scatter hop is 8 jobs of 64 tiles = 512 tiles in one launch."""
    N, n = 8, 1 << 21
    c = z.Context(n, N)
    send = fields.rank_fields(N, n, base_seed=300, kind="smooth")
    want, wrc = oracle.sim_allreduce(send, oracle.EB_REL, 1e-3)
    recv = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(N)]
    c.sim_allreduce([dev(a) for a in send], recv, z.EB_REL, 1e-3)
    assert c.status() == wrc
    for r in range(N):
        assert_same_bits(recv[r].cpu().numpy(), want[r])
    c.close()


def test_resolve_range_on_the_device(z, ctx):
    """zccl_resolve_range + ZCCL_EB_RESOLVED give the stream a relative bound over the combined range gives: the pair
    is put together from two arrays' pairs on the device, as two ranks of a ring would, and the oracle resolves the
    same bound from the concatenated data."""
    a = fields.smooth_1d(50_000, seed=3)
    b = (fields.smooth_1d(50_000, seed=4) * np.float32(1.7)).astype(np.float32)
    xa, xb = dev(a), dev(b)
    ma = torch.zeros(2, dtype=torch.float32, device="cuda")
    mb = torch.zeros(2, dtype=torch.float32, device="cuda")
    ctx.range(xa, ma)
    ctx.range(xb, mb)
    mm = torch.stack([torch.minimum(ma[0], mb[0]), torch.maximum(ma[1], mb[1])])
    ea_dev = torch.zeros(1, dtype=torch.float32, device="cuda")
    ctx.resolve_range(mm, 1e-3, ea_dev)
    ea, s, r = oracle.resolve(oracle.EB_REL, 1e-3, np.concatenate([a, b]))
    for arr, x in ((a, xa), (b, xb)):     # the block keeps its contents from call to call
        cap = z.compress_bound(arr.size)
        out = torch.empty(cap, dtype=torch.uint8, device="cuda")
        nb = torch.zeros(1, dtype=torch.int64, device="cuda")
        ctx.compress(x, z.EB_RESOLVED, 0.0, out, nb)
        assert ctx.check() in (z.OK, z.W_PRECISION)
        want, _ = oracle.compress_core(arr, ea, s, r)
        assert np.array_equal(out[: int(nb.item())].cpu().numpy(), want)
    assert np.float32(ea_dev.item()) == np.float32(ea)
    # a pair without extent: the device reports it, nothing is written
    ctx.resolve_range(torch.tensor([2.0, 2.0], device="cuda"), 1e-3, ea_dev)
    out = torch.empty(z.compress_bound(a.size), dtype=torch.uint8, device="cuda")
    nb = torch.ones(1, dtype=torch.int64, device="cuda")
    ctx.compress(xa, z.EB_RESOLVED, 0.0, out, nb)
    assert ctx.status() == z.E_DEGENERATE
    assert int(nb.item()) == 0 and float(ea_dev.item()) == 0.0
    with pytest.raises(z.ZcclError):
        ctx.resolve_range(mm, 0.0)


def test_two_contexts_on_two_streams_run_hops_side_by_side(z):
    """Fused hops of two contexts enqueued on two streams without any ordering between them: whichever share of the
    device each launch gets, and in whichever order their blocks run, both results are the oracle's.  (No block of
    the hop's launches waits for another block, so there is nothing for co-scheduling to break.)"""
    n = 3_000_000
    ctxs = [z.Context(n, 0), z.Context(n, 0)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    cases = []
    for k in range(2):
        a = fields.smooth_1d(n, seed=10 + k)
        b = fields.smooth_1d(n, seed=20 + k)
        ea, s, r = oracle.resolve(oracle.EB_REL, 1e-3, np.concatenate([a, b]))
        sa, _ = oracle.compress_core(a, ea, s, r)
        want, _, wraw = oracle.drc(sa, local=b, want_raw=True)
        cap = z.compress_bound(n)
        cases.append(dict(sa=torch.from_numpy(sa.copy()).cuda(), b=dev(b), want=want, wraw=wraw,
                          out=[torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(6)],
                          nb=[torch.zeros(1, dtype=torch.int64, device="cuda") for _ in range(6)],
                          raw=[torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(6)]))
    torch.cuda.synchronize()
    for rep in range(6):                      # interleaved enqueues: the launches of the two streams overlap on the device
        for k in range(2):
            c = cases[k]
            with torch.cuda.stream(streams[k]):
                ctxs[k].decompress_reduce_compress(c["sa"], n, c["out"][rep], c["nb"][rep], local=c["b"], raw_out=c["raw"][rep],
                                                   stream=streams[k])
    torch.cuda.synchronize()
    for k in range(2):
        assert ctxs[k].check() in (z.OK, z.W_PRECISION)
        c = cases[k]
        for rep in range(6):
            got = c["out"][rep][: int(c["nb"][rep].item())].cpu().numpy()
            assert np.array_equal(got, c["want"])
            assert_same_bits(c["raw"][rep].cpu().numpy(), c["wraw"])


def test_launches_from_several_threads(z):
    """Four host threads, each with a context and a stream of its own, compress and decompress at the same time: the
    launchers share no mutable state, so every thread gets the oracle's stream."""
    import threading
    n = 400_000
    arrs = [fields.smooth_1d(n, seed=30 + k) for k in range(4)]
    wants = [oracle.compress(a, oracle.EB_ABS, 1e-3)[0] for a in arrs]
    errors = []

    def work(k):
        try:
            torch.cuda.set_device(0)
            st = torch.cuda.Stream()
            ctx = z.Context(n, 0)
            x = torch.from_numpy(arrs[k]).cuda()
            cap = z.compress_bound(n)
            for _ in range(8):
                out = torch.empty(cap, dtype=torch.uint8, device="cuda")
                nb = torch.zeros(1, dtype=torch.int64, device="cuda")
                y = torch.empty(n, dtype=torch.float32, device="cuda")
                with torch.cuda.stream(st):
                    ctx.compress(x, z.EB_ABS, 1e-3, out, nb, stream=st)
                    ctx.decompress(out, y, stream=st)
                st.synchronize()
                if ctx.check(stream=st) not in (z.OK, z.W_PRECISION):
                    errors.append((k, "status"))
                if not np.array_equal(out[: int(nb.item())].cpu().numpy(), wants[k]):
                    errors.append((k, "stream"))
                if not np.array_equal(y.cpu().numpy(), oracle.decompress(wants[k])):
                    errors.append((k, "values"))
        except Exception as exc:   # a thread's exception must fail the test
            errors.append((k, repr(exc)))

    threads = [threading.Thread(target=work, args=(k,)) for k in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


@pytest.mark.parametrize("tiles", [3, 40, 200, 700])
def test_large_blobs_are_staged_a_window_at_a_time(z, ctx, tiles):
    """Tiles whose blobs are larger than a 4 KiB staging buffer (code lengths 9 to 24, up to 12 KiB per tile): the
    decoder and the hop move a window over them; few tiles make the hop start its warps inside tiles (units of one or
    two rounds, which skip over the rounds in front through the window), many make it take whole tiles.  Both operands
    compressed as well (the second one is read in place)."""
    n = tiles * 4096 - 777
    rng = np.random.default_rng(tiles)
    scale = np.repeat(10.0 ** rng.uniform(-0.5, 4.0, (n + 1023) // 1024), 1024)[:n]      # the code length changes from round to round
    a = (rng.standard_normal(n) * scale).astype(np.float32)
    b = (rng.standard_normal(n) * scale[::-1]).astype(np.float32)
    ea, s, r = oracle.resolve(oracle.EB_ABS, 2e-3)
    sa, _ = oracle.compress_core(a, ea, s, r)
    assert sa.size > 1.5 * 4096 * tiles                                                 # blobs above the buffer on average
    got_y, rcd = gpu_decompress(z, ctx, sa, n)
    assert rcd == z.OK
    assert_same_bits(got_y, oracle.decompress(sa))
    want, wrc, wraw = oracle.drc(sa, local=b, want_raw=True)
    got, rc, raw = _drc_gpu(z, ctx, sa, n, local=b, raw=True)
    assert rc == wrc and np.array_equal(got, want)
    assert_same_bits(raw, wraw)
    sb, _ = oracle.compress_core(b, ea, s, r)
    want2, wrc2 = oracle.drc(sa, local_c=sb)
    got2, rc2, _ = _drc_gpu(z, ctx, sa, n, local_c=sb)
    assert rc2 == wrc2 and np.array_equal(got2, want2)
    # and the compressor on the same data
    st, rcc = gpu_compress(z, ctx, a, z.EB_ABS, 2e-3)
    assert np.array_equal(st, sa)
