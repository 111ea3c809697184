"""The allocation-free compressor (zccl_compress_noalloc), through the C-ABI, against the context-based entry
point it mirrors and against the CPU oracle.  Some callers of this library cannot allocate device memory (work captured into a CUDA graph,
plug-ins with a fixed memory budget, out-of-memory handlers), so they cannot create a context; this entry point
keeps its scan workspace in a fixed array inside the library instead.  The array is shared by all calls and keeps
the previous call's contents, hence the check on two calls in a row with different inputs.

Collected last on purpose: if it fails, a run that stops at the first failure has already run every other test."""
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


def _reference_stream(z, ctx, dx, eb_abs):
    out = torch.empty(z.compress_bound(dx.numel()), dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    ctx.compress(dx, z.EB_ABS, eb_abs, out, nbytes)
    assert ctx.status() >= 0
    return out[: int(nbytes.item())].cpu().numpy()


def test_noalloc_matches_context_entry_point_on_two_calls_in_a_row(z):
    ctx = z.Context(1 << 21, 0)
    cases = [(fields.smooth_1d(300_000 + 77, seed=5), 2e-3),          # 74 tiles, ragged tail
             (fields.gradient_like(123_457, seed=6), 1e-5)]           # different data, size and bound right after
    for x, eb in cases + cases[:1]:
        dx = torch.from_numpy(x).cuda()
        want = _reference_stream(z, ctx, dx, eb)
        out = torch.full((z.compress_bound(x.size) + 64,), 0xEE, dtype=torch.uint8, device="cuda")
        nbytes = torch.full((1,), -1, dtype=torch.int64, device="cuda")
        rc = z.compress_noalloc(dx, eb, out[: z.compress_bound(x.size)], nbytes)
        assert rc == z.OK
        torch.cuda.synchronize()
        got = out[: int(nbytes.item())].cpu().numpy()
        assert got.size == want.size
        assert np.array_equal(got, want)                              # same bytes as zccl_compress
        assert np.array_equal(got, oracle.compress(x, oracle.EB_ABS, eb)[0])   # and as the CPU oracle
        assert bool((out[z.compress_bound(x.size):] == 0xEE).all())   # nothing written past the capacity
    ctx.close()


def test_noalloc_rejects_what_it_cannot_place(z):
    x = torch.zeros(1000, dtype=torch.float32, device="cuda")
    out = torch.empty(z.compress_bound(1000), dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    assert z.compress_noalloc(x, 1e-3, out, nbytes, n=z.NOALLOC_MAX_ELEMS + 1) == z.E_TOO_LARGE   # nothing enqueued
    assert z.compress_noalloc(x, 0.0, out, nbytes) == z.E_ARG
    assert z.compress_noalloc(x, 1e-3, out[:16], nbytes) == z.E_CAPACITY
    # a device-side error (capacity overrun) is reported as a zero length
    y = torch.from_numpy(fields.smooth_1d(50_000, seed=9)).cuda()
    small = torch.empty(32 + 4 * 13 + 64, dtype=torch.uint8, device="cuda")
    assert z.compress_noalloc(y, 1e-4, small, nbytes) == z.OK
    torch.cuda.synchronize()
    assert int(nbytes.item()) == 0
    # and the next call is unaffected by it
    big = torch.empty(z.compress_bound(50_000), dtype=torch.uint8, device="cuda")
    assert z.compress_noalloc(y, 1e-4, big, nbytes) == z.OK
    torch.cuda.synchronize()
    assert int(nbytes.item()) > 32


def test_noalloc_inside_a_captured_graph(z):
    # the case the entry point exists for: after one call outside any capture (which resolves the array's address),
    # a call is captured into a CUDA graph and replayed; every replay produces the context entry point's bytes
    ctx = z.Context(1 << 20, 0)
    x = fields.smooth_1d(150_000 + 5, seed=15)
    eb = 1e-3
    dx = torch.from_numpy(x).cuda()
    want = _reference_stream(z, ctx, dx, eb)
    cap = z.compress_bound(x.size)
    out = torch.zeros(cap, dtype=torch.uint8, device="cuda")
    nbytes = torch.zeros(1, dtype=torch.int64, device="cuda")
    assert z.compress_noalloc(dx, eb, out, nbytes) == z.OK          # first call: outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            assert z.compress_noalloc(dx, eb, out, nbytes) == z.OK
    torch.cuda.synchronize()
    for _ in range(3):
        out.zero_()
        nbytes.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(out[: int(nbytes.item())].cpu().numpy(), want)
    ctx.close()
