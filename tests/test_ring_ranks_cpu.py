"""The real-rank collectives (paper_2502_18554_b200.ring) as gloo processes on CPU.  The codec steps are taken by
the oracle here (a host stand-in with the methods of DeviceCodec), so what these tests check is everything around
them: which chunk meets which at which hop, the split into pieces, the byte counts and payloads that cross between
the ranks, the bound resolved once over all ranks' data, the binomial tree.  The expected values are those of the
oracle's own emulated collectives (Sections 3.1.1, 3.1.2, 3.2)."""
import os
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


class HostCodec:
    """Oracle-backed codec on host tensors, for tests only."""

    def __init__(self):
        import oracle
        self.o = oracle
        self.device = torch.device("cpu")

    def bound(self, n):
        return self.o.compress_bound(n)

    def minmax(self, x):
        a = x.numpy()
        return torch.tensor([a.min(), a.max()], dtype=torch.float32) if a.size else torch.tensor([np.inf, -np.inf])

    def _put(self, stream, out, out_bytes):
        out[: stream.size] = torch.from_numpy(stream)
        out_bytes[0] = stream.size

    def compress(self, x, eb_abs, out, out_bytes):
        ea, s, r = self.o.resolve(self.o.EB_ABS, eb_abs)
        stream, _ = self.o.compress_core(x.numpy(), ea, s, r)
        self._put(stream, out, out_bytes)

    def drc(self, in_c, n, local, out, out_bytes, raw_out, flags):
        res = self.o.drc(in_c.numpy(), local=local.numpy(), flags=flags, want_raw=raw_out is not None)
        self._put(res[0], out, out_bytes)
        if raw_out is not None:
            raw_out.copy_(torch.from_numpy(res[2]))

    def decompress(self, in_c, y):
        y.copy_(torch.from_numpy(self.o.decompress(in_c.numpy())))

    def scale(self, y, divisor):
        y.copy_(torch.from_numpy(y.numpy() / np.float32(divisor)))

    def finish(self):
        return 0


def _inputs(world, n):
    from paper_2502_18554_b200 import fields
    return [fields.smooth_1d(n, seed=40 + r) * np.float32(1 + r) for r in range(world)]


def _worker(rank, world, port, n, segments, transport, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, str(ROOT))
    try:
        import oracle
        from paper_2502_18554_b200 import ring, zccl as z
        dist.init_process_group("gloo", rank=rank, world_size=world)
        xs = _inputs(world, n)
        x = torch.from_numpy(xs[rank].copy())
        R = ring.Ring(n * world, codec=HostCodec(), segments=segments, transport=transport)
        res = {}
        out = torch.zeros(n)
        R.allreduce(x, out, z.EB_REL, 1e-3)
        res["allreduce"] = (out.numpy().copy(), R.sent_bytes)
        out = torch.zeros(n)
        R.allreduce(x, out, z.EB_ABS, 2e-3, flags=z.OP_AVG | z.CONSISTENT_OWNER)
        res["allreduce_avg"] = (out.numpy().copy(), R.sent_bytes)
        out = torch.zeros(ring.chunk_span(n, world, rank)[1])
        R.reduce_scatter(x, out, z.EB_REL, 1e-3)
        res["reduce_scatter"] = (out.numpy().copy(), R.sent_bytes)
        out = torch.zeros(world * n)
        R.allgather(x, out, z.EB_REL, 1e-2)
        res["allgather"] = (out.numpy().copy(), R.sent_bytes)
        root = world - 1
        xb = torch.from_numpy(xs[root].copy()) if rank == root else torch.zeros(n)
        R.bcast(xb, root, z.EB_REL, 1e-3)
        res["bcast"] = (xb.numpy().copy(), R.sent_bytes)
        q.put((rank, res, None))
        dist.barrier()
        dist.destroy_process_group()
    except Exception as e:                          # the parent must not wait for a rank that died
        import traceback
        q.put((rank, None, traceback.format_exc()))
        raise e


def _run(world, n, segments, transport):
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29700 + (os.getpid() * 7 + world * 13 + segments * 3 + len(transport)) % 900
    procs = [ctx.Process(target=_worker, args=(r, world, port, n, segments, transport, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = {}
    for _ in range(world):
        rank, res, err = q.get(timeout=300)
        assert err is None, err
        got[rank] = res
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    return got


@pytest.mark.parametrize("world,n,segments,transport", [(2, 20000, 1, "host"), (3, 20000, 2, "host"), (4, 9001, 3, "direct"),
                                                       (3, 2, 1, "host"), (2, 30000, 2, "direct"), (3, 20000, 1, "direct"),
                                                       (2, 5000, 8, "direct")])     # more pieces than tiles: empty pieces travel too
def test_real_rank_collectives_match_the_emulated_ones(world, n, segments, transport):
    """"direct" keeps the payload messages in flight behind the codec steps and waits for each where its data is
    needed (the bookkeeping an NCCL group runs with); "host" waits for every message where it is posted."""
    import oracle
    from paper_2502_18554_b200 import ring, zccl as z
    got = _run(world, n, segments, transport)
    xs = _inputs(world, n)

    exp, _ = oracle.sim_allreduce(xs, oracle.EB_REL, 1e-3)
    for r in range(world):
        np.testing.assert_array_equal(got[r]["allreduce"][0], exp[r])
    exp, _ = oracle.sim_allreduce(xs, oracle.EB_ABS, 2e-3, flags=oracle.OP_AVG | oracle.FLAG_CONSISTENT_OWNER)
    for r in range(world):
        np.testing.assert_array_equal(got[r]["allreduce_avg"][0], exp[r])
    exp, _, hop = oracle.sim_reduce_scatter(xs, oracle.EB_REL, 1e-3)
    for r in range(world):
        np.testing.assert_array_equal(got[r]["reduce_scatter"][0], exp[r])
    exp, _, sizes = oracle.sim_allgather(xs, oracle.EB_REL, 1e-2)
    for r in range(world):
        np.testing.assert_array_equal(got[r]["allgather"][0], exp[r])
    root = world - 1
    exp, _, stream_bytes = oracle.sim_bcast(xs[root], world - 1, oracle.EB_REL, 1e-3)
    for r in range(world):
        np.testing.assert_array_equal(got[r]["bcast"][0], xs[root] if r == root else exp[0])

    if segments == 1:
        # what crossed the links: with one piece per chunk the streams are the emulated ring's own
        # reduce-scatter: steps 0 .. N-2 of every rank are sent on (the last hop's output stays with its owner)
        for r in range(world):
            assert got[r]["reduce_scatter"][1] == int(hop[: world - 1, r].sum())
        # allgather: every rank sends its own stream and forwards N - 2 foreign ones: all streams but rank r+1's
        for r in range(world):
            assert got[r]["allgather"][1] == int(sizes.sum() - sizes[(r + 1) % world])
        # bcast over the binomial tree: N - 1 copies of the one stream cross in total
        assert sum(got[r]["bcast"][1] for r in range(world)) == (world - 1) * stream_bytes


def test_piece_spans_cover_a_chunk_in_whole_tiles():
    from paper_2502_18554_b200 import ring
    for length in (0, 1, 4095, 4096, 4097, 20000, 1 << 20):
        for S in (1, 2, 3, 7):
            sp = ring.piece_spans(length, S)
            assert len(sp) == S and sum(l for _, l in sp) == length
            pos = 0
            for off, l in sp:
                assert off == pos or l == 0
                pos += l
            assert all(l % ring.TILE == 0 for _, l in sp[:-1] if l and (_ + l) < length)
            assert max(l for _, l in sp) == sp[0][1]
    for n, N in ((10, 4), (4096 * 8, 8), (7, 8), (0, 3)):
        spans = [ring.chunk_span(n, N, c) for c in range(N)]
        assert sum(l for _, l in spans) == n and spans[0][1] == -(-n // N)
