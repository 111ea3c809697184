"""Compression-enabled collectives between real ranks: one process per GPU, `torch.distributed` for transport.

The schedules are those of the collective computation framework (Section 3.1.2, Figure 3: every hop of the
reduce-scatter stage decompresses the stream it received, combines it with the rank's own chunk and recompresses)
and of the collective data movement framework (Section 3.1.1: a contribution is compressed once, compressed bytes
travel, receivers decompress).  Every codec step is one call of the C boundary on the rank's own GPU; what crosses
the links are the compressed streams, with their byte counts sent ahead because the two sides of a message must
agree on its length.  The error bound is resolved once per collective over the data of all ranks (Section 3.2), so
the result on rank r equals what the emulated ring computes for rank r, bit for bit.

Overlap (the GPU analogue of polling the network between the chunks of the pipelined compressor, Section 3.5.2):
with `segments` = S > 1 every ring chunk is cut into S balanced pieces that are compressed, sent and reduced
independently, so that piece i is on the wire while piece i+1 is in the codec, and the next hop's work on piece i
starts as soon as it has arrived.  A remote stream always lands in this rank's memory before a kernel reads it.

The codec is an object with the methods of `DeviceCodec`; tests substitute one that works on host tensors, which is
how the schedules and the transport are checked without GPUs.
"""
from __future__ import annotations

import contextlib

import numpy as np
import torch
import torch.distributed as dist

from . import zccl as z

TILE = 4096


def chunk_span(n: int, N: int, c: int) -> tuple[int, int]:
    """Offset and length of ring chunk c: n elements in N chunks of ceil(n / N), the last ones shorter."""
    m = (n + N - 1) // N
    off = min(c * m, n)
    return off, min(m, n - off)


def piece_spans(length: int, S: int) -> list[tuple[int, int]]:
    """S balanced pieces of a chunk, every piece but the last a whole number of codec tiles.  Trailing pieces may
    be empty: an empty piece still travels, as a header-only stream, so that all ranks agree on the message count."""
    per = -(-length // S)
    per = -(-per // TILE) * TILE
    out = []
    for i in range(S):
        off = min(i * per, length)
        out.append((off, min(per, length - off)))
    return out


class DegenerateRange(ValueError):
    """A relative bound over data whose range is zero, infinite or not a number."""


RESOLVED = object()   # stands for "the bound the codec resolved on the device" where an absolute bound is expected


class DeviceCodec:
    """The per-rank codec steps on the rank's GPU; each method enqueues one call of the C boundary."""

    def __init__(self, max_elems: int):
        self.ctx = z.Context(max_elems, 1)          # raises when the library or the GPU is missing
        self.device = torch.device("cuda", torch.cuda.current_device())
        self._none = torch.zeros(1, dtype=torch.float32, device=self.device)   # operand of an empty piece

    def bound(self, n: int) -> int:
        return z.compress_bound(n)

    def minmax(self, x: torch.Tensor) -> torch.Tensor:
        out = torch.empty(2, dtype=torch.float32, device=self.device)
        self.ctx.range(x, out)
        return out

    def resolve(self, minmax: torch.Tensor, eb_rel: float):
        """The relative bound over a (min, max) pair that is on the device, resolved on the device: no value comes
        back to the host.  Returns the token that compress takes in place of an absolute bound."""
        self.ctx.resolve_range(minmax, eb_rel)
        return RESOLVED

    def compress(self, x, eb_abs, out, out_bytes):
        if eb_abs is RESOLVED:
            self.ctx.compress(x, z.EB_RESOLVED, 0.0, out, out_bytes)
        else:
            self.ctx.compress(x, z.EB_ABS, eb_abs, out, out_bytes)

    def drc(self, in_c, n: int, local, out, out_bytes, raw_out, flags: int):
        if n == 0:
            local, raw_out = self._none, None
        self.ctx.decompress_reduce_compress(in_c, n, out, out_bytes, local=local, raw_out=raw_out, flags=flags)

    def decompress(self, in_c, y):
        self.ctx.decompress(in_c, y)

    def scale(self, y, divisor: float):
        self.ctx.scale(y, divisor)

    def finish(self) -> int:
        """Waits for the enqueued work and raises on a device-side error; returns the warning code, if any."""
        try:
            return self.ctx.check()
        except z.ZcclError as exc:
            if exc.code == z.E_DEGENERATE:
                raise DegenerateRange("relative bound over data without a finite, non-zero range") from exc
            raise


class _Msg:
    """The outstanding work of one posted group.  With NCCL a wait makes the current stream wait, and two streams
    may each have to (the codec's and the one messages are issued from); elsewhere a wait blocks the host and is
    taken once."""

    def __init__(self, works, stream_side: bool):
        self.works, self.stream_side, self.done = works, stream_side, False

    def wait(self):
        if self.stream_side or not self.done:
            for w in self.works:
                w.wait()
            self.done = True


class _Link:
    """Point-to-point transport inside one process group.  NCCL moves device memory; any other backend is given
    the bytes in host memory."""

    def __init__(self, group, device: torch.device, transport: str = "auto"):
        self.group = group
        self.rank = dist.get_rank(group)
        self.N = dist.get_world_size(group)
        nccl = dist.get_backend(group) == "nccl"
        if transport not in ("auto", "direct", "host"):
            raise ValueError("transport must be auto, direct or host")
        # direct: the backend is handed the codec's own buffers and payloads stay in flight while the codec works;
        # host: payloads are copied to host memory and each message is waited for.  NCCL needs direct, a backend
        # that moves host memory only can be direct when the codec's buffers are host memory too.
        self.direct = nccl or transport == "direct" if transport != "host" else False
        if nccl and (device.type != "cuda" or transport == "host"):
            raise ValueError("an NCCL group needs the direct transport and a codec on a CUDA device")
        if self.direct and not nccl and device.type != "cpu":
            raise ValueError("this backend moves host memory only: use transport='host'")
        self.msg_device = device if self.direct else torch.device("cpu")
        # messages are issued from a stream of their own, so that a send waits for the piece it carries (the host
        # has seen that piece's event) and not for whatever else the codec stream has queued behind it
        self.comm_stream = torch.cuda.Stream(device) if nccl else None

    def peer(self, r: int) -> int:
        r %= self.N
        return dist.get_global_rank(self.group, r) if self.group is not None else r

    def issuing(self):
        return torch.cuda.stream(self.comm_stream) if self.comm_stream is not None else contextlib.nullcontext()

    def post(self, send, dst, recv, src):
        """One send (to dst) and one receive (from src) as a single group, either of which may be absent: a ring
        of two has the same peer on both sides, and a send must not wait behind it for the matching receive."""
        ops = []
        if dst is not None:
            ops.append(dist.P2POp(dist.isend, send, self.peer(dst), self.group))
        if src is not None:
            ops.append(dist.P2POp(dist.irecv, recv, self.peer(src), self.group))
        return [_Msg(dist.batch_isend_irecv(ops), self.comm_stream is not None)] if ops else []

    @staticmethod
    def wait(reqs):
        """For NCCL the current stream waits, not the host; other backends block until the message is through."""
        for q in reqs:
            q.wait()

    def swap_sizes(self, nbytes: int, dst, src) -> int:
        out = torch.tensor([nbytes], dtype=torch.int64, device=self.msg_device)
        inc = torch.zeros(1, dtype=torch.int64, device=self.msg_device)
        self.wait(self.post(out, dst, inc, src))
        return int(inc.item())

    def all_max(self, t: torch.Tensor) -> torch.Tensor:
        m = t.to(self.msg_device)
        dist.all_reduce(m, op=dist.ReduceOp.MAX, group=self.group)
        return m


class _Piece:
    """Buffers and outstanding work of one piece: two streams it produces in turn, two it receives in turn."""

    def __init__(self, codec, cap: int):
        dev = codec.device
        cuda = dev.type == "cuda"
        self.out = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(2)]
        self.inc = [torch.empty(cap, dtype=torch.uint8, device=dev) for _ in range(2)]
        self.out_bytes = torch.zeros(1, dtype=torch.int64, device=dev)
        self.host_bytes = torch.zeros(1, dtype=torch.int64, pin_memory=cuda)
        self.produced = torch.cuda.Event() if cuda else None
        self.inc_read = [None, None]      # event after the last kernel that reads inc[side]
        self.out_sends = [[], []]         # messages that read out[side]
        self.inc_sends = [[], []]         # messages that read inc[side] (forwarding)
        self.recvs = [[], []]             # message that writes inc[side]
        self.nin = [0, 0]


class Ring:
    """Ring Allreduce, Reduce-scatter and Allgather, binomial-tree Bcast, of fp32 arrays held one per rank.

    max_elems: largest array a collective will be given (sizes the codec's workspace).
    group:     process group (default: the world); its backend decides the transport.
    segments:  pieces per ring chunk (see the module text).
    transport: "auto" (direct for NCCL, through host memory otherwise), "direct" or "host"."""

    def __init__(self, max_elems: int, group=None, codec=None, segments: int = 1, transport: str = "auto"):
        if segments < 1:
            raise ValueError("segments must be at least 1")
        self.codec = codec if codec is not None else DeviceCodec(max_elems)
        self.link = _Link(group, self.codec.device, transport)
        self.rank, self.N = self.link.rank, self.link.N
        self.S = segments
        self.max_elems = max_elems
        self.sent_bytes = 0      # compressed bytes this rank put on the wire in the last collective

    # ------------------------------------------------------------------------------------------------ the bound

    def resolve(self, x: torch.Tensor, eb_mode: int, eb: float, collective: bool = True):
        """eb -> absolute bound.  A relative bound refers to the range of the data of all ranks (of x alone when
        `collective` is false): eb_abs = fl32(eb * fl32(max - min)).  A codec that can resolve on the device gets
        the combined (min, max) there and the host never waits for it (a range without extent then shows up as
        DegenerateRange when the collective finishes, on every rank alike); otherwise the host forms the bound."""
        if not (eb > 0) or not np.isfinite(eb):
            raise ValueError("the error bound must be a positive finite number")
        if eb_mode == z.EB_ABS:
            return float(np.float32(eb))
        if eb_mode != z.EB_REL:
            raise ValueError("eb_mode")
        mm = self.codec.minmax(x)
        t = torch.stack([-mm[0], mm[1]])
        if collective and self.N > 1:
            t = self.link.all_max(t)
        if hasattr(self.codec, "resolve"):
            pair = torch.stack([-t[0], t[1]]).to(mm.device)   # back on the codec's device when the messages go through the host
            return self.codec.resolve(pair, float(np.float32(eb)))
        rc, ea, _, _ = z.resolve_range_host(float(-t[0].item()), float(t[1].item()), float(np.float32(eb)))
        if rc != z.OK:
            raise DegenerateRange("relative bound over data without a finite, non-zero range")
        return ea

    # ------------------------------------------------------------------------------------------------ one message

    def _pieces(self, longest: int) -> list[_Piece]:
        cap = -(-self.codec.bound(piece_spans(longest, self.S)[0][1]) // 256) * 256
        return [_Piece(self.codec, cap) for _ in range(self.S)]

    @staticmethod
    def _mark_produced(p: _Piece):
        """After the codec call that wrote one of p.out and p.out_bytes."""
        p.host_bytes.copy_(p.out_bytes, non_blocking=True)
        if p.produced is not None:
            p.produced.record()

    @staticmethod
    def _produced_view(p: _Piece, side: int) -> torch.Tensor:
        """The stream in out[side]; the host waits for the codec call that produced it (it needs the length)."""
        if p.produced is not None:
            p.produced.synchronize()
        return p.out[side][: int(p.host_bytes.item())]

    def _exchange(self, p: _Piece, what, origin, dst, recv_side, src):
        """Sends the stream `what` to rank dst (origin = ("out", side) or ("inc", side): the buffer of p it lives
        in) and posts the receive of the next stream from rank src into p.inc[recv_side].  Either direction may be
        None.  Blocks the host for the exchange of the byte counts only; the payload stays in flight."""
        link = self.link
        ns = what.numel() if dst is not None else 0
        with link.issuing():
            nin = link.swap_sizes(ns, dst, src)
            if src is not None and nin > p.inc[recv_side].numel():
                raise RuntimeError(f"incoming stream of {nin} bytes exceeds the bound {p.inc[recv_side].numel()}")
            self.sent_bytes += ns
            if link.direct:
                if src is not None:       # the buffer to be overwritten: its last reader and its last forward
                    if p.inc_read[recv_side] is not None:
                        torch.cuda.current_stream().wait_event(p.inc_read[recv_side])
                    link.wait(p.inc_sends[recv_side])
                    p.inc_sends[recv_side] = []
                if dst is not None and origin[0] == "inc":
                    link.wait(p.recvs[origin[1]])         # forward only what has arrived
                reqs = link.post(what, dst, p.inc[recv_side][:nin] if src is not None else None, src)
            else:
                hs = what.cpu() if dst is not None else None
                hr = torch.empty(nin, dtype=torch.uint8) if src is not None else None
                link.wait(link.post(hs, dst, hr, src))
                if src is not None:
                    p.inc[recv_side][:nin].copy_(hr)
                reqs = []
        if dst is not None:
            sends = p.out_sends if origin[0] == "out" else p.inc_sends
            sends[origin[1]] = sends[origin[1]] + reqs
        if src is not None:
            p.recvs[recv_side] = reqs
            p.nin[recv_side] = nin

    def _incoming(self, p: _Piece, side: int) -> torch.Tensor:
        """The stream received into inc[side]; the codec stream waits for it, the host does not."""
        self.link.wait(p.recvs[side])
        return p.inc[side][: p.nin[side]]

    @staticmethod
    def _mark_read(p: _Piece, side: int):
        """After the codec call that read inc[side]."""
        if p.produced is not None:
            e = torch.cuda.Event()
            e.record()
            p.inc_read[side] = e

    def _before_overwrite_out(self, p: _Piece, side: int):
        self.link.wait(p.out_sends[side])
        p.out_sends[side] = []

    def _drain(self, pieces):
        """The caller's stream waits for every message still in flight."""
        for p in pieces:
            for side in (0, 1):
                self.link.wait(p.out_sends[side])
                self.link.wait(p.inc_sends[side])
                self.link.wait(p.recvs[side])

    # ------------------------------------------------------------------------------------------------ stages

    def _reduce_scatter_stage(self, x, n, ea, flags, shift, raw_of):
        """N - 1 fused hops.  At step 0 rank r compresses chunk r - shift; at hop k it receives chunk
        r - shift - k - 1 from rank r - 1, combines it with its own and recompresses; the last hop also writes the
        uncompressed result through raw_of(chunk, piece offset, piece length).  Returns the pieces and the side of
        p.out that holds the stream of the chunk this rank ends up owning."""
        N, r, S, codec = self.N, self.rank, self.S, self.codec
        pieces = self._pieces((n + N - 1) // N)
        off0, len0 = chunk_span(n, N, (r - shift) % N)
        side = 0
        for p, (po, pl) in zip(pieces, piece_spans(len0, S)):
            codec.compress(x[off0 + po: off0 + po + pl], ea, p.out[side], p.out_bytes)
            self._mark_produced(p)
        for k in range(N - 1):
            rs = k & 1
            for p in pieces:
                self._exchange(p, self._produced_view(p, side), ("out", side), r + 1, rs, r - 1)
            c = (r - shift - k - 1) % N
            off, length = chunk_span(n, N, c)
            for p, (po, pl) in zip(pieces, piece_spans(length, S)):
                inc = self._incoming(p, rs)
                self._before_overwrite_out(p, side ^ 1)
                codec.drc(inc, pl, x[off + po: off + po + pl], p.out[side ^ 1], p.out_bytes,
                          raw_of(c, po, pl) if k == N - 2 else None, flags)
                self._mark_produced(p)
                self._mark_read(p, rs)
            side ^= 1
        return pieces, side

    def _forward_stage(self, pieces, own, own_side, deliver):
        """N - 1 forwarding hops of compressed streams.  own[i]: this rank's stream of piece i, in out[own_side].  At hop h the rank
        sends on what it holds (its own at h = 0, else what it received at hop h - 1) and receives the stream that
        rank r - h - 1 put in; deliver(h, i, stream) enqueues its decompression."""
        r = self.rank
        for h in range(self.N - 1):
            rs = h & 1
            for i, p in enumerate(pieces):
                if h == 0:
                    self._exchange(p, own[i], ("out", own_side), r + 1, rs, r - 1)
                else:
                    self._exchange(p, p.inc[rs ^ 1][: p.nin[rs ^ 1]], ("inc", rs ^ 1), r + 1, rs, r - 1)
            for i, p in enumerate(pieces):
                deliver(h, i, self._incoming(p, rs))
                self._mark_read(p, rs)

    # ------------------------------------------------------------------------------------------------ collectives

    def _check(self, x, out, out_elems, what):
        if x.dtype != torch.float32 or out.dtype != torch.float32 or not x.is_contiguous() or not out.is_contiguous():
            raise ValueError(f"{what}: contiguous float32 tensors expected")
        if x.numel() > self.max_elems or out.numel() != out_elems:
            raise ValueError(f"{what}: sizes do not fit (x {x.numel()}, out {out.numel()}, expected {out_elems})")
        self.sent_bytes = 0

    def allreduce(self, x: torch.Tensor, out: torch.Tensor, eb_mode: int, eb: float, flags: int = 0) -> int:
        """out <- reduction over the ranks of x, element by element (Sum unless flags carry another operation).
        Ring reduce-scatter with fused hops, then a ring allgather of the reduced chunks' streams."""
        n, N, r, S, codec = x.numel(), self.N, self.rank, self.S, self.codec
        self._check(x, out, n, "allreduce")
        ea = self.resolve(x, eb_mode, eb)
        if N == 1:
            out.copy_(x)
            return codec.finish()

        def raw_of(c, po, pl):
            return out[chunk_span(n, N, c)[0] + po:][:pl]

        pieces, side = self._reduce_scatter_stage(x, n, ea, flags, 0, raw_of)

        def deliver(h, i, stream):          # the stream of the chunk that rank r - h - 1 owns: chunk r - h
            off, length = chunk_span(n, N, (r - h) % N)
            po, pl = piece_spans(length, S)[i]
            codec.decompress(stream, out[off + po: off + po + pl])

        self._forward_stage(pieces, [self._produced_view(p, side) for p in pieces], side, deliver)
        if (flags & z.OP_AVG) == z.OP_AVG:
            codec.scale(out, float(N))
        self._drain(pieces)
        return codec.finish()

    def reduce_scatter(self, x: torch.Tensor, out: torch.Tensor, eb_mode: int, eb: float, flags: int = 0) -> int:
        """out <- chunk r of the reduction over the ranks of x (chunks of ceil(n / N) elements).  The ring is
        shifted by one so that the last hop of chunk r ends on rank r, which keeps the uncompressed result."""
        n, N, r = x.numel(), self.N, self.rank
        self._check(x, out, chunk_span(n, N, r)[1], "reduce_scatter")
        ea = self.resolve(x, eb_mode, eb)
        if N == 1:
            out.copy_(x)
            return self.codec.finish()
        pieces, _ = self._reduce_scatter_stage(x, n, ea, flags, 1, lambda c, po, pl: out[po: po + pl])
        self._drain(pieces)
        return self.codec.finish()

    def allgather(self, x: torch.Tensor, out: torch.Tensor, eb_mode: int, eb: float) -> int:
        """out[q * n : (q + 1) * n] <- rank q's x.  Every contribution is compressed once; a rank keeps its own
        uncompressed."""
        n, N, r, S, codec = x.numel(), self.N, self.rank, self.S, self.codec
        self._check(x, out, N * n, "allgather")
        ea = self.resolve(x, eb_mode, eb)
        out[r * n: (r + 1) * n].copy_(x)
        if N == 1:
            return codec.finish()
        pieces = self._pieces(n)
        spans = piece_spans(n, S)
        for p, (po, pl) in zip(pieces, spans):
            codec.compress(x[po: po + pl], ea, p.out[0], p.out_bytes)
            self._mark_produced(p)

        def deliver(h, i, stream):
            q = (r - h - 1) % N
            po, pl = spans[i]
            codec.decompress(stream, out[q * n + po: q * n + po + pl])

        self._forward_stage(pieces, [self._produced_view(p, 0) for p in pieces], 0, deliver)
        self._drain(pieces)
        return codec.finish()

    def bcast(self, x: torch.Tensor, root: int, eb_mode: int, eb: float) -> int:
        """x on every rank but the root <- the root's x as its one compression reconstructs it.  Binomial tree:
        in the round with distance d = 1, 2, 4, ... every rank that already holds the streams hands them to the
        rank d places further (relative to the root); a relative bound refers to the root's data."""
        n, N, S, codec = x.numel(), self.N, self.S, self.codec
        self._check(x, x, n, "bcast")
        rel = (self.rank - root) % N
        pieces = self._pieces(n)
        spans = piece_spans(n, S)
        held = None
        if rel == 0:
            ea = self.resolve(x, eb_mode, eb, collective=False)
            for p, (po, pl) in zip(pieces, spans):
                codec.compress(x[po: po + pl], ea, p.out[0], p.out_bytes)
                self._mark_produced(p)
            held = [self._produced_view(p, 0) for p in pieces]
        d = 1
        while d < N:
            if rel < d and rel + d < N:
                for p, s in zip(pieces, held):
                    self._exchange(p, s, ("out", 0) if rel == 0 else ("inc", 0), root + rel + d, None, None)
            elif d <= rel < 2 * d:
                for p in pieces:
                    self._exchange(p, None, None, None, 0, root + rel - d)
                held = []
                for p, (po, pl) in zip(pieces, spans):
                    s = self._incoming(p, 0)
                    codec.decompress(s, x[po: po + pl])
                    self._mark_read(p, 0)
                    held.append(s)
            d <<= 1
        self._drain(pieces)
        return codec.finish()
