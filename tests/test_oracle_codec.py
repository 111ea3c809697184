"""Pins for the CPU oracle's codec (no GPU).  Every check here is something other than the oracle itself:
hand-computed byte vectors, closed forms written in numpy, an independently written stream parser, invariants
the paper states (error bound, constant-block rule), brute force on tiny inputs.
"""
import glob
import itertools
import re
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2502_18554_b200 import fields

GOLDEN = Path(__file__).resolve().parent / "golden"
f32 = np.float32


# ----------------------------------------------------------------------------- helpers independent of the oracle

def pointwise_quantiser(x, s, r):
    """Closed form of one round trip: Lorenzo + packing are lossless on integers, so decompress(compress(x))
    must equal fl32(float(rint(fl32(x*r))) * s) element by element (Section 3.3: quantisation is a multiply)."""
    t = (x.astype(f32) * f32(r)).astype(f32)
    q = np.rint(t).astype(np.int64)     # round half to even; the code is an integer, so -0.3 gives +0
    return (q.astype(f32) * f32(s)).astype(f32), q


def closed_form_size(q, n, T):
    """32 + 4 nT + sum_t (4 + pad4(nblk_t)) + sum_b [L_b > 0] 4 (1 + L_b), L_b by brute force from the codes."""
    nT = -(-n // T)
    total = 32 + 4 * nT
    n_const = n_blocks = 0
    for t in range(nT):
        qt = q[t * T:(t + 1) * T]
        d = np.diff(qt, prepend=qt[:1])
        nb = -(-len(qt) // 32)
        d = np.concatenate([d, np.zeros(nb * 32 - len(d), np.int64)]).reshape(nb, 32)
        mx = np.abs(d).max(axis=1)
        L = np.array([int(m).bit_length() for m in mx])
        total += 4 + ((nb + 3) & ~3) + int((4 * (1 + L[L > 0])).sum())
        n_const += int((L == 0).sum())
        n_blocks += nb
    return total, n_const, n_blocks


def parse_stream(buf: bytes):
    """Independent pure-Python reader of the stream layout; returns (header dict, list of integer codes)."""
    u32 = lambda o: int.from_bytes(buf[o:o + 4], "little")
    assert buf[:4] == b"ZCL1"
    assert u32(4) == 0x05000001
    n = int.from_bytes(buf[8:16], "little")
    s = np.frombuffer(buf[20:24], f32)[0]
    eb_abs = np.frombuffer(buf[16:20], f32)[0]
    T, nT = u32(24), u32(28)
    assert nT == -(-n // T)
    codes = []
    blob0 = 32 + 4 * nT
    prev = 0
    for t in range(nT):
        end_w = u32(32 + 4 * t)
        pos = blob0 + 4 * prev
        ln = min(T, n - t * T)
        nb = -(-ln // 32)
        acc = int.from_bytes(buf[pos:pos + 4], "little", signed=True)
        Ls = buf[pos + 4: pos + 4 + nb]
        assert all(b == 0 for b in buf[pos + 4 + nb: pos + 4 + ((nb + 3) & ~3)])
        p = pos + 4 + ((nb + 3) & ~3)
        for b in range(nb):
            L = Ls[b]
            assert L <= 31
            sign = 0
            planes = []
            if L:
                sign = u32(p)
                planes = [u32(p + 4 * (1 + k)) for k in range(L)]
                assert planes[L - 1] != 0, "top plane of a block must be non-empty (L is the exact bit length)"
                p += 4 * (1 + L)
            for j in range(32):
                mag = sum(((planes[k] >> j) & 1) << k for k in range(L))
                d = -mag if (sign >> j) & 1 else mag
                if b * 32 + j < ln:
                    acc += d
                    codes.append(acc)
                else:
                    assert d == 0 and not (sign >> j) & 1, "padding lanes carry zero deltas"
        assert p == blob0 + 4 * end_w
        prev = end_w
    assert len(buf) == blob0 + 4 * prev
    return dict(n=n, s=s, eb_abs=eb_abs, T=T, nT=nT), codes


def load_golden(path):
    kv, key = {}, None
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        if line[0].isspace() and key:
            kv[key] += " " + line.strip()
            continue
        key, v = line.split("=", 1)
        key = key.strip()
        kv[key] = v.strip()
    return kv


# ----------------------------------------------------------------------------- hand-computed byte vectors

@pytest.mark.parametrize("path", sorted(glob.glob(str(GOLDEN / "*.txt"))), ids=lambda p: Path(p).stem)
def test_golden_vectors(path):
    kv = load_golden(path)
    x = np.array(eval(kv["x"]), dtype=f32)
    want = bytes.fromhex(re.sub(r"\s", "", kv["bytes"]))
    st, rc = oracle.compress_core(x, float(kv["eb_abs"]), float(kv["s"]), float(kv["r"]), int(kv["T"]))
    assert rc == oracle.OK
    assert st.tobytes() == want
    assert int(kv["n"]) == x.size
    y = oracle.decompress(np.frombuffer(want, np.uint8))
    ref, _ = pointwise_quantiser(x, float(kv["s"]), float(kv["r"]))
    assert np.array_equal(y, ref)


# ----------------------------------------------------------------------------- bound resolution

def test_resolve_matches_stated_reading():
    x = fields.smooth_1d(50_000, seed=11)
    ea, s, r = oracle.resolve(oracle.EB_REL, 1e-3, x)
    rng_ = f32(x.max()) - f32(x.min())
    assert ea == f32(f32(1e-3) * rng_)
    assert s == f32(2) * f32(ea * f32(0.984375))
    assert r == f32(1) / s
    ea2, s2, r2 = oracle.resolve(oracle.EB_ABS, 1e-5)
    assert ea2 == f32(1e-5) and s2 == f32(2) * f32(f32(1e-5) * f32(0.984375)) and r2 == f32(1) / s2


def test_resolve_rejects():
    with pytest.raises(oracle.OracleError) as e:
        oracle.resolve(oracle.EB_REL, 1e-3, np.full(100, 3.0, f32))
    assert e.value.code == oracle.E_DEGENERATE
    for bad in (0.0, -1.0, float("nan"), float("inf")):
        with pytest.raises(oracle.OracleError) as e:
            oracle.resolve(oracle.EB_ABS, bad)
        assert e.value.code == oracle.E_ARG
    with pytest.raises(oracle.OracleError):
        oracle.resolve(7, 1e-3, np.arange(4, dtype=f32))


# ----------------------------------------------------------------------------- round trip == pointwise quantiser; bound

def _roundtrip_checks(x, eb_mode, eb, T=oracle.DEFAULT_TILE):
    ea, s, r = oracle.resolve(eb_mode, eb, x)
    st, rc = oracle.compress(x, eb_mode, eb, T)
    y, q = oracle.decompress(st, want_codes=True)
    ref, qref = pointwise_quantiser(x, s, r)
    assert np.array_equal(q.astype(np.int64), qref)
    assert np.array_equal(y.view(np.uint32), ref.view(np.uint32))
    if rc == oracle.OK:    # strict bound whenever no precision warning was raised
        err = np.abs(x.astype(np.float64) - y.astype(np.float64))
        assert err.max(initial=0.0) <= float(ea)
    size, n_const, n_blocks = closed_form_size(qref, x.size, T)
    assert st.size == size
    hdr, codes = parse_stream(st.tobytes())
    assert hdr["n"] == x.size and hdr["T"] == T and hdr["s"] == s and hdr["eb_abs"] == ea
    assert np.array_equal(np.array(codes, np.int64), qref)
    return st, rc, (ea, s, r)


def test_config0_roundtrip_bound_size():
    x = fields.smooth_1d(1 << 20, seed=0)
    st, rc, _ = _roundtrip_checks(x, oracle.EB_REL, 1e-3)
    assert rc == oracle.OK
    assert 10.0 < x.nbytes / st.size < 20.0     # smooth field at REL 1e-3: ratio of order 14


@pytest.mark.parametrize("rel", [1e-2, 1e-3, 1e-4])
def test_fourier_field_small(rel):
    x = fields.fourier_field_3d(48, seed=5)     # 110592 elements: 27 tiles
    _roundtrip_checks(x, oracle.EB_REL, rel)


def test_gradient_like_abs_bound():
    x = fields.gradient_like(300_001, seed=3)
    st, rc, _ = _roundtrip_checks(x, oracle.EB_ABS, 1e-5)
    assert rc == oracle.OK


def test_adversarial_values_meet_bound():
    ea, s, r = oracle.resolve(oracle.EB_ABS, 1e-3)
    k = np.arange(-3000, 3000, dtype=np.float64)
    half = ((k + 0.5) * float(s)).astype(f32)                  # quantisation-cell edges
    near = np.nextafter(half, f32(np.inf))
    near2 = np.nextafter(half, f32(-np.inf))
    small = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-38, -1e-38, 1.17549435e-38], f32)   # zeros and denormals
    big = (np.array([32768, -32768, 32767.5, 20000.25, -31000.75], np.float64) * float(s)).astype(f32)
    x = np.concatenate([half, near, near2, small, big])
    rng = np.random.default_rng(0)
    rng.shuffle(x)
    st, rc, _ = _roundtrip_checks(x, oracle.EB_ABS, 1e-3)
    assert rc == oracle.OK


def test_large_offset_up_to_precondition():
    # |q| <= 2^15 is the stated precondition of the strict bound: a field riding on a large offset
    ea, s, r = oracle.resolve(oracle.EB_ABS, 1e-2)
    rng = np.random.default_rng(5)
    x = (32000.0 * float(s) + rng.normal(0, 5 * float(s), 200_000)).astype(f32)
    x = np.minimum(x, f32(32767.0 * float(s)))
    st, rc, _ = _roundtrip_checks(x, oracle.EB_ABS, 1e-2)
    assert rc == oracle.OK


def test_precision_warning_and_range_error():
    ea, s, r = oracle.resolve(oracle.EB_ABS, 1e-3)
    x = np.array([0.0, 40000.0 * float(s)], f32)
    st, rc = oracle.compress(x, oracle.EB_ABS, 1e-3)
    assert rc == oracle.W_PRECISION
    y = oracle.decompress(st)
    assert np.array_equal(y, pointwise_quantiser(x, s, r)[0])
    with pytest.raises(oracle.OracleError) as e:
        oracle.compress(np.array([0.0, 3e6], f32), oracle.EB_ABS, 1e-3)    # |x*r| >= 2^30
    assert e.value.code == oracle.E_RANGE
    just_ok = np.array([f32(2 ** 30 - 64) * s], f32)
    if abs(float(just_ok[0] * r)) < 2 ** 30:
        _, rc2 = oracle.compress(just_ok, oracle.EB_ABS, 1e-3)
        assert rc2 == oracle.W_PRECISION


def test_constant_block_rule_and_ratio_limit():
    # code length 0 => only the one-byte code length is stored (Section 3.3) => closed-form minimum size
    T = 4096
    for v in (0.0, 3.25, -17.0):
        x = np.full(10 * T, v, f32)
        st, rc = oracle.compress(x, oracle.EB_ABS, 1e-2)
        assert st.size == 32 + 10 * (4 + 4 + T // 32)
    assert x.nbytes / (st.size - 32) == 4 * T / (8 + T / 32)             # -> 120.47 for T = 4096 (header aside)
    hdr, codes = parse_stream(st.tobytes())
    assert len(set(codes)) == 1


def test_ratio_falls_with_constant_block_share():
    # Table 3's relation: a tighter bound leaves fewer constant blocks and a lower ratio
    x = fields.fourier_field_3d(64, seed=2)
    ratios, shares = [], []
    for rel in (1e-1, 1e-2, 1e-3, 1e-4):
        ea, s, r = oracle.resolve(oracle.EB_REL, rel, x)
        st, _ = oracle.compress(x, oracle.EB_REL, rel)
        _, qref = pointwise_quantiser(x, s, r)
        _, n_const, n_blocks = closed_form_size(qref, x.size, 4096)
        ratios.append(x.nbytes / st.size)
        shares.append(n_const / n_blocks)
    assert ratios == sorted(ratios, reverse=True)
    assert shares == sorted(shares, reverse=True)


# ----------------------------------------------------------------------------- brute force on tiny inputs

def test_tiny_alphabet_brute_force():
    s = f32(0.25)
    r = f32(4.0)
    alphabet = [0.0, 0.5 * s, -0.5 * s, s, -s, 1.5 * s, -1.5 * s, 7 * s, -7 * s, 1000 * s, -1000 * s]
    for n in range(1, 5):
        for combo in itertools.product(alphabet, repeat=n):
            x = np.array(combo, f32)
            st, rc = oracle.compress_core(x, 0.125, s, r)
            ref, qref = pointwise_quantiser(x, s, r)
            assert np.array_equal(oracle.decompress(st), ref)
            assert st.size == closed_form_size(qref, n, 4096)[0]
    rng = np.random.default_rng(1)
    for _ in range(3000):
        x = rng.choice(np.array(alphabet, f32), 5)
        st, rc = oracle.compress_core(x, 0.125, s, r)
        ref, qref = pointwise_quantiser(x, s, r)
        assert np.array_equal(oracle.decompress(st), ref)
        hdr, codes = parse_stream(st.tobytes())
        assert codes == list(qref)


def test_every_length_small_tiles():
    # every n in 0 .. 2T+33 for a small tile, random walk data: decode(encode) == closed form, size == closed form
    T = 64
    rng = np.random.default_rng(2)
    base = np.cumsum(rng.normal(0, 3.0, 2 * T + 40)).astype(f32)
    ea, s, r = oracle.resolve(oracle.EB_ABS, 0.5)
    for n in range(0, 2 * T + 34):
        x = base[:n]
        st, rc = oracle.compress_core(x, ea, s, r, T)
        ref, qref = pointwise_quantiser(x, s, r)
        assert np.array_equal(oracle.decompress(st), ref)
        assert st.size == closed_form_size(qref, n, T)[0]
        hdr, codes = parse_stream(st.tobytes())
        assert codes == list(qref)


@pytest.mark.parametrize("n", [0, 1, 31, 32, 33, 4095, 4096, 4097, 8191, 8192, 8225])
def test_ragged_lengths_default_tile(n):
    rng = np.random.default_rng(n)
    x = np.cumsum(rng.normal(0, 1e-2, n)).astype(f32)
    if n:
        _roundtrip_checks(x, oracle.EB_ABS, 1e-3)
    else:
        st, rc = oracle.compress(x, oracle.EB_ABS, 1e-3)
        assert st.size == 32 and oracle.decompress(st).size == 0


def test_paper_chunk_size_is_expressible():
    # the paper's PIPE-fZ-light chunk of 5120 points (Section 3.5.2) as the tile size
    x = fields.smooth_1d(3 * 5120 + 77, seed=9)
    _roundtrip_checks(x, oracle.EB_REL, 1e-3, T=5120)


def test_wide_deltas_use_long_codes():
    # white noise at a tight bound: code lengths above 16 bits, still lossless on the integers
    rng = np.random.default_rng(4)
    x = rng.normal(0, 1.0, 5000).astype(f32)
    st, rc, (ea, s, r) = _roundtrip_checks(x, oracle.EB_ABS, 1e-6)
    assert rc == oracle.W_PRECISION
    hdr, codes = parse_stream(st.tobytes())
    assert max(abs(a - b) for a, b in zip(codes[1:], codes[:-1])) > (1 << 16)


# ----------------------------------------------------------------------------- capacity and malformed streams

def test_capacity_is_respected():
    x = fields.smooth_1d(10_000, seed=3)
    ea, s, r = oracle.resolve(oracle.EB_REL, 1e-3, x)
    full, _ = oracle.compress_core(x, ea, s, r)
    for cap in (0, 31, 32 + 4 * 3 - 1, full.size - 1, full.size // 2):
        with pytest.raises(oracle.OracleError) as e:
            oracle.compress_core(x, ea, s, r, cap=cap)
        assert e.value.code == oracle.E_CAPACITY
    st, _ = oracle.compress_core(x, ea, s, r, cap=full.size)
    assert np.array_equal(st, full)
    assert full.size <= oracle.compress_bound(x.size)


def test_compress_bound_is_worst_case():
    T = 4096
    for n in (0, 1, 32, 33, 4096, 4097, 10_000):
        nT = -(-n // T)
        nB = -(-n // 32)
        pad = sum(((-(-min(T, n - t * T) // 32)) + 3) & ~3 for t in range(nT))
        assert oracle.compress_bound(n) == 32 + 4 * nT + 4 * nT + pad + nB * 128
    rng = np.random.default_rng(8)
    x = (rng.integers(-2 ** 29, 2 ** 29, 5000).astype(np.float64)).astype(f32)   # deltas up to 31 bits
    st, rc = oracle.compress_core(x, 0.5, 1.0, 1.0)
    assert st.size <= oracle.compress_bound(x.size)
    assert st.size > 0.9 * oracle.compress_bound(x.size)


def test_malformed_streams_are_rejected():
    x = fields.smooth_1d(9000, seed=4)
    st, _ = oracle.compress(x, oracle.EB_REL, 1e-3)

    def bad(mut):
        b = st.copy()
        mut(b)
        with pytest.raises(oracle.OracleError) as e:
            oracle.decompress(b)
        assert e.value.code == oracle.E_BAD_STREAM

    bad(lambda b: b.__setitem__(0, 0x00))                       # magic
    bad(lambda b: b.__setitem__(4, 0x02))                       # version
    bad(lambda b: b.__setitem__(slice(24, 28), [0, 0, 0, 0]))   # T = 0
    bad(lambda b: b.__setitem__(slice(28, 32), [9, 0, 0, 0]))   # nT inconsistent with n
    bad(lambda b: b.__setitem__(slice(32, 36), [0xFF, 0xFF, 0xFF, 0x7F]))   # index not monotone / beyond buffer
    bad(lambda b: b.__setitem__(32 + 4 * 3 + 4, 40))            # code length > 31
    bad(lambda b: b.__setitem__(32 + 4 * 3 + 4, b[32 + 4 * 3 + 4] + 1))   # blob size no longer matches index
    for cut in (10, 33, st.size - 1):
        with pytest.raises(oracle.OracleError):
            oracle.decompress(st[:cut])


# ----------------------------------------------------------------------------- the reduce-scatter hop

def test_drc_is_decompress_add_compress():
    rng = np.random.default_rng(6)
    a = fields.smooth_1d(20_000, seed=1)
    b = fields.smooth_1d(20_000, seed=2)
    ea, s, r = oracle.resolve(oracle.EB_REL, 1e-3, np.concatenate([a, b]))
    sa, _ = oracle.compress_core(a, ea, s, r)
    out, rc, raw = oracle.drc(sa, local=b, want_raw=True)
    # composition written out in numpy: dequantise (one multiply), add (one add, decoded operand on the left), quantise
    a_hat, _ = pointwise_quantiser(a, s, r)
    y = (a_hat + b).astype(f32)
    assert np.array_equal(raw.view(np.uint32), y.view(np.uint32))
    ref, _ = oracle.compress_core(y, ea, s, r)
    assert np.array_equal(out, ref)
    y_hat, _ = pointwise_quantiser(y, s, r)
    assert np.array_equal(oracle.decompress(out), y_hat)
    # error chain of Eq. 2 for two ranks: two compressions
    exact = a.astype(np.float64) + b.astype(np.float64)
    assert np.abs(oracle.decompress(out).astype(np.float64) - exact).max() <= 2 * float(ea) * (1 + 1e-6)
    # consistent-owner flag returns the dequantised sum instead of the raw one
    out2, rc2, raw2 = oracle.drc(sa, local=b, want_raw=True, flags=oracle.FLAG_CONSISTENT_OWNER)
    assert np.array_equal(out2, out) and np.array_equal(raw2, y_hat)
    # two-compressed variant: both operands decoded first
    sb, _ = oracle.compress_core(b, ea, s, r)
    out3, rc3, raw3 = oracle.drc(sa, local_c=sb, want_raw=True)
    b_hat, _ = pointwise_quantiser(b, s, r)
    y3 = (a_hat + b_hat).astype(f32)
    assert np.array_equal(raw3, y3)
    assert np.array_equal(out3, oracle.compress_core(y3, ea, s, r)[0])


def test_drc_argument_checks():
    a = fields.smooth_1d(5000, seed=1)
    sa, _ = oracle.compress(a, oracle.EB_ABS, 1e-3)
    with pytest.raises(oracle.OracleError):
        oracle.drc(sa)                                   # neither operand
    with pytest.raises(oracle.OracleError):
        oracle.drc(sa, local=a, local_c=sa)              # both operands
    sb, _ = oracle.compress(a[:4000], oracle.EB_ABS, 1e-3)
    with pytest.raises(oracle.OracleError) as e:
        oracle.drc(sa, local_c=sb)                       # length mismatch between the two streams
    assert e.value.code == oracle.E_BAD_STREAM
    sc, _ = oracle.compress(a, oracle.EB_ABS, 2e-3)
    with pytest.raises(oracle.OracleError):
        oracle.drc(sa, local_c=sc)                       # different steps
