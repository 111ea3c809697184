"""Pins of the binary64 oracle (oracle/zccl_oracle_f64.c) against things other than itself: hand-computed byte
vectors of the stated layout, the closed form of one round trip in numpy's binary64 arithmetic, the error bound in
exact rational arithmetic on adversarial values, and the stated reading of bound and step (Section 3.3)."""
import glob
import re
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2502_18554_b200 import fields

GOLDEN = Path(__file__).resolve().parent / "golden" / "f64"


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


@pytest.mark.parametrize("path", sorted(glob.glob(str(GOLDEN / "*.txt"))), ids=lambda p: Path(p).stem)
def test_golden_vectors_f64(path):
    kv = load_golden(path)
    x = np.array(eval(kv["x"]), dtype=np.float64)
    want = bytes.fromhex(re.sub(r"\s", "", kv["bytes"]))
    assert int(kv["n"]) == x.size
    st = oracle.compress_f64(x, oracle.EB_ABS, float(kv["eb_abs"]), int(kv["T"]))
    assert st.tobytes() == want
    y, q = oracle.decompress_f64(np.frombuffer(want, np.uint8), want_codes=True)
    assert np.array_equal(q, x.astype(np.int64))                     # the codes are the integers themselves
    assert np.array_equal(y, x * (1.0 - 2.0 ** -20))                 # and the values are code * step


def test_bound_and_step_as_stated():
    ea, s, r = oracle.resolve_f64(oracle.EB_ABS, 0.25)
    assert ea == 0.25 and s == 0.5 - 2.0 ** -21 and r == 1.0 / s     # 0.25 * (1 - 2^-20) is exact in binary64
    ea, s, r = oracle.resolve_f64(oracle.EB_REL, 1e-3, -3.5, 12.25)
    assert ea == 1e-3 * 15.75 and s == 2.0 * (ea * (1.0 - 2.0 ** -20)) and r == 1.0 / s
    for bad in ((oracle.EB_REL, 1e-3, 2.0, 2.0), (oracle.EB_REL, 1e-3, 3.0, 2.0), (oracle.EB_REL, 1e-3, 0.0, float("inf"))):
        with pytest.raises(oracle.OracleError) as e:
            oracle.resolve_f64(*bad)
        assert e.value.code == oracle.E_DEGENERATE
    with pytest.raises(oracle.OracleError):
        oracle.resolve_f64(oracle.EB_ABS, 0.0)


def closed_form(x, s, r):
    """One round trip, element by element: Lorenzo and the bit planes are lossless on integers, so decompress(compress(x))
    is fl64(rint(fl64(x * r)) * s) (numpy's binary64 multiplication is IEEE, rint rounds ties to even)."""
    q = np.rint(x * r)
    return q * s, q.astype(np.int64)


@pytest.mark.parametrize("n,eb", [(1, 1e-3), (33, 1e-9), (4096, 1e-6), (4097, 4e-10), (100_003, 3e-7)])
def test_round_trip_is_the_pointwise_quantiser(n, eb):
    rng = np.random.default_rng(n)
    x = np.cumsum(rng.standard_normal(n)) * 1e-3 + rng.standard_normal(n) * 1e-7
    ea, s, r = oracle.resolve_f64(oracle.EB_ABS, eb)
    y, q = oracle.decompress_f64(oracle.compress_f64(x, oracle.EB_ABS, eb), want_codes=True)
    want_y, want_q = closed_form(x, s, r)
    assert np.array_equal(q, want_q)
    assert np.array_equal(y, want_y)
    assert np.array_equal(oracle.quantise_f64(x, r), want_q)
    assert float(np.abs(x - y).max()) <= eb


def test_relative_bound_uses_the_range_in_binary64():
    x = fields.smooth_1d(20_000, seed=4).astype(np.float64) * 1.000000123
    st = oracle.compress_f64(x, oracle.EB_REL, 1e-4)
    ea, s, r = oracle.resolve_f64(oracle.EB_REL, 1e-4, float(x.min()), float(x.max()))
    assert np.frombuffer(st[16:24].tobytes(), np.float64)[0] == s
    assert np.array_equal(oracle.decompress_f64(st), closed_form(x, s, r)[0])


def test_error_bound_holds_exactly_on_adversarial_values():
    """|x - x'| <= eb_abs in exact rational arithmetic: ties at (k + 1/2) s and their neighbours in binary64, values
    next to the largest code, denormals, zeros of both signs, and magnitudes spread over the whole code range."""
    eb = 1e-5
    ea, s, r = oracle.resolve_f64(oracle.EB_ABS, eb)
    rng = np.random.default_rng(3)
    ks = np.concatenate([np.arange(-40, 40), rng.integers(-(2 ** 30) + 2, 2 ** 30 - 2, 400), [2 ** 30 - 2, -(2 ** 30) + 2]]).astype(np.float64)
    ties = (ks + 0.5) * s
    vals = [ties, np.nextafter(ties, np.inf), np.nextafter(ties, -np.inf), ks * s, np.nextafter(ks * s, np.inf),
            np.array([0.0, -0.0, 5e-324, -5e-324, 2.2250738585072014e-308, 1e-300]),
            rng.standard_normal(500) * 10.0 ** rng.uniform(-12, 3.9, 500)]
    x = np.concatenate(vals)
    x = x[np.abs(x * r) < 2.0 ** 30]
    y = oracle.decompress_f64(oracle.compress_f64(x, oracle.EB_ABS, eb, T=32))
    bound = Fraction(eb)
    worst = Fraction(0)
    for a, b in zip(x.tolist(), y.tolist()):
        err = abs(Fraction(a) - Fraction(b))
        assert err <= bound, (a, b)
        worst = max(worst, err)
    assert worst > bound * Fraction(99, 100)      # the ties come close to it: the step is not needlessly small


def test_out_of_range_and_foreign_streams():
    ea, s, r = oracle.resolve_f64(oracle.EB_ABS, 1e-3)
    with pytest.raises(oracle.OracleError) as e:
        oracle.compress_f64(np.array([0.0, 2.0 ** 30 * s * 1.01]), oracle.EB_ABS, 1e-3)
    assert e.value.code == oracle.E_RANGE
    st64 = oracle.compress_f64(np.arange(100, dtype=np.float64), oracle.EB_ABS, 0.5)
    st32, _ = oracle.compress(np.arange(100, dtype=np.float32), oracle.EB_ABS, 0.5)
    with pytest.raises(oracle.OracleError):
        oracle.decompress(st64)           # the binary32 decoder refuses the other data type
    with pytest.raises(oracle.OracleError):
        oracle.decompress_f64(st32)
    assert st64[32:].tobytes() != b"" and st64.size > 32
