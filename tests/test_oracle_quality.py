"""Pins for the oracle's quality metrics (no GPU): closed forms, a library cross-check, the degenerate cases, and
the link between the error bound and the metrics on a compressed field (Section 4.1: NRMSE, PSNR, bit rate)."""
import math

import numpy as np

import oracle
from paper_2502_18554_b200 import fields

f32 = np.float32


def test_constant_offset_closed_form():
    # y = x + c with x spanning [0, 8] exactly: every error is c, so MSE = c^2, NRMSE = c / 8, PSNR = 20 log10(8 / c)
    x = np.linspace(0.0, 8.0, 4097).astype(f32)
    c = 0.25                                           # exactly representable; x + c is exact for these values
    q = oracle.quality(x, (x + f32(c)).astype(f32))
    assert q["max_abs_err"] == c
    assert q["mse"] == c * c
    assert q["min"] == 0.0 and q["max"] == 8.0
    assert math.isclose(q["nrmse"], c / 8.0, rel_tol=1e-15)
    assert math.isclose(q["psnr"], 20.0 * math.log10(8.0 / c), rel_tol=1e-15)


def test_alternating_error_and_sign():
    # errors +e and -e alternate: MSE = e^2 whatever the signs, max error e
    x = np.arange(1000, dtype=f32)
    e = 0.5
    y = (x + np.where(np.arange(1000) % 2 == 0, e, -e)).astype(f32)
    q = oracle.quality(x, y)
    assert q["max_abs_err"] == e and q["mse"] == e * e
    assert math.isclose(q["nrmse"], e / 999.0, rel_tol=1e-15)


def test_against_numpy_fp64():
    rng = np.random.default_rng(3)
    x = rng.normal(0, 3, 100_003).astype(f32)
    y = (x + rng.normal(0, 1e-3, x.size)).astype(f32)
    q = oracle.quality(x, y)
    d = x.astype(np.float64) - y.astype(np.float64)
    rng_x = float(x.max()) - float(x.min())
    assert q["max_abs_err"] == float(np.max(np.abs(d)))
    assert math.isclose(q["mse"], float(np.mean(d * d)), rel_tol=1e-12)
    assert math.isclose(q["nrmse"], math.sqrt(float(np.mean(d * d))) / rng_x, rel_tol=1e-12)
    assert math.isclose(q["psnr"], 20 * math.log10(rng_x / math.sqrt(float(np.mean(d * d)))), rel_tol=1e-12)


def test_degenerate_cases():
    x = fields.smooth_1d(5000, seed=2)
    q = oracle.quality(x, x)
    assert q["mse"] == 0.0 and q["max_abs_err"] == 0.0 and q["nrmse"] == 0.0 and q["psnr"] == math.inf
    c = np.full(100, 3.5, f32)
    q = oracle.quality(c, c + f32(1))
    assert q["mse"] == 1.0 and math.isnan(q["nrmse"]) and math.isnan(q["psnr"])


def test_uniform_quantisation_error_statistics():
    # a quantiser with step s leaves errors spread over [-s/2, s/2]: MSE close to s^2 / 12 on a field that is rough at
    # the scale of s, and never above (s/2)^2; with a relative bound eps the NRMSE is then near eps / sqrt(3)
    x = fields.smooth_1d(1 << 18, seed=9)
    rel = 1e-3
    st, rc = oracle.compress(x, oracle.EB_REL, rel)
    y = oracle.decompress(st)
    ea, s, _ = oracle.resolve(oracle.EB_REL, rel, x)
    q = oracle.quality(x, y)
    assert q["max_abs_err"] <= float(ea)
    assert q["mse"] <= (float(s) / 2) ** 2 * (1 + 1e-6)
    assert 0.5 < q["mse"] / (float(s) ** 2 / 12) < 1.5
    assert 0.5 * rel / math.sqrt(3) < q["nrmse"] < 1.05 * rel / math.sqrt(3)
    assert math.isclose(q["psnr"], -20 * math.log10(q["nrmse"]), rel_tol=1e-12)


# ----------------------------------------------------------------------------- code-length statistics of a stream

def _brute_force_hist(x, ea_s_r, T):
    """Histogram of code lengths straight from the definition: quantise, deltas inside each tile (the first element
    of a tile has none), bit length of the largest magnitude of every block of 32."""
    _, s, r = ea_s_r
    q, _ = oracle.quantise(x, r)
    q = q.astype(np.int64)
    hist = np.zeros(33, np.uint64)
    for t0 in range(0, q.size, T):
        qt = q[t0:t0 + T]
        d = np.diff(qt, prepend=qt[:1])
        for b0 in range(0, d.size, 32):
            L = int(np.abs(d[b0:b0 + 32]).max()).bit_length()
            hist[L] += 1
            hist[32] += 1
    return hist


def test_stream_stats_constant_field_is_all_constant_blocks():
    # Section 3.3: code length 0 = constant block, stored as its one byte; a constant array has nothing else
    x = np.full(3 * 4096 + 100, 2.5, np.float32)
    st, _ = oracle.compress(x, oracle.EB_ABS, 1e-3)
    h = oracle.stream_stats(st)
    nblk = 3 * 128 + 4
    assert h[0] == nblk and h[32] == nblk and h[1:32].sum() == 0


def test_stream_stats_match_brute_force_and_stream_size():
    for T in (4096, 5120):
        for seed, n, eb in ((1, 20000, 1e-3), (2, 4096 * 3, 1e-2), (3, 5000, 1e-5)):
            x = fields.smooth_1d(n, seed=seed)
            x[n // 2: n // 2 + 700] += np.random.default_rng(seed).normal(0, 0.3, 700).astype(np.float32)
            st, _ = oracle.compress(x, oracle.EB_REL, eb, T)
            h = oracle.stream_stats(st)
            want = _brute_force_hist(x, oracle.resolve(oracle.EB_REL, eb, x), T)
            assert np.array_equal(h, want)
            # the histogram fixes the stream's length: header, one index entry and one outlier per tile, the padded
            # code-length bytes, a sign word and L plane words per non-constant block
            nT = -(-n // T)
            size = 32 + 4 * nT
            for t in range(nT):
                nb = -(-min(T, n - t * T) // 32)
                size += 4 + ((nb + 3) & ~3)
            size += sum(4 * (1 + L) * int(h[L]) for L in range(1, 32))
            assert size == st.size


def test_stream_stats_rejects_a_damaged_stream():
    x = fields.smooth_1d(9000, seed=5)
    st, _ = oracle.compress(x, oracle.EB_ABS, 1e-3)
    bad = st.copy()
    bad[0] ^= 0xFF
    try:
        oracle.stream_stats(bad)
        assert False, "a stream without the magic word must be refused"
    except oracle.OracleError as e:
        assert e.code == oracle.E_BAD_STREAM
