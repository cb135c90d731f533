"""Pins for the oracle's random numbers, the quantiser Q_(delta,b) (Section 3.1) and the bit packer.

Nothing here touches the CUDA library.  Each test checks the oracle against something other than
itself: published known answers, exact rational arithmetic, brute force, or the paper's own
statements (code range, unbiasedness, the variance bound of the appendix's first lemma).
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")
F32 = np.float32


# ---------------------------------------------------------------------------------------------------
# Philox
# ---------------------------------------------------------------------------------------------------
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt")) if not l.startswith("#") and l.strip()]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        assert list(oracle.philox4x32_10(v[0:4], v[4:6])) == v[6:10]


def _philox_bigint(ctr, key):
    """Independent restatement with Python integers: the bijection as two 32x32->64 products per round."""
    c = list(ctr); k = list(key)
    for r in range(10):
        hi0, lo0 = divmod(0xD2511F53 * c[0], 1 << 32)
        hi1, lo1 = divmod(0xCD9E8D57 * c[2], 1 << 32)
        c = [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]
        k = [(k[0] + 0x9E3779B9) % (1 << 32), (k[1] + 0xBB67AE85) % (1 << 32)]
    return c


def test_philox_against_bigint_restatement():
    g = np.random.default_rng(11)
    for _ in range(3000):
        ctr = [int(x) for x in g.integers(0, 1 << 32, 4)]
        key = [int(x) for x in g.integers(0, 1 << 32, 2)]
        assert [int(x) for x in oracle.philox4x32_10(ctr, key)] == _philox_bigint(ctr, key)


def test_uniform_lane_layout():
    """Coordinate i: Philox counter (i>>3, round, worker, stream), key = seed halves; word (i&7)>>1;
    16-bit draw = low/high half for even/odd i; 15-bit draw = its top 15 bits."""
    seed, rnd, wk, st = 0x1234_5678_9ABC_DEF0, 77, 5, 1
    for i in list(range(40)) + [2 ** 27 - 1, 2 ** 31 + 5]:
        out = _philox_bigint([i >> 3, rnd, wk, st], [seed & 0xFFFFFFFF, seed >> 32])
        w = out[(i & 7) >> 1]
        assert oracle.u16(seed, rnd, wk, st, i) == ((w >> 16) if i & 1 else (w & 0xFFFF))
        assert oracle.u15(seed, rnd, wk, st, i) == ((w >> 17) if i & 1 else ((w & 0xFFFF) >> 1))


def test_uniform_chi_square():
    n, bins = 1 << 18, 256
    u = np.array([oracle.u15(9, 3, 1, 1, i) for i in range(n)])
    assert u.min() >= 0 and u.max() < (1 << 15)
    cnt = np.bincount(u >> 7, minlength=bins)
    chi2 = ((cnt - n / bins) ** 2 / (n / bins)).sum()
    assert chi2 < 255 + 6 * np.sqrt(2 * 255)            # mean 255, sd sqrt(510)
    # independence of neighbouring coordinates (same Philox call): correlation ~ N(0, 1/n)
    a, b = u[0::2].astype(np.float64), u[1::2].astype(np.float64)
    assert abs(np.corrcoef(a, b)[0, 1]) < 6 / np.sqrt(n / 2)


# ---------------------------------------------------------------------------------------------------
# scale factors
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("b", [2, 3, 4, 8])
def test_scales(b):
    L = 2 ** (b - 1) - 1
    g = np.random.default_rng(b)
    nrms = list(np.abs(g.standard_normal(200)).astype(F32) * F32(10.0) ** g.integers(-20, 20, 200).astype(F32))
    nrms += [F32(1e-45), F32(1.2e-38), F32(3.0e38), F32(1.0), F32(L), F32(0.1)]
    for nrm in nrms:
        nrm = F32(nrm)
        if nrm == 0 or not np.isfinite(nrm):
            continue
        assert oracle.scale_delta(nrm, b) == F32(nrm) / F32(L)        # delta = ||v||_inf / (2^(b-1)-1)
        c = oracle.scale_inv(nrm, b)
        assert np.isfinite(c) and c > 0
        assert Fraction(float(c)) * Fraction(float(nrm)) <= L          # keeps every |v_i| <= nrm inside the hull
        up = np.nextafter(c, F32(np.inf), dtype=F32)
        assert (not np.isfinite(up)) or Fraction(float(up)) * Fraction(float(nrm)) > L   # and is the largest such


# ---------------------------------------------------------------------------------------------------
# Q: one coordinate, exact
# ---------------------------------------------------------------------------------------------------
def _fixed_point_shape(b):
    """(offset 2^(e-1) on the code axis, fractional bits) of the fixed-point position: e = 8 up to 8-bit codes, else b."""
    e = 8 if b <= 8 else b
    return 1 << (e - 1), 23 - e


def _exact_fixed_point(v, inv, b=8):
    """(t + offset) * 2^fbits rounded to nearest-even, from exact rationals."""
    off, fb = _fixed_point_shape(b)
    t = Fraction(float(v)) * Fraction(float(inv))
    s = (t + off) * (1 << fb)
    fl = s.numerator // s.denominator
    rem = s - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return fl, t


@pytest.mark.parametrize("b", [2, 3, 4, 5, 6, 7, 8, 9, 10, 11])
def test_q_code_is_stochastic_rounding_with_exact_probability(b):
    """Rule (i): the code is floor(t) or floor(t)+1 and, over ALL values of the uniform draw, it is rounded up
    exactly frac*2^fbits times, with frac the fractional part of t at the fixed-point resolution (15 fractional
    bits up to 8-bit codes, 14/13/12 for 9/10/11 bits; the draw's top bits are used)."""
    L = 2 ** (b - 1) - 1
    off, fb = _fixed_point_shape(b)
    g = np.random.default_rng(100 + b)
    nrm = F32(3.7)
    inv = oracle.scale_inv(nrm, b)
    us = [0, 1, 2, 12345, (1 << 14), (1 << 15) - 2, (1 << 15) - 1]
    for v in list((g.uniform(-1, 1, 60) * float(nrm)).astype(F32)) + [nrm, -nrm, F32(0.0), F32(1e-30)]:
        F, t = _exact_fixed_point(v, inv, b)
        z = F >> fb                                                   # floor at the fixed-point resolution, + offset
        frac = F & ((1 << fb) - 1)
        assert abs(Fraction(F, 1 << fb) - off - t) <= Fraction(1, 1 << (fb + 1))      # resolution of the position
        for u in us:
            k = oracle.q_code(v, inv, b, u)
            assert -L <= k <= L
            assert k == z - off + (1 if (u >> (15 - fb)) + frac >= (1 << fb) else 0)
        # exact count of round-ups over the whole uniform range, on a few values
    for v in (g.uniform(-1, 1, 3 if b in (2, 4, 8, 11) else 1) * float(nrm)).astype(F32):
        F, _ = _exact_fixed_point(v, inv, b)
        ks = np.array([oracle.q_code(v, inv, b, u) for u in range(1 << 15)])
        assert set(np.unique(ks)) <= {(F >> fb) - off, (F >> fb) - off + 1}
        assert int((ks == (F >> fb) - off + 1).sum()) == (F & ((1 << fb) - 1)) << (15 - fb)


@pytest.mark.parametrize("b", [2, 3, 4, 7, 8, 9, 10, 11])
def test_q_rule_ii_clamps_to_dom(b):
    """Rule (ii): outside the hull of dom(delta,b) the nearest member: -2^(b-1) below, 2^(b-1)-1 above."""
    inv = oracle.scale_inv(F32(1.0), b)
    for u in (0, 77, (1 << 15) - 1):
        assert oracle.q_code(F32(50.0), inv, b, u) == 2 ** (b - 1) - 1
        assert oracle.q_code(F32(-50.0), inv, b, u) == -(2 ** (b - 1))
        assert oracle.q_code(F32(1.0), inv, b, u) in (2 ** (b - 1) - 2, 2 ** (b - 1) - 1)     # the hull's own end stays inside
        assert oracle.q_code(F32(1e30), inv, b, u) == 2 ** (b - 1) - 1


# ---------------------------------------------------------------------------------------------------
# Q: vectors
# ---------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("b", [2, 3, 4, 5, 6, 7, 8, 9, 10, 11])
def test_code_range_and_neighbours(b):
    L = 2 ** (b - 1) - 1
    g = np.random.default_rng(b)
    for trial in range(20):
        d = int(g.integers(1, 300))
        v = g.standard_normal(d).astype(F32) * F32(10.0 ** g.integers(-30, 30))
        if trial % 3 == 0:
            v[g.integers(0, d)] *= F32(100)
        codes, delta, rc = oracle.quantize(v, b, 5, trial, 2, oracle.STREAM_GRAD)
        assert rc == 0 and np.abs(codes).max() <= L
        nrm = np.abs(v).max()
        assert delta == nrm / F32(L)
        inv = oracle.scale_inv(nrm, b)
        t = np.array([float(Fraction(float(x)) * Fraction(float(inv))) for x in v])
        res = float(1 << _fixed_point_shape(b)[1])
        fl = np.floor(np.round(t * res) / res)                          # t is a multiple of the resolution after rounding
        assert np.all((codes == fl) | (codes == fl + 1))
        i = int(np.argmax(np.abs(v)))
        assert abs(codes[i]) >= L - 1                                   # the max coordinate sits at the end of the grid


def test_grid_points_are_fixed_points():
    """A vector already on the grid k*delta is reproduced exactly whatever the random draw."""
    for b in (2, 4, 8):
        L = 2 ** (b - 1) - 1
        k = np.arange(-L, L + 1, dtype=np.int32)
        v = (k * 0.125).astype(F32)                                    # nrm = L/8, delta = 1/8 exactly
        for rnd in range(5):
            codes, delta, rc = oracle.quantize(v, b, 1, rnd, 0, oracle.STREAM_GRAD)
            assert rc == 0 and delta == F32(0.125)
            assert np.array_equal(codes, k)
            assert np.array_equal(codes.astype(F32) * delta, v)


def test_zero_and_nonfinite():
    codes, delta, rc = oracle.quantize(np.zeros(17, F32), 4, 1, 1, 1, 1)
    assert rc == 0 and delta == 0 and not codes.any()
    for bad in (np.nan, np.inf, -np.inf):
        v = np.ones(9, F32); v[4] = bad
        assert oracle.quantize(v, 4, 1, 1, 1, 1)[2] == oracle.ERR_NONFINITE


@pytest.mark.parametrize("b", [2, 4, 8, 5, 11])
def test_unbiased_and_variance(b):
    """E[Q(v)] = v (Section 3.1 rule (i)) and E||Q(v)-v||^2 <= d delta^2/4 with per-coordinate variance
    (x-z)(z+delta-x) (appendix, first lemma and its proof)."""
    L = 2 ** (b - 1) - 1
    g = np.random.default_rng(40 + b)
    d, N = 48, 20000
    v = g.standard_normal(d).astype(F32)
    v[3] = 0.0
    acc = np.zeros(d); acc2 = np.zeros(d)
    delta = None
    for rnd in range(N):
        codes, delta, rc = oracle.quantize(v, b, 2024, rnd, 1, oracle.STREAM_GRAD)
        q = codes.astype(np.float64) * float(delta)
        acc += q; acc2 += (q - v) ** 2
    delta = float(delta)
    mean, mse = acc / N, acc2 / N
    z = np.floor(v / delta) * delta
    var_exact = (v - z) * (z + delta - v)
    sd = np.sqrt(np.maximum(var_exact, 1e-30))
    resol = delta * 2.0 ** -_fixed_point_shape(b)[1]  # fixed-point position + fp32 scale rounding
    assert np.all(np.abs(mean - v) <= 5 * sd / np.sqrt(N) + resol)
    assert np.all(var_exact <= delta ** 2 / 4 + 1e-12)
    assert np.all(np.abs(mse - var_exact) <= 0.05 * delta ** 2 / 4 + resol * delta)
    assert mse.sum() <= d * delta ** 2 / 4
    assert mean[3] == 0.0


def test_rounding_streams_differ():
    v = np.random.default_rng(1).standard_normal(4096).astype(F32)
    base = oracle.quantize(v, 8, 7, 10, 3, oracle.STREAM_GRAD)[0]
    for args in [(8, 10, 3, oracle.STREAM_GRAD), (7, 11, 3, oracle.STREAM_GRAD), (7, 10, 4, oracle.STREAM_GRAD),
                 (7, 10, 3, oracle.STREAM_MODEL)]:
        other = oracle.quantize(v, 8, *args)[0]
        assert 0.2 < np.mean(other != base) < 0.8      # seed, round, worker and stream all key the draw
    assert np.array_equal(base, oracle.quantize(v, 8, 7, 10, 3, oracle.STREAM_GRAD)[0])


# ---------------------------------------------------------------------------------------------------
# pack / unpack
# ---------------------------------------------------------------------------------------------------
def _pack_bigint(codes, b, nbytes):
    """The message as ONE little-endian integer: coordinate j occupies bits [j*b, (j+1)*b)."""
    word = 0
    for j, k in enumerate(codes):
        word |= (int(k) % (1 << b)) << (j * b)
    return np.frombuffer(word.to_bytes(nbytes, "little"), dtype=np.uint8)


@pytest.mark.parametrize("b", [2, 3, 4, 5, 6, 7, 8, 9, 10, 11])
def test_pack_matches_bit_by_bit_and_roundtrips(b):
    g = np.random.default_rng(b)
    lo, hi = -(2 ** (b - 1)), 2 ** (b - 1) - 1
    for d in range(1, 258):
        codes = g.integers(lo, hi + 1, d).astype(np.int32)
        buf = oracle.pack(codes, b)
        assert buf.size % 16 == 0 and buf.size >= (d * b + 7) // 8
        assert np.array_equal(buf, _pack_bigint(codes, b, buf.size))    # includes zero tail/padding
        assert np.array_equal(oracle.unpack(buf, d, b), codes)
    for lane in range(8):                                               # every code value at every bit phase of a byte
        for k in (range(lo, hi + 1) if b <= 8 else list(range(lo, lo + 40)) + list(range(-20, 20)) + list(range(hi - 40, hi + 1))):
            codes = np.zeros(8, np.int32); codes[lane] = k
            buf = oracle.pack(codes, b)
            assert int.from_bytes(buf.tobytes(), "little") == (k % (1 << b)) << (lane * b)
            assert oracle.unpack(buf, 8, b)[lane] == k
