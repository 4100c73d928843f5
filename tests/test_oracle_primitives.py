"""Pins for the oracle's building blocks: Philox, the elementary functions, the
noise distributions and the compressors.  CPU only."""
import os
from fractions import Fraction

import numpy as np
import pytest
from scipy import stats

from oracle import oracle as orc
from paper_1907_07346_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- Philox
def _philox_numpy(ctr, key):
    """Second, independently written Philox4x32-10 (numpy uint64 arithmetic),
    vectorised over leading dimensions."""
    c = [np.asarray(v, dtype=np.uint64) for v in ctr]
    k = [np.uint64(key[0]), np.uint64(key[1])]
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        prod_a = np.uint64(0xD2511F53) * c[0]
        prod_b = np.uint64(0xCD9E8D57) * c[2]
        c = [(prod_b >> np.uint64(32)) ^ c[1] ^ k[0], prod_b & mask,
             (prod_a >> np.uint64(32)) ^ c[3] ^ k[1], prod_a & mask]
        k = [(k[0] + np.uint64(0x9E3779B9)) & mask, (k[1] + np.uint64(0xBB67AE85)) & mask]
    return [v.astype(np.uint32) for v in c]


def test_philox_known_answers():
    rows = [ln.split() for ln in open(os.path.join(GOLD, "philox4x32_10_kat.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 2
    for r in rows:
        vals = [int(t, 16) for t in r]
        out = orc.philox(vals[0:4], vals[4:6])
        assert [int(v) for v in out] == vals[6:10]


def test_philox_matches_second_implementation():
    rng = np.random.default_rng(5)
    for _ in range(200):
        ctr = rng.integers(0, 2**32, size=4, dtype=np.uint64)
        key = rng.integers(0, 2**32, size=2, dtype=np.uint64)
        ref = _philox_numpy([ctr[0], ctr[1], ctr[2], ctr[3]], key)
        out = orc.philox(ctr.astype(np.uint32), key.astype(np.uint32))
        assert [int(v) for v in out] == [int(v) for v in ref]


def test_stream_addressing_of_rounding_words():
    """rnd24 of element k is word k%4 of block k/4, counter
    (block, node, step low, (step>>32)<<8 | 1), key (seed low, seed high)."""
    seed, node, step = 0x1234_5678_9ABC_DEF0, 5, (7 << 32) | 99
    k = np.arange(64)
    blocks = (k >> 2).astype(np.uint64)
    w = _philox_numpy([blocks, np.full(64, node), np.full(64, step & 0xFFFFFFFF),
                       np.full(64, ((step >> 32) << 8) | 1)],
                      (seed & 0xFFFFFFFF, seed >> 32))
    word = np.choose(k & 3, w)
    expect = (word >> np.uint32(8)).astype(np.float64) / 2.0**24
    got = orc.rnd24_row(seed, node, step, 0, 64)
    assert np.array_equal(got.astype(np.float64), expect)
    # a different node, step or seed gives a different stream
    assert not np.array_equal(got, orc.rnd24_row(seed, node + 1, step, 0, 64))
    assert not np.array_equal(got, orc.rnd24_row(seed, node, step + 1, 0, 64))
    assert not np.array_equal(got, orc.rnd24_row(seed + 1, node, step, 0, 64))
    # a row read from an offset is the same stream
    assert np.array_equal(got[13:], orc.rnd24_row(seed, node, step, 13, 51))


# ------------------------------------------------- elementary functions
def _ulp_err(got32, ref64):
    ref32 = ref64.astype(np.float32)
    ulp = np.spacing(np.abs(ref32)).astype(np.float64)
    return np.abs(got32.astype(np.float64) - ref64) / ulp


def test_log_exhaustive_accuracy():
    """All 2^24 arguments j 2^-24: within 3 ulp of ln in float64."""
    worst = 0.0
    total = 1 << 24
    blk = 1 << 22
    for j0 in range(1, total + 1, blk):
        cnt = min(blk, total + 1 - j0)
        got = orc.log_u24_array(j0, cnt)
        j = np.arange(j0, j0 + cnt, dtype=np.float64)
        ref = np.log(j) - 24.0 * np.log(2.0)
        ok = ref != 0
        worst = max(worst, float(_ulp_err(got[ok], ref[ok]).max()))
        assert np.all(got[~ok] == 0.0)           # ln(1) = 0 exactly
        assert np.all(got <= 0.0)
    assert worst <= 3.0, worst


def test_sincos_exhaustive_accuracy():
    """All 2^24 angles: absolute error <= 2^-23, and <= 3 ulp away from the
    axes crossings; cos^2 + sin^2 = 1 within 3e-7; exact values on the axes."""
    total = 1 << 24
    blk = 1 << 22
    worst_abs = 0.0
    for k0 in range(0, total, blk):
        c, s = orc.sincos_u24_array(k0, blk)
        ang = 2.0 * np.pi * np.arange(k0, k0 + blk, dtype=np.float64) / total
        worst_abs = max(worst_abs, float(np.abs(c - np.cos(ang)).max()),
                        float(np.abs(s - np.sin(ang)).max()))
        assert np.abs(c.astype(np.float64)**2 + s.astype(np.float64)**2 - 1).max() < 3e-7
    assert worst_abs <= 2.0**-23, worst_abs
    c, s = orc.sincos_u24_array(0, 1)
    assert (c[0], s[0]) == (1.0, 0.0)
    c, s = orc.sincos_u24_array(1 << 22, 1)
    assert (c[0], s[0]) == (0.0, 1.0)
    c, s = orc.sincos_u24_array(1 << 23, 1)
    assert (c[0], s[0]) == (-1.0, 0.0)
    c, s = orc.sincos_u24_array(3 << 22, 1)
    assert (c[0], s[0]) == (0.0, -1.0)
    # 45 degrees
    c, s = orc.sincos_u24_array(1 << 21, 1)
    assert abs(c[0] - np.sqrt(0.5)) < 1.2e-7 and abs(s[0] - np.sqrt(0.5)) < 1.2e-7


# -------------------------------------------------------- distributions
def test_gauss_noise_is_standard_normal():
    z = orc.noise_row(I.NOISE_GAUSS, 2024, 3, 17, 0, 1 << 20).astype(np.float64)
    assert abs(z.mean()) < 4e-3
    assert abs(z.var() - 1.0) < 6e-3
    assert abs((z**3).mean()) < 2e-2
    assert abs((z**4).mean() - 3.0) < 5e-2
    assert stats.kstest(z[:200_000], "norm").pvalue > 1e-3
    # the four elements of a block are uncorrelated
    zz = z.reshape(-1, 4)
    corr = np.corrcoef(zz.T)
    assert np.abs(corr - np.eye(4)).max() < 1e-2


def test_student_t3_noise_distribution():
    t = orc.noise_row(I.NOISE_STUDENT_T3, 77, 1, 4, 0, 1 << 19).astype(np.float64)
    assert stats.kstest(t[:200_000], "t", args=(3,)).pvalue > 1e-3
    assert stats.kstest(t[1::2][:200_000], "t", args=(3,)).pvalue > 1e-3      # the sine halves alone
    assert abs(np.median(np.abs(t)) - stats.t.ppf(0.75, 3)) < 1e-2


def test_student_t3_pairs_are_spherical_bivariate_t():
    """(t_a, t_b) of a pair is a spherical bivariate t(3) vector: its squared
    radius over 2 is F(2, 3)-distributed, its angle is uniform, and neither the
    elements of a pair nor neighbouring pairs are correlated (checked on the
    bounded transform tanh so that the heavy tails do not swamp the estimate)."""
    t = orc.noise_row(I.NOISE_STUDENT_T3, 5, 0, 9, 0, 1 << 19).astype(np.float64).reshape(-1, 2)
    rad2 = (t**2).sum(axis=1) / 2.0
    assert stats.kstest(rad2[:200_000], "f", args=(2, 3)).pvalue > 1e-3
    ang = np.arctan2(t[:, 1], t[:, 0])
    assert stats.kstest(ang[:200_000], "uniform", args=(-np.pi, 2 * np.pi)).pvalue > 1e-3
    b = np.tanh(t)
    assert abs(np.corrcoef(b[:, 0], b[:, 1])[0, 1]) < 1e-2
    assert abs(np.corrcoef(b[:-1, 1], b[1:, 0])[0, 1]) < 1e-2


def test_student_t3_radius_accuracy_all_arguments():
    """rho(j) = sqrt(3 ((j 2^-24)^(-2/3) - 1)) for every j = 1 .. 2^24 against
    binary64: within 8 ulp, exact 0 at u = 1, largest value at j = 1."""
    total = 1 << 24
    blk = 1 << 22
    worst = 0.0
    for j0 in range(1, total + 1, blk):
        got = orc.t3_radius_u24_array(j0, blk)
        u = np.arange(j0, j0 + blk, dtype=np.float64) / total
        ref = np.sqrt(3.0 * np.expm1(-(2.0 / 3.0) * np.log(u)))
        ok = ref > 0
        worst = max(worst, float(_ulp_err(got[ok], ref[ok]).max()))
        assert np.all(got >= 0) and np.all(np.isfinite(got))
    assert worst <= 8.0, worst
    assert orc.t3_radius_u24_array(total, 1)[0] == 0.0
    assert abs(orc.t3_radius_u24_array(1, 1)[0] - np.sqrt(3.0 * (2.0**16 - 1))) < 1e-3


def test_student_t3_element_mapping():
    """Element k takes words (0,1) or (2,3) of noise block k/4; the cosine
    goes to the even element of the pair, the sine to the odd one."""
    seed, node, step, N = 1234, 2, 7, 64
    t = orc.noise_row(I.NOISE_STUDENT_T3, seed, node, step, 0, N)
    for k in range(0, N, 2):
        ctr = np.array([k >> 2, node, step, 0], dtype=np.uint32)
        w = orc.philox(ctr, np.array([seed, 0], dtype=np.uint32))
        pair = (k >> 1) & 1
        rho = orc.t3_radius_u24_array((int(w[2 * pair]) >> 8) + 1, 1)[0]
        c, s = orc.sincos_u24_array(int(w[2 * pair + 1]) >> 8, 1)
        assert t[k] == np.float32(rho) * c[0] and t[k + 1] == np.float32(rho) * s[0]


def test_student_t3_iid_distribution_and_independence():
    """The independent-coordinates Student-t(3) noise: every element is t(3), and, unlike the
    spherical pairs, neighbouring elements are INDEPENDENT: their squares are uncorrelated
    (for a spherical pair they share the radius: the same statistic is far from zero there)."""
    t = orc.noise_row(I.NOISE_STUDENT_T3_IID, 77, 1, 4, 0, 1 << 19).astype(np.float64)
    assert stats.kstest(t[:200_000], "t", args=(3,)).pvalue > 1e-3
    assert abs(np.median(np.abs(t)) - stats.t.ppf(0.75, 3)) < 1e-2
    b = np.tanh(t) ** 2                     # bounded, so the heavy tails do not swamp the estimate
    assert abs(np.corrcoef(b[0::2], b[1::2])[0, 1]) < 1e-2
    assert abs(np.corrcoef(b[:-1], b[1:])[0, 1]) < 1e-2
    pairs = np.tanh(orc.noise_row(I.NOISE_STUDENT_T3, 77, 1, 4, 0, 1 << 19).astype(np.float64)) ** 2
    assert np.corrcoef(pairs[0::2], pairs[1::2])[0, 1] > 0.05       # the contrast: a shared radius


def test_student_t3_iid_element_mapping():
    """Element k owns block k of the noise stream: words (0,1) give Z0, Z1 and (2,3) give Z2, Z3
    by Box-Muller (cosine first), and t = Z0 / sqrt((Z1^2 + Z2^2 + Z3^2)/3) -- rebuilt here from the
    oracle's Philox, logarithm and sine/cosine with numpy binary32 arithmetic, and, as a looser
    check of the formula itself, in binary64."""
    seed, node, step, N = 4321, 1, 9, 48
    t = orc.noise_row(I.NOISE_STUDENT_T3_IID, seed, node, step, 0, N)
    f = np.float32
    for k in range(N):
        w = orc.philox(np.array([k, node, step, 0], dtype=np.uint32), np.array([seed, 0], dtype=np.uint32))
        z = []
        for a, b in ((0, 1), (2, 3)):
            lg = orc.log_u24_array((int(w[a]) >> 8) + 1, 1)[0]
            rho = np.sqrt(f(-2.0) * lg, dtype=np.float32)
            c, s = orc.sincos_u24_array(int(w[b]) >> 8, 1)
            z += [f(rho * c[0]), f(rho * s[0])]
        z64 = [float(v) for v in z]
        want64 = z64[0] / np.sqrt((z64[1] ** 2 + z64[2] ** 2 + z64[3] ** 2) / 3.0)
        assert abs(float(t[k]) - want64) <= 1e-5 * max(1.0, abs(want64))
        # binary32, operation by operation (the two fma's as exact binary64 products rounded once)
        q = f(float(z[3]) * float(z[3]) + float(f(float(z[2]) * float(z[2]) + float(f(z[1] * z[1])))))
        want = f(z[0] / np.sqrt(f(q / f(3.0)), dtype=np.float32))
        assert t[k] == want, (k, t[k], want)


def test_noise_none_is_zero():
    assert np.all(orc.noise_row(I.NOISE_NONE, 1, 0, 0, 0, 100) == 0)


def test_rnd24_uniform():
    r = orc.rnd24_row(9, 0, 0, 0, 1 << 20).astype(np.float64)
    assert r.min() >= 0.0 and r.max() < 1.0
    assert np.all(r * 2**24 == np.floor(r * 2**24))
    assert stats.kstest(r[:200_000], "uniform").pvalue > 1e-3


# ----------------------------------------------------------- compressors
def test_levels_grid():
    for b in (1, 2, 4, 8):
        L = (1 << b) - 1
        lv = np.array([orc.level(b, q) for q in range(L + 1)], dtype=np.float64)
        assert lv[0] == -1.0 and lv[-1] == 1.0
        assert np.allclose(np.diff(lv), 2.0 / L, atol=1e-7)
        assert np.allclose(lv, -lv[::-1], atol=0)          # symmetric grid


def test_sign_compressor_closed_forms():
    """C = sign(v) * mean|v|; error energy ||v - C||^2 = ||v||^2 - m s^2, hence
    alpha^2 = 1 - ||v||_1^2 / (m ||v||^2) < 1 (Assumption 1, bounded
    signal-to-noise factor)."""
    rng = np.random.default_rng(1)
    for m in (1, 7, 32, 1000):
        v = rng.standard_normal(m).astype(np.float32)
        s, q, Cv = orc.compress_chunk(I.COMP_SIGN1_L1, 1, v)
        v64 = v.astype(np.float64)
        assert s == np.float32(np.abs(v64).sum() / m)
        assert np.array_equal(q, (v >= 0).astype(np.uint32))
        assert np.array_equal(Cv, np.where(v >= 0, np.float32(s), -np.float32(s)))
        err = ((v64 - Cv) ** 2).sum()
        assert err == pytest.approx((v64**2).sum() - m * s**2, rel=1e-5, abs=1e-6)
        alpha2 = err / (v64**2).sum()
        assert alpha2 < 1.0
        assert alpha2 == pytest.approx(1 - np.abs(v64).sum()**2 / (m * (v64**2).sum()), abs=1e-5)


def test_sign_of_zero_and_nan():
    v = np.array([0.0, -0.0, np.nan, -1.0, 2.0], dtype=np.float32)
    s, q, Cv = orc.compress_chunk(I.COMP_SIGN1_L1, 1, v[[0, 1, 3, 4]])
    assert list(q) == [1, 1, 0, 1]
    s, q, Cv = orc.compress_chunk(I.COMP_SIGN1_L1, 1, v)
    assert q[2] == 0


def _uniform_numpy(v, r, b):
    """Independent restatement of the b-bit quantiser in numpy."""
    L = (1 << b) - 1
    s = np.float32(np.abs(v).max())
    y = (v / s).astype(np.float32)                       # IEEE binary32 division
    hl = np.float32(0.5 * L)
    u = (y.astype(np.float64) * float(hl) + float(hl)).astype(np.float32)  # exact product and sum -> one rounding
    t = np.floor((u + r).astype(np.float32))
    q = np.clip(t, 0, L).astype(np.uint32)
    lv = ((2.0 * q.astype(np.float64) - L) / L).astype(np.float32)
    return s, q, (s * lv).astype(np.float32)


@pytest.mark.parametrize("b", [1, 2, 4, 8])
def test_uniform_quantiser_matches_restatement_and_bounds(b):
    rng = np.random.default_rng(b)
    L = (1 << b) - 1
    for m in (1, 5, 64, 513):
        v = (rng.standard_normal(m) * 10.0 ** rng.uniform(-3, 3)).astype(np.float32)
        r = (rng.integers(0, 2**24, size=m) / 2.0**24).astype(np.float32)
        s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_STOCH_MAXABS, b, v, r)
        s2, q2, C2 = _uniform_numpy(v, r, b)
        assert s == s2 and np.array_equal(q, q2) and np.array_equal(Cv, C2)
        assert q.max() <= L
        # quantisation error below one grid step, extremes coded exactly
        assert np.abs(Cv.astype(np.float64) - v).max() <= 2.0 * s / L * (1 + 1e-6)
        top = np.abs(v) == np.float32(s)
        assert np.array_equal(Cv[top], v[top])


def test_uniform_hand_case():
    rows = [ln.split() for ln in open(os.path.join(GOLD, "hand_case_uniform2bit.txt"))
            if ln.strip() and not ln.startswith("#")]
    v = None
    for r in rows:
        if r[0] == "v":
            v = np.array([float(Fraction(t)) for t in r[1:]], dtype=np.float32)
        elif r[0] == "r":
            rr = np.full(v.shape[0], float(Fraction(r[1])), dtype=np.float32)
            s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_STOCH_MAXABS, 2, v, rr)
            assert s == 1.0
            want = [int(t) for t in r[3:]]
            assert list(q) == want
            assert np.allclose(Cv, [(2 * t - 3) / 3 for t in want], atol=1e-7)
            if Fraction(r[1]) == Fraction(1, 2):
                packed = orc.pack_codes(2, q)
                gold = [x for x in rows if x[0] == "packed_r_half"][0]
                assert int(packed[0]) == int(gold[1], 16)
        elif r[0] == "levels":
            assert np.allclose([orc.level(2, k) for k in range(4)],
                               [float(Fraction(t)) for t in r[1:]], atol=1e-7)


def test_uniform_is_unbiased():
    """E C_k = v_k over the rounding stream (Monte Carlo over seeds)."""
    v = np.array([0.9, -0.37, 0.05, -1.0, 0.61, 0.0, 0.123, -0.77], dtype=np.float32)
    trials = 10_000
    for b in (2, 4):
        acc = np.zeros(8)
        sq = np.zeros(8)
        for t in range(trials):
            r = orc.rnd24_row(1000 + t, 0, 0, 0, 8)
            _, _, Cv = orc.compress_chunk(I.COMP_UNIFORM_STOCH_MAXABS, b, v, r)
            acc += Cv
            sq += Cv.astype(np.float64) ** 2
        mean = acc / trials
        sd = np.sqrt(np.maximum(sq / trials - mean**2, 0) / trials)
        assert np.all(np.abs(mean - v) <= 4.5 * sd + 1e-6), (mean - v, sd)


def test_uniform_degenerate_chunks():
    s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_STOCH_MAXABS, 4, np.zeros(9, np.float32),
                                  np.full(9, 0.5, np.float32))
    assert s == 0.0 and np.all(q == 0) and np.all(Cv == 0.0)
    v = np.array([1.0, np.inf, -2.0], dtype=np.float32)
    s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_STOCH_MAXABS, 4, v, np.zeros(3, np.float32))
    assert s == 0.0 and np.all(q == 0) and np.all(Cv == 0.0)
    v = np.array([1.0, np.nan, -2.0], dtype=np.float32)        # NaN ignored by the max, codes to 0
    s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_STOCH_MAXABS, 4, v, np.zeros(3, np.float32))
    assert s == 2.0 and q[1] == 0 and q[2] == 0 and q[0] == 11   # floor(7.5*0.5+7.5) = 11


def test_identity_compressor():
    v = np.array([1.5, -2.25, 0.0], dtype=np.float32)
    s, q, Cv = orc.compress_chunk(I.COMP_IDENTITY, 32, v)
    assert np.array_equal(Cv, v) and np.array_equal(q.view(np.float32), v)


@pytest.mark.parametrize("b", [1, 2, 4, 8])
def test_pack_layout_and_volume(b):
    """Element k sits at bit (k*b)%32 of word (k*b)/32; the packed size is
    b/32 of the float32 size (Section 5: 4 bits save 7/8, 2 bits 93.75 %)."""
    rng = np.random.default_rng(b)
    m = 1000
    q = rng.integers(0, 1 << b, size=m, dtype=np.uint32)
    words = orc.pack_codes(b, q)
    assert words.shape[0] == (m * b + 31) // 32
    big = 0
    for k in range(m):
        big |= int(q[k]) << (k * b)
    for w in range(words.shape[0]):
        assert int(words[w]) == (big >> (32 * w)) & 0xFFFFFFFF
    assert I.code_words(1 << 20, b) * 32 == (1 << 20) * b
    assert I.code_words(1 << 20, 4) / (1 << 20) == 1 / 8
    assert I.code_words(1 << 20, 2) / (1 << 20) == 1 / 16


# ------------------------------- the paper's own compressor (norm-matched)
@pytest.mark.parametrize("b", [2, 4])
def test_nearest_l2_compressor(b):
    """Section 5, "Compression": b bits per element plus the Euclidean norm; the
    decoded tensor is rescaled to that norm.  Pins: the decoded chunk has the
    norm that was sent; codes are the nearest grid level (brute force over all
    levels); C is proportional to the unit levels; b/32 of the volume."""
    rng = np.random.default_rng(10 + b)
    L = (1 << b) - 1
    levels = np.array([orc.level(b, q) for q in range(L + 1)], dtype=np.float64)
    for m in (1, 9, 64, 512):
        v = (rng.standard_normal(m) * 10.0 ** rng.uniform(-2, 2)).astype(np.float32)
        s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_NEAREST_L2, b, v)
        v64 = v.astype(np.float64)
        assert s == pytest.approx(np.sqrt((v64**2).sum()), rel=2e-7)            # what is sent
        assert np.sqrt((Cv.astype(np.float64)**2).sum()) == pytest.approx(s, rel=1e-6)   # norm matched
        g = np.abs(v64).max()
        nearest = np.abs(v64[:, None] / g - levels[None, :]).argmin(axis=1)
        dist = np.abs(v64[:, None] / g - levels[None, :])
        ties = np.sort(dist, axis=1)
        clear = (ties[:, 1] - ties[:, 0]) > 1e-5 if L > 0 else np.ones(m, bool)
        assert np.array_equal(q[clear], nearest[clear].astype(np.uint32))
        unit = levels[q]
        ratio = s / np.sqrt((unit**2).sum())
        assert np.allclose(Cv, ratio * unit, rtol=3e-7, atol=0)
    # deterministic: the rounding stream is not used
    v = rng.standard_normal(100).astype(np.float32)
    a1 = orc.compress_chunk(I.COMP_UNIFORM_NEAREST_L2, b, v, np.zeros(100, np.float32))
    a2 = orc.compress_chunk(I.COMP_UNIFORM_NEAREST_L2, b, v, np.full(100, 0.9, np.float32))
    assert a1[0] == a2[0] and np.array_equal(a1[1], a2[1]) and np.array_equal(a1[2], a2[2])
    # degenerate chunk
    s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_NEAREST_L2, b, np.zeros(7, np.float32))
    assert s == 0.0 and np.all(q == 0) and np.all(Cv == 0.0)


def test_nearest_l2_hand_case():
    """v = (3, -4, 0, 1) with 2 bits: g = 4, y = (3/4, -1, 0, 1/4), u = 3/2 y + 3/2 =
    (21/8, 0, 3/2, 15/8), codes floor(u + 1/2) = (3, 0, 2, 2), unit levels (1, -1, 1/3, 1/3),
    ||v|| = sqrt(26), ||l|| = sqrt(2 + 2/9) = sqrt(20)/3, C = l * 3 sqrt(26/20)."""
    v = np.array([3.0, -4.0, 0.0, 1.0], dtype=np.float32)
    s, q, Cv = orc.compress_chunk(I.COMP_UNIFORM_NEAREST_L2, 2, v)
    assert list(q) == [3, 0, 2, 2]
    assert s == pytest.approx(np.sqrt(26.0), rel=1e-7)
    ratio = 3.0 * np.sqrt(26.0 / 20.0)
    assert np.allclose(Cv, ratio * np.array([1.0, -1.0, 1 / 3, 1 / 3]), rtol=3e-7)
