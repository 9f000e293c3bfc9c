"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-uses the oracle's own arithmetic to produce the expected
value: expectations come from published known-answer vectors, exact rational
arithmetic (fractions), closed forms of the paper's Eq. 4 / Lemma 1, grid fixed
points, brute-force enumeration, numpy library routines and finite differences.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import qesgd_ref as q

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F = Fraction


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as fh:
        return [ln.strip() for ln in fh if ln.strip() and not ln.startswith("#")]


# ----------------------------------------------------------------- Philox --
def test_philox_known_answers():
    rows = _golden_lines("philox4x32_10_kat.txt")
    assert len(rows) == 3
    for row in rows:
        v = [int(x, 16) for x in row.split()]
        out = q.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_draw_is_a_pure_function_of_seed_worker_epoch_element():
    seed, worker, epoch = 0x0123456789ABCDEF, 7, 3
    for block in (0, 1, 12345, (1 << 29) + 5, (1 << 33) + 9):
        x = q.philox4x32_10([block & 0xFFFFFFFF, block >> 32, worker, epoch],
                            [seed & 0xFFFFFFFF, seed >> 32])
        halves = [q.draw16(seed, worker, epoch, 8 * block + j) for j in range(8)]
        words = [halves[2 * w] | (halves[2 * w + 1] << 16) for w in range(4)]
        assert words == [int(v) for v in x]
    base = [q.draw16(seed, worker, epoch, i) for i in range(64)]
    assert base != [q.draw16(seed + 1, worker, epoch, i) for i in range(64)]
    assert base != [q.draw16(seed, worker + 1, epoch, i) for i in range(64)]
    assert base != [q.draw16(seed, worker, epoch + 1, i) for i in range(64)]
    assert base != [q.draw16(seed ^ (1 << 40), worker, epoch, i) for i in range(64)]


def test_draws_look_uniform():
    h = np.array([q.draw16(11, 0, 0, i) for i in range(1 << 16)], dtype=np.float64)
    assert abs(h.mean() / 65536 - 0.5) < 4 / math.sqrt(12 * h.size)
    hist = np.bincount((h // 4096).astype(int), minlength=16)
    expected = h.size / 16
    assert ((hist - expected) ** 2 / expected).sum() < 45  # chi^2, 15 dof, p ~ 1e-4


# -------------------------------------------- rounding probabilities, Eq. 4 --
def _levels_over_all_draws(a, inv, s):
    return np.array([q.level(a, inv, s, h) for h in range(0, 65536)], dtype=np.int64)


@pytest.mark.parametrize("v_over_delta", ["0", "1/3", "5/2", "6.999", "7", "2.0000305", "0.5",
                                          "3.99999", "1e-7", "6.25", "262147/131072",
                                          "65535/131072", "1/131072"])
def test_rounding_probability_matches_eq4(v_over_delta):
    """P(ceil) = (v - delta*floor(v/delta))/delta, P(floor) = 1 - that (Eq. 4),
    realised with 16-bit draws: the count of 'up' draws is exactly the number of
    h with (h + 1/2)/2^16 < p, so it is within 2^-17 of p."""
    s = 7
    scale = np.float32(0.4375)          # delta = scale/s = 1/16 exactly
    inv = np.float32(s) / scale         # 16 exactly
    delta = F(1, 16)
    a = np.float32(float(F(v_over_delta) * delta))
    r_exact = F(float(a)) / delta       # exact because inv is a power of two
    lo = math.floor(r_exact)
    p = r_exact - lo
    lv = _levels_over_all_draws(a, inv, s)
    assert set(np.unique(lv)) <= {lo, lo + 1}
    ups = int((lv == lo + 1).sum())
    expected = sum(1 for h in range(65536) if F(2 * h + 1, 131072) < p)
    assert ups == expected
    assert abs(F(ups, 65536) - p) <= F(1, 131072)
    if p == 0:
        assert ups == 0                 # grid points never move


def test_inverse_spacing_is_the_nearest_float_and_the_top_of_the_range_is_a_fixed_point():
    """inv = fl32(s / scale) is the float nearest to the exact quotient.  For the largest
    coordinate a bucket can hold (|z| = scale) the fp32 product |z| * inv is s or one ulp above
    it (at most 2^-22 above where inv is subnormal, which needs s < 4); Eq. 4's first branch (the
    min) takes it back to s, and even without that branch the overshoot is too small to move a
    draw: ceil(r * 2^16 - 1/2) = s * 2^16 because the overshoot is at most 2^-17 for s <= 127."""
    rng = np.random.default_rng(77)
    for s in (1, 3, 7, 100, 127):
        for trial in range(400):
            scale = np.float32(np.exp(rng.uniform(-40, 40)))
            if trial >= 300:                                  # inv = s / scale is subnormal here
                scale = np.float32(2.0 ** rng.uniform(126, 128) * 0.999)
            inv = q.inv(s, scale)
            exact = F(s) / F(float(scale))
            lo, hi = np.nextafter(inv, np.float32(0)), np.nextafter(inv, np.float32(np.inf))
            assert abs(F(float(inv)) - exact) <= min(abs(F(float(lo)) - exact), abs(F(float(hi)) - exact))
            r = scale * inv                                   # numpy fp32 multiply
            assert r.dtype == np.float32
            assert float(r) - s <= max(float(np.spacing(np.float32(s))), 2.0 ** -22)
            assert math.ceil(F(float(r)) * 65536 - F(1, 2)) <= s * 65536
            for h in (0, 1, 32767, 65535):
                if r >= s:
                    assert q.level(scale, inv, s, h) == s


def test_level_monotone_in_draw_and_bounded():
    rng = np.random.default_rng(5)
    for s in (1, 7, 127):
        for _ in range(20):
            scale = np.float32(rng.uniform(0.01, 3.0))
            inv = np.float32(s) / scale
            a = np.float32(rng.uniform(0, float(scale)))
            lv = _levels_over_all_draws(a, inv, s)[::97]
            assert (np.diff(lv) <= 0).all()      # small h rounds up, large h down
            assert lv.max() <= s and lv.min() >= 0
        # the top of the range is absorbing (first branch of Eq. 4)
        assert q.level(np.float32(10.0), np.float32(s), s, 0) == s


# ------------------------------------------------------------------ scale --
def test_scale_exact_cases():
    z = np.zeros(64, dtype=np.float32)
    z[3], z[40] = 3.0, -4.0
    assert q.bucket_scale(z, q.SCALE_NORM) == np.float32(5.0)
    assert q.bucket_scale(z, q.SCALE_MAX) == np.float32(4.0)
    z = np.zeros(128, dtype=np.float32)
    z[:49] = np.float32(2.0 ** -20)
    assert q.bucket_scale(z, q.SCALE_NORM) == np.float32(7 * 2.0 ** -20)
    z = np.zeros(512, dtype=np.float32)
    z[511] = -1.25e-3
    assert q.bucket_scale(z, q.SCALE_NORM) == np.float32(1.25e-3)
    assert q.bucket_scale(np.zeros(64, np.float32), q.SCALE_NORM) == 0.0


@pytest.mark.parametrize("B", [64, 256, 4096])
def test_norm_scale_within_one_ulp_of_exact(B):
    rng = np.random.default_rng(B)
    for trial in range(6):
        z = (rng.standard_normal(B) * 10.0 ** rng.integers(-6, 3)).astype(np.float32)
        exact = sum(F(float(v)) ** 2 for v in z)
        got = q.bucket_scale(z, q.SCALE_NORM)
        lo, hi = np.nextafter(got, np.float32(0)), np.nextafter(got, np.float32(np.inf))
        assert F(float(lo)) ** 2 < exact < F(float(hi)) ** 2
        assert got >= np.abs(z).max()           # every coordinate inside the range (Lemma 2)
        assert q.bucket_scale(z, q.SCALE_MAX) == np.abs(z).max()


def test_norm_scale_uses_balanced_tree():
    """fp64 sums depend on order; the oracle's is the balanced tree on index
    order.  numpy adding adjacent pairs level by level is that tree."""
    rng = np.random.default_rng(9)
    differs = 0
    for trial in range(40):
        z = (rng.standard_normal(512) * np.exp(rng.uniform(-8, 8, 512))).astype(np.float32)
        x = z.astype(np.float64) ** 2
        seq = 0.0
        for v in x:
            seq += v
        while x.size > 1:
            x = x[0::2] + x[1::2]
        tree = np.float32(np.sqrt(x[0]))
        assert q.bucket_scale(z, q.SCALE_NORM) == tree
        assert q.bucket_sumsq(z) == float(x[0])      # the fp64 sum itself, bit for bit
        differs += float(x[0]) != seq
    assert differs > 0   # the test can tell a tree from a running sum


# ----------------------------------------------------- encode: fixed points --
def _unpack(codes, n, bits):
    per = 32 // bits
    e = np.arange(n)
    return (codes[e // per] >> ((e % per) * bits).astype(np.uint32)) & np.uint32((1 << bits) - 1)


def _signed_levels(codes, n, bits):
    c = _unpack(codes, n, bits).astype(np.int64)
    lv = c & ((1 << (bits - 1)) - 1)
    return np.where(c >> (bits - 1), -lv, lv)


def test_packing_golden_examples():
    for row in _golden_lines("pack_examples.txt"):
        bits_s, levels_s, words_s = [p.strip() for p in row.split("|")]
        bits = int(bits_s)
        k = np.array([int(v) for v in levels_s.split(",")], dtype=np.int64)
        s = (1 << (bits - 1)) - 1
        # on-grid input in max mode: delta = 2^-9, one element pinned at +s*delta
        z = np.zeros(64, dtype=np.float32)
        z[:k.size] = k * 2.0 ** -9
        z[63] = s * 2.0 ** -9
        codes, scales, status = q.encode(z, None, 64, s, bits, q.SCALE_MAX, 1, 0, 0)
        assert status == 0 and scales[0] == np.float32(s * 2.0 ** -9)
        nwords = k.size * bits // 32
        assert [f"{int(w):08x}" for w in codes[:nwords]] == words_s.split()


@pytest.mark.parametrize("bits", [2, 4, 8])
def test_grid_points_are_fixed_points_for_every_seed(bits):
    s = (1 << (bits - 1)) - 1
    rng = np.random.default_rng(bits)
    for seed in range(5):
        n = 64 * 3 + 17
        k = rng.integers(-s, s + 1, size=n)
        k[::64] = s                                     # every bucket reaches the top level
        z = (k * 2.0 ** -12).astype(np.float32)
        codes, scales, status = q.encode(z, None, 64, s, bits, q.SCALE_MAX, seed, seed, 2)
        assert status == 0
        assert (scales == np.float32(s * 2.0 ** -12)).all()
        assert (_signed_levels(codes, n, bits) == k).all()
        assert (_unpack(codes, 4 * 64, bits)[n:] == 0).all()   # padding codes are zero
        assert (q.decode(codes, scales, n, 64, s, bits) == z).all()
    # every one of the 2^bits - 1 used codes round-trips (the "-0" code is never produced)
    k = np.arange(-s, s + 1)
    z = np.zeros(512, dtype=np.float32)
    z[:k.size] = k * 0.5
    codes, scales, _ = q.encode(z, None, 512, s, bits, q.SCALE_MAX, 3, 0, 0)
    assert (_signed_levels(codes, k.size, bits) == k).all()
    assert sorted(set(_unpack(codes, 512, bits).tolist())) == \
        sorted(set(range(0, s + 1)) | set(range((1 << (bits - 1)) + 1, (1 << (bits - 1)) + s + 1)))


def test_no_negative_zero_code():
    """A negative value that rounds to level 0 is encoded as plain 0: the grid has one zero."""
    for bits, s in ((2, 1), (4, 7), (8, 127)):
        z = np.zeros(64, dtype=np.float32)
        z[0] = 1.0
        z[1:40] = -1e-9          # level 0 for every draw that matters
        z[40] = -0.0
        for seed in range(4):
            codes, scales, _ = q.encode(z, None, 64, s, bits, q.SCALE_MAX, seed, 0, 0)
            c = _unpack(codes, 64, bits)
            assert c[0] == s and (c[1:] == 0).all()


def test_norm_mode_single_nonzero_is_exact():
    z = np.zeros(256, dtype=np.float32)
    z[5], z[64 + 9], z[128], z[255] = 0.3, -1e-4, 7.5, -2.0 ** -30
    codes, scales, status = q.encode(z, None, 64, 127, 8, q.SCALE_NORM, 9, 1, 1)
    assert (scales == np.abs(z[[5, 73, 128, 255]])).all()
    lv = _signed_levels(codes, 256, 8)
    assert lv[5] == 127 and lv[73] == -127 and lv[128] == 127 and lv[255] == -127
    assert np.count_nonzero(lv) == 4
    assert (q.decode(codes, scales, 256, 64, 127, 8) == z).all()


def test_delta_is_taken_against_the_anchor():
    """Sec. 2.2: what is compressed is z = u - w_t, formed in fp32."""
    rng = np.random.default_rng(1)
    w = rng.standard_normal(300).astype(np.float32)
    u = (w + 1e-3 * rng.standard_normal(300)).astype(np.float32)
    a = q.encode(u, w, 128, 7, 4, q.SCALE_NORM, 5, 2, 1)
    b = q.encode(u - w, None, 128, 7, 4, q.SCALE_NORM, 5, 2, 1)
    assert (a[0] == b[0]).all() and (a[1] == b[1]).all()
    c = q.encode(w, w, 128, 7, 4, q.SCALE_NORM, 5, 2, 1)
    assert not c[0].any() and not c[1].any()      # zero delta: zero scale, zero codes


def test_slices_with_global_offset_reproduce_the_whole():
    rng = np.random.default_rng(2)
    z = (1e-3 * rng.standard_normal(64 * 9 + 5)).astype(np.float32)
    full = q.encode(z, None, 64, 7, 4, q.SCALE_NORM, 77, 3, 4)
    lo = 64 * 4
    part = q.encode(z[lo:], None, 64, 7, 4, q.SCALE_NORM, 77, 3, 4, i0=lo)
    assert (part[0] == full[0][lo * 4 // 32:]).all() and (part[1] == full[1][4:]).all()
    other = q.encode(z[lo:], None, 64, 7, 4, q.SCALE_NORM, 77, 3, 4, i0=0)
    assert (other[0] != part[0]).any()            # the draw really depends on the global index


def test_nonfinite_and_vanishing_buckets():
    z = (1e-3 * np.random.default_rng(3).standard_normal(256)).astype(np.float32)
    z[70] = np.inf
    z[130] = np.nan
    z[192:] = np.float32(2.0 ** -120)
    for mode in (q.SCALE_NORM, q.SCALE_MAX):
        codes, scales, status = q.encode(z, None, 64, 7, 4, mode, 1, 0, 0)
        assert status == q.STATUS_NONFINITE
        assert scales[0] > 0 and scales[1] == 0 and scales[2] == 0 and scales[3] == 0
        lv = _signed_levels(codes, 256, 4)
        assert lv[:64].any() and not lv[64:].any()
    huge = np.full(64, 3e38, dtype=np.float32)      # norm overflows fp32
    codes, scales, status = q.encode(huge, None, 64, 7, 4, q.SCALE_NORM, 1, 0, 0)
    assert status == q.STATUS_NONFINITE and scales[0] == 0 and not codes.any()
    codes, scales, status = q.encode(huge, None, 64, 7, 4, q.SCALE_MAX, 1, 0, 0)
    assert status == 0 and scales[0] == np.float32(3e38)
    assert (_signed_levels(codes, 64, 4) == 7).all()


# ------------------------------------- unbiasedness, variance (Lemma 1) ------
def _exact_up_probability(a, scale, s):
    """P(ceil) of Eq. 4 in exact rationals, delta = scale/s."""
    delta = F(float(scale)) / s
    r = F(float(a)) / delta
    return math.floor(r), r - math.floor(r), delta


@pytest.mark.parametrize("mode", [q.SCALE_NORM, q.SCALE_MAX])
@pytest.mark.parametrize("s,bits", [(1, 2), (7, 4), (127, 8)])
def test_brute_force_expectation_small_d(mode, s, bits):
    """d <= 8: enumerate all 2^d floor/ceil outcomes with the probabilities of
    Eq. 4 and check E[Q(z)] = z; the oracle's per-element up-frequency over all
    65 536 draws must agree with those probabilities."""
    z = np.array([0.31, -0.77, 0.05, 0.0, -0.2, 0.9, -0.001, 0.45], dtype=np.float32) * 1e-3
    d = z.size
    zz = np.zeros(64, dtype=np.float32)
    zz[:d] = z
    _, scales, _ = q.encode(zz, None, 64, s, bits, mode, 0, 0, 0)
    scale = scales[0]
    inv = q.inv(s, scale)
    floors, probs = [], []
    for i in range(d):
        lo, p, delta = _exact_up_probability(abs(z[i]), scale, s)
        lv = _levels_over_all_draws(abs(z[i]), inv, s)
        # the oracle rounds between the two grid points around its fp32 r = |z| * inv ...
        r_fp = np.float32(abs(z[i])) * inv
        assert set(np.unique(lv)) <= {math.floor(r_fp), math.floor(r_fp) + 1}
        # ... and its mean level is the exact r = |z| / delta up to 2^-17 from the draw
        # resolution and two fp32 roundings (inv and the product), each a factor within
        # 1 +- 2^-24: |r_fp - r| <= r * ((1 + 2^-24)^2 - 1) = r * (2^-23 + 2^-48)
        mean_level = F(int(lv.sum()), 65536)
        assert abs(mean_level - (lo + p)) <= F(1, 131072) + (lo + p) * (F(1, 1 << 23) + F(1, 1 << 48))
        floors.append(lo)
        probs.append(p)
    mean = [F(0)] * d
    total = F(0)
    for outcome in itertools.product((0, 1), repeat=d):
        pr = F(1)
        for i, up in enumerate(outcome):
            pr *= probs[i] if up else 1 - probs[i]
        total += pr
        for i, up in enumerate(outcome):
            mean[i] += pr * (floors[i] + up) * delta
    assert total == 1
    for i in range(d):
        assert mean[i] == F(float(abs(z[i])))        # exact: E[Q(v)] = v inside the range


def test_monte_carlo_unbiased_and_variance_closed_form():
    """Over many epochs (the epoch is part of the counter) the decoded mean
    tends to z and the per-coordinate variance to delta^2 p(1-p) <= delta^2/4
    (proof of Lemma 1); E||Q(z)-z||^2 <= d delta^2/4 (proof of Theorem 1)."""
    rng = np.random.default_rng(4)
    d, B, s, bits, N = 48, 64, 7, 4, 3000
    z = (1e-3 * rng.standard_normal(d)).astype(np.float32)
    acc = np.zeros(d)
    acc2 = np.zeros(d)
    for epoch in range(N):
        codes, scales, _ = q.encode(z, None, B, s, bits, q.SCALE_NORM, 2024, 1, epoch)
        v = q.decode(codes, scales, d, B, s, bits).astype(np.float64)
        acc += v
        acc2 += (v - z) ** 2
    delta = float(scales[0]) / s
    r = np.abs(z.astype(np.float64)) / delta
    p = r - np.floor(r)
    var = delta ** 2 * p * (1 - p)
    mean = acc / N
    assert (np.abs(mean - z) <= 5 * np.sqrt(var / N) + delta * 2.0 ** -16).all()
    emp = acc2 / N
    # (v - z)^2 is a two-point variable: (p delta)^2 w.p. 1-p, ((1-p) delta)^2 w.p. p
    sd = np.abs((p * delta) ** 2 - ((1 - p) * delta) ** 2) * np.sqrt(p * (1 - p))
    assert (np.abs(emp - var) <= 5 * sd / math.sqrt(N) + 1e-6 * delta ** 2).all()
    assert (var <= delta ** 2 / 4).all() and (emp <= delta ** 2 / 4 * 1.05).all()
    assert emp.sum() <= d * delta ** 2 / 4


@pytest.mark.parametrize("mode", [q.SCALE_NORM, q.SCALE_MAX])
@pytest.mark.parametrize("s,bits", [(1, 2), (7, 4), (5, 4), (127, 8)])
def test_error_below_one_grid_step_and_levels_in_range(mode, s, bits):
    rng = np.random.default_rng(s)
    n = 512 * 3 + 100
    z = (1e-3 * rng.standard_normal(n)).astype(np.float32)
    z[rng.random(n) < 0.01] *= 100
    codes, scales, status = q.encode(z, None, 512, s, bits, mode, 8, 0, 0)
    assert status == 0
    lv = _signed_levels(codes, n, bits)
    assert np.abs(lv).max() <= s
    v = q.decode(codes, scales, n, 512, s, bits).astype(np.float64)
    step = np.repeat(scales.astype(np.float64) / s, 512)[:n]
    assert (np.abs(v - z) < step * (1 + 1e-6)).all()
    assert (np.sign(v) * np.sign(z) >= 0).all()
    if mode == q.SCALE_MAX:
        assert (np.abs(lv).reshape(-1)[:512 * 3].reshape(3, 512).max(axis=1) == s).all()


# ---------------------------------------------------------------- decode -----
def test_decode_by_hand():
    # one bucket of 64, 4-bit, s = 7, scale = 0.875 -> delta = 1/8
    k = np.array([0, 1, -1, 7, -7, 3, -4, 2] + [0] * 56)
    words = np.zeros(8, dtype=np.uint32)
    for e, kk in enumerate(k):
        code = (8 if kk < 0 else 0) | abs(int(kk))
        words[e // 8] |= np.uint32(code << (4 * (e % 8)))
    out = q.decode(words, np.array([0.875], np.float32), 64, 64, 7, 4)
    assert (out == k / 8.0).all()
    # delta = fl32(scale / s) with one rounding, value = fl32(level * delta)
    scale = np.float32(0.1)
    out = q.decode(words, np.array([scale], np.float32), 64, 64, 7, 4)
    delta = np.float32(F(float(scale)) / 7)            # correctly rounded quotient
    assert out[3] == np.float32(F(float(delta)) * 7) and out[4] == -out[3]


# ------------------------------------------------ decode-average-apply (A8) --
def test_average_apply_k1_on_grid_returns_the_local_parameter():
    rng = np.random.default_rng(6)
    n, s, bits = 64 * 5, 127, 8
    k = rng.integers(-s, s + 1, n)
    k[::64] = s
    z = (k * 2.0 ** -10).astype(np.float32)
    w = (rng.integers(-1000, 1000, n) * 2.0 ** -10).astype(np.float32)   # w + z exact in fp32
    codes, scales, _ = q.encode(w + z, w, 64, s, bits, q.SCALE_MAX, 1, 0, 0)
    out = q.decode_average_apply(w, codes[None, :], scales[None, :], 64, s, bits)
    assert (out == w + z).all()


def test_average_apply_matches_fp64_mean_of_decoded_workers():
    """Last line of the server task of Algorithm 3: w + (1/K) sum_k z_k."""
    rng = np.random.default_rng(7)
    n, K, B, s, bits = 64 * 4 + 11, 5, 64, 7, 4
    w = (0.05 * rng.standard_normal(n)).astype(np.float32)
    codes, scales, dec = [], [], []
    for k in range(K):
        u = (w + 1e-3 * rng.standard_normal(n)).astype(np.float32)
        c, sc, _ = q.encode(u, w, B, s, bits, q.SCALE_NORM, 3, k, 0)
        codes.append(c)
        scales.append(sc)
        dec.append(q.decode(c, sc, n, B, s, bits).astype(np.float64))
    out = q.decode_average_apply(w, np.stack(codes), np.stack(scales), B, s, bits)
    expect = (w.astype(np.float64) + np.sum(dec, axis=0) / K).astype(np.float32)
    assert (out == expect).all()
    # K copies of one worker average to that worker; order of workers is irrelevant
    same = q.decode_average_apply(w, np.stack([codes[0]] * 4), np.stack([scales[0]] * 4), B, s, bits)
    one = q.decode_average_apply(w, codes[0][None], scales[0][None], B, s, bits)
    assert (same == one).all()
    perm = [3, 1, 4, 0, 2]
    out2 = q.decode_average_apply(w, np.stack([codes[i] for i in perm]),
                                  np.stack([scales[i] for i in perm]), B, s, bits)
    assert np.abs(out2.astype(np.float64) - out).max() <= 2.0 ** -23 * np.abs(out).max()


# ------------------------------------------------ fixed grid spacing (Eq. 4) --
def test_fixed_delta_clips_at_the_top_level():
    """With delta chosen by the caller (Sec. 4, last paragraph) values beyond
    the range take the outermost grid point (first and last branch of Eq. 4)."""
    s, bits, delta = 7, 4, np.float32(2.0 ** -8)
    z = np.zeros(64, dtype=np.float32)
    z[0], z[1], z[2], z[3], z[4] = 1.0, -1.0, 7 * delta, 3 * delta, -2.5 * delta
    ups = 0
    for epoch in range(200):
        codes, scales, status = q.encode(z, None, 64, s, bits, q.SCALE_FIXED, 5, 0, epoch,
                                         fixed_delta=float(delta))
        assert status == 0 and scales[0] == 7 * delta
        lv = _signed_levels(codes, 64, bits)
        assert lv[0] == 7 and lv[1] == -7 and lv[2] == 7 and lv[3] == 3
        assert lv[4] in (-2, -3)
        ups += lv[4] == -3
    assert 60 < ups < 140        # p = 1/2


def test_fixed_delta_nonfinite_values_are_handled_element_by_element():
    """Caller-given spacing, non-finite input (first and last branch of Eq. 4 read on the
    extended reals): +Inf lies above the range and takes the top grid point +s, -Inf the
    bottom one -s, for every draw; NaN is no point of the line at all: code 0 and the
    NONFINITE status.  Nothing couples the elements of a bucket in this mode, so the finite
    neighbours must come out exactly as they do when the non-finite values are replaced by
    zeros, draw for draw."""
    s, bits, delta, B = 7, 4, np.float32(2.0 ** -8), 64
    rng = np.random.default_rng(11)
    base = (rng.standard_normal(2 * B) * 3 * delta).astype(np.float32)
    base[5], base[B + 9] = 2.5 * delta, -6.25 * delta          # known neighbours
    pos, neg, nan = [3, B + 1], [17, B + 40], [30, B + 63]
    bad = base.copy()
    bad[pos], bad[neg], bad[nan] = np.inf, -np.inf, np.nan
    clean = base.copy()
    clean[pos + neg + nan] = 0.0
    seen_5, seen_9 = set(), set()
    for epoch in range(64):
        codes, scales, status = q.encode(bad, None, B, s, bits, q.SCALE_FIXED, 9, 2, epoch,
                                         fixed_delta=float(delta))
        ref_codes, ref_scales, ref_status = q.encode(clean, None, B, s, bits, q.SCALE_FIXED, 9, 2,
                                                     epoch, fixed_delta=float(delta))
        assert status == q.STATUS_NONFINITE and ref_status == 0
        assert (scales == np.float32(s) * delta).all() and (ref_scales == scales).all()
        raw = _unpack(codes, 2 * B, bits)
        lv, ref_lv = _signed_levels(codes, 2 * B, bits), _signed_levels(ref_codes, 2 * B, bits)
        assert (lv[pos] == s).all() and (raw[pos] == s).all()              # +Inf -> +s
        assert (lv[neg] == -s).all() and (raw[neg] == (8 | s)).all()       # -Inf -> -s, sign bit set
        assert (raw[nan] == 0).all()                                       # NaN -> code 0
        others = np.setdiff1d(np.arange(2 * B), pos + neg + nan)
        assert (lv[others] == ref_lv[others]).all()                        # neighbours untouched
        assert lv[5] in (2, 3) and lv[B + 9] in (-6, -7)
        seen_5.add(int(lv[5]))
        seen_9.add(int(lv[B + 9]))
    assert seen_5 == {2, 3} and seen_9 == {-6, -7}     # the neighbours' draws are alive
    # a bucket with only NaN flags, a bucket with only +-Inf does not
    only_inf = np.zeros(B, dtype=np.float32)
    only_inf[0], only_inf[1] = np.inf, -np.inf
    codes, _, status = q.encode(only_inf, None, B, s, bits, q.SCALE_FIXED, 1, 0, 0, fixed_delta=float(delta))
    assert status == 0 and list(_signed_levels(codes, B, bits)[:3]) == [s, -s, 0]
    # decode gives +-s*delta back for the clipped infinities
    out = q.decode(codes, np.full(1, np.float32(s) * delta, dtype=np.float32), B, B, s, bits)
    assert out[0] == s * delta and out[1] == -s * delta and not out[2:].any()


# --------------------------------------------- logistic regression, Eq. 2 ----
def _lr_data(m, d, seed):
    rng = np.random.default_rng(seed)
    X = (rng.standard_normal((m, d)) / np.sqrt(d)).astype(np.float32)
    y = np.where(rng.random(m) < 0.5, 1.0, -1.0).astype(np.float32)
    return X, y


def test_lr_loss_values():
    X, y = _lr_data(9, 33, 0)
    assert abs(q.lr_loss(X, y, np.zeros(33, np.float32)) - math.log(2.0)) < 1e-15
    w = np.random.default_rng(1).standard_normal(33).astype(np.float32)
    t = -(y.astype(np.float64) * (X.astype(np.float64) @ w.astype(np.float64)))
    assert abs(q.lr_loss(X, y, w) - np.logaddexp(0.0, t).mean()) < 1e-13


def test_lr_step_is_gradient_step_of_the_loss():
    """u_new - u = -lr * grad(mean loss): checked by central differences of an
    independent (numpy, fp64) evaluation of the loss of Sec. 1."""
    m, d, lr = 7, 12, 0.25
    X, y = _lr_data(m, d, 2)
    u = (0.5 * np.random.default_rng(3).standard_normal(d)).astype(np.float32)
    Xd, yd = X.astype(np.float64), y.astype(np.float64)

    def loss(w):
        return np.logaddexp(0.0, -yd * (Xd @ w)).mean()

    grad = np.zeros(d)
    eps = 1e-6
    for i in range(d):
        e = np.zeros(d)
        e[i] = eps
        grad[i] = (loss(u.astype(np.float64) + e) - loss(u.astype(np.float64) - e)) / (2 * eps)
    new = q.lr_sgd_step(X, y, lr, u)
    assert np.abs((new.astype(np.float64) - u) + lr * grad).max() < 2e-7


def test_lr_step_from_zero_closed_form_and_epoch_descends():
    m, d, lr = 64, 40, 0.1
    X, y = _lr_data(m * 4, d, 4)
    u0 = np.zeros(d, dtype=np.float32)
    new = q.lr_sgd_step(X[:m], y[:m], lr, u0)
    # at u = 0 every c_j = -y_j/2, so u_1 = lr/(2m) sum_j y_j x_j
    expect = (lr / (2 * m)) * (y[:m, None].astype(np.float64) * X[:m].astype(np.float64)).sum(0)
    assert np.abs(new - expect).max() <= 2.0 ** -24 * np.abs(expect).max() * 1.01
    # a local epoch = consecutive steps in row order, the last batch with its own size
    ep = q.lr_local_epoch(X[:150], y[:150], 64, lr, u0)
    manual = u0
    for lo in (0, 64, 128):
        manual = q.lr_sgd_step(X[lo:min(lo + 64, 150)], y[lo:min(lo + 64, 150)], lr, manual)
    assert (ep == manual).all()
    rate_rng = np.random.default_rng(5)
    w_star = rate_rng.standard_normal(d)
    y2 = np.sign(X.astype(np.float64) @ w_star).astype(np.float32)
    u = np.zeros(d, np.float32)
    before = q.lr_loss(X, y2, u)
    for _ in range(30):
        u = q.lr_local_epoch(X, y2, 64, 2.0, u)
    assert q.lr_loss(X, y2, u) < before - 0.05 and abs(before - math.log(2)) < 1e-12


def test_lr_gradient_against_finite_differences_and_the_step():
    m, d, lr = 9, 14, 0.3
    X, y = _lr_data(m, d, 11)
    w = (0.4 * np.random.default_rng(12).standard_normal(d)).astype(np.float32)
    Xd, yd = X.astype(np.float64), y.astype(np.float64)

    def loss(v):
        return np.logaddexp(0.0, -yd * (Xd @ v)).mean()

    fd = np.zeros(d)
    eps = 1e-6
    for i in range(d):
        e = np.zeros(d)
        e[i] = eps
        fd[i] = (loss(w.astype(np.float64) + e) - loss(w.astype(np.float64) - e)) / (2 * eps)
    g = q.lr_gradient(X, y, w)
    assert np.abs(g - fd).max() < 2e-7
    # Eq. 2: the step is w - lr * g
    step = q.lr_sgd_step(X, y, lr, w)
    assert np.abs(step - (w.astype(np.float64) - lr * g.astype(np.float64))).max() < 1e-7


def test_average_axpy_is_linear_in_alpha_and_reduces_to_average_apply():
    """w + alpha * mean_k g_k: alpha = 1 is the averaging line of Algorithm 3; alpha = -lr is the
    SGD step of Eq. 2 on the mean of the decoded (quantised) gradients."""
    rng = np.random.default_rng(21)
    n, K, B, s, bits = 64 * 3 + 7, 4, 64, 7, 4
    w = (0.05 * rng.standard_normal(n)).astype(np.float32)
    codes, scales, dec = [], [], []
    for k in range(K):
        g = (1e-2 * rng.standard_normal(n)).astype(np.float32)
        c, sc, _ = q.encode(g, None, B, s, bits, q.SCALE_NORM, 3, k, 0)
        codes.append(c)
        scales.append(sc)
        dec.append(q.decode(c, sc, n, B, s, bits).astype(np.float64))
    codes, scales = np.stack(codes), np.stack(scales)
    mean = np.sum(dec, axis=0) / K
    assert (q.decode_average_axpy(w, codes, scales, B, s, bits, 1.0)
            == q.decode_average_apply(w, codes, scales, B, s, bits)).all()
    for alpha in (-0.1, 0.5, -2.0):
        got = q.decode_average_axpy(w, codes, scales, B, s, bits, alpha)
        want = (w.astype(np.float64) + np.float64(np.float32(alpha)) * mean).astype(np.float32)
        assert (got == want).all()
    assert (q.decode_average_axpy(w, codes, scales, B, s, bits, 0.0) == w).all()


# ----------------------------------------- per-step QESGD (Algorithms 2 and 3) --
def test_requantize_is_encode_decode_and_add():
    rng = np.random.default_rng(31)
    n, B, s, bits = 64 * 3 + 9, 64, 7, 4
    w = (0.05 * rng.standard_normal(n)).astype(np.float32)
    u = (w + 1e-3 * rng.standard_normal(n)).astype(np.float32)
    zsum = (1e-3 * rng.standard_normal(n)).astype(np.float32)
    u2, z2, codes, scales, st = q.requantize(u, w, B, s, bits, q.SCALE_NORM, 5, 0, 3, zsum=zsum)
    c, sc, _ = q.encode(u, w, B, s, bits, q.SCALE_NORM, 5, 0, 3)
    v = q.decode(c, sc, n, B, s, bits)
    assert st == 0 and (codes == c).all() and (scales == sc).all()
    assert (u2 == w + v).all() and (z2 == zsum + v).all()         # numpy fp32 adds
    assert np.abs(u2 - u).max() < scales.max() / s                 # moved by less than one grid step
    # a point already on the grid (and exactly representable after the add) stays put
    k = rng.integers(-7, 8, 64)
    k[0] = 7
    wg = (rng.integers(-100, 100, 64) * 2.0 ** -8).astype(np.float32)
    ug = (wg + k * 2.0 ** -8).astype(np.float32)
    u3, _, _, _, _ = q.requantize(ug, wg, 64, 7, 4, q.SCALE_MAX, 1, 0, 0)
    assert (u3 == ug).all()


def test_qesgd_epoch_average_and_eight_bits_track_sgd():
    """Algorithm 2 on a small logistic problem: w_{t+1} = (1/K_t) sum_{k<K_t} u_{t,k}
    = w_t + (1/K_t) sum_k z_{t,k}; with 8 bits the epoch ends close to Epoch-SGD (Algorithm 1),
    as the end of Sec. 4 says."""
    m, d, Kt, lr = 16, 256, 12, 0.5
    rng = np.random.default_rng(41)
    X = (rng.standard_normal((m * Kt, d)) / np.sqrt(d)).astype(np.float32)
    y = np.sign(X.astype(np.float64) @ rng.standard_normal(d)).astype(np.float32)
    w = np.zeros(d, dtype=np.float32)
    delta = 5e-4                                   # grid spacing; the range +-127 * delta is never left
    u, u_sgd = w.copy(), w.copy()
    zsum = np.zeros(d, dtype=np.float32)
    iterates, iterates_sgd = [], []
    for k in range(Kt):
        iterates.append(u.astype(np.float64))
        iterates_sgd.append(u_sgd.astype(np.float64))
        rows = slice(k * m, (k + 1) * m)
        u = q.lr_sgd_step(X[rows], y[rows], lr, u)
        u_sgd = q.lr_sgd_step(X[rows], y[rows], lr, u_sgd)
        acc = zsum if k + 1 < Kt else None         # z_{t,K_t} is not part of the average
        u, znew, _, _, st = q.requantize(u, w, 256, 127, 8, q.SCALE_FIXED, 7, 0, k, zsum=acc,
                                         fixed_delta=delta)
        assert st == 0
        if znew is not None:
            zsum = znew
    w_next = w.astype(np.float64) + zsum.astype(np.float64) / Kt
    assert np.abs(w_next - np.mean(iterates, axis=0)).max() < 1e-6
    w_sgd = np.mean(iterates_sgd, axis=0)
    # quantisation noise per step is at most delta/2 per coordinate and does not accumulate
    assert np.abs(w_next - w_sgd).max() < 4 * delta
    assert abs(q.lr_loss(X, y, w_next.astype(np.float32)) - q.lr_loss(X, y, w_sgd.astype(np.float32))) < 1e-3


def test_invalid_arguments_are_rejected():
    z = np.zeros(64, np.float32)
    for kw in (dict(bucket=48), dict(bucket=32), dict(bucket=16384), dict(bits=3),
               dict(s=8, bits=4), dict(s=0), dict(mode=3), dict(i0=5)):
        args = dict(bucket=64, s=7, bits=4, mode=q.SCALE_NORM, i0=0)
        args.update(kw)
        with pytest.raises(ValueError):
            q.encode(z, None, args["bucket"], args["s"], args["bits"], args["mode"], 0, 0, 0,
                     i0=args["i0"])
