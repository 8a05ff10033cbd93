"""Pins of the oracle's quantiser (Eq. 4, Eq. 5, Section IV-A binning) against things other
than itself: hand-worked rational level tables and decision points (tests/golden), a brute
force nearest-level search, exact round trips, symmetry and limits."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import lqsgd_oracle as orc


def _rows(path):
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


def test_level_tables_match_hand_worked_rationals(golden_dir):
    n = 0
    for bits, alpha, k, num, den in _rows(f"{golden_dir}/quantizer_levels.txt"):
        bits, k = int(bits), int(k)
        want = float(Fraction(int(num), int(den)))
        got = orc.level_values(bits, float(alpha))[k]
        assert got == pytest.approx(want, rel=1e-13, abs=0), (bits, alpha, k)
        n += 1
    assert n >= 20


def test_levels_round_trip_exactly_through_the_code(golden_dir):
    """Every level s*l_k quantises to k and dequantises (W=1) back to s*l_k; sign kept."""
    for bits, alpha, k, num, den in _rows(f"{golden_dir}/quantizer_levels.txt"):
        bits, k, alpha = int(bits), int(k), float(alpha)
        for s in (1.0, 0.03125, 3.0):
            for sign in (1.0, -1.0):
                x = np.float32(sign * s * int(num) / int(den))
                # the fp32 rounding of x may not sit exactly on the level; keep cases whose
                # level index is unambiguous (all of them: levels are far from thresholds)
                code = orc.log_quantize(np.array([x]), np.float32(s), bits, alpha)[0]
                neg = 1 if x < 0 else 0
                assert code == (neg << (bits - 1)) | k
                back = orc.average_dequantize([np.array([code])], np.float32(s), bits, alpha)[0]
                want = sign * float(np.float32(s)) * int(num) / int(den)
                if k == 0:
                    assert back == 0.0
                else:
                    assert back == pytest.approx(want, rel=1e-12)


def test_decision_points_match_hand_worked_cases(golden_dir):
    n = 0
    for bits, alpha, s, x, code in _rows(f"{golden_dir}/quantizer_thresholds.txt"):
        got = orc.log_quantize(np.array([float(x)], dtype=np.float32), np.float32(float(s)),
                               int(bits), float(alpha))[0]
        assert int(got) == int(code), (bits, alpha, s, x)
        n += 1
    assert n >= 35


@pytest.mark.parametrize("bits,alpha", [(2, 127.0), (3, 7.0), (4, 127.0), (5, 10.0), (8, 127.0), (8, 255.0)])
def test_nearest_neighbour_matching_brute_force(bits, alpha):
    """Section IV-A: precomputed levels + nearest-neighbour matching.  Brute force over the
    explicit level grid in the companded domain must give the same index as the oracle."""
    rng = np.random.default_rng(bits * 1000 + int(alpha))
    L = 1 << (bits - 1)
    x = np.concatenate([rng.standard_normal(4000), rng.standard_t(3, 4000) * 0.1,
                        [0.0, 1e-30, -1e-30]]).astype(np.float32)
    s = np.float32(np.max(np.abs(x)))
    codes = orc.log_quantize(x, s, bits, alpha)
    t = (np.abs(x) / s).astype(np.float32).astype(np.float64)
    # Eq. 4 written out with plain logs, independently of the oracle's log1p form
    q = np.log(1.0 + alpha * t) / np.log(1.0 + alpha)
    grid = np.arange(L) / (L - 1)
    k_brute = np.argmin(np.abs(q[:, None] - grid[None, :]), axis=1)
    k = codes & (L - 1)
    dist = np.abs(q * (L - 1) - np.floor(q * (L - 1)) - 0.5)
    clear = dist > 1e-9                      # away from exact ties
    assert np.array_equal(k[clear], k_brute[clear])
    assert clear.mean() > 0.999
    assert np.array_equal(codes >> (bits - 1), (x < 0).astype(np.uint8))


def test_compander_pair_closed_form_properties():
    for alpha in (0.5, 7.0, 127.0, 255.0, 1e4):
        x = np.linspace(-1, 1, 2001)
        q = orc.compand(x, alpha)
        assert np.allclose(orc.expand(q, alpha), x, rtol=0, atol=1e-14)      # Eq. 5 inverts Eq. 4
        assert np.array_equal(q, -orc.compand(-x, alpha))                    # odd
        assert np.all(np.diff(q) > 0)                                        # strictly increasing
        assert orc.compand(0.0, alpha) == 0.0
        assert orc.compand(1.0, alpha) == pytest.approx(1.0, abs=1e-15)
        assert orc.compand(-1.0, alpha) == pytest.approx(-1.0, abs=1e-15)
        # concave on [0,1]: more resolution near zero (the stated purpose of the mapping)
        qp = orc.compand(np.linspace(0, 1, 101), alpha)
        assert np.all(np.diff(qp, 2) < 0)
    # alpha -> 0: the mapping tends to the identity
    x = np.linspace(-1, 1, 11)
    assert np.allclose(orc.compand(x, 1e-9), x, atol=1e-8)
    # known values: q(1/ (1+alpha)... ) use alpha = 3: q(1/3) = log 2 / log 4 = 1/2
    assert orc.compand(1.0 / 3.0, 3.0) == pytest.approx(0.5, abs=1e-15)
    assert orc.expand(0.5, 3.0) == pytest.approx(1.0 / 3.0, abs=1e-15)
    assert orc.compand(-3.0 / 15.0, 15.0) == pytest.approx(-0.5, abs=1e-15)


def test_zero_scale_sign_of_zero_and_idempotence():
    x = np.array([0.0, -0.0, 0.0], dtype=np.float32)
    assert np.array_equal(orc.log_quantize(x, np.float32(0), 4, 127.0), [0, 0, 0])
    # negative value that lands on level 0 keeps its sign bit but dequantises to exactly 0
    c = orc.log_quantize(np.array([-1e-6], np.float32), np.float32(1), 4, 127.0)
    assert c[0] == 8
    assert orc.average_dequantize([c], np.float32(1), 4, 127.0)[0] == 0.0
    rng = np.random.default_rng(5)
    x = rng.standard_normal(5000).astype(np.float32)
    for bits in (2, 3, 4, 8):
        s = orc.factor_scale([x])
        c1 = orc.log_quantize(x, s, bits, 127.0)
        y = orc.average_dequantize([c1], s, bits, 127.0).astype(np.float32)
        s2 = orc.factor_scale([y])
        assert s2 == s                                  # full scale is a level
        c2 = orc.log_quantize(y, s2, bits, 127.0)
        k1, k2 = c1 & ((1 << (bits - 1)) - 1), c2 & ((1 << (bits - 1)) - 1)
        assert np.array_equal(k1, k2)                   # quantise(dequantise(quantise)) = quantise
        # x and its level lie between the same two neighbouring levels: the error is below the
        # widest gap between adjacent levels, and relative to |x| it is below sqrt-of-ratio - 1
        lv = orc.level_values(bits, 127.0) * float(s)
        assert np.max(np.abs(y.astype(np.float64) - x)) < np.max(np.diff(lv))


def test_worker_average_is_exact_integer_mean():
    rng = np.random.default_rng(11)
    bits, alpha, W = 4, 127.0, 5
    xs = [rng.standard_normal(300).astype(np.float32) for _ in range(W)]
    s = orc.factor_scale(xs)
    codes = [orc.log_quantize(x, s, bits, alpha) for x in xs]
    a = orc.average_dequantize(codes, s, bits, alpha)
    b = orc.average_dequantize(codes[::-1], s, bits, alpha)
    assert np.array_equal(a, b)                                           # order-independent
    same = orc.average_dequantize([codes[0]] * W, s, bits, alpha)
    one = orc.average_dequantize([codes[0]], s, bits, alpha)
    assert np.array_equal(same, one)                                      # W identical workers = 1 worker
    # hand case: W=2, b=4, alpha=127, codes k=+3 and k=-1 -> S=2, q=2/14=1/7 -> 128^(1/7)=2 -> 1/127
    v = orc.average_dequantize([np.array([3], np.uint8), np.array([8 | 1], np.uint8)],
                               np.float32(2.0), 4, 127.0)
    assert v[0] == pytest.approx(2.0 * 1.0 / 127.0, rel=1e-13)
    # k=+7 and k=+7 with k=-7,-7: mean 0
    v = orc.average_dequantize([np.array([7], np.uint8), np.array([15], np.uint8)], np.float32(1), 4, 127.0)
    assert v[0] == 0.0


def test_value_domain_average_variant():
    """Eq. 5 per worker, then the mean (the parameter-server reading): hand cases with
    b = 4, alpha = 127 (levels (2^k - 1)/127), the one-worker case, and the convexity relation
    to Algorithm 1's order."""
    # k = +3 and k = -1, s = 2:  (7/127 - 1/127) / 2 * 2 = 6/127
    v = orc.dequantize_average([np.array([3], np.uint8), np.array([8 | 1], np.uint8)], np.float32(2.0), 4, 127.0)
    assert v[0] == pytest.approx(6.0 / 127.0, rel=1e-13)
    # k = +7 and k = 0: half of full scale, where the code-domain mean gives (128^(1/2) - 1)/127
    v = orc.dequantize_average([np.array([7], np.uint8), np.array([0], np.uint8)], np.float32(1), 4, 127.0)
    c = orc.average_dequantize([np.array([7], np.uint8), np.array([0], np.uint8)], np.float32(1), 4, 127.0)
    assert v[0] == pytest.approx(0.5, rel=1e-13)
    assert c[0] == pytest.approx((np.sqrt(128.0) - 1) / 127.0, rel=1e-13)
    rng = np.random.default_rng(5)
    bits, alpha, W = 5, 50.0, 6
    xs = [rng.standard_normal(400).astype(np.float32) for _ in range(W)]
    s = orc.factor_scale(xs)
    codes = [orc.log_quantize(x, s, bits, alpha) for x in xs]
    # one worker: both orders are the plain dequantisation
    assert np.array_equal(orc.dequantize_average(codes[:1], s, bits, alpha), orc.average_dequantize(codes[:1], s, bits, alpha))
    # it is the mean of the per-worker dequantised values, whatever the order of the workers
    per = np.stack([orc.average_dequantize([c], s, bits, alpha) for c in codes])
    assert np.allclose(orc.dequantize_average(codes, s, bits, alpha), per.mean(axis=0), rtol=1e-13, atol=1e-13 * float(s))
    assert np.allclose(orc.dequantize_average(codes[::-1], s, bits, alpha), per.mean(axis=0), rtol=1e-13, atol=1e-13 * float(s))
    # expand() is convex on [0, 1] and odd: where all workers agree in sign, averaging after
    # dequantisation is at least as large in magnitude as dequantising the average
    sg = np.stack([orc.signed_levels(c, bits) for c in codes])
    same_sign = (sg >= 0).all(axis=0) | (sg <= 0).all(axis=0)
    a = np.abs(orc.dequantize_average(codes, s, bits, alpha))[same_sign]
    b = np.abs(orc.average_dequantize(codes, s, bits, alpha))[same_sign]
    assert same_sign.sum() > 5 and np.all(a >= b * (1 - 1e-14))
    # exchange_factor routes to it
    x = orc.exchange_factor(xs, bits, alpha, average="values")
    assert np.array_equal(x["mean"], orc.dequantize_average(codes, s, bits, alpha))


def test_column_scales_variant():
    """One scale per column: every column is quantised exactly as if it were a factor of its own
    with the scalar rule; a zero column gets scale 0 and codes 0; the levels of each column
    round-trip with that column's scale."""
    rng = np.random.default_rng(12)
    bits, alpha, W = 4, 127.0, 3
    fs = [(rng.standard_normal((40, 5)) * np.array([1.0, 10.0, 0.01, 0.0, 3.0])).astype(np.float32) for _ in range(W)]
    s = orc.factor_scale(fs, per_column=True)
    assert s.shape == (5,) and s.dtype == np.float32 and s[3] == 0
    assert np.array_equal(s, np.array([orc.factor_scale([f[:, j:j + 1] for f in fs]) for j in range(5)], np.float32))
    x = orc.exchange_factor(fs, bits, alpha, column_scales=True)
    for j in range(5):
        xj = orc.exchange_factor([f[:, j:j + 1] for f in fs], bits, alpha)
        for w in range(W):
            assert np.array_equal(x["codes"][w][:, j], xj["codes"][w][:, 0])
        assert np.array_equal(x["mean"][:, j], xj["mean"][:, 0])
    assert np.all(x["mean"][:, 3] == 0) and all(np.all(c[:, 3] == 0) for c in x["codes"])
    lev = orc.level_values(4, 127.0)
    one = np.stack([np.float32(2.0) * lev, np.float32(0.5) * lev[::-1]], axis=1).astype(np.float32)
    y = orc.exchange_factor([one], 4, 127.0, column_scales=True)
    assert np.array_equal(y["scale"], np.array([2.0, 0.5], np.float32))
    assert np.allclose(y["mean"], one.astype(np.float64), rtol=1e-6, atol=0)
    assert orc.payload_bytes(((6, 5), (1, 9)), 2, 4, 4, column_scales=True) == 6 + 5 + 16 + 36


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 8])
def test_pack_layout_and_size(bits):
    rng = np.random.default_rng(bits)
    for count in (0, 1, 7, 8, 9, 333):
        codes = rng.integers(0, 1 << bits, size=count).astype(np.uint8)
        stream = orc.pack_codes(codes, bits)
        assert stream.size == (count * bits + 7) // 8            # r(n+m)b bits, padded to a byte
        assert np.array_equal(orc.unpack_codes(stream, count, bits), codes)
        # independent statement of the layout: one big little-endian integer
        big = 0
        for i, c in enumerate(codes):
            big |= int(c) << (i * bits)
        assert stream.tobytes() == big.to_bytes(stream.size, "little")
    if bits == 4:
        assert orc.pack_codes(np.array([0x1, 0xF, 0x7], np.uint8), 4).tolist() == [0xF1, 0x07]
    if bits == 3:
        # 5,1,7 -> bits 101 | 001<<3 | 111<<6 = 0b1_1100_1101 -> bytes CD 01
        assert orc.pack_codes(np.array([5, 1, 7], np.uint8), 3).tolist() == [0xCD, 0x01]


def test_near_threshold_count_on_a_hand_worked_threshold():
    """b = 2, alpha = 3: the single decision point sits at compand = 1/2, i.e. |x|/s = (sqrt(4) - 1)/3 = 1/3
    exactly.  fp32(1/3) lies just above 1/3, so of nine consecutive fp32 numbers centred on it exactly two
    have neighbours on both sides of the threshold: fp32(1/3) itself and the number below it."""
    c = np.float32(1.0) / np.float32(3.0)
    assert float(c) > 1.0 / 3.0
    xs = [c]
    for _ in range(4):
        xs.insert(0, np.nextafter(xs[0], np.float32(0)))
        xs.append(np.nextafter(xs[-1], np.float32(1)))
    flags = [orc.near_threshold_count(np.array([x], dtype=np.float32), np.float32(1), 2, 3.0) for x in xs]
    assert flags == [0, 0, 0, 1, 1, 0, 0, 0, 0]
    # the sign and the scale do not matter (|x|/s is the same fp32 number for a power-of-two scale)
    assert orc.near_threshold_count(-np.array(xs, dtype=np.float32) * np.float32(8), np.float32(8), 2, 3.0) == 2
    # zero, a zero scale, and values far from every threshold count nothing
    assert orc.near_threshold_count(np.zeros(5, dtype=np.float32), np.float32(1), 4, 127.0) == 0
    assert orc.near_threshold_count(np.ones(5, dtype=np.float32), np.float32(0), 4, 127.0) == 0
    assert orc.near_threshold_count(np.array([1.0, 0.5], dtype=np.float32), np.float32(1), 2, 3.0) == 0


def test_near_threshold_count_agrees_with_brute_force_over_the_thresholds():
    """Against the definition written with exact thresholds: an entry counts when some decision point b_k
    satisfies below(t) < b_k <= above(t).  Values are planted on and next to every threshold of several
    quantisers, among random ones."""
    rng = np.random.default_rng(5)
    for bits, alpha in [(2, 3.0), (3, 15.0), (4, 127.0), (8, 127.0)]:
        L = orc.magnitude_levels(bits)
        b = np.expm1((np.arange(L - 1) + 0.5) / (L - 1) * np.log1p(alpha)) / alpha          # exact decision points
        near = np.float32(b)
        planted = np.concatenate([near, np.nextafter(near, np.float32(0)), np.nextafter(near, np.float32(2)),
                                  np.nextafter(np.nextafter(near, np.float32(2)), np.float32(2))])
        x = np.concatenate([planted, rng.random(2000).astype(np.float32)]).astype(np.float32)
        lo = np.where(x > 0, np.nextafter(x, np.float32(-1)), np.float32(0)).astype(np.float64)
        hi = np.nextafter(x, np.float32(2)).astype(np.float64)
        want = int(np.count_nonzero(((lo[:, None] < b[None, :]) & (b[None, :] <= hi[:, None])).any(axis=1)))
        assert want >= 2 * (L - 1)
        assert orc.near_threshold_count(x, np.float32(1), bits, alpha) == want, (bits, alpha)
