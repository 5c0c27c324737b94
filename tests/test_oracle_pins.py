"""Pins for the CPU oracle: values the paper prints, closed forms, brute force, invariants.

None of these re-type the oracle's formula and compare it with itself: each pins the oracle to
something fixed by the paper or by arithmetic that a plausible mistake (a dropped zero point, a
wrong level count, a mirrored bit order, a flipped comparison in Eq. 7) would break.
"""
import os

import numpy as np
import pytest

import oracle
import workloads
from oracle import (LAYOUT_BITPLANE, LAYOUT_INTERLEAVED, RANGE_ABSMAX, RANGE_MINMAX, ROUND_NEAREST,
                    ROUND_STOCHASTIC)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
LAYOUTS = [LAYOUT_INTERLEAVED, LAYOUT_BITPLANE]


def ks_for(layout):
    return (2, 4, 8) if layout == LAYOUT_INTERLEAVED else (2, 3, 4, 8)


# ------------------------------------------------------------------ independent bit-at-a-time reader


def brute_read_code(payload_words, i, chunk, k, layout):
    """Code of element i read one bit at a time straight from the stream definition."""
    m, t = divmod(i, chunk)
    base_word = m * (chunk * k // 32)
    code = 0
    for j in range(k):
        if layout == LAYOUT_INTERLEAVED:
            bitpos = k * t + j
            word, bit = base_word + bitpos // 32, bitpos % 32
        else:
            g, lane = divmod(t, 32)
            word, bit = base_word + g * k + j, lane
        code |= ((int(payload_words[word]) >> bit) & 1) << j
    return code


# ------------------------------------------------------------------ the paper's worked example


def _read_example():
    vals = {}
    with open(os.path.join(GOLDEN, "forward_encoder_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *rest = line.split()
            vals[key] = [int(v) for v in rest]
    return vals["value"][0], vals["bits_lsb_first"]


def test_forward_encoder_worked_example_54():
    """Eight one-bit values -> (00110110)_2 = 54 (Forward Encoder example)."""
    value, bits = _read_example()
    assert sum(b << t for t, b in enumerate(bits)) == value == 54
    # put the example's bits on binary digit 1 of eight 2-bit codes; digit 0 gets the complement
    codes = np.zeros(32, dtype=np.uint8)
    for t, b in enumerate(bits):
        codes[t] = (b << 1) | (1 - b)
    words = oracle.pack(codes, 32, 2, LAYOUT_BITPLANE)
    assert words.size == 2
    assert int(words[1]) & 0xFF == 54            # plane of digit 1: the paper's integer
    assert int(words[0]) & 0xFF == (~54) & 0xFF  # plane of digit 0: its complement
    assert int(words[0]) >> 8 == 0 and int(words[1]) >> 8 == 0


def test_k4_two_codes_per_byte_and_k8_plain_bytes():
    """Backward Encoder: two 4-bit codes share an 8-bit integer; 8-bit codes travel as they are."""
    codes4 = np.arange(32, dtype=np.uint8) % 16
    b = oracle.pack(codes4, 32, 4, LAYOUT_INTERLEAVED).view(np.uint8)
    assert b.size == 16
    for i in range(16):
        assert {int(b[i]) & 0xF, int(b[i]) >> 4} == {int(codes4[2 * i]), int(codes4[2 * i + 1])}
        assert int(b[i]) & 0xF == int(codes4[2 * i])  # even element in the low half (this build's reading)
    codes8 = (np.arange(64, dtype=np.uint32) * 37 % 256).astype(np.uint8)
    assert np.array_equal(oracle.pack(codes8, 64, 8, LAYOUT_INTERLEAVED).view(np.uint8), codes8)


# ------------------------------------------------------------------ sizes: Eq. 8 and the size table


def test_payload_size_closed_form():
    """k bits per element, no redundant bits (Eq. 8 with n a multiple of 8)."""
    for n in (32, 64, 4096, 1 << 20):
        for k in (2, 3, 4, 8):
            assert oracle.payload_bytes(n, k) * 8 == n * k
    # padding to whole groups: ceil(n/32) groups of k words
    assert oracle.payload_bytes(1, 3) == 12
    assert oracle.payload_bytes(33, 2) == 16
    # stream = header + one {s,o} pair per chunk (+ pad to 16) + payload
    for n, c, k in [(100, 32, 2), (4096, 4096, 8), (5000, 1024, 4), (1 << 20, 1 << 20, 3)]:
        m = -(-n // c)
        off = -(-(32 + 8 * m) // 16) * 16
        assert oracle.payload_offset(n, c) == off
        assert oracle.stream_bytes(n, c, k) == off + 4 * k * (-(-n // 32))


def test_paper_size_table():
    """The paper's transmitted sizes = N*k/8 bytes + a constant framing of about 1 KB."""
    with open(os.path.join(GOLDEN, "table_transmission_sizes.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for name, orig_kb, s2, s3, s4, su in rows:
        n = int(float(orig_kb) * 1024 / 4)  # fp32 elements
        framing = []
        for k, printed in ((2, s2), (3, s3), (4, s4)):
            payload_kb = oracle.payload_bytes(n, k) / 1024
            assert payload_kb == float(orig_kb) * k / 32
            framing.append(float(printed) - payload_kb)
        # forward: the same framing for every k up to the table's one-decimal rounding
        assert max(framing) - min(framing) <= 0.11 and 0.9 <= min(framing) <= 1.3
        back = float(su) - oracle.payload_bytes(n, 4) / 1024
        assert 0.3 <= back <= 0.7
        # compression ratio tends to 32/k (text after Eq. 8): one range for the whole tensor
        for k in (2, 3, 4):
            ratio = 4 * n / oracle.stream_bytes(n, max(32, -(-n // 32) * 32), k)
            assert abs(ratio - 32 / k) / (32 / k) < 1e-3


# ------------------------------------------------------------------ quantizer against hand-worked values


def test_absmax_codes_by_hand_k4():
    """c = 7 makes s = 1 exactly (k = 4: L = 7); codes are rint(x) + 8, ties to even."""
    x = np.zeros(32, dtype=np.float32)
    hand = [(7.0, 15), (-7.0, 1), (0.0, 8), (0.5, 8), (1.5, 10), (2.5, 10), (-0.5, 8), (-1.5, 6),
            (-2.5, 6), (3.49, 11), (3.51, 12), (-6.6, 1), (6.4, 14), (0.49999, 8), (1.0, 9), (-1.0, 7)]
    for i, (v, _) in enumerate(hand):
        x[i] = v
    codes, meta, flag = oracle.quantize(x, 32, 4)
    assert flag == 0 and meta[0, 0] == 1.0 and meta[0, 1] == 0.0
    assert [int(c) for c in codes[:len(hand)]] == [u for _, u in hand]
    assert all(int(c) == 8 for c in codes[len(hand):])
    xhat = oracle.dequantize(codes, meta, 32, 4, RANGE_ABSMAX)
    assert [float(v) for v in xhat[:4]] == [7.0, -7.0, 0.0, 0.0]
    assert float(xhat[4]) == 2.0 and float(xhat[7]) == -2.0


@pytest.mark.parametrize("k", [2, 3, 4, 8])
def test_absmax_scale_and_extremes(k):
    """s = c/(2^(k-1)-1); the largest-magnitude element gets code +-L and decodes to +-c."""
    L = 2 ** (k - 1) - 1
    x = workloads.random_tensor(256, 7 + k, "normal")
    x[17] = -9.25  # the abs-max, negative on purpose
    codes, meta, _ = oracle.quantize(x, 256, k)
    assert meta[0, 0] == np.float32(np.float32(9.25) / np.float32(L))
    assert int(codes[17]) == 2 ** (k - 1) - L  # = 1: the code -L, never -2^(k-1)
    assert codes.min() >= 1 and codes.max() <= 2 ** k - 1
    xhat = oracle.dequantize(codes, meta, 256, k, RANGE_ABSMAX)
    assert abs(float(xhat[17]) + 9.25) <= 9.25 * 2 ** -23


def test_minmax_codes_by_hand():
    """lo = -1, hi = 2, k = 2: L = 3, s = 1, codes rint(x+1), decode u*1 + (-1)."""
    x = np.full(32, -1.0, dtype=np.float32)
    x[:6] = [2.0, -1.0, 0.0, 0.4, 0.6, 1.5]
    codes, meta, _ = oracle.quantize(x, 32, 2, RANGE_MINMAX)
    assert meta[0, 0] == 1.0 and meta[0, 1] == -1.0
    assert [int(c) for c in codes[:6]] == [3, 0, 1, 1, 2, 2]  # 2.5 -> 2 (ties to even)
    xhat = oracle.dequantize(codes, meta, 32, 2, RANGE_MINMAX)
    assert [float(v) for v in xhat[:6]] == [2.0, -1.0, 0.0, 0.0, 1.0, 1.0]


def test_reciprocal_scale_is_the_quotient_rounded_toward_zero():
    """inv = L / r rounded toward zero, against exact rational arithmetic: inv <= L/r < next float above inv,
    hence r * inv <= L and no product x * inv with |x| <= r can leave the code range (checked in exact
    arithmetic too, and in fp32 on the extreme element)."""
    from fractions import Fraction
    rng = np.random.default_rng(11)
    ranges = np.concatenate([np.exp2(rng.uniform(-100, 100, 3000)), rng.uniform(0.5, 2.0, 3000), [1.0, 3.0, 7.0, 127.0, 255.0]])
    for L in (1.0, 3.0, 7.0, 15.0, 127.0, 255.0):
        for r in ranges.astype(np.float32):
            inv = np.float32(oracle.reciprocal_toward_zero(L, float(r)))
            exact = Fraction(L) / Fraction(float(r))
            assert Fraction(float(inv)) <= exact < Fraction(float(np.nextafter(inv, np.float32(np.inf))))
            assert Fraction(float(r)) * Fraction(float(inv)) <= Fraction(L)
            assert np.float32(r) * inv <= np.float32(L)  # the fp32 product of the extreme element


def test_extreme_element_takes_the_top_code_under_every_draw_of_eq7():
    """With |x * inv| <= L the largest element sits exactly on or just below the top level: stochastic rounding
    gives it L or L - 1, never L + 1 (which a clamp would have to repair), and -L or -L + 1 on the low side."""
    for k in (2, 4, 8):
        L = 2 ** (k - 1) - 1
        zp = 2 ** (k - 1)
        for c in (0.1, 1.0 / 3.0, 0.7, 3.0, 1e-3, 12345.678):
            x = np.array([c, -c, c / 2, 0.0] * 8, dtype=np.float32)
            for seed in range(200):
                codes = oracle.quantize(x, x.size, k, RANGE_ABSMAX, ROUND_STOCHASTIC, seed, 0)[0].astype(int) - zp
                assert set(codes[0::4]) <= {L, L - 1} and set(codes[1::4]) <= {-L, -L + 1}


@pytest.mark.parametrize("k", [2, 4, 8])
def test_per_tensor_range_matches_true_division(k):
    """One chunk >= N is the paper's per-tensor quantizer: codes = round(g / s), s = max|g|/L.
    The oracle multiplies by L/c instead of dividing by s; against float64 true division the codes
    may differ only for values within an ulp of a rounding boundary, and then by one step."""
    g = workloads.generate("cfg2_grad", 0, 1 << 18)
    n = g.size
    codes, meta, _ = oracle.quantize(g, n, k)
    L = 2 ** (k - 1) - 1
    c = np.abs(g).max()
    assert meta[0, 0] == np.float32(c / np.float32(L))
    s64 = float(c) / L
    ref = np.rint(g.astype(np.float64) / s64) + 2 ** (k - 1)
    diff = np.abs(codes.astype(np.int64) - ref.astype(np.int64))
    assert diff.max() <= 1
    assert (diff != 0).mean() < 1e-5


@pytest.mark.parametrize("range_", [RANGE_ABSMAX, RANGE_MINMAX])
@pytest.mark.parametrize("k", [2, 3, 4, 8])
def test_nearest_error_bound_and_monotone(k, range_):
    """|x - xhat| <= s/2 per element (plus rounding slack); codes are monotone in x within a chunk."""
    chunk = 1024
    for kind in ("normal", "relu", "wide"):
        x = workloads.random_tensor(5 * chunk + 100, 3, kind)
        codes, meta, flag = oracle.quantize(x, chunk, k, range_)
        assert flag == 0
        xhat = oracle.dequantize(codes, meta, chunk, k, range_).astype(np.float64)
        s = np.repeat(meta[:, 0].astype(np.float64), chunk)[:x.size]
        levels = 2 ** k
        slack = s * levels * 2.0 ** -21 + np.abs(x.astype(np.float64)) * 2.0 ** -22
        assert np.all(np.abs(x.astype(np.float64) - xhat) <= s / 2 + slack)
        for m in range(meta.shape[0]):
            xs = x[m * chunk:(m + 1) * chunk]
            cs = codes[m * chunk:(m + 1) * chunk].astype(np.int64)
            order = np.argsort(xs, kind="stable")
            assert np.all(np.diff(cs[order]) >= 0)


def test_absmax_decoded_values_are_multiples_of_s():
    x = workloads.random_tensor(4096, 11, "normal")
    codes, meta, _ = oracle.quantize(x, 4096, 4)
    xhat = oracle.dequantize(codes, meta, 4096, 4, RANGE_ABSMAX)
    s = meta[0, 0]
    allowed = {np.float32(np.float32(j) * s) for j in range(-8, 8)}
    assert set(np.unique(xhat)).issubset(allowed)


# ------------------------------------------------------------------ degenerate and non-finite chunks


def test_degenerate_chunks():
    x = np.zeros(96, dtype=np.float32)
    x[32:64] = 3.5            # constant chunk
    x[64:96] = 1e-45          # range so small that L/c overflows
    for k in (2, 4, 8):
        codes, meta, flag = oracle.quantize(x, 32, k)
        assert flag == 0
        assert np.all(codes[:32] == 2 ** (k - 1)) and meta[0, 0] == 0
        assert np.all(codes[64:] == 2 ** (k - 1)) and meta[2, 0] == 0
        assert np.all(codes[32:64] == 2 ** k - 1)  # constant nonzero chunk: every value is +c
        codes, meta, flag = oracle.quantize(x, 32, k, RANGE_MINMAX)
        assert np.all(codes[:64] == 0) and meta[1, 0] == 0 and meta[1, 1] == 3.5
        xhat = oracle.dequantize(codes, meta, 32, k, RANGE_MINMAX)
        assert np.all(xhat[32:64] == 3.5) and np.all(xhat[:32] == 0)


def test_negative_zero_offset_is_canonical():
    x = np.full(32, -0.0, dtype=np.float32)
    _, meta, _ = oracle.quantize(x, 32, 4, RANGE_MINMAX)
    assert meta[0, 1] == 0 and not np.signbit(meta[0, 1])


@pytest.mark.parametrize("bad", [np.nan, np.inf, -np.inf])
@pytest.mark.parametrize("range_", [RANGE_ABSMAX, RANGE_MINMAX])
def test_nonfinite_chunk_flagged_and_degenerate(bad, range_):
    x = workloads.random_tensor(128, 5, "normal")
    x[40] = bad
    codes, meta, flag = oracle.quantize(x, 32, 4, range_)
    assert flag == 1
    zero_point = 8 if range_ == RANGE_ABSMAX else 0
    assert np.all(codes[32:64] == zero_point) and meta[1, 0] == 0 and meta[1, 1] == 0
    assert meta[0, 0] > 0 and meta[2, 0] > 0  # the other chunks are untouched
    xhat = oracle.dequantize(codes, meta, 32, 4, range_)
    assert np.all(xhat[32:64] == 0) and np.all(np.isfinite(xhat))


def test_minmax_range_overflow_is_flagged():
    x = np.zeros(32, dtype=np.float32)
    x[0], x[1] = 3e38, -3e38
    _, meta, flag = oracle.quantize(x, 32, 8, RANGE_MINMAX)
    assert flag == 1 and meta[0, 0] == 0


# ------------------------------------------------------------------ stochastic rounding (Eq. 7)


def test_stochastic_codes_are_floor_or_floor_plus_one_and_integers_fixed():
    """c = L makes t = x exactly: the code is floor(x) or floor(x)+1, and integers never move."""
    k, L = 4, 7
    x = workloads.random_tensor(4096, 21, "uniform") * np.float32(6.9)
    x[0] = 7.0  # pins c = L, inv = 1
    x[1:9] = [-3.0, 2.0, 0.0, 6.0, -7.0, 1.0, -1.0, 5.0]
    for seed in range(5):
        codes, meta, _ = oracle.quantize(x, 4096, k, RANGE_ABSMAX, ROUND_STOCHASTIC, seed, 0)
        assert meta[0, 0] == 1.0
        q = codes.astype(np.int64) - 8
        fl = np.floor(x.astype(np.float64)).astype(np.int64)
        assert np.all((q == fl) | (q == fl + 1))
        assert [int(v) for v in q[:9]] == [7, -3, 2, 0, 6, -7, 1, -1, 5]


def test_stochastic_rounding_is_unbiased_and_uses_the_fraction():
    """Mean of the decoded value over many seeds tends to x; P(round up) = t - floor(t)."""
    k = 8
    x = np.zeros(64, dtype=np.float32)
    x[0] = 127.0  # c = L = 127 -> s = 1, t = x
    fr = np.array([0.25, -0.25, 0.9, -0.9, 3.125, -3.125, 0.5, -0.5, 0.03125, -0.03125, 100.75],
                  dtype=np.float32)
    x[1:1 + fr.size] = fr
    trials = 4096
    acc = np.zeros(64, dtype=np.float64)
    for seed in range(trials):
        codes, meta, _ = oracle.quantize(x, 64, k, RANGE_ABSMAX, ROUND_STOCHASTIC, 1000 + seed, 0)
        acc += codes.astype(np.float64) - 128
    mean = acc / trials
    p = x.astype(np.float64) - np.floor(x.astype(np.float64))
    sigma = np.sqrt(p * (1 - p) / trials)
    assert np.all(np.abs(mean - x) <= 4.5 * sigma + 1e-12)
    # a flipped comparison (U > pr) would give mean = floor + 1 - p: far outside for p = 0.25
    assert abs(mean[1] - 0.25) < 0.05 and abs(mean[2] + 0.25) < 0.05


def test_stochastic_is_deterministic_and_counter_based():
    x = workloads.generate("cfg2_grad", 0, 8192)
    a, _, _ = oracle.quantize(x, 1024, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, 42, 0)
    b, _, _ = oracle.quantize(x, 1024, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, 42, 0)
    c, _, _ = oracle.quantize(x, 1024, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, 43, 0)
    d, _, _ = oracle.quantize(x, 1024, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, 42, 8192)
    assert np.array_equal(a, b) and not np.array_equal(a, c) and not np.array_equal(a, d)
    # the draw of element i depends on rng_offset + i only: coding the second half on its own
    # with rng_offset = 4096 reproduces the second half of the full call
    e, _, _ = oracle.quantize(x[4096:], 1024, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, 42, 4096)
    assert np.array_equal(a[4096:], e)


def test_rng_uniformity():
    """Chi-square over 64 bins for consecutive counters, a few seeds; U in [0,1) on a 2^-24 grid."""
    n, bins = 1 << 16, 64
    for seed in (0, 1, 2 ** 40 + 12345):
        u = np.array([oracle.rng_uniform(seed, 7 * 2 ** 32 - n // 2 + i) for i in range(n)])
        assert u.min() >= 0 and u.max() < 1
        assert np.all(u * 2 ** 24 == np.floor(u * 2 ** 24))
        hist = np.bincount((u * bins).astype(int), minlength=bins)
        chi2 = ((hist - n / bins) ** 2 / (n / bins)).sum()
        assert chi2 < 120  # 63 dof: mean 63, sd 11.2; 120 is > 5 sd
        assert abs(u.mean() - 0.5) < 0.01
        # neighbouring counters are uncorrelated
        assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.02
    # all 32 hash bits move: each bit is set about half of the time
    h = np.array([oracle.rng_hash(9, i) for i in range(1 << 14)], dtype=np.uint64)
    for b in range(32):
        assert abs(((h >> np.uint64(b)) & np.uint64(1)).mean() - 0.5) < 0.03


def fmix32_py(h):
    """MurmurHash3's 32-bit finaliser as published (two multiplies, three xor-shifts)."""
    h ^= h >> 16
    h = (h * 0x85EBCA6B) & 0xFFFFFFFF
    h ^= h >> 13
    h = (h * 0xC2B2AE35) & 0xFFFFFFFF
    h ^= h >> 16
    return h


LANE_MUL = (1, 0x9E3779B1, 0x85EBCA77, 0xC2B2AE3D)


def test_rng_quad_structure_and_finaliser():
    """Counters 4j .. 4j+3 share one finaliser output; counter 4j+m is that word times the m-th odd
    constant (a bijection, so each stays uniform); seed 0 / counter 0 does not sit on fmix32(0) = 0."""
    assert fmix32_py(0) == 0 and fmix32_py(1) == 0x514E28B7  # published finaliser: fixed point and one value
    for seed, j in [(0, 0), (5, 77), (2 ** 63 + 9, 2 ** 40 + 3)]:
        inner = fmix32_py(((j >> 32) ^ (seed & 0xFFFFFFFF) ^ 0x9E3779B9) & 0xFFFFFFFF)
        h = fmix32_py(((j & 0xFFFFFFFF) ^ inner ^ (seed >> 32)) & 0xFFFFFFFF)
        for m in range(4):
            assert oracle.rng_hash(seed, 4 * j + m) == (h * LANE_MUL[m]) & 0xFFFFFFFF
    assert all(oracle.rng_hash(0, m) != 0 for m in range(4)) and all(v % 2 == 1 for v in LANE_MUL)


def test_rng_quads_are_jointly_uniform():
    """The four numbers of a quad, pair by pair: no correlation, and a 16 x 16 chi-square."""
    n = 1 << 16
    u = np.array([oracle.rng_uniform(3, i) for i in range(4 * n)]).reshape(n, 4)
    for a in range(4):
        for b in range(a + 1, 4):
            assert abs(np.corrcoef(u[:, a], u[:, b])[0, 1]) < 0.02
            cells = (u[:, a] * 16).astype(int) * 16 + (u[:, b] * 16).astype(int)
            hist = np.bincount(cells, minlength=256)
            chi2 = ((hist - n / 256) ** 2 / (n / 256)).sum()
            assert chi2 < 360, (a, b, chi2)  # 255 dof: mean 255, sd 22.6
    # sums of the four numbers of a quad behave like sums of independent uniforms (variance 4/12)
    assert abs(u.sum(axis=1).var() - 4 / 12) < 0.01
    # the low bits of the 24 used are as balanced as the high ones
    r = (u * 2 ** 24).astype(np.int64)
    for b in range(24):
        assert abs(((r >> b) & 1).mean() - 0.5) < 0.01


# The reading shares one hash among the four counters of a quad: counter 4j+m takes h * M_m.  Eq. 7 needs each
# U on its own to be uniform (that is what makes the rounding unbiased); what the reading gives up is the
# independence of the four numbers of a quad, which lie on the lattice {h * (M_0, M_1, M_2, M_3) mod 2^32}.
# The pins below are as fine as that reading is bold: the lattice itself is measured (spectral test, exact, over
# the whole period), and the statistics are taken at a resolution where a coarse lattice would show.


def _quad_words(seed, n_quads, first_quad=0):
    return oracle.rng_words(seed, 4 * first_quad, 4 * n_quads).reshape(n_quads, 4)


def _chi2(cells, n_cells):
    hist = np.bincount(cells, minlength=n_cells).astype(np.float64)
    expect = cells.size / n_cells
    return ((hist - expect) ** 2 / expect).sum()


def test_rng_bulk_words_match_single_calls():
    w = oracle.rng_words(2 ** 63 + 5, 2 ** 32 - 6, 12)
    assert [int(v) for v in w] == [oracle.rng_hash(2 ** 63 + 5, 2 ** 32 - 6 + i) for i in range(12)]


def test_rng_quad_pairs_fine_grid():
    """All six pairs of lanes: chi-square over 256 x 256 cells on 2^22 quads (64 per cell)."""
    n = 1 << 22
    top = (_quad_words(11, n) >> 24).astype(np.int64)  # the leading 8 of the 24 bits U uses
    for a in range(4):
        for b in range(a + 1, 4):
            chi2 = _chi2(top[:, a] * 256 + top[:, b], 65536)
            assert abs(chi2 - 65535) < 5 * 362, (a, b, chi2)  # 65535 dof: sd 362


def test_rng_quads_four_dimensional_grid():
    """The four lanes together: chi-square over 8^4 cells on 2^22 quads; a short relation between the lane
    constants would leave whole cells empty."""
    n = 1 << 22
    oct_ = (_quad_words(12, n) >> 29).astype(np.int64)
    cells = ((oct_[:, 0] * 8 + oct_[:, 1]) * 8 + oct_[:, 2]) * 8 + oct_[:, 3]
    chi2 = _chi2(cells, 4096)
    assert abs(chi2 - 4095) < 5 * 90.5, chi2
    # and at 16^4 cells (64 per cell)
    hex_ = (_quad_words(13, n) >> 28).astype(np.int64)
    cells = ((hex_[:, 0] * 16 + hex_[:, 1]) * 16 + hex_[:, 2]) * 16 + hex_[:, 3]
    chi2 = _chi2(cells, 65536)
    assert abs(chi2 - 65535) < 5 * 362, chi2


def test_rng_neighbouring_quads_are_unrelated():
    """Lane m of quad j against lane m' of quad j+1, all sixteen combinations: correlation and a 64 x 64 chi-square."""
    n = 1 << 20
    w = _quad_words(14, n + 1, first_quad=2 ** 30 - n // 2)  # the quad index crosses 2^30: counters cross 2^32
    u = (w >> 8).astype(np.float64) / 2 ** 24
    six = (w >> 26).astype(np.int64)
    for a in range(4):
        for b in range(4):
            assert abs(np.corrcoef(u[:-1, a], u[1:, b])[0, 1]) < 5 / np.sqrt(n), (a, b)
            chi2 = _chi2(six[:-1, a] * 64 + six[1:, b], 4096)
            assert abs(chi2 - 4095) < 5 * 90.5, (a, b, chi2)


def test_rng_quad_lanes_bit_by_bit():
    """Each of the 24 bits U uses of lane a against each of lane b (six pairs of lanes): a pair of bits is
    (1, 1) a quarter of the time, as for independent fair bits -- for every pair of DIFFERENT bit positions
    within 5.5 standard errors.  Bits at the SAME position of two lanes are where the reading shows: bit i of
    h * M is bit i of h plus a carry out of the bits below, and that carry is set slightly more or less than
    half of the time, so P(1, 1) misses 1/4 by up to 0.0096 (a correlation of 0.04 between single bits, largest
    for the lowest bit, i.e. at the 2^-24 end of U).  That bound is pinned too: 0.012."""
    n = 1 << 20
    r = (_quad_words(15, n) >> 8).astype(np.int64)
    bits = [((r[:, m, None] >> np.arange(24)) & 1).astype(np.float32) for m in range(4)]
    sd = np.sqrt(3.0 / 16.0 / n)
    same = np.eye(24, dtype=bool)
    for m in range(4):
        assert np.all(np.abs(bits[m].mean(axis=0) - 0.5) < 5 * 0.5 / np.sqrt(n))
    for a in range(4):
        for b in range(a + 1, 4):
            miss = np.abs(bits[a].T @ bits[b] / n - 0.25)  # 24 x 24 table of P(bit i of a = 1 and bit j of b = 1) - 1/4
            assert np.all(miss[~same] < 5.5 * sd), (a, b, float(miss[~same].max()))
            assert np.all(miss[same] < 0.012), (a, b, float(miss[same].max()))


def _lane_constants():
    """The lane multipliers, recovered from the oracle's own words (a quad whose hash is odd, hence invertible)."""
    j = next(j for j in range(64) if oracle.rng_hash(21, 4 * j) & 1)
    h = oracle.rng_hash(21, 4 * j)
    inv = pow(h, -1, 1 << 32)
    return [(oracle.rng_hash(21, 4 * j + m) * inv) % (1 << 32) for m in range(4)]


def _shortest_relation(mults, reach):
    """Length of the shortest non-zero integer vector c with sum_i c_i * mults[i] = 0 (mod 2^32): the lanes of
    every quad lie on hyperplanes 1 / length apart (the spectral test of a multiplicative lattice), exactly,
    over the whole period.  c_0 is solved for; the others run over [-reach, reach]."""
    mod = 1 << 32
    inv0 = pow(mults[0], -1, mod)
    rng_ = np.arange(-reach, reach + 1, dtype=np.int64)
    grids = np.meshgrid(*([rng_] * min(2, len(mults) - 1)), indexing="ij")
    best = float("inf")
    outer = range(0, reach + 1) if len(mults) == 4 else [None]
    for d in outer:
        s = sum(g * m for g, m in zip(grids, mults[1:]))
        n2 = sum(g * g for g in grids)
        if d is not None:
            s = s + d * mults[3]
            n2 = n2 + d * d
        c0 = (-(s % mod) * inv0) % mod
        c0 = np.where(c0 >= mod // 2, c0 - mod, c0)
        n2 = n2 + c0 * c0
        zero = np.ones_like(n2, dtype=bool)
        for g in grids:
            zero &= g == 0
        if d in (None, 0):
            n2 = np.where(zero, np.int64(1) << 62, n2)
        best = min(best, float(np.sqrt(n2.min())))
    return best


def test_rng_lane_constants_span_a_fine_lattice():
    """Spectral test of the reading: in 2, 3 and 4 dimensions the lanes of a quad lie on hyperplanes that are
    closer than 2^-14.5, 2^-8.5 and 2^-7.5 of the unit cube (the best any lattice of 2^32 points can do is
    about 2^-16.1, 2^-10.8, 2^-8.2): far finer than a k <= 8 bit rounding decision resolves."""
    import itertools
    m = _lane_constants()
    assert m[0] == 1 and all(v % 2 == 1 for v in m) and len(set(m)) == 4
    # a relation shorter than the bound has every coefficient below the bound: that is how far the search reaches
    for a, b in itertools.combinations(range(4), 2):
        assert _shortest_relation([m[a], m[b]], 23171) >= 2 ** 14.5, (a, b)
    for t in itertools.combinations(range(4), 3):
        assert _shortest_relation([m[i] for i in t], 363) >= 2 ** 8.5, t
    assert _shortest_relation(m, 182) >= 2 ** 7.5


# ------------------------------------------------------------------ packing: round trip and brute force


@pytest.mark.parametrize("layout", LAYOUTS)
def test_pack_unpack_every_code_in_every_position(layout):
    for k in ks_for(layout):
        chunk = 64
        for pos in range(chunk):
            for code in range(2 ** k):
                codes = np.zeros(chunk + 32, dtype=np.uint8)  # second (partial) chunk of 32
                codes[pos] = code
                words = oracle.pack(codes, chunk, k, layout)
                assert sum(bin(int(w)).count("1") for w in words) == bin(code).count("1")
                assert np.array_equal(oracle.unpack(words, codes.size, chunk, k, layout), codes)
                assert brute_read_code(words, pos, chunk, k, layout) == code


@pytest.mark.parametrize("layout", LAYOUTS)
def test_stream_against_bit_at_a_time_reader(layout):
    """Whole stream of a ragged tensor: header words, side words and every code read bit by bit."""
    n, chunk = 3 * 96 + 41, 96  # partial last chunk, n not a multiple of 32
    x = workloads.random_tensor(n, 99, "normal")
    for k in ks_for(layout):
        stream, flag = oracle.compress(x, chunk, k, RANGE_ABSMAX, ROUND_NEAREST, layout)
        assert stream.size == oracle.stream_bytes(n, chunk, k) and flag == 0
        header, meta, payload = oracle.split_stream(stream, n, chunk)
        assert [int(h) for h in header] == [0x54504341, 1, n, 0, chunk, k, layout << 16, 0]
        codes, meta_q, _ = oracle.quantize(x, chunk, k)
        assert np.array_equal(meta, meta_q)
        got = [brute_read_code(payload, i, chunk, k, layout) for i in range(n)]
        assert got == [int(c) for c in codes]
        # padding bits are zero: total set bits = set bits of the codes
        assert sum(bin(int(w)).count("1") for w in payload) == sum(bin(int(c)).count("1") for c in codes)
        # decoder + dequantizer reproduce dequantize(codes)
        xhat = oracle.decompress(stream, n)
        assert np.array_equal(xhat, oracle.dequantize(codes, meta, chunk, k, RANGE_ABSMAX))


def test_decompress_rejects_bad_headers():
    x = workloads.random_tensor(100, 1, "normal")
    stream, _ = oracle.compress(x, 32, 4)
    with pytest.raises(ValueError):
        oracle.decompress(stream, 101)
    bad = stream.copy()
    bad[0] ^= 1
    with pytest.raises(ValueError):
        oracle.decompress(bad, 100)
    with pytest.raises(ValueError):
        oracle.decompress(stream[:-4], 100)


def test_chunking_is_local():
    """Chunks are independent: coding a chunk on its own gives the same codes and side words."""
    x = workloads.generate("cfg1_act", 4096 * 3, 4096 * 4)
    codes, meta, _ = oracle.quantize(x, 4096, 8)
    for m in range(4):
        c1, m1, _ = oracle.quantize(x[m * 4096:(m + 1) * 4096], 4096, 8)
        assert np.array_equal(c1, codes[m * 4096:(m + 1) * 4096]) and np.array_equal(m1[0], meta[m])


def test_bitwidth_schedule():
    """Forward 2 -> 3 -> 4 (cap); backward 8 -> 4 at the first learning-rate change."""
    assert [oracle.bitwidth_schedule(False, c) for c in range(5)] == [2, 3, 4, 4, 4]
    assert [oracle.bitwidth_schedule(True, c) for c in range(4)] == [8, 4, 4, 4]
