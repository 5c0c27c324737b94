"""Pins for the oracle's forward quantizer (multi-bit quantization, Eq. 1-5): the paper's level set,
library least squares, brute-force nearest level, closed forms and exact-recovery cases."""
import os

import numpy as np
import pytest

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def signs(codes, k):
    """B in {-1,+1}^(n x k) from codes (bit j set <-> +1)."""
    return ((codes[:, None] >> np.arange(k)) & 1).astype(np.float64) * 2 - 1


def test_level_set_of_the_paper_k2():
    rows = dict((l.split()[0], [float(v) for v in l.split()[1:]])
                for l in open(os.path.join(GOLDEN, "mbq_level_set_k2.txt")) if l.strip() and not l.startswith("#"))
    levels = oracle.mbq_levels(rows["alpha"])
    a1, a2 = rows["alpha"]
    assert sorted(levels.tolist()) == sorted([-a1 - a2, a1 - a2, -a1 + a2, a1 + a2]) == sorted(rows["levels"])
    # code bit j set <-> +alpha_j
    assert levels.tolist() == [-a1 - a2, a1 - a2, -a1 + a2, a1 + a2]


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_levels_are_B_alpha(k):
    alpha = np.array([1.7, 0.9, 0.41, 0.2][:k], dtype=np.float32)
    codes = np.arange(1 << k, dtype=np.uint8)
    want = signs(codes, k) @ alpha.astype(np.float64)
    assert np.allclose(oracle.mbq_levels(alpha), want, rtol=0, atol=1e-6)


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_nearest_level_against_brute_force(k):
    rng = np.random.default_rng(k)
    alpha = np.abs(rng.standard_normal(k)).astype(np.float32) + 0.05
    x = workloads.random_tensor(5000, 40 + k, "normal") * np.float32(1.5)
    codes = oracle.mbq_assign_nearest(x, alpha)
    levels = oracle.mbq_levels(alpha).astype(np.float64)
    dist = np.abs(x.astype(np.float64)[:, None] - levels[None, :])
    assert np.array_equal(dist[np.arange(x.size), codes], dist.min(axis=1))
    # a value equal to a level gets that level; a midpoint goes to the lower one
    lv = np.sort(oracle.mbq_levels(np.array([2.0, 1.0][:min(k, 2)], dtype=np.float32)))
    a = np.array([2.0, 1.0][:min(k, 2)], dtype=np.float32)
    probe = np.concatenate([lv, (lv[:-1] + lv[1:]) / 2]).astype(np.float32)
    got = oracle.mbq_levels(a)[oracle.mbq_assign_nearest(probe, a)]
    assert np.array_equal(got[:lv.size], lv) and np.array_equal(got[lv.size:], lv[:-1])


@pytest.mark.parametrize("alpha", [[0.9, 0.5, 0.27, 0.14], [3e-30, 1.4e-30, 0.6e-30], [2e37, 1e37], [1.0, 0.5, 0.2500001]])
def test_nearest_level_is_exact_against_rational_arithmetic(alpha):
    """The closest level, decided in exact rational arithmetic, for values whose distances to two
    levels differ by less than any rounding of the differences could show: next to every midpoint,
    next to zero (between the two innermost levels), and at the far ends of the fp32 range."""
    from fractions import Fraction
    alpha = np.array(alpha, dtype=np.float32)
    levels = oracle.mbq_levels(alpha)
    lv = np.unique(levels).astype(np.float64)
    mid = ((lv[:-1] + lv[1:]) / 2).astype(np.float32)
    probe = [mid]
    up, down = mid.copy(), mid.copy()
    for _ in range(2):
        up, down = np.nextafter(up, np.float32(np.inf)), np.nextafter(down, np.float32(-np.inf))
        probe += [up.copy(), down.copy()]
    tiny = np.float32(1e-45)
    probe.append(np.array([0.0, tiny, -tiny, 1e-38, -1e-38, 1e-20, -1e-20, 3e38, -3e38, 1e10, -1e10, 7.0, -7.0],
                          dtype=np.float32))
    probe = np.concatenate(probe).astype(np.float32)
    codes = oracle.mbq_assign_nearest(probe, alpha)
    exact = [Fraction(float(v)) for v in levels]
    for x, c in zip(probe, codes):
        fx = Fraction(float(x))
        dist = [abs(fx - l) for l in exact]
        best = min(dist)
        # among the levels at the smallest distance: the lowest level, then the smallest code
        want = min((i for i, d in enumerate(dist) if d == best), key=lambda i: (exact[i], i))
        assert c == want, (x, c, want)


def test_duplicate_levels_pick_the_smallest_code():
    alpha = np.array([1.0, 1.0], dtype=np.float32)  # codes 1 and 2 both give level 0
    codes = oracle.mbq_assign_nearest(np.array([0.0, 0.1, -0.1, 0.9], dtype=np.float32), alpha)
    assert codes.tolist() == [1, 1, 1, 1]


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_alpha_update_is_least_squares_plus_moving_average(k):
    """Eq. 3 against numpy's least squares, Eq. 4 with beta = min(0.9, (1+t)/(10+t))."""
    x = workloads.random_tensor(20000, 7, "normal")
    alpha_prev = np.array([0.8, 0.45, 0.25, 0.12][:k], dtype=np.float32)
    codes = oracle.mbq_assign_nearest(x, alpha_prev)
    B = signs(codes, k)
    cur = np.linalg.lstsq(B, x.astype(np.float64), rcond=None)[0]
    for t, beta in [(0, 0.1), (1, 2 / 11), (8, 0.5), (80, 0.9), (1000, 0.9)]:
        want = beta * alpha_prev.astype(np.float64) + (1 - beta) * cur
        got = oracle.mbq_update_alpha(x, codes, alpha_prev, t)
        assert np.allclose(got, want, rtol=2e-7, atol=0)


def test_singular_gram_matrix_keeps_alpha():
    x = np.abs(workloads.random_tensor(512, 3, "normal")) + 10  # far above every level: all signs +1
    alpha_prev = np.array([1.0, 0.5], dtype=np.float32)
    codes = oracle.mbq_assign_nearest(x, alpha_prev)
    assert np.all(codes == 3)
    assert np.array_equal(oracle.mbq_update_alpha(x, codes, alpha_prev, 5), alpha_prev)


@pytest.mark.parametrize("k", [2, 3, 4])
def test_exact_recovery_when_the_data_lies_on_the_levels(k):
    """x drawn from P: the signs are recovered, least squares returns alpha, no error, no bias."""
    alpha = np.array([2.0, 1.0, 0.5, 0.25][:k], dtype=np.float32)  # sums are exact in fp32
    rng = np.random.default_rng(5)
    true_codes = rng.integers(0, 1 << k, 4096).astype(np.uint8)
    x = oracle.mbq_levels(alpha)[true_codes]
    codes = oracle.mbq_assign_nearest(x, alpha)
    assert np.array_equal(codes, true_codes)
    assert np.array_equal(oracle.mbq_update_alpha(x, codes, alpha, 3), alpha)
    assert oracle.mbq_bias(x, codes, alpha) == 0.0
    stream, nxt = oracle.mbq_compress(x, k, 3, False, alpha)
    assert np.array_equal(nxt, alpha) and np.array_equal(oracle.mbq_decompress(stream, x.size), x)


def test_bias_is_the_mean_quantization_error():
    """Eq. 5: m_q = E[x_hat - x]; subtracting it makes the reconstruction's mean equal the data's."""
    x = workloads.generate("cfg1_act", 0, 1 << 15)  # post-ReLU: strongly biased under symmetric levels
    alpha = np.array([0.6, 0.3], dtype=np.float32)
    codes = oracle.mbq_assign_nearest(x, alpha)
    want = (signs(codes, 2) @ alpha.astype(np.float64) - x.astype(np.float64)).mean()
    assert abs(oracle.mbq_bias(x, codes, alpha) - want) <= 1e-7 * max(1.0, abs(want))
    stream, nxt = oracle.mbq_compress(x, 2, 4, False, alpha)
    xhat = oracle.mbq_decompress(stream, x.size)
    assert abs(xhat.astype(np.float64).mean() - x.astype(np.float64).mean()) < 1e-6
    lv = oracle.mbq_levels(nxt).astype(np.float64)
    m_q = float(stream[32 + 8:32 + 12].view(np.float32)[0])
    assert set(np.unique(xhat)).issubset({np.float32(np.float32(v) - np.float32(m_q)) for v in oracle.mbq_levels(nxt)})
    assert lv.size == 4


def test_residue_initialisation():
    """k = 1 is the closed form (sign, mean |x|); more bases never increase the residual energy."""
    x = workloads.random_tensor(10000, 9, "normal")
    codes, a = oracle.mbq_assign_residue(x, 1)
    assert np.array_equal(codes, (x >= 0).astype(np.uint8))
    assert abs(a[0] - np.abs(x.astype(np.float64)).mean()) < 1e-7
    prev = None
    for k in (1, 2, 3, 4):
        codes, a = oracle.mbq_assign_residue(x, k)
        err = np.linalg.norm(signs(codes, k) @ a.astype(np.float64) - x)
        assert prev is None or err < prev
        assert np.all(np.diff(a) < 0) and np.all(a > 0)
        prev = err
    # first basis and coefficient do not depend on k
    assert np.array_equal(codes & 1, (x >= 0).astype(np.uint8))


def test_residue_initialisation_worked_by_hand_k2():
    """Eight values, two bases, every number worked by hand (all of them exact in binary):
         x   =  3     -1     0.5   -2.5    1    -0.5    2    -3.5      sum |x| = 14   -> alpha_0 = 1.75
         b_0 =  +      -      +     -      +     -      +     -
         r_1 =  1.25   0.75  -1.25 -0.75  -0.75  1.25   0.25 -1.75     sum |r_1| = 8  -> alpha_1 = 1
         b_1 =  +      +      -     -      -     +      +     -
       code = [b_0 = +] + 2 [b_1 = +]."""
    x = np.array([3, -1, 0.5, -2.5, 1, -0.5, 2, -3.5], dtype=np.float32)
    codes, alpha = oracle.mbq_assign_residue(x, 2)
    assert alpha.tolist() == [1.75, 1.0]
    assert codes.tolist() == [3, 2, 1, 0, 1, 2, 3, 0]
    # the levels of these coefficients and the reconstruction B alpha of every element, again by hand
    assert oracle.mbq_levels(alpha).tolist() == [-2.75, 0.75, -0.75, 2.75]
    stream, nxt = oracle.mbq_compress(x, 2, 0, True)
    assert nxt.tolist() == [1.75, 1.0]
    # B alpha = 2.75 -0.75 0.75 -2.75 0.75 -0.75 2.75 -2.75; mean(B alpha - x) = (-0.25+0.25+0.25-0.25-0.25-0.25+0.75+0.75)/8
    m_q = float(stream[32 + 8:32 + 12].view(np.float32)[0])
    assert m_q == 1.0 / 8
    assert oracle.mbq_decompress(stream, 8).tolist() == [2.625, -0.875, 0.625, -2.875, 0.625, -0.875, 2.625, -2.875]


def _fraction_sum(values):
    from fractions import Fraction
    return float(sum((Fraction(float(v)) for v in values), Fraction(0)))  # Fraction -> float rounds to nearest, ties to even


def test_exact_sums_against_rational_arithmetic():
    """The sums behind Eq. 3 and Eq. 5 are exact and rounded once: against Python's rational arithmetic and
    math.fsum on magnitudes spread over the whole fp32 range, on sums that cancel, on subnormals, and on exact
    ties between two doubles (which go to the even one)."""
    import math
    rng = np.random.default_rng(2024)
    cases = [
        rng.standard_normal(3000).astype(np.float32),
        (rng.standard_normal(3000) * 10.0 ** rng.uniform(-44, 38, 3000)).astype(np.float32),
        np.float32([2.0 ** 53, 1.0]),                 # 2^53 + 1: tie, the even neighbour is 2^53
        np.float32([2.0 ** 53, 2.0, 1.0]),            # 2^53 + 3: tie, the even neighbour is 2^53 + 4
        np.float32([2.0 ** 53, 1.0, 2.0 ** -149]),    # just above the tie: rounds up
        np.float32([2.0 ** 100, -(2.0 ** 100), 2.0 ** -149, 2.0 ** -149]),
        np.float32([3.0e38] * 500 + [-3.0e38] * 499 + [1e-45] * 7),
        (rng.integers(-(1 << 22), 1 << 22, 999).astype(np.float64) * 2.0 ** -149).astype(np.float32),
    ]
    v = rng.standard_normal(2000).astype(np.float32)
    cases.append(np.concatenate([v, -v[::-1], np.float32([1e-30])]))
    for x in cases:
        x = x[np.isfinite(x)]
        want = _fraction_sum(x)
        assert oracle.exact_sum(x) == want == math.fsum(float(t) for t in x)
        assert oracle.exact_abs_sum(x) == _fraction_sum(np.abs(x))
        codes = rng.integers(0, 4, x.size).astype(np.uint8)
        for p in (0, 1):
            signed = np.where((codes >> p) & 1, x, -x)
            assert oracle.exact_signed_sum(x, codes, p) == _fraction_sum(signed)
    assert oracle.exact_sum(np.float32([2.0 ** 53, 1.0])) == 2.0 ** 53
    assert oracle.exact_sum(np.float32([2.0 ** 53, 2.0, 1.0])) == 2.0 ** 53 + 4
    # an order-independent result: any permutation gives the same bits
    x = cases[1]
    assert oracle.exact_sum(x) == oracle.exact_sum(x[::-1]) == oracle.exact_sum(np.sort(x))


def test_alpha_update_does_not_depend_on_the_order_of_the_elements():
    """Eq. 3-5 are sums over the tensor: permuting the elements (and their codes with them) leaves alpha^t and m_q
    unchanged bit for bit, also where a plain left-to-right float sum would not."""
    rng = np.random.default_rng(8)
    x = (rng.standard_normal(20000) * 10.0 ** rng.uniform(-6, 6, 20000)).astype(np.float32)
    alpha_prev = np.array([40.0, 9.0, 1.5], dtype=np.float32)
    codes = oracle.mbq_assign_nearest(x, alpha_prev)
    a0 = oracle.mbq_update_alpha(x, codes, alpha_prev, 4)
    m0 = oracle.mbq_bias(x, codes, a0)
    for seed in (1, 2, 3):
        perm = np.random.default_rng(seed).permutation(x.size)
        assert np.array_equal(oracle.mbq_update_alpha(x[perm], codes[perm], alpha_prev, 4).view(np.uint32), a0.view(np.uint32))
        assert oracle.mbq_bias(x[perm], codes[perm], a0) == m0


@pytest.mark.parametrize("k", [2, 3, 4])
def test_stream_layout_and_size(k):
    """Side words: alpha (k floats) and m_q, the 32(k+1) bits of Eq. 8; payload k bits per element as planes."""
    n = 1000
    x = workloads.random_tensor(n, k, "normal")
    stream, alpha = oracle.mbq_compress(x, k, 0, True)
    assert stream.size == oracle.mbq_stream_bytes(n, k) == -(-(32 + 4 * (k + 1)) // 16) * 16 + 4 * k * 32
    hdr = stream[:32].view(np.uint32)
    assert [int(v) for v in hdr] == [0x54504341, 1, n, 0, 0, k, 0, 1]
    assert np.array_equal(stream[32:32 + 4 * k].view(np.float32), alpha)
    codes, _ = oracle.mbq_assign_residue(x, k)
    payload = stream[oracle.mbq_payload_offset(k):].view(np.uint32)
    for i in (0, 1, 31, 32, 500, 999):
        got = sum(((int(payload[(i // 32) * k + j]) >> (i % 32)) & 1) << j for j in range(k))
        assert got == int(codes[i])
    # the paper's table: largest MobileNetV2 output, 4096 KB -> 256/384/512 KB of planes (+ framing)
    big = 4096 * 1024 // 4
    assert oracle.mbq_stream_bytes(big, k) - oracle.mbq_payload_offset(k) == big * k // 8
    assert abs(4 * big / oracle.mbq_stream_bytes(big, k) - 32 / k) < 1e-3 * 32 / k


def test_alternating_updates_reduce_the_error():
    """A few batches of the same data: nearest assignment + least squares never increases the error much
    and ends below the residue initialisation (the alternating scheme the paper follows)."""
    x = workloads.generate("cfg1_act", 0, 1 << 15)
    k = 3
    stream, alpha = oracle.mbq_compress(x, k, 0, True)
    e0 = np.linalg.norm(oracle.mbq_decompress(stream, x.size) - x)
    for t in range(1, 30):
        stream, alpha = oracle.mbq_compress(x, k, t, False, alpha)
    e1 = np.linalg.norm(oracle.mbq_decompress(stream, x.size) - x)
    assert e1 < e0
