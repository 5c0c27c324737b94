"""GPU parity of the forward quantizer (multi-bit quantization) against the oracle, through the C ABI.

Bar: the whole stream bit-exact -- header, bit planes (the sign decisions are taken in the same
arithmetic on both sides) and the side words alpha_next and m_q: the sums of Eq. 3 and Eq. 5 are taken
without rounding on both sides and rounded once, so they do not depend on the order in which either
side adds; given the same stream, the receiver's output is bit-exact.
"""
import numpy as np
import pytest

import oracle
import workloads
from tests import gpu_util

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _A():
    import paper_2311_05827_b200 as A
    return A


def gpu_mbq_compress(x, k, t, init, alpha_prev):
    A = _A()
    p = A.MbqParams(x.size, k, t, init)
    g_x = gpu_util.guarded_input(torch, x)
    g_prev = None if alpha_prev is None else gpu_util.guarded_input(torch, np.asarray(alpha_prev, dtype=np.float32))
    g_next = gpu_util.guarded_floats(torch, k)
    g_stream = gpu_util.guarded_stream(A, torch, p, 0x77)
    g_ws = gpu_util.guarded_workspace(A, torch, p)
    d_stream, d_ws, d_next = g_stream.bytes, g_ws.view(torch.int32), g_next.view(torch.float32)
    A.accept_mbq_compress(p, g_x.view(torch.float32), None if g_prev is None else g_prev.view(torch.float32), d_next,
                          d_stream, d_ws)
    status = A.accept_last_device_status(d_ws)
    for g, what in ((g_x, "input"), (g_prev, "alpha_prev"), (g_next, "alpha_next"), (g_stream, "stream"), (g_ws, "workspace")):
        if g is not None:
            g.check(what)
    # the call leaves everything but the status word and the residue coefficients of its workspace zeroed
    assert not bool(d_ws.view(torch.uint8)[64:].any()), "exact sums not cleared"
    return p, d_stream, d_next.cpu().numpy(), status, d_ws


def check_mbq(x, k, t, init, alpha_prev):
    A = _A()
    ref_stream, ref_alpha = oracle.mbq_compress(x, k, t, init, alpha_prev)
    p, d_stream, alpha_next, status, d_ws = gpu_mbq_compress(x, k, t, init, alpha_prev)
    got = d_stream.cpu().numpy()
    assert status == 0 and got.size == ref_stream.size
    off = A.accept_mbq_payload_offset(p)
    assert off == oracle.mbq_payload_offset(k)
    assert np.array_equal(got[:32], ref_stream[:32]), "header"
    side_g, side_r = got[32:32 + 4 * (k + 1)].view(np.float32), ref_stream[32:32 + 4 * (k + 1)].view(np.float32)
    assert np.array_equal(side_g.view(np.uint32), side_r.view(np.uint32)), f"side words {side_g} vs {side_r}"
    assert np.array_equal(side_g[:k], alpha_next) and np.array_equal(alpha_next.view(np.uint32), ref_alpha.view(np.uint32))
    assert np.all(got[32 + 4 * (k + 1):off] == 0), "padding"
    bad = np.nonzero(got[off:].view(np.uint32) != ref_stream[off:].view(np.uint32))[0]
    assert bad.size == 0, f"{bad.size} plane words differ, first {bad[:5]}"
    # receiver: the GPU decodes its own stream; the oracle decodes the same bytes
    g_xhat = gpu_util.guarded_floats(torch, x.size)
    d_xhat = g_xhat.view(torch.float32)
    A.accept_mbq_decompress(p, d_stream, d_xhat, d_ws)
    assert A.accept_last_device_status(d_ws) == 0
    g_xhat.check("reconstruction")
    want = oracle.mbq_decompress(got, x.size)
    assert np.array_equal(d_xhat.cpu().numpy().view(np.uint32), want.view(np.uint32))
    return alpha_next, side_g


@pytest.mark.parametrize("k", [2, 3, 4])
@pytest.mark.parametrize("n", [1, 31, 32, 33, 1000, 8192, 8193, 8192 * 5 + 777, 1 << 20])
def test_mbq_parity_shapes(k, n):
    x = workloads.random_tensor(n, 100 + k, "normal")
    alpha_prev = np.array([0.9, 0.5, 0.27, 0.14][:k], dtype=np.float32)
    check_mbq(x, k, 3, False, alpha_prev)
    check_mbq(x, k, 0, True, None)


@pytest.mark.parametrize("k", [2, 3, 4])
def test_mbq_chained_batches_follow_the_oracle(k):
    """Residue initialisation, then batches whose alpha is chained on the device."""
    A = _A()
    n = 8192 * 7 + 100
    alpha = None
    for t in range(0, 6):
        x = workloads.generate("cfg1_act", t * n, n)
        alpha, side = check_mbq(x, k, t, t == 0, alpha)
        assert np.all(np.isfinite(side))
    assert np.all(alpha > 0)


def test_mbq_ties_duplicates_and_unsorted_coefficients():
    """Values exactly on levels and midpoints; equal and unordered coefficients; a zero coefficient."""
    for alpha_prev in ([2.0, 1.0], [1.0, 1.0], [0.25, 2.0, 1.0], [1.0, 0.0, 0.5], [0.5, 0.5, 0.5, 0.5], [3.0, -1.0, 0.5]):
        alpha_prev = np.array(alpha_prev, dtype=np.float32)
        k = alpha_prev.size
        lv = np.unique(oracle.mbq_levels(alpha_prev))
        probe = np.concatenate([lv, (lv[:-1] + lv[1:]) / 2, lv + 1e-6, lv - 1e-6,
                                workloads.random_tensor(5000, k, "normal") * 2]).astype(np.float32)
        check_mbq(probe, k, 2, False, alpha_prev)


@pytest.mark.parametrize("alpha_prev", [
    [0.9, 0.5, 0.27, 0.14],                # well separated levels: the grid search is used
    [1.5829446, 0.88997394, 0.48820832, 0.29352355],
    [1.0, 0.5, 0.25, 0.125 + 1e-4],        # two thresholds 2e-4 apart share a cell: threshold search instead
    [1.0, 0.5, 0.2500001],                 # nearly coinciding levels
    [3e-30, 1.4e-30, 0.6e-30],             # tiny coefficients (the grid's scale is near 1e29)
    [2e37, 1e37],                          # huge ones (levels up to 3e37)
    [1e-39, 4e-40],                        # subnormal coefficients: scale overflows, no grid
    [0.7, 0.3],
])
def test_mbq_level_search_at_thresholds_and_extremes(alpha_prev):
    """Every decision of the nearest-level search: values on, just below and just above each midpoint
    between neighbouring levels, a dense sweep over the span of the levels, and the extremes of fp32."""
    alpha_prev = np.array(alpha_prev, dtype=np.float32)
    k = alpha_prev.size
    lv = np.unique(oracle.mbq_levels(alpha_prev)).astype(np.float64)
    mid = ((lv[:-1] + lv[1:]) / 2).astype(np.float32)
    near = [mid]
    up, down = mid.copy(), mid.copy()
    for _ in range(3):
        up, down = np.nextafter(up, np.float32(np.inf)), np.nextafter(down, np.float32(-np.inf))
        near += [up.copy(), down.copy()]
    span = float(np.abs(lv).max())
    sweep = np.linspace(-1.25 * span, 1.25 * span, 150001).astype(np.float32)
    tiny = np.float32(1e-45)
    extremes = np.array([0.0, -0.0, tiny, -tiny, 1e-38, -1e-38, 3e38, -3e38, 1.0, -1.0], dtype=np.float32)
    probe = np.concatenate(near + [sweep, extremes, lv.astype(np.float32),
                                   workloads.random_tensor(4000, k, "wide") * np.float32(span * 2.0 ** -20)]).astype(np.float32)
    probe = probe[np.isfinite(probe)]
    check_mbq(probe, k, 4, False, alpha_prev)


@pytest.mark.parametrize("i", range(16))
def test_mbq_parity_random_configurations(i):
    """Seeded random (n, k, batch index, coefficients, value distribution), sizes around the 4096-element
    tiles and the 296 groups of the encode pass."""
    rng = np.random.default_rng([20231107, i])
    n = int(rng.choice([int(rng.integers(1, 5000)), int(rng.integers(5000, 300000)), 4096 * 296 + int(rng.integers(-40, 9000)),
                        4096 * int(rng.integers(1, 700))]))
    k = int(rng.integers(2, 5))
    t = int(rng.integers(1, 60))
    kind = str(rng.choice(["normal", "relu", "uniform"]))
    x = workloads.random_tensor(n, 9500 + i, kind) * np.float32(rng.choice([1.0, 1e-3, 37.0]))
    alpha_prev = (np.abs(rng.standard_normal(k)) + 0.02).astype(np.float32) * np.float32(np.abs(x).mean() + 1e-6)
    check_mbq(x, k, t, False, alpha_prev)
    if i % 4 == 0:
        check_mbq(x, k, 0, True, None)


@pytest.mark.parametrize("k", [2, 3, 4])
@pytest.mark.parametrize("kind", ["decades", "cancel", "subnormal", "huge"])
def test_mbq_side_words_are_exact_for_any_magnitudes(k, kind):
    """The sums behind alpha_next and m_q are exact whatever the values: magnitudes spread over the whole
    fp32 range (nearly every value misses the kernel's accumulation window), sums that cancel to a tiny
    remainder, subnormals only, values near the top of the fp32 range.  Side words compared bit for bit."""
    rng = np.random.default_rng([77, k, len(kind)])
    n = 4096 * 9 + 321
    if kind == "decades":
        x = (rng.standard_normal(n) * 10.0 ** rng.uniform(-44, 35, n)).astype(np.float32)
    elif kind == "cancel":
        half = (rng.standard_normal(n // 2) * 10.0 ** rng.uniform(-3, 30, n // 2)).astype(np.float32)
        x = np.concatenate([half, -half, np.float32([1e-30] * (n - 2 * (n // 2)))])
        x = x[rng.permutation(x.size)]
    elif kind == "subnormal":
        x = (rng.integers(-(1 << 22), 1 << 22, n).astype(np.float64) * 2.0 ** -149).astype(np.float32)
    else:
        x = (rng.uniform(-1, 1, n) * 2.0e37).astype(np.float32)  # level sums stay below the fp32 maximum
    x = x[np.isfinite(x)].astype(np.float32)
    scale = np.float32(max(float(np.abs(x.astype(np.float64)).mean()), 1e-40))
    alpha_prev = (np.array([0.9, 0.5, 0.27, 0.14][:k]) * float(scale)).astype(np.float32)
    check_mbq(x, k, 3, False, alpha_prev)
    check_mbq(x, k, 0, True, None)
    # coefficients far from the data: every value falls outside the window placed around the levels
    check_mbq(x, k, 7, False, np.array([1.0, 0.5, 0.25, 0.125][:k], dtype=np.float32))


def test_mbq_singular_system_keeps_alpha():
    x = np.abs(workloads.random_tensor(5000, 3, "normal")) + 10
    alpha_prev = np.array([1.0, 0.5], dtype=np.float32)
    alpha_next, _ = check_mbq(x, 2, 5, False, alpha_prev)
    assert np.array_equal(alpha_next, alpha_prev)


@pytest.mark.parametrize("name,k", [("cfg3_act", 4), ("cfg1_act", 2), ("cfg1_act", 3)])
def test_mbq_workloads(name, k):
    """Post-ReLU activations of the workloads at full size (cfg3: 51M elements), every plane word compared."""
    x = workloads.generate(name)
    stream0, alpha0 = oracle.mbq_compress(x[:1 << 20], k, 0, True)
    check_mbq(x, k, 1, False, alpha0)


def test_mbq_header_mismatch_and_bad_arguments():
    A = _A()
    x = workloads.random_tensor(5000, 1, "normal")
    p, d_stream, _, _, d_ws = gpu_mbq_compress(x, 3, 0, True, None)
    d_xhat = torch.empty(5000, dtype=torch.float32, device="cuda")
    A.accept_mbq_decompress(A.MbqParams(5000, 3), d_stream, d_xhat, d_ws)
    assert A.accept_last_device_status(d_ws) == 0
    big = torch.zeros(A.accept_mbq_compressed_size(A.MbqParams(5000, 4)), dtype=torch.uint8, device="cuda")
    big[:d_stream.numel()] = d_stream
    A.accept_mbq_decompress(A.MbqParams(5000, 4), big, d_xhat, d_ws)
    assert A.accept_last_device_status(d_ws) == A.DEV_BAD_HEADER
    assert A.accept_mbq_check_params(A.MbqParams(0, 3)) == 9
    assert A.accept_mbq_check_params(A.MbqParams(10, 5)) == 2
    assert A.accept_mbq_check_params(A.MbqParams(10, 1)) == 2
    with pytest.raises(A.AcceptError):
        A.accept_mbq_compress(A.MbqParams(5000, 3, 1, False), torch.from_numpy(x).cuda(), None,
                              torch.empty(3, device="cuda"), d_stream, d_ws)


def test_mbq_nonfinite_input_sets_the_status_bit():
    x = workloads.random_tensor(20000, 1, "normal")
    x[777] = np.inf
    _, _, _, status, _ = gpu_mbq_compress(x, 2, 1, False, np.array([1.0, 0.5], dtype=np.float32))
    assert status & 1
