"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Bar: the whole compressed stream (header words, per-chunk side words, packed payload) is
bit-exact; reconstructed floats agree within 1e-6 * (chunk max - chunk min) -- and are in fact
required to be bit-exact too, since decoding is a fixed sequence of rounded fp32 operations.
"""
import numpy as np
import pytest

import oracle
import workloads
from tests import gpu_util
from oracle import (LAYOUT_BITPLANE, LAYOUT_INTERLEAVED, RANGE_ABSMAX, RANGE_MINMAX, ROUND_NEAREST,
                    ROUND_STOCHASTIC)

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _lib():
    import paper_2311_05827_b200 as A
    return A


def gpu_compress(x_np, chunk, k, range_, round_, layout, seed=0, rng_offset=0, x_dev=None):
    """Every buffer of the call is exactly as large as the size queries say and sits between guard bands
    (tests/gpu_util.py) that must come back untouched: each parity test is a bounds test on the write side."""
    A = _lib()
    n = x_np.size if x_dev is None else x_dev.numel()
    p = A.Params(n, chunk, k, range_, round_, layout, seed, rng_offset)
    g_x = gpu_util.guarded_input(torch, x_np) if x_dev is None else None
    d_x = g_x.view(torch.float32) if x_dev is None else x_dev
    g_stream = gpu_util.guarded_stream(A, torch, p)  # stale bytes inside: all of them must be overwritten
    g_ws = gpu_util.guarded_workspace(A, torch, p)
    d_stream, d_ws = g_stream.bytes, g_ws.view(torch.int32)
    A.accept_compress(p, d_x, d_stream, d_ws)
    status = A.accept_last_device_status(d_ws)
    g_stream.check("stream")
    g_ws.check("workspace")
    if g_x is not None:
        g_x.check("input")
        assert np.array_equal(d_x.cpu().numpy().view(np.uint32), np.ascontiguousarray(x_np).reshape(-1).view(np.uint32)), "input modified"
    return d_stream.cpu().numpy(), status, p, d_stream, d_ws


def gpu_decompress(p, stream_np_or_dev, d_ws=None):
    """The receiver's workspace is 16 bytes (the status word) whatever the parameters; guards as in gpu_compress."""
    A = _lib()
    if torch.is_tensor(stream_np_or_dev):
        d_stream, g_stream = stream_np_or_dev, None
    else:
        g_stream = gpu_util.Guarded(torch, stream_np_or_dev.size)
        g_stream.bytes.copy_(torch.from_numpy(stream_np_or_dev))
        d_stream = g_stream.bytes
    g_xhat = gpu_util.guarded_floats(torch, p.n_elems)
    d_xhat = g_xhat.view(torch.float32)
    g_ws = gpu_util.guarded_workspace(A, torch, p, 16)
    A.accept_decompress(p, d_stream, d_xhat, g_ws.view(torch.int32))
    status = A.accept_last_device_status(g_ws.view(torch.int32))
    g_xhat.check("reconstruction")
    g_ws.check("receiver workspace")
    if g_stream is not None:
        g_stream.check("received stream")
    return d_xhat.cpu().numpy(), status


def assert_float_parity(xhat_gpu, xhat_ref, x, chunk):
    """Stated tolerance (1e-6 of the chunk's max - min), then the stricter bit-exact check."""
    n = x.size
    m = -(-n // chunk)
    pad = m * chunk - n
    xp = np.concatenate([x, np.full(pad, x[-1], dtype=np.float32)]).reshape(m, chunk).astype(np.float64)
    span = np.repeat(xp.max(axis=1) - xp.min(axis=1), chunk)[:n]
    assert np.all(np.abs(xhat_gpu.astype(np.float64) - xhat_ref.astype(np.float64)) <= 1e-6 * span)
    assert np.array_equal(xhat_gpu.view(np.uint32), xhat_ref.view(np.uint32))


def check_roundtrip(x, chunk, k, range_, round_, layout, seed=0, rng_offset=0):
    ref_stream, ref_flag = oracle.compress(x, chunk, k, range_, round_, layout, seed, rng_offset)
    got_stream, status, p, d_stream, d_ws = gpu_compress(x, chunk, k, range_, round_, layout, seed, rng_offset)
    assert got_stream.size == ref_stream.size
    if not np.array_equal(got_stream, ref_stream):
        hdr_g, meta_g, pay_g = oracle.split_stream(got_stream, x.size, chunk)
        hdr_r, meta_r, pay_r = oracle.split_stream(ref_stream, x.size, chunk)
        assert np.array_equal(hdr_g, hdr_r), "header words differ"
        bad = np.nonzero(meta_g.view(np.uint32) != meta_r.view(np.uint32))
        assert bad[0].size == 0, f"side words differ first at chunk {bad[0][:4]}: {meta_g[bad[0][:4]]} vs {meta_r[bad[0][:4]]}"
        badw = np.nonzero(pay_g != pay_r)[0]
        assert badw.size == 0, f"{badw.size} payload words differ, first {badw[:8]}"
        raise AssertionError("streams differ outside header/meta/payload (padding)")
    assert (status & 1) == ref_flag
    xhat_ref = oracle.decompress(ref_stream, x.size)
    xhat_gpu, status2 = gpu_decompress(p, d_stream)
    assert status2 == 0
    if ref_flag == 0:
        assert_float_parity(xhat_gpu, xhat_ref, x, chunk)
    else:
        assert np.array_equal(xhat_gpu.view(np.uint32), xhat_ref.view(np.uint32))


def modes():
    out = []
    for layout in (LAYOUT_INTERLEAVED, LAYOUT_BITPLANE):
        for k in ((2, 4, 8) if layout == LAYOUT_INTERLEAVED else (2, 3, 4, 8)):
            for range_ in (RANGE_ABSMAX, RANGE_MINMAX):
                for round_ in (ROUND_NEAREST, ROUND_STOCHASTIC):
                    out.append((k, range_, round_, layout))
    return out


MODE_IDS = [f"k{k}-{'absmax' if r == 0 else 'minmax'}-{'rn' if d == 0 else 'sr'}-{'il' if l == 0 else 'bp'}"
            for k, r, d, l in modes()]


# ------------------------------------------------------------------ shapes spanning tiles and ragged tails


@pytest.mark.parametrize("mode", modes(), ids=MODE_IDS)
@pytest.mark.parametrize("chunk,n", [
    (4096, 4096 * 37 + 1234),   # register path (2 rounds, 256 threads per chunk) + partial chunk
    (1024, 1024 * 131 + 1),     # 64 threads per chunk, four chunks per block, last block part idle
    (512, 512 * 9),             # one warp per chunk
    (256, 256 * 21 + 77),       # one round
    (2048, 2048 * 5 + 2047),
    (96, 96 * 50 + 40),         # any-shape coder only
    (32, 1000),
])
def test_parity_shapes(mode, chunk, n):
    k, range_, round_, layout = mode
    x = workloads.random_tensor(n, 17 * chunk + k, "normal")
    check_roundtrip(x, chunk, k, range_, round_, layout, seed=0x1234567890ABCDEF, rng_offset=3)


@pytest.mark.parametrize("chunk", [8192, 16384, 32768, 1 << 20])
@pytest.mark.parametrize("mode", [(4, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_BITPLANE),
                                  (8, RANGE_MINMAX, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED)])
def test_parity_large_chunks(chunk, mode):
    """512- and 1024-thread groups, four rounds, and a chunk far larger than a block holds."""
    k, range_, round_, layout = mode
    n = min(3 * chunk + 333, (1 << 21) + 333)
    x = workloads.random_tensor(n, chunk, "relu")
    check_roundtrip(x, chunk, k, range_, round_, layout, seed=5)


@pytest.mark.parametrize("mode", modes(), ids=MODE_IDS)
@pytest.mark.parametrize("chunk,n", [
    (32800, 32800 * 5 + 12345),      # not a power of two: blocks of the range pass straddle chunk boundaries
    (65536, 65536 * 3 + 8191),       # n not a multiple of 8: a partly filled last octet
    (1 << 18, (1 << 18) + 33),
    (1 << 21, 1500003),              # one range for the whole tensor (chunk >= n)
])
def test_parity_wide_chunks(mode, chunk, n):
    """Chunks above 32768 elements: ranges gathered in the workspace, constants, then encode."""
    k, range_, round_, layout = mode
    x = workloads.random_tensor(n, chunk + k, "normal")
    check_roundtrip(x, chunk, k, range_, round_, layout, seed=77, rng_offset=2 ** 32 - 70000)


@pytest.mark.parametrize("bad", [np.nan, -np.inf])
def test_wide_chunks_degenerate_and_nonfinite(bad):
    chunk = 40000 // 32 * 32
    x = workloads.random_tensor(chunk * 6 + 5, 3, "normal")
    x[:chunk] = 0.0                  # all-zero chunk
    x[chunk:2 * chunk] = 1e-42       # L/c overflows
    x[2 * chunk:3 * chunk] = -7.0    # constant chunk
    for range_ in (RANGE_ABSMAX, RANGE_MINMAX):
        check_roundtrip(x, chunk, 4, range_, ROUND_NEAREST, LAYOUT_BITPLANE)
        check_roundtrip(x, chunk, 8, range_, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, seed=3)
    x[4 * chunk + 17] = bad
    x[-1] = bad                      # also in the partial last chunk
    for range_ in (RANGE_ABSMAX, RANGE_MINMAX):
        check_roundtrip(x, chunk, 4, range_, ROUND_NEAREST, LAYOUT_INTERLEAVED)
        check_roundtrip(x, chunk, 2, range_, ROUND_STOCHASTIC, LAYOUT_BITPLANE, seed=4)


def test_per_tensor_range_on_a_large_tensor():
    """The paper's granularity (one scaling factor per tensor) on the 205 MB gradient, every element."""
    spec = workloads.TENSORS["cfg3_grad"]
    x = workloads.generate("cfg3_grad")
    chunk = (x.size + 31) // 32 * 32
    check_roundtrip(x, chunk, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, seed=spec.seed)
    check_roundtrip(x, chunk, 8, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_INTERLEAVED)


@pytest.mark.parametrize("n", [1, 2, 7, 8, 9, 31, 32, 33, 63, 255, 257, 4095, 4097])
def test_parity_tiny_and_ragged(n):
    for k, range_, round_, layout in [(2, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_INTERLEAVED),
                                      (3, RANGE_MINMAX, ROUND_NEAREST, LAYOUT_BITPLANE),
                                      (4, RANGE_ABSMAX, ROUND_STOCHASTIC, LAYOUT_BITPLANE),
                                      (8, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_INTERLEAVED)]:
        x = workloads.random_tensor(n, n + k, "normal")
        for chunk in (32, 256, 4096):
            check_roundtrip(x, chunk, k, range_, round_, layout, seed=n)


def test_per_tensor_range_is_one_chunk():
    """chunk >= N reproduces the paper's one-range-per-tensor scheme."""
    x = workloads.generate("cfg2_grad", 0, 100000)
    for k in (4, 8):
        check_roundtrip(x, 100000 // 32 * 32 + 32, k, RANGE_ABSMAX, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, seed=9)


# ------------------------------------------------------------------ degenerate values


def edge_tensor(chunk):
    x = workloads.random_tensor(chunk * 12, 77, "normal")
    x[0 * chunk:1 * chunk] = 0.0                      # all-zero chunk
    x[1 * chunk:2 * chunk] = -2.5                     # constant chunk
    x[2 * chunk:3 * chunk] = np.float32(1e-42)        # denormals only: L/c overflows
    x[3 * chunk + 5] = np.float32(3e38)               # one huge outlier
    x[4 * chunk:5 * chunk:2] = -0.0                   # negative zeros among values
    x[5 * chunk:6 * chunk] = -0.0                     # all negative zero
    x[6 * chunk:7 * chunk] *= np.float32(1e-39)       # denormal-scale values
    x[7 * chunk + 1] = np.float32(-3e38)
    x[7 * chunk + 2] = np.float32(3e38)               # min/max range overflows
    x[8 * chunk:9 * chunk] = np.abs(x[8 * chunk:9 * chunk])
    x[9 * chunk + 3] = np.float32(1e-30)
    x[9 * chunk:10 * chunk] *= np.float32(1e-30)
    return x


@pytest.mark.parametrize("chunk", [32, 512, 4096])
@pytest.mark.parametrize("mode", modes(), ids=MODE_IDS)
def test_parity_degenerate_values(chunk, mode):
    k, range_, round_, layout = mode
    check_roundtrip(edge_tensor(chunk), chunk, k, range_, round_, layout, seed=11)


@pytest.mark.parametrize("bad", [np.nan, np.inf, -np.inf])
@pytest.mark.parametrize("chunk", [64, 1024, 4096])
def test_nonfinite_input_sets_status_and_writes_degenerate_chunk(bad, chunk):
    x = workloads.random_tensor(chunk * 6 + 50, 3, "normal")
    x[chunk + 9] = bad
    x[chunk * 6 + 7] = bad  # also in the partial chunk
    for range_ in (RANGE_ABSMAX, RANGE_MINMAX):
        for layout, k in ((LAYOUT_INTERLEAVED, 4), (LAYOUT_BITPLANE, 3)):
            ref_stream, flag = oracle.compress(x, chunk, k, range_, ROUND_NEAREST, layout)
            got, status, p, d_stream, _ = gpu_compress(x, chunk, k, range_, ROUND_NEAREST, layout)
            assert flag == 1 and status == 1
            assert np.array_equal(got, ref_stream)
            xhat, st2 = gpu_decompress(p, d_stream)
            assert st2 == 0 and np.all(np.isfinite(xhat))
            assert np.array_equal(xhat.view(np.uint32), oracle.decompress(ref_stream, x.size).view(np.uint32))


def test_rng_counter_wraps_32_bits():
    """Random-number counters that cross a multiple of 2^32 inside the tensor."""
    x = workloads.random_tensor(4096 * 3, 5, "uniform")
    for off in (2 ** 32 - 4096 - 5, 2 ** 32 - 3, 2 ** 64 - 100):
        check_roundtrip(x, 4096, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, seed=2 ** 63 + 12345, rng_offset=off)
        check_roundtrip(x[:1000], 96, 2, RANGE_MINMAX, ROUND_STOCHASTIC, LAYOUT_BITPLANE, seed=7, rng_offset=off)


def test_unaligned_device_pointers_take_the_any_shape_path():
    A = _lib()
    n, chunk, k = 4096 * 5 + 100, 4096, 4
    x = workloads.random_tensor(n, 1, "normal")
    big = torch.zeros(n + 16, dtype=torch.float32, device="cuda")
    d_x = big[4:4 + n]  # 16-byte but not 32-byte aligned
    d_x.copy_(torch.from_numpy(x))
    for layout in (LAYOUT_INTERLEAVED, LAYOUT_BITPLANE):
        ref, _ = oracle.compress(x, chunk, k, RANGE_ABSMAX, ROUND_NEAREST, layout)
        got, status, p, d_stream, d_ws = gpu_compress(x, chunk, k, RANGE_ABSMAX, ROUND_NEAREST, layout, x_dev=d_x)
        assert np.array_equal(got, ref) and status == 0
        out = torch.zeros(n + 16, dtype=torch.float32, device="cuda")
        A.accept_decompress(p, d_stream, out[4:4 + n], d_ws)
        assert np.array_equal(out[4:4 + n].cpu().numpy().view(np.uint32), oracle.decompress(ref, n).view(np.uint32))
        assert float(out[:4].abs().sum()) == 0 and float(out[4 + n:].abs().sum()) == 0


def test_decompress_flags_header_mismatch():
    A = _lib()
    x = workloads.random_tensor(5000, 2, "normal")
    ref, _ = oracle.compress(x, 1024, 4, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_INTERLEAVED)
    p_ok = A.Params(5000, 1024, 4)
    xhat, st = gpu_decompress(p_ok, ref)
    assert st == 0
    # same sizes, other layout: the kernel reads inside the buffers and reports the mismatch
    p_bad = A.Params(5000, 1024, 4, layout=LAYOUT_BITPLANE)
    _, st = gpu_decompress(p_bad, ref)
    assert st == A.DEV_BAD_HEADER
    # a stream coded with stochastic rounding decodes under parameters that say nearest
    ref_sr, _ = oracle.compress(x, 1024, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, 3, 0)
    _, st = gpu_decompress(p_ok, ref_sr)
    assert st == 0
    # the host parser recovers the parameters from the 32 header bytes
    got = A.accept_parse_header(bytes(ref_sr[:32]))
    assert (got.n_elems, got.chunk_elems, got.k, got.range, got.round, got.layout) == (5000, 1024, 4, 0, 1, 0)


def test_output_canaries_untouched():
    """Nothing is written past the compressed size or the N floats."""
    A = _lib()
    n, chunk, k = 4096 * 3 + 1001, 4096, 3
    x = workloads.random_tensor(n, 8, "normal")
    p = A.Params(n, chunk, k, layout=LAYOUT_BITPLANE)
    size = A.accept_compressed_size(p)
    d_stream = torch.full((size + 256,), 0x5A, dtype=torch.uint8, device="cuda")
    d_ws = A.new_workspace(p)
    A.accept_compress(p, torch.from_numpy(x).cuda(), d_stream, d_ws)
    host = d_stream.cpu().numpy()
    assert np.all(host[size:] == 0x5A)
    assert np.array_equal(host[:size], oracle.compress(x, chunk, k, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_BITPLANE)[0])
    d_out = torch.full((n + 64,), 7.0, dtype=torch.float32, device="cuda")
    A.accept_decompress(p, d_stream, d_out, d_ws)
    assert A.accept_last_device_status(d_ws) == 0
    assert bool((d_out[n:] == 7.0).all())


def test_host_buffer_entry_points():
    A = _lib()
    n, chunk, k = 1 << 18, 4096, 8
    x = workloads.generate("cfg1_act", 0, n)
    p = A.Params(n, chunk, k)
    h_x = torch.from_numpy(x).pin_memory()
    h_stream = torch.empty(A.accept_compressed_size(p), dtype=torch.uint8).pin_memory()
    h_xhat = torch.empty(n, dtype=torch.float32).pin_memory()
    d_x = torch.empty(n, dtype=torch.float32, device="cuda")
    d_xhat = torch.empty(n, dtype=torch.float32, device="cuda")
    d_stream, d_ws = A.new_stream_buffer(p), A.new_workspace(p)
    A.accept_compress_host(p, h_x, h_stream, d_x, d_stream, d_ws)
    A.accept_decompress_host(p, h_stream, h_xhat, d_stream, d_xhat, d_ws)
    assert A.accept_last_device_status(d_ws) == 0
    ref, _ = oracle.compress(x, chunk, k)
    assert np.array_equal(h_stream.numpy(), ref)
    assert np.array_equal(h_xhat.numpy().view(np.uint32), oracle.decompress(ref, n).view(np.uint32))


# ------------------------------------------------------------------ the five workloads


def _modes_of(spec):
    return [(m.k, m.range, m.round, m.layout) for m in spec.headline + spec.also]


@pytest.mark.parametrize("mode", modes(), ids=MODE_IDS)
def test_parity_extreme_ranges(mode):
    """Chunks whose range sits at the ends of fp32: the reciprocal scale is subnormal (range near 3e38 with
    k = 2), overflows (range below ~4e-37: a degenerate chunk) or is about to; values from full scale down
    to subnormals inside each chunk."""
    k, range_, round_, layout = mode
    chunk = 1024
    rng = np.random.default_rng(99)
    parts = []
    for top in (3.0e38, 1.2e38, 2.0e-36, 5.0e-37, 1.0e-38, 1.0e-42, 1.0):
        v = (rng.uniform(-1, 1, chunk) * top).astype(np.float32)
        v[:8] = np.array([top, -top, top / 2, top * 2.0 ** -30, 1e-45, -1e-45, 0.0, top * 0.999999], dtype=np.float32)
        parts.append(v)
    x = np.concatenate(parts).astype(np.float32)
    assert np.all(np.isfinite(x))
    check_roundtrip(x, chunk, k, range_, round_, layout, seed=17, rng_offset=3)


def _random_case(i):
    """Seeded draw of (n, chunk, mode, seed, counter offset, value kind) for the property test."""
    rng = np.random.default_rng([20231105, i])
    n = int(rng.choice([rng.integers(1, 600), rng.integers(600, 70000), rng.integers(70000, 400000)]))
    chunk = int(rng.choice([32, 64, 96, 256, 512, 1024, 1504, 2048, 4096, 8192, 16384, 32768, 33024, 65536,
                            32 * int(rng.integers(1, 3000))]))
    mode = modes()[int(rng.integers(0, len(modes())))]
    seed = int(rng.integers(0, 2 ** 63)) * 2 + int(rng.integers(0, 2))
    offset = int(rng.choice([0, int(rng.integers(0, 2 ** 20)), 2 ** 32 - int(rng.integers(0, 5000)),
                             2 ** 64 - int(rng.integers(1, 300000))]))
    kind = str(rng.choice(["normal", "relu", "wide", "uniform"]))
    return n, chunk, mode, seed, offset, kind


@pytest.mark.parametrize("i", range(48))
def test_parity_random_configurations(i):
    """Property test over random (n, chunk, k, range rule, rounding, layout, seed, counter offset, value
    distribution): stream and reconstruction bit-exact against the oracle, whatever path the sizes select
    (register-resident chunks, the any-shape coder, chunks wider than 32768, a ragged tail)."""
    n, chunk, (k, range_, round_, layout), seed, offset, kind = _random_case(i)
    x = workloads.random_tensor(n, 7000 + i, kind)
    if i % 7 == 3 and n > chunk:  # a constant chunk and an all-zero chunk somewhere inside
        x[:chunk] = x[0]
        x[-chunk:] = 0.0
    check_roundtrip(x, chunk, k, range_, round_, layout, seed, offset)


@pytest.mark.parametrize("name", ["cfg1_act", "cfg2_grad", "cfg5_64KB", "cfg5_1MB", "cfg5_16MB"])
def test_workloads_full_parity_small(name):
    spec = workloads.TENSORS[name]
    x = workloads.generate(name)
    for k, range_, round_, layout in _modes_of(spec):
        check_roundtrip(x, spec.chunk, k, range_, round_, layout, seed=spec.seed)


@pytest.mark.parametrize("name", ["cfg3_act", "cfg3_grad", "cfg4_hidden"])
def test_workloads_full_parity_large(name):
    """Full-size tensors in the launch configuration the benchmark times; every element compared."""
    spec = workloads.TENSORS[name]
    x = workloads.generate(name)
    for m in spec.headline:
        check_roundtrip(x, spec.chunk, m.k, m.range, m.round, m.layout, seed=spec.seed)


def _host_threads():
    import os
    return max(1, len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1))


def _in_threads(fn, jobs):
    """fn over jobs on one thread per host core (numpy and the oracle's C code release the interpreter lock)."""
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=_host_threads()) as pool:
        return list(pool.map(fn, jobs))


def _oracle_in_slices(x, chunk, m, seed):
    """The oracle over disjoint runs of whole chunks (chunks are independent and the random-number counter is
    the element index, so a run can be coded on its own): -> side words, payload words, reconstruction of
    the whole tensor, exactly what one call over the whole tensor would give."""
    n = x.size
    per = -(-(-(-n // chunk)) // (4 * _host_threads())) * chunk

    def one(lo):
        hi = min(lo + per, n)
        ref, flag = oracle.compress(x[lo:hi], chunk, m.k, m.range, m.round, m.layout, seed, lo)
        assert flag == 0
        _, meta, payload = oracle.split_stream(ref, hi - lo, chunk)
        return meta.copy(), payload.copy(), oracle.decompress(ref, hi - lo)

    parts = _in_threads(one, range(0, n, per))
    return (np.concatenate([p[0] for p in parts]), np.concatenate([p[1] for p in parts]),
            np.concatenate([p[2] for p in parts]))


@pytest.mark.parametrize("name", ["cfg5_256MB", "cfg5_1GB"])
def test_workloads_full_parity_sweep(name):
    """The two large points of the size sweep at full size, in the launch configuration the benchmark times:
    every side word, every payload word and every reconstructed value against the oracle."""
    A = _lib()
    spec = workloads.TENSORS[name]
    n, chunk = spec.n, spec.chunk
    step = 1 << 22
    x = np.concatenate(_in_threads(lambda s0: workloads.generate(name, s0, min(step, n - s0)), range(0, n, step)))
    g_x = gpu_util.guarded_input(torch, x)
    d_x = g_x.view(torch.float32)
    for m in spec.headline:
        p = A.Params(n, chunk, m.k, m.range, m.round, m.layout, spec.seed, 0)
        g_stream, g_ws = gpu_util.guarded_stream(A, torch, p), gpu_util.guarded_workspace(A, torch, p)
        g_xhat = gpu_util.guarded_floats(torch, n)
        d_stream, d_ws, d_xhat = g_stream.bytes, g_ws.view(torch.int32), g_xhat.view(torch.float32)
        A.accept_compress(p, d_x, d_stream, d_ws)
        A.accept_decompress(p, d_stream, d_xhat, d_ws)
        assert A.accept_last_device_status(d_ws) == 0
        for g, what in ((g_x, "input"), (g_stream, "stream"), (g_ws, "workspace"), (g_xhat, "reconstruction")):
            g.check(what)
        got = d_stream.cpu().numpy()
        hdr, meta_g, pay_g = oracle.split_stream(got, n, chunk)
        assert [int(v) for v in hdr] == [0x54504341, 1, n & 0xFFFFFFFF, n >> 32, chunk, m.k, m.range | m.round << 8 | m.layout << 16, 0]
        meta_r, pay_r, xhat_r = _oracle_in_slices(x, chunk, m, spec.seed)
        assert np.array_equal(meta_g.view(np.uint32), meta_r.view(np.uint32)), "side words"
        assert pay_g.size == pay_r.size and np.array_equal(pay_g, pay_r), "payload"
        assert not got[32 + 8 * meta_g.shape[0]:A.accept_payload_offset(p)].any(), "padding"
        xhat_g = d_xhat.cpu().numpy()
        assert np.array_equal(xhat_g.view(np.uint32), xhat_r.view(np.uint32)), "reconstruction"
        # the stated tolerance, on a run of chunks (the bit-exact comparison above is the stricter bar)
        assert_float_parity(xhat_g[:64 * chunk], xhat_r[:64 * chunk], x[:64 * chunk], chunk)
        del g_stream, g_xhat, got, xhat_g, xhat_r, pay_r
        torch.cuda.empty_cache()


def test_parity_beyond_32_bit_element_indices():
    """A tensor of more than 2^32 elements (17 GB): element indices, byte offsets and random-number
    counters all pass 2^32.  Values are drawn on the GPU; the oracle recomputes runs of chunks around
    the interesting indices from slices copied back (chunks are independent, counters are indices)."""
    A = _lib()
    free, _ = torch.cuda.mem_get_info()
    n, chunk = (1 << 32) + 4096 * 5 + 123, 4096
    if free < 45 * (1 << 30):
        pytest.skip("needs about 40 GB of free device memory")
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234)
    d_x = torch.empty(n, dtype=torch.float32, device="cuda")
    step = 1 << 28
    for s in range(0, n, step):
        d_x[s:s + step].normal_(generator=gen)
    for k, round_, layout in [(4, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED), (2, ROUND_NEAREST, LAYOUT_BITPLANE)]:
        p = A.Params(n, chunk, k, RANGE_ABSMAX, round_, layout, seed=99, rng_offset=0)
        d_stream, d_ws = A.new_stream_buffer(p), A.new_workspace(p)
        A.accept_compress(p, d_x, d_stream, d_ws)
        d_xhat = torch.empty(n, dtype=torch.float32, device="cuda")
        A.accept_decompress(p, d_stream, d_xhat, d_ws)
        assert A.accept_last_device_status(d_ws) == 0
        off = A.accept_payload_offset(p)
        wpc = chunk * k // 32
        n_chunks = -(-n // chunk)
        for c0 in (0, (1 << 31) // chunk - 2, (1 << 32) // chunk - 3, n_chunks - 4):
            c1 = min(c0 + 4, n_chunks)
            e0, e1 = c0 * chunk, min(c1 * chunk, n)
            xs = d_x[e0:e1].cpu().numpy()
            ref, _ = oracle.compress(xs, chunk, k, RANGE_ABSMAX, round_, layout, 99, e0)
            _, meta_r, pay_r = oracle.split_stream(ref, xs.size, chunk)
            meta_g = d_stream[32 + 8 * c0:32 + 8 * c1].cpu().numpy().view(np.float32).reshape(-1, 2)
            assert np.array_equal(meta_g.view(np.uint32), meta_r.view(np.uint32))
            b0 = off + 4 * wpc * c0
            pay_g = d_stream[b0:b0 + 4 * pay_r.size].cpu().numpy().view(np.uint32)
            assert np.array_equal(pay_g, pay_r)
            want = oracle.decompress(ref, xs.size)
            assert np.array_equal(d_xhat[e0:e1].cpu().numpy().view(np.uint32), want.view(np.uint32))
        hdr = d_stream[:32].cpu().numpy().view(np.uint32)
        assert int(hdr[2]) == n & 0xFFFFFFFF and int(hdr[3]) == 1
        del d_stream, d_xhat
        torch.cuda.empty_cache()
