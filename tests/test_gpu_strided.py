"""GPU parity of pack groups along the batch dimension (the paper's own grouping) against the oracle."""
import numpy as np
import pytest

import oracle
import workloads
from tests import gpu_util
from oracle import (LAYOUT_BITPLANE, LAYOUT_INTERLEAVED, RANGE_ABSMAX, RANGE_MINMAX, ROUND_NEAREST,
                    ROUND_STOCHASTIC)

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def modes():
    out = []
    for layout in (LAYOUT_INTERLEAVED, LAYOUT_BITPLANE):
        for k in ((2, 4, 8) if layout == LAYOUT_INTERLEAVED else (2, 3, 4, 8)):
            for range_ in (RANGE_ABSMAX, RANGE_MINMAX):
                for round_ in (ROUND_NEAREST, ROUND_STOCHASTIC):
                    out.append((k, range_, round_, layout))
    return out


def check(x, chunk, stride, k, range_, round_, layout, seed=0, rng_offset=0):
    import paper_2311_05827_b200 as A
    n = x.size
    ref, flag = oracle.compress_strided(x, chunk, k, stride, range_, round_, layout, seed, rng_offset)
    p = A.Params(n, chunk, k, range_, round_, layout, seed, rng_offset, group_stride=stride)
    assert A.accept_compressed_size(p) == ref.size
    g_x = gpu_util.guarded_input(torch, x)
    g_stream = gpu_util.guarded_stream(A, torch, p, 0x3C)
    g_ws = gpu_util.guarded_workspace(A, torch, p)
    d_stream, d_ws = g_stream.bytes, g_ws.view(torch.int32)
    A.accept_compress(p, g_x.view(torch.float32), d_stream, d_ws)
    assert (A.accept_last_device_status(d_ws) & 1) == flag
    for g, what in ((g_x, "input"), (g_stream, "stream"), (g_ws, "workspace")):
        g.check(what)
    got = d_stream.cpu().numpy()
    if not np.array_equal(got, ref):
        off = oracle.payload_offset(n, chunk)
        assert np.array_equal(got[:32], ref[:32]), "header"
        assert np.array_equal(got[32:off], ref[32:off]), "side words"
        bad = np.nonzero(got[off:].view(np.uint32) != ref[off:].view(np.uint32))[0]
        raise AssertionError(f"{bad.size} payload words differ, first {bad[:8]}")
    g_xhat = gpu_util.guarded_floats(torch, n)
    d_xhat = g_xhat.view(torch.float32)
    g_ws16 = gpu_util.guarded_workspace(A, torch, p, 16)  # the receiver needs the status word only
    A.accept_decompress(p, d_stream, d_xhat, g_ws16.view(torch.int32))
    assert A.accept_last_device_status(g_ws16.view(torch.int32)) == 0
    g_xhat.check("reconstruction")
    g_ws16.check("receiver workspace")
    want = oracle.decompress_strided(ref, n)
    assert np.array_equal(d_xhat.cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert A.accept_parse_header(bytes(got[:32])).group_stride == stride


@pytest.mark.parametrize("range_", [RANGE_ABSMAX, RANGE_MINMAX])
@pytest.mark.parametrize("rows,stride,chunk", [
    (40, 1000, 256),         # one octet per thread, a warp per chunk, four chunks per block; ragged last chunk
    (40, 1000, 512),         # two octets per thread
    (40, 1000, 1024),        # four octets per thread, a warp per chunk
    (40, 1000, 12800),       # two octets per thread, 800 threads per chunk (a block of its own)
    (48, 2048, 24576),       # four octets per thread, 768 threads per chunk
    (48, 2048, 32768),       # the largest chunk a block holds: 1024 threads
    (40, 1000, 4000),        # no register-resident geometry: every chunk goes through the plain loop
    (40, 1000, 39968),       # more than 32768: ranges by atomics, constants pass (the whole tensor is 40000)
])
def test_strided_parity_chunk_geometries(range_, rows, stride, chunk):
    """The one-launch pass for ranges, side words and constants under every launch shape it has, and the
    atomics + constants passes that wider chunks take; side words and payload against the oracle."""
    x = workloads.random_tensor(rows * stride, chunk % 97, "normal")
    x[5] = 7.5  # not the largest magnitude of its chunk's neighbours by accident
    check(x, chunk, stride, 4, range_, ROUND_NEAREST, LAYOUT_BITPLANE)
    check(x, chunk, stride, 8, range_, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, seed=3, rng_offset=17)


@pytest.mark.parametrize("mode", modes())
@pytest.mark.parametrize("rows,stride,chunk", [
    (64, 24, 64 * 24),       # one range for the whole tensor, two full batch groups
    (40, 16, 96),            # partly filled second batch group, small chunks
    (33, 2056, 4096),        # chunk boundaries inside rows, more than one block of feature octets
    (128, 4096, 4096),       # chunk = one sample
])
def test_strided_parity(mode, rows, stride, chunk):
    k, range_, round_, layout = mode
    x = workloads.random_tensor(rows * stride, rows + k, "normal")
    check(x, chunk, stride, k, range_, round_, layout, seed=21, rng_offset=5)


@pytest.mark.parametrize("mode", modes())
@pytest.mark.parametrize("rows,stride,chunk", [
    (70, 1, 32),             # one value per sample: the groups are runs of the only column
    (33, 7, 64),             # rows start at any multiple of four bytes
    (96, 12, 96 * 12),       # one range for the whole tensor
    (40, 50, 512),
    (65, 2060, 4096),        # the 2056 + 4 case: more than one block of features, ragged last block
])
def test_strided_parity_any_values_per_sample(mode, rows, stride, chunk):
    """Values per sample that are not a multiple of eight (Sec. 4.3.1's smaller outputs need not be): the
    feature-per-thread kernels, every mode, eight bit planes included."""
    k, range_, round_, layout = mode
    x = workloads.random_tensor(rows * stride, rows + stride + k, "normal")
    check(x, chunk, stride, k, range_, round_, layout, seed=33, rng_offset=2 ** 32 - 1000)


@pytest.mark.parametrize("i", range(24))
def test_strided_parity_random_configurations(i):
    """Seeded random (batch rows, values per sample, chunk, mode, seed, counter offset): rows that do not fill
    the last batch group, feature counts that do not fill the last block of 64 octets, chunks of any
    multiple of 32 (boundaries anywhere inside rows), counters next to the 2^32 and 2^64 wraps."""
    rng = np.random.default_rng([20231106, i])
    rows = int(rng.choice([1, 2, 31, 32, 33, int(rng.integers(1, 200))]))
    stride = 8 * int(rng.choice([1, 3, 63, 64, 65, int(rng.integers(1, 1200))]))
    if i % 3 == 2:
        stride += int(rng.integers(1, 8))  # not a multiple of eight: the feature-per-thread kernels
    n = rows * stride
    chunk = int(rng.choice([32, 96, 1024, 4096, 32 * int(rng.integers(1, 2000)), (n + 31) // 32 * 32]))
    k, range_, round_, layout = modes()[int(rng.integers(0, len(modes())))]
    seed = int(rng.integers(0, 2 ** 63)) * 2 + 1
    offset = int(rng.choice([0, int(rng.integers(0, 2 ** 20)), 2 ** 32 - int(rng.integers(0, 5000)),
                             2 ** 64 - int(rng.integers(1, 300000))]))
    x = workloads.random_tensor(n, 9000 + i, str(rng.choice(["normal", "relu", "wide"])))
    check(x, chunk, stride, k, range_, round_, layout, seed=seed, rng_offset=offset)


@pytest.mark.parametrize("k,layout", [(2, LAYOUT_INTERLEAVED), (3, LAYOUT_BITPLANE), (4, LAYOUT_INTERLEAVED), (8, LAYOUT_INTERLEAVED),
                                      (8, LAYOUT_BITPLANE)])
@pytest.mark.parametrize("position", [0, 1, 2, 3])
@pytest.mark.parametrize("stride", [1536, 1531])
def test_strided_stochastic_counter_wraps(k, layout, position, stride):
    """Eq. 7 draws in the octet-per-thread encoder: the counter of every octet's first value sits at `position` of
    its group of four counters (the host picks the kernel by it); counter ranges that cross 2^34 (the low word of
    the group index wraps: the key changes inside an octet) and 2^64 (the counter itself wraps)."""
    rows, chunk = 40, 1024   # (stride 1531: the feature-per-thread kernels, which keep the key from one counter to the next)
    x = workloads.random_tensor(rows * stride, 77 + position, "normal")
    n = x.size
    for base in (0, 2 ** 34 - n // 2 - 4, 2 ** 64 - n // 3 - 8, 2 ** 34 - 8):
        offset = base // 4 * 4 + position
        check(x, chunk, stride, k, RANGE_ABSMAX, ROUND_STOCHASTIC, layout, seed=0xC0FFEE + k, rng_offset=offset)
    check(x, chunk, stride, k, RANGE_MINMAX, ROUND_STOCHASTIC, layout, seed=5, rng_offset=(2 ** 34 - n // 2) // 4 * 4 + position)


def test_strided_largest_latent_output_of_the_paper():
    """Batch 128, 8192 values per sample (the 4096 KB output of Sec. 4.3.1), per-tensor range, both encoders."""
    x = workloads.generate("cfg2_grad").reshape(32, -1)
    x = np.concatenate([x, x * np.float32(0.5), -x, x * np.float32(0.25)]).reshape(-1)  # 128 x 32768
    n = x.size
    check(x, n, 32768, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, seed=3)
    check(x, n, 32768, 2, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_BITPLANE)


def test_strided_nonfinite_and_bad_arguments():
    import paper_2311_05827_b200 as A
    x = workloads.random_tensor(64 * 64, 2, "normal")
    x[70] = np.nan
    check(x, 1024, 64, 4, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_BITPLANE)
    assert A.accept_check_params(A.Params(64 * 63, 1024, 4, group_stride=63)) == 0      # any number of values per sample
    assert A.accept_check_params(A.Params(64 * 64 + 8, 1024, 4, group_stride=64)) == 9  # n not a multiple of F
    assert A.accept_check_params(A.Params(64 * 64, 1024, 8, layout=LAYOUT_BITPLANE, group_stride=64)) == 0
    assert A.accept_workspace_size(A.Params(64 * 64, 1024, 4, group_stride=64)) == 16 + 16 * 4
