"""Pins for the oracle's grouping along the batch dimension (the paper's own grouping)."""
import numpy as np
import pytest

import oracle
import workloads
from oracle import LAYOUT_BITPLANE, LAYOUT_INTERLEAVED, RANGE_ABSMAX, ROUND_NEAREST


def test_forward_encoder_example_along_the_batch_dimension():
    """Forward Encoder example: an 8 x 1 x 1 x 1 x 4 binary tensor becomes 1 x 1 x 1 x 1 x 4 integers;
    eight one-bit values of eight batch neighbours give (00110110)_2 = 54."""
    bits = [0, 1, 1, 0, 1, 1, 0, 0]  # digits of 54, least significant first
    F, nb, k = 8, 8, 4
    # feature 3: binary digit 2 of the eight samples spells the example; other digits/features are 0
    x = np.zeros((nb, F), dtype=np.float32)
    x[:, 3] = [4.0 * b for b in bits]          # MINMAX over the tensor: lo = 0, hi = 15 -> code = value
    x[0, 0] = 15.0
    stream, _ = oracle.compress_strided(x, nb * F, k, F, oracle.RANGE_MINMAX, ROUND_NEAREST, LAYOUT_BITPLANE)
    payload = stream[oracle.payload_offset(nb * F, nb * F):].view(np.uint32)
    assert payload.size == k * F                  # ceil(8/32) = 1 batch group per feature, k words each
    assert int(payload[3 * k + 2]) == 54          # feature 3, digit 2
    assert [int(payload[3 * k + j]) for j in (0, 1, 3)] == [0, 0, 0]
    assert int(payload[0 * k + 0]) == 1 and int(payload[0 * k + 3]) == 1   # x[0,0] = 15 -> sample 0, all digits


@pytest.mark.parametrize("layout", [LAYOUT_INTERLEAVED, LAYOUT_BITPLANE])
def test_strided_grouping_is_the_contiguous_one_on_the_transposed_tensor(layout):
    """Grouping batch neighbours of a (n_b x F) tensor = grouping consecutive values of its transpose,
    feature by feature: same codes, words regrouped."""
    nb, F, chunk = 64, 24, 64 * 24
    x = workloads.random_tensor(nb * F, 3, "normal").reshape(nb, F)
    for k in ((2, 4, 8) if layout == LAYOUT_INTERLEAVED else (2, 3, 4)):
        s_str, _ = oracle.compress_strided(x, chunk, k, F, RANGE_ABSMAX, ROUND_NEAREST, layout)
        codes, meta, _ = oracle.quantize(x, chunk, k)
        pay = s_str[oracle.payload_offset(nb * F, chunk):].view(np.uint32).reshape(nb // 32, F, k)
        ct = codes.reshape(nb, F)
        for f in (0, 5, 23):
            col = np.ascontiguousarray(ct[:, f])                      # the feature's codes over the batch
            want = oracle.pack(col, nb, k, layout).reshape(nb // 32, k)
            assert np.array_equal(pay[:, f, :], want)
        assert np.array_equal(oracle.decompress_strided(s_str, nb * F),
                              oracle.dequantize(codes, meta, chunk, k, RANGE_ABSMAX))


def test_strided_sizes_and_padding():
    """ceil(n_b/32) batch groups per feature (Eq. 8's ceil(n/8) with words of 32); rows past n_b are zero bits."""
    nb, F, k = 40, 16, 4
    x = np.abs(workloads.random_tensor(nb * F, 1, "normal")).reshape(nb, F) + 1
    s, _ = oracle.compress_strided(x, 640, k, F, RANGE_ABSMAX, ROUND_NEAREST, LAYOUT_BITPLANE)
    assert s.size == oracle.strided_stream_bytes(nb * F, 640, k, F) == oracle.payload_offset(640, 640) + 4 * k * 2 * F
    pay = s[oracle.payload_offset(640, 640):].view(np.uint32).reshape(2, F, k)
    assert np.all(pay[1] >> 8 == 0)     # second batch group holds rows 32..39 only
    hdr = s[:32].view(np.uint32)
    assert int(hdr[7]) == F and int(hdr[4]) == 640
    # the paper's table: batch 128, 4096 KB original, 4-bit -> 512 KB of packed integers
    assert oracle.strided_stream_bytes(1 << 20, 1 << 20, 4, 8192) - oracle.payload_offset(1 << 20, 1 << 20) == 512 * 1024
