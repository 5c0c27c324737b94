"""accept_compress_static: the compress entry point for callers that cannot allocate.

Some users of the codec have no allocator to turn to when a call is made: a pipeline stage on a device
whose memory was handed out once at start-up, or a plug-in inside a framework that owns all device memory.
They cannot create the small workspace accept_compress wants, so the library carries one itself.  This
test drives that entry point through the C ABI twice in a row -- the built-in scratch is shared by all
calls and keeps what the last call left -- and requires, both times, exactly the stream that
accept_compress writes with a caller-owned workspace (the parity tests' bar: bit-exact), and the status
bits of that call alone.  Collected last so that a run stopping at the first failure has already run
everything else.
"""
import ctypes

import numpy as np
import pytest

import oracle
import workloads

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _reference(A, p, d_x):
    d_stream = A.new_stream_buffer(p)
    d_stream.fill_(0x11)
    d_ws = A.new_workspace(p)
    A.accept_compress(p, d_x, d_stream, d_ws)
    return d_stream.cpu().numpy(), A.accept_last_device_status(d_ws)


def test_static_scratch_entry_point_matches_accept_compress_twice_in_a_row():
    import paper_2311_05827_b200 as A

    n, chunk = 4096 * 21 + 777, 4096
    x1 = workloads.random_tensor(n, 31, "normal")
    x1[5000] = np.nan                      # first call: one non-finite chunk -> status bit set
    x2 = workloads.random_tensor(n, 32, "relu")  # second call: clean input -> the stale bit must be gone
    calls = [
        (x1, A.Params(n, chunk, 4, A.RANGE_ABSMAX, A.ROUND_STOCHASTIC, A.LAYOUT_INTERLEAVED, seed=5, rng_offset=9)),
        (x2, A.Params(n, chunk, 3, A.RANGE_MINMAX, A.ROUND_NEAREST, A.LAYOUT_BITPLANE)),
    ]
    launches = A.accept_launch_count()
    for i, (x, p) in enumerate(calls):
        d_x = torch.from_numpy(x).cuda()
        want_stream, want_status = _reference(A, p, d_x)
        d_stream = A.new_stream_buffer(p)
        d_stream.fill_(0xEE)
        d_status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        A.accept_compress_static(p, d_x, d_stream, d_status)
        torch.cuda.synchronize()
        got_stream = d_stream.cpu().numpy()
        assert np.array_equal(got_stream, want_stream), f"call {i}: stream differs from accept_compress"
        ref, flag = oracle.compress(x, p.chunk_elems, p.k, p.range, p.round, p.layout, p.seed, p.rng_offset)
        assert np.array_equal(got_stream, ref) and flag == want_status, f"call {i}: stream differs from the oracle's"
        assert int(d_status.item()) == want_status == (1 if i == 0 else 0)
    assert A.accept_launch_count() - launches == 4  # two reference launches, two static launches

    # the status output is optional
    x, p = calls[1]
    d_stream = A.new_stream_buffer(p)
    A.accept_compress_static(p, torch.from_numpy(x).cuda(), d_stream)
    torch.cuda.synchronize()
    assert np.array_equal(d_stream.cpu().numpy(), _reference(A, p, torch.from_numpy(x).cuda())[0])


def test_static_scratch_holds_the_chunk_records_of_wide_chunks_and_batch_groups():
    """Calls whose chunk records really live in the built-in array (bytes 16..255: at most 15 chunks): chunks
    wider than a block holds, and pack groups along the batch dimension.  Two calls in a row of each kind; every
    stream against the oracle's and against accept_compress with a caller-owned workspace, bit for bit."""
    import paper_2311_05827_b200 as A

    n, chunk = 15 * 65536, 65536
    x1 = workloads.random_tensor(n, 41, "normal")
    x2 = workloads.random_tensor(n, 42, "relu")
    x2[3 * chunk + 5] = np.inf  # second call: one non-finite chunk; its bit must not leak anywhere else
    rows, stride = 48, 1280     # 61440 values, 15 chunks of 4096
    x3 = workloads.random_tensor(rows * stride, 43, "normal")
    calls = [
        (x1, A.Params(n, chunk, 4, A.RANGE_ABSMAX, A.ROUND_STOCHASTIC, A.LAYOUT_INTERLEAVED, seed=5, rng_offset=9), None),
        (x2, A.Params(n, chunk, 3, A.RANGE_MINMAX, A.ROUND_NEAREST, A.LAYOUT_BITPLANE), None),
        (x3, A.Params(x3.size, 4096, 4, A.RANGE_ABSMAX, A.ROUND_NEAREST, A.LAYOUT_BITPLANE, group_stride=stride), stride),
        (x3, A.Params(x3.size, 4096, 8, A.RANGE_MINMAX, A.ROUND_STOCHASTIC, A.LAYOUT_INTERLEAVED, seed=7, group_stride=stride), stride),
    ]
    for i, (x, p, group_stride) in enumerate(calls):
        assert 16 < A.accept_workspace_size(p) <= 256
        d_x = torch.from_numpy(x).cuda()
        want_stream, want_status = _reference(A, p, d_x)
        if group_stride is None:
            ref, flag = oracle.compress(x, p.chunk_elems, p.k, p.range, p.round, p.layout, p.seed, p.rng_offset)
        else:
            ref, flag = oracle.compress_strided(x, p.chunk_elems, p.k, group_stride, p.range, p.round, p.layout, p.seed, p.rng_offset)
        d_stream = A.new_stream_buffer(p)
        d_stream.fill_(0xEE)
        d_status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        A.accept_compress_static(p, d_x, d_stream, d_status)
        torch.cuda.synchronize()
        got = d_stream.cpu().numpy()
        assert np.array_equal(got, ref), f"call {i}: stream differs from the oracle's"
        assert np.array_equal(got, want_stream), f"call {i}: stream differs from accept_compress"
        assert int(d_status.item()) == want_status == flag == (1 if i == 1 else 0)
    # one chunk more than the array holds is refused on the host
    with pytest.raises(A.AcceptError) as err:
        A.accept_compress_static(A.Params(16 * 65536, 65536, 4), torch.zeros(16 * 65536, device="cuda"),
                                 torch.zeros(1 << 20, dtype=torch.uint8, device="cuda"))
    assert err.value.code == 11


def test_static_scratch_entry_point_rejects_bad_arguments_on_the_host():
    import paper_2311_05827_b200 as A
    from paper_2311_05827_b200 import binding
    lib = binding.lib()
    p = A.Params(1000, 32, 4).c()
    size = A.accept_compressed_size(A.Params(1000, 32, 4))
    good = 0x10000
    before = A.accept_launch_count()
    assert lib.accept_compress_static(ctypes.byref(p), None, good, size, None, None) == 1
    assert lib.accept_compress_static(ctypes.byref(p), good, good, size - 1, None, None) == 5
    assert lib.accept_compress_static(ctypes.byref(p), good, good, size, good + 2, None) == 10
    bad = A.Params(1000, 32, 5).c()
    assert lib.accept_compress_static(ctypes.byref(bad), good, good, size, None, None) == 2
    assert A.accept_launch_count() == before
