"""Stand-ins for a memory checker and a fault injector, in the forms this library allows on a shared GPU.

1. The checking build (the same sources with -DACCEPT_BOUNDS_CHECK): every access of every kernel to caller
   memory is compared with the byte ranges of the call; an access outside is counted and skipped, never
   performed.  The parity cases that select every launch path are run against it and must report zero
   skipped accesses (reads included, which guard bands cannot see) and still be bit-exact.
2. The checker checked: with the writable ranges cut short on purpose (an environment switch of the
   checking build only) the last stores of a call must be reported, and left undone.
3. The bounded wait of the staged batch-group encoder, made to run out: a build in which a stage announces
   bytes that never arrive.  The kernel must give up within milliseconds, report ACCEPT_DEV_COPY_TIMEOUT
   and leave the GPU usable: the next ordinary call is bit-exact again.
"""
import os

import numpy as np
import pytest

import oracle
import workloads
from oracle import (LAYOUT_BITPLANE, LAYOUT_INTERLEAVED, RANGE_ABSMAX, RANGE_MINMAX, ROUND_NEAREST,
                    ROUND_STOCHASTIC)
from tests import gpu_util
from tests import test_gpu_mbq, test_gpu_parity, test_gpu_strided

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _report():
    import paper_2311_05827_b200 as A
    return A.accept_bounds_check_report()


def test_the_product_build_checks_nothing():
    code, count, _, _, _ = _report()
    assert code == 12 and count == 0  # ACCEPT_ERR_UNCHECKED_BUILD


def test_every_launch_path_stays_inside_its_buffers():
    with gpu_util.library_variant("bounds"):
        assert _report()[:2] == (0, 0)
        # consecutive layout: register-resident chunks of every geometry, the any-shape coder, ragged tails
        for k, range_, round_, layout in test_gpu_parity.modes():
            for chunk, n in [(4096, 4096 * 5 + 1234), (1024, 1024 * 13 + 1), (512, 512 * 9), (256, 256 * 5 + 77),
                             (96, 96 * 20 + 40), (32, 1000), (8192, 8192 * 2 + 333)]:
                x = workloads.random_tensor(n, chunk + k, "normal")
                test_gpu_parity.check_roundtrip(x, chunk, k, range_, round_, layout, seed=5, rng_offset=2 ** 32 - 3000)
            # chunks wider than a block holds: range pass, constants, encode
            for chunk, n in [(32800, 32800 * 3 + 12345), (1 << 18, (1 << 18) + 33), (1 << 20, 300003)]:
                x = workloads.random_tensor(n, chunk + k, "relu")
                test_gpu_parity.check_roundtrip(x, chunk, k, range_, round_, layout, seed=6)
        for n in (1, 7, 33, 255, 4097):
            x = workloads.random_tensor(n, n, "normal")
            test_gpu_parity.check_roundtrip(x, 256, 3, RANGE_MINMAX, ROUND_NEAREST, LAYOUT_BITPLANE)
        assert _report()[:2] == (0, 0), "consecutive layout"
        # pack groups along the batch dimension
        for k, range_, round_, layout in test_gpu_strided.modes():
            for rows, stride, chunk in [(64, 24, 64 * 24), (40, 16, 96), (33, 2056, 4096), (70, 520, 1024), (33, 7, 64), (65, 2060, 4096)]:
                x = workloads.random_tensor(rows * stride, rows + k, "normal")
                test_gpu_strided.check(x, chunk, stride, k, range_, round_, layout, seed=21, rng_offset=5)
        assert _report()[:2] == (0, 0), "batch groups"
        # forward quantizer: residue initialisation, grid search, threshold search, ragged sizes
        for k in (2, 3, 4):
            for n in (1, 33, 8193, 8192 * 5 + 777, 4096 * 300 + 5):
                x = workloads.random_tensor(n, 100 + k, "normal")
                test_gpu_mbq.check_mbq(x, k, 3, False, np.array([0.9, 0.5, 0.27, 0.14][:k], dtype=np.float32))
                test_gpu_mbq.check_mbq(x, k, 0, True, None)
            x = workloads.random_tensor(20000, k, "wide")
            test_gpu_mbq.check_mbq(x, k, 2, False, np.array([1.0, 0.5, 0.25, 0.125 + 1e-4][:k], dtype=np.float32))
        code, count, addr, size, write = _report()
        assert (code, count) == (0, 0), f"forward quantizer: {count} accesses outside, first at {addr:#x} ({size} bytes, write={write})"


def test_the_checker_reports_and_skips_stores_past_a_shortened_range():
    import paper_2311_05827_b200 as A
    n, chunk, k = 4096 * 6, 4096, 8
    x = workloads.random_tensor(n, 3, "normal")
    ref, _ = oracle.compress(x, chunk, k)
    p = A.Params(n, chunk, k)
    with gpu_util.library_variant("bounds"):
        assert _report()[:2] == (0, 0)
        os.environ["ACCEPT_BOUNDS_TEST_SHRINK"] = "64"
        try:
            g_stream = gpu_util.guarded_stream(A, torch, p, 0xA5)
            d_ws = torch.zeros(64, dtype=torch.int32, device="cuda")  # larger than the 64 bytes cut off
            A.accept_compress(p, torch.from_numpy(x).cuda(), g_stream.bytes, d_ws)
            code, count, addr, size, write = _report()
        finally:
            del os.environ["ACCEPT_BOUNDS_TEST_SHRINK"]
        g_stream.check("stream")
        got = g_stream.bytes.cpu().numpy()
        end = g_stream.bytes.data_ptr() + got.size
        # k = 8, consecutive layout: the payload is stored eight bytes per thread, so the last 64 bytes are eight stores
        assert code == 0 and count == 8 and write and size == 8 and end - 64 <= addr < end
        assert np.array_equal(got[:-64], ref[:-64]) and np.all(got[-64:] == 0xA5)
        assert _report()[:2] == (0, 0)  # a report clears the count


@pytest.mark.parametrize("k,layout", [(4, LAYOUT_BITPLANE), (8, LAYOUT_INTERLEAVED)])
def test_bounded_copy_wait_runs_out_and_the_gpu_stays_usable(k, layout):
    import paper_2311_05827_b200 as A
    rows, stride, chunk = 96, 4096, 4096
    x = workloads.random_tensor(rows * stride, 12, "normal")
    p = A.Params(x.size, chunk, k, RANGE_ABSMAX, ROUND_NEAREST, layout, group_stride=stride)
    d_x = torch.from_numpy(x).cuda()
    with gpu_util.library_variant("stall"):
        g_stream = gpu_util.guarded_stream(A, torch, p)
        g_ws = gpu_util.guarded_workspace(A, torch, p)
        # a call of this build that stages nothing first: loading its kernels onto the GPU is not what is timed
        warm = A.Params(x.size, chunk, k, RANGE_ABSMAX, ROUND_NEAREST, layout)
        A.accept_compress(warm, d_x, gpu_util.guarded_stream(A, torch, warm).bytes, gpu_util.guarded_workspace(A, torch, warm).view(torch.int32))
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        A.accept_compress(p, d_x, g_stream.bytes, g_ws.view(torch.int32))
        t1.record()
        status = A.accept_last_device_status(g_ws.view(torch.int32))
        assert status == A.DEV_COPY_TIMEOUT
        assert t0.elapsed_time(t1) < 200.0  # milliseconds: three waits of 2 ms per block, all blocks resident at once
        g_stream.check("stream")
        g_ws.check("workspace")
    # the ordinary library, same process, same GPU: the same call is bit-exact
    test_gpu_strided.check(x, chunk, stride, k, RANGE_ABSMAX, ROUND_NEAREST, layout)
    test_gpu_parity.check_roundtrip(x[:4096 * 7 + 5], 4096, 4, RANGE_ABSMAX, ROUND_STOCHASTIC, LAYOUT_INTERLEAVED, seed=1)


def test_bounded_copy_wait_of_the_forward_quantizer_runs_out_cleanly():
    """The staged encode pass of the forward quantizer under the same stalled copies: the status word reports it,
    the workspace is left clean (the block that ends last still closes the batch), and the ordinary library
    then codes the same tensor bit for bit like the oracle, on the very workspace the failed call used."""
    import paper_2311_05827_b200 as A
    n, k = 8192 * 40 + 123, 3
    x = workloads.random_tensor(n, 5, "relu")
    alpha_prev = np.array([0.9, 0.5, 0.27], dtype=np.float32)
    p = A.MbqParams(n, k, 2, False)
    d_x = torch.from_numpy(x).cuda()
    d_prev = torch.from_numpy(alpha_prev).cuda()
    d_next = torch.zeros(k, dtype=torch.float32, device="cuda")
    g_stream = gpu_util.guarded_stream(A, torch, p)
    g_ws = gpu_util.guarded_workspace(A, torch, p)
    d_ws = g_ws.view(torch.int32)
    with gpu_util.library_variant("stall"):
        A.accept_mbq_compress(p, d_x, d_prev, d_next, g_stream.bytes, d_ws)
        assert A.accept_last_device_status(d_ws) & A.DEV_COPY_TIMEOUT
        g_stream.check("stream")
        g_ws.check("workspace")
    assert not bool(d_ws.view(torch.uint8)[32:].any()), "sums, counters or tickets left behind"
    d_ws.zero_()  # the caller clears the status word
    A.accept_mbq_compress(p, d_x, d_prev, d_next, g_stream.bytes, d_ws)
    assert A.accept_last_device_status(d_ws) == 0
    ref, ref_alpha = oracle.mbq_compress(x, k, 2, False, alpha_prev)
    assert np.array_equal(g_stream.bytes.cpu().numpy(), ref)
    assert np.array_equal(d_next.cpu().numpy().view(np.uint32), ref_alpha.view(np.uint32))
