"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates arguments before touching CUDA, and sizes streams like the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def A():
    from paper_2311_05827_b200 import build
    build.build()
    import paper_2311_05827_b200 as pkg
    return pkg


def declared_functions():
    text = open(os.path.join(ROOT, "include", "accept.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(accept_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(A):
    from paper_2311_05827_b200 import binding
    names = declared_functions()
    assert len(names) >= 12
    lib = binding.lib()
    for name in names:
        assert hasattr(lib, name), f"{name} declared in accept.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_params_struct_matches_header_layout(A):
    from paper_2311_05827_b200.binding import CParams
    assert ctypes.sizeof(CParams) == 48
    assert CParams.seed.offset == 32 and CParams.rng_offset.offset == 40 and CParams.range.offset == 16


@pytest.mark.parametrize("n,chunk,k", [(1, 32, 2), (100, 32, 3), (5000, 1024, 4), (4096, 4096, 8),
                                       (1 << 20, 1 << 20, 2), (51380224, 4096, 4), (268435456, 4096, 8),
                                       (2 ** 33 + 5, 4096, 2)])
def test_size_queries_match_oracle(A, n, chunk, k):
    layout = A.LAYOUT_BITPLANE if k == 3 else A.LAYOUT_INTERLEAVED
    p = A.Params(n, chunk, k, layout=layout)
    assert A.accept_check_params(p) == 0
    assert A.accept_compressed_size(p) == oracle.stream_bytes(n, chunk, k)
    assert A.accept_payload_offset(p) == oracle.payload_offset(n, chunk)
    assert A.accept_workspace_size(p) == 16 + (16 * -(-n // chunk) if chunk > 32768 else 0)


def test_workspace_grows_with_wide_chunks_and_static_scratch_refuses_them(A):
    """16 bytes, plus a 16-byte record per chunk once chunks exceed 32768 elements; the built-in
    256-byte scratch of accept_compress_static holds 15 such records and refuses more."""
    from paper_2311_05827_b200 import binding
    assert A.accept_workspace_size(A.Params(10 ** 6, 32768, 4)) == 16
    assert A.accept_workspace_size(A.Params(10 ** 6, 32800, 4)) == 16 + 16 * 31
    assert A.accept_workspace_size(A.Params(10 ** 6, 1 << 20, 4)) == 32
    lib = binding.lib()
    good = 0x10000
    for n, chunk, want in [(10 ** 6, 32800, 11), (15 * 65536, 65536, 1)]:  # 31 records: refused; 15 fit (then NULL input)
        p = A.Params(n, chunk, 4)
        size = A.accept_compressed_size(p)
        x_ptr = good if want == 11 else None
        assert lib.accept_compress_static(ctypes.byref(p.c()), x_ptr, good, size, None, None) == want


def test_mbq_size_queries_match_oracle(A):
    for n, k in [(1, 2), (1000, 3), (1 << 20, 4), (51380224, 4)]:
        p = A.MbqParams(n, k)
        assert A.accept_mbq_check_params(p) == 0
        assert A.accept_mbq_compressed_size(p) == oracle.mbq_stream_bytes(n, k)
        assert A.accept_mbq_payload_offset(p) == oracle.mbq_payload_offset(k)
        assert A.accept_mbq_workspace_size(p) == 64 + 8 * 5 * 12 + 80  # status and coefficients, five exact sums of 12 digits, ten counts
    assert A.accept_mbq_compressed_size(A.MbqParams(10, 7)) == 0


def test_invalid_params_are_rejected(A):
    P = A.Params
    assert A.accept_check_params(P(0, 32, 4)) == 9
    assert A.accept_check_params(P(10, 0, 4)) == 3
    assert A.accept_check_params(P(10, 48, 4)) == 3
    assert A.accept_check_params(P(10, 32, 5)) == 2
    assert A.accept_check_params(P(10, 32, 3)) == 2                       # k = 3 needs BITPLANE
    assert A.accept_check_params(P(10, 32, 3, layout=A.LAYOUT_BITPLANE)) == 0
    assert A.accept_check_params(P(10, 32, 4, range=2)) == 4
    assert A.accept_check_params(P(10, 32, 4, round=-1)) == 4
    assert A.accept_check_params(P(10, 32, 4, layout=7)) == 4
    for bad in (P(0, 32, 4), P(10, 33, 4), P(10, 32, 1)):
        assert A.accept_compressed_size(bad) == 0 and A.accept_workspace_size(bad) == 0


def test_entry_points_validate_before_launching(A):
    """Bad arguments return an error code without any CUDA call (this machine has no GPU)."""
    from paper_2311_05827_b200 import binding
    lib = binding.lib()
    before = A.accept_launch_count()
    p = A.Params(1000, 32, 4).c()
    size = oracle.stream_bytes(1000, 32, 4)
    good = 0x10000  # never dereferenced on the host
    assert lib.accept_compress(ctypes.byref(p), None, good, size, good, 16, None) == 1
    assert lib.accept_compress(ctypes.byref(p), good, None, size, good, 16, None) == 1
    assert lib.accept_compress(ctypes.byref(p), good, good, size, None, 16, None) == 1
    assert lib.accept_compress(ctypes.byref(p), good, good, size - 1, good, 16, None) == 5
    assert lib.accept_compress(ctypes.byref(p), good, good, size, good, 15, None) == 5
    assert lib.accept_compress(ctypes.byref(p), good + 4, good, size, good, 16, None) == 10
    assert lib.accept_decompress(ctypes.byref(p), good, size, None, good, 16, None) == 1
    assert lib.accept_decompress(ctypes.byref(p), good, size - 1, good, good, 16, None) == 5
    bad = A.Params(1000, 32, 7).c()
    assert lib.accept_compress(ctypes.byref(bad), good, good, size, good, 16, None) == 2
    assert lib.accept_compress_host(ctypes.byref(p), None, good, size, good, good, good, 16, None) == 1
    assert lib.accept_decompress_host(ctypes.byref(p), good, size, None, good, good, good, 16, None) == 1
    assert A.accept_launch_count() == before


def test_parse_header_reads_an_oracle_stream(A):
    x = workloads.random_tensor(777, 4, "normal")
    stream, _ = oracle.compress(x, 96, 3, oracle.RANGE_MINMAX, oracle.ROUND_STOCHASTIC, oracle.LAYOUT_BITPLANE, 5, 6)
    p = A.accept_parse_header(bytes(stream[:32]))
    assert (p.n_elems, p.chunk_elems, p.k, p.range, p.round, p.layout) == (777, 96, 3, 1, 1, 1)
    broken = stream[:32].copy()
    broken[1] ^= 0x40
    with pytest.raises(A.AcceptError):
        A.accept_parse_header(bytes(broken))
    broken = stream[:32].copy()
    broken[20] = 6  # k = 6
    with pytest.raises(A.AcceptError):
        A.accept_parse_header(bytes(broken))


def test_bitwidth_schedule_matches_the_paper(A):
    assert [A.accept_bitwidth_schedule(False, c) for c in range(5)] == [2, 3, 4, 4, 4]
    assert [A.accept_bitwidth_schedule(True, c) for c in range(4)] == [8, 4, 4, 4]
    for back in (False, True):
        for c in range(-1, 6):
            assert A.accept_bitwidth_schedule(back, c) == oracle.bitwidth_schedule(back, c)


def test_workload_generator_is_sliceable_and_seeded():
    a = workloads.generate("cfg3_act", (1 << 20) - 100, 300)
    b = workloads.generate("cfg3_act", (1 << 20) - 100, 300)
    whole = workloads.generate("cfg3_act", 0, (1 << 20) + 500)
    assert np.array_equal(a, b) and np.array_equal(a, whole[(1 << 20) - 100:(1 << 20) + 200])
    x = workloads.generate("cfg1_act")
    assert x.size == 32 * 64 * 32 * 32 and 0.45 < (x == 0).mean() < 0.55 and x.min() >= 0
    g = workloads.generate("cfg2_grad")
    assert abs(np.abs(g).max() - 0.05) < 1e-6 and 0.0005 < (np.abs(g) == np.float32(0.05)).mean() < 0.002
    h = workloads.generate("cfg4_hidden", 0, 4096 * 4)
    assert np.allclose(h[:4096].std() / h[4096:8192].std(), 1, atol=0.2)


def test_recorded_traffic_is_quoted_only_for_unchanged_sources(tmp_path, monkeypatch):
    """bench.py's roofline.traffic: the stored ncu bytes are returned while the files the captured kernel is
    compiled from are the captured ones, and None as soon as one of them differs."""
    import json
    import bench
    files = ["accept_api.cu", "accept_device.cuh", "accept_kernels.cuh"]
    table = {"captures": {"w": {"accept_compress": {"dram_bytes_per_launch": 123.0, "sources": files,
                                                    "sources_digest": bench.kernel_sources_digest(files)},
                                "accept_decompress": {"dram_bytes_per_launch": 5.0, "sources": files,
                                                      "sources_digest": "0" * 16}}}}
    (tmp_path / "profiles").mkdir()
    (tmp_path / "profiles" / "traffic.json").write_text(json.dumps(table))
    real_root = bench.ROOT
    real_digest = bench.kernel_sources_digest(files)
    monkeypatch.setattr(bench, "kernel_sources_digest", lambda f=None: real_digest)
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    assert bench.recorded_traffic("w", "accept_compress") == 123.0
    assert bench.recorded_traffic("w", "accept_decompress") is None      # another digest: the kernel has changed
    assert bench.recorded_traffic("w", "accept_mbq_compress") is None    # never captured
    assert bench.recorded_traffic("other", "accept_compress") is None
    monkeypatch.setattr(bench, "ROOT", real_root)
    monkeypatch.undo()
    # the committed table: rows are well formed (whether they are current is the bench's business)
    with open(os.path.join(real_root, "profiles", "traffic.json")) as f:
        committed = json.load(f)
    for rows in committed["captures"].values():
        for row in rows.values():
            assert row["dram_bytes_per_launch"] == row["read"] + row["written"]
            assert all(os.path.exists(os.path.join(real_root, "paper_2311_05827_b200", "csrc", s)) for s in row["sources"])
