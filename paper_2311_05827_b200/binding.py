"""Thin ctypes binding of the C ABI in ``include/accept.h``: argument marshalling only.

Every function below passes device (or host) pointers and sizes straight to the shared library;
no step of the codec runs in Python or in torch.  Torch is used for device memory and for the
current CUDA stream.  Loading fails loudly when the library has not been built.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaccept.so")

RANGE_ABSMAX, RANGE_MINMAX = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
LAYOUT_INTERLEAVED, LAYOUT_BITPLANE = 0, 1
HEADER_BYTES = 32

OK = 0
DEV_NONFINITE, DEV_BAD_HEADER, DEV_COPY_TIMEOUT = 1, 2, 4

STATUS_NAMES = {
    0: "ACCEPT_OK", 1: "ACCEPT_ERR_NULL", 2: "ACCEPT_ERR_BAD_K", 3: "ACCEPT_ERR_BAD_CHUNK",
    4: "ACCEPT_ERR_BAD_ENUM", 5: "ACCEPT_ERR_TOO_SMALL", 6: "ACCEPT_ERR_BAD_STREAM_HEADER",
    7: "ACCEPT_ERR_CUDA", 8: "ACCEPT_ERR_NONFINITE", 9: "ACCEPT_ERR_BAD_SIZE", 10: "ACCEPT_ERR_MISALIGNED",
    11: "ACCEPT_ERR_SCRATCH_LIMIT", 12: "ACCEPT_ERR_UNCHECKED_BUILD",
}

EXPORTS = [
    "accept_check_params", "accept_compressed_size", "accept_payload_offset", "accept_workspace_size",
    "accept_compress", "accept_decompress", "accept_compress_host", "accept_decompress_host",
    "accept_last_device_status", "accept_parse_header", "accept_bitwidth_schedule", "accept_launch_count",
    "accept_compress_static", "accept_bounds_check_report", "accept_launch_null",
    "accept_mbq_check_params", "accept_mbq_compressed_size", "accept_mbq_payload_offset", "accept_mbq_workspace_size",
    "accept_mbq_compress", "accept_mbq_decompress",
]


class AcceptError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)}")


class CParams(ctypes.Structure):
    _fields_ = [("n_elems", ctypes.c_uint64), ("chunk_elems", ctypes.c_uint32), ("k", ctypes.c_uint32),
                ("range", ctypes.c_int32), ("round", ctypes.c_int32), ("layout", ctypes.c_int32),
                ("group_stride", ctypes.c_uint32), ("seed", ctypes.c_uint64), ("rng_offset", ctypes.c_uint64)]


@dataclass(frozen=True)
class Params:
    n_elems: int
    chunk_elems: int
    k: int
    range: int = RANGE_ABSMAX
    round: int = ROUND_NEAREST
    layout: int = LAYOUT_INTERLEAVED
    seed: int = 0
    rng_offset: int = 0
    group_stride: int = 0

    def __post_init__(self):
        # the C struct is built once: calls only pass a reference to it
        object.__setattr__(self, "_c", CParams(self.n_elems, self.chunk_elems, self.k, self.range, self.round,
                                               self.layout, self.group_stride, self.seed & (2**64 - 1),
                                               self.rng_offset & (2**64 - 1)))

    def c(self) -> CParams:
        return self._c


class CMbqParams(ctypes.Structure):
    _fields_ = [("n_elems", ctypes.c_uint64), ("k", ctypes.c_uint32), ("batch_index", ctypes.c_uint32),
                ("init", ctypes.c_uint32), ("reserved", ctypes.c_uint32)]


@dataclass(frozen=True)
class MbqParams:
    n_elems: int
    k: int
    batch_index: int = 0
    init: bool = False

    def c(self) -> CMbqParams:
        return CMbqParams(self.n_elems, self.k, self.batch_index, 1 if self.init else 0, 0)


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2311_05827_b200.build`")
    _lib = load(LIB_PATH)
    return _lib


def load(path: str) -> ctypes.CDLL:
    """Loads a build of the library (the product, or one of the tests-only variants of build.py) and
    declares the argument types of its entry points."""
    L = ctypes.CDLL(path)
    P, vp, sz, u64 = ctypes.POINTER(CParams), ctypes.c_void_p, ctypes.c_size_t, ctypes.c_uint64
    L.accept_check_params.restype = ctypes.c_int
    L.accept_check_params.argtypes = [P]
    for name in ("accept_compressed_size", "accept_payload_offset", "accept_workspace_size"):
        getattr(L, name).restype = sz
        getattr(L, name).argtypes = [P]
    L.accept_compress.restype = ctypes.c_int
    L.accept_compress.argtypes = [P, vp, vp, sz, vp, sz, vp]
    L.accept_decompress.restype = ctypes.c_int
    L.accept_decompress.argtypes = [P, vp, sz, vp, vp, sz, vp]
    L.accept_compress_host.restype = ctypes.c_int
    L.accept_compress_host.argtypes = [P, vp, vp, sz, vp, vp, vp, sz, vp]
    L.accept_decompress_host.restype = ctypes.c_int
    L.accept_decompress_host.argtypes = [P, vp, sz, vp, vp, vp, vp, sz, vp]
    L.accept_last_device_status.restype = ctypes.c_int
    L.accept_last_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    L.accept_parse_header.restype = ctypes.c_int
    L.accept_parse_header.argtypes = [vp, P]
    L.accept_bitwidth_schedule.restype = ctypes.c_int
    L.accept_bitwidth_schedule.argtypes = [ctypes.c_int, ctypes.c_int]
    L.accept_compress_static.restype = ctypes.c_int
    L.accept_compress_static.argtypes = [P, vp, vp, sz, vp, vp]
    MP = ctypes.POINTER(CMbqParams)
    L.accept_mbq_check_params.restype = ctypes.c_int
    L.accept_mbq_check_params.argtypes = [MP]
    for name in ("accept_mbq_compressed_size", "accept_mbq_payload_offset", "accept_mbq_workspace_size"):
        getattr(L, name).restype = sz
        getattr(L, name).argtypes = [MP]
    L.accept_mbq_compress.restype = ctypes.c_int
    L.accept_mbq_compress.argtypes = [MP, vp, vp, vp, vp, sz, vp, sz, vp]
    L.accept_mbq_decompress.restype = ctypes.c_int
    L.accept_mbq_decompress.argtypes = [MP, vp, sz, vp, vp, sz, vp]
    L.accept_launch_count.restype = u64
    L.accept_launch_count.argtypes = []
    L.accept_launch_null.restype = ctypes.c_int
    L.accept_launch_null.argtypes = [ctypes.c_uint32, ctypes.c_uint32, vp]
    L.accept_bounds_check_report.restype = ctypes.c_int
    L.accept_bounds_check_report.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(u64), ctypes.POINTER(u64)]
    return L


def _check(code: int, where: str) -> None:
    if code != OK:
        raise AcceptError(code, where)


def _stream_handle(stream=None) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


# ---- size queries (host only) -------------------------------------------------------------

def accept_check_params(p: Params) -> int:
    return int(lib().accept_check_params(ctypes.byref(p.c())))


def accept_compressed_size(p: Params) -> int:
    return int(lib().accept_compressed_size(ctypes.byref(p.c())))


def accept_payload_offset(p: Params) -> int:
    return int(lib().accept_payload_offset(ctypes.byref(p.c())))


def accept_workspace_size(p: Params) -> int:
    return int(lib().accept_workspace_size(ctypes.byref(p.c())))


def accept_bitwidth_schedule(is_backward: bool, n_lr_changes: int) -> int:
    return int(lib().accept_bitwidth_schedule(int(is_backward), int(n_lr_changes)))


def accept_launch_count() -> int:
    return int(lib().accept_launch_count())


def accept_parse_header(header_bytes: bytes) -> Params:
    buf = ctypes.create_string_buffer(bytes(header_bytes[:HEADER_BYTES]), HEADER_BYTES)
    out = CParams()
    _check(lib().accept_parse_header(ctypes.cast(buf, ctypes.c_void_p), ctypes.byref(out)), "accept_parse_header")
    return Params(out.n_elems, out.chunk_elems, out.k, out.range, out.round, out.layout, group_stride=out.group_stride)


# ---- device entry points -------------------------------------------------------------------

def accept_compress(p: Params, d_x, d_stream, d_ws, stream=None) -> None:
    """d_x: float32 CUDA tensor (n_elems); d_stream: uint8 CUDA tensor; d_ws: CUDA workspace tensor."""
    _check(lib().accept_compress(ctypes.byref(p.c()), d_x.data_ptr(), d_stream.data_ptr(),
                                 d_stream.numel() * d_stream.element_size(), d_ws.data_ptr(),
                                 d_ws.numel() * d_ws.element_size(), _stream_handle(stream)), "accept_compress")


def accept_compress_static(p: Params, d_x, d_stream, d_status_out=None, stream=None) -> None:
    """accept_compress with the library's built-in scratch: for callers that cannot allocate a workspace.
    d_status_out: optional int32/uint32 CUDA tensor (>= 1 element) that receives this call's status bits."""
    _check(lib().accept_compress_static(ctypes.byref(p.c()), d_x.data_ptr(), d_stream.data_ptr(),
                                        d_stream.numel() * d_stream.element_size(),
                                        None if d_status_out is None else d_status_out.data_ptr(),
                                        _stream_handle(stream)), "accept_compress_static")


def accept_decompress(p: Params, d_stream, d_xhat, d_ws, stream=None) -> None:
    _check(lib().accept_decompress(ctypes.byref(p.c()), d_stream.data_ptr(),
                                   d_stream.numel() * d_stream.element_size(), d_xhat.data_ptr(),
                                   d_ws.data_ptr(), d_ws.numel() * d_ws.element_size(),
                                   _stream_handle(stream)), "accept_decompress")


def accept_compress_host(p: Params, h_x, h_stream, d_x, d_stream, d_ws, stream=None) -> None:
    """h_x / h_stream: host tensors (pinned for asynchronous copies); d_*: device staging buffers."""
    _check(lib().accept_compress_host(ctypes.byref(p.c()), h_x.data_ptr(), h_stream.data_ptr(),
                                      d_stream.numel() * d_stream.element_size(), d_x.data_ptr(),
                                      d_stream.data_ptr(), d_ws.data_ptr(), d_ws.numel() * d_ws.element_size(),
                                      _stream_handle(stream)), "accept_compress_host")


def accept_decompress_host(p: Params, h_stream, h_xhat, d_stream, d_xhat, d_ws, stream=None) -> None:
    _check(lib().accept_decompress_host(ctypes.byref(p.c()), h_stream.data_ptr(),
                                        d_stream.numel() * d_stream.element_size(), h_xhat.data_ptr(),
                                        d_stream.data_ptr(), d_xhat.data_ptr(), d_ws.data_ptr(),
                                        d_ws.numel() * d_ws.element_size(), _stream_handle(stream)),
           "accept_decompress_host")


def accept_launch_null(blocks: int, threads: int, stream=None) -> None:
    _check(lib().accept_launch_null(blocks, threads, _stream_handle(stream)), "accept_launch_null")


def accept_bounds_check_report(stream=None):
    """-> (return code, skipped accesses, address of the first, its size, whether it was a write)."""
    count, addr, info = ctypes.c_uint32(0), ctypes.c_uint64(0), ctypes.c_uint64(0)
    code = lib().accept_bounds_check_report(_stream_handle(stream), ctypes.byref(count), ctypes.byref(addr), ctypes.byref(info))
    return int(code), int(count.value), int(addr.value), int(info.value & 0xFFFFFFFF), bool(info.value >> 32)


def accept_last_device_status(d_ws, stream=None) -> int:
    bits = ctypes.c_uint32(0)
    _check(lib().accept_last_device_status(d_ws.data_ptr(), _stream_handle(stream), ctypes.byref(bits)),
           "accept_last_device_status")
    return int(bits.value)


# ---- multi-bit quantization (forward path) ----------------------------------------------------

def accept_mbq_check_params(p: MbqParams) -> int:
    return int(lib().accept_mbq_check_params(ctypes.byref(p.c())))


def accept_mbq_compressed_size(p: MbqParams) -> int:
    return int(lib().accept_mbq_compressed_size(ctypes.byref(p.c())))


def accept_mbq_payload_offset(p: MbqParams) -> int:
    return int(lib().accept_mbq_payload_offset(ctypes.byref(p.c())))


def accept_mbq_workspace_size(p: MbqParams) -> int:
    return int(lib().accept_mbq_workspace_size(ctypes.byref(p.c())))


def accept_mbq_compress(p: MbqParams, d_x, d_alpha_prev, d_alpha_next, d_stream, d_ws, stream=None) -> None:
    """d_alpha_prev (may be None when p.init) and d_alpha_next: float32 CUDA tensors of k elements."""
    _check(lib().accept_mbq_compress(ctypes.byref(p.c()), d_x.data_ptr(),
                                     None if d_alpha_prev is None else d_alpha_prev.data_ptr(),
                                     d_alpha_next.data_ptr(), d_stream.data_ptr(),
                                     d_stream.numel() * d_stream.element_size(), d_ws.data_ptr(),
                                     d_ws.numel() * d_ws.element_size(), _stream_handle(stream)), "accept_mbq_compress")


def accept_mbq_decompress(p: MbqParams, d_stream, d_xhat, d_ws, stream=None) -> None:
    _check(lib().accept_mbq_decompress(ctypes.byref(p.c()), d_stream.data_ptr(),
                                       d_stream.numel() * d_stream.element_size(), d_xhat.data_ptr(),
                                       d_ws.data_ptr(), d_ws.numel() * d_ws.element_size(),
                                       _stream_handle(stream)), "accept_mbq_decompress")


# ---- small conveniences for callers (allocation only) -----------------------------------------

def new_stream_buffer(p, device="cuda"):
    import torch
    size = accept_mbq_compressed_size(p) if isinstance(p, MbqParams) else accept_compressed_size(p)
    return torch.empty(size, dtype=torch.uint8, device=device)


def new_workspace(p, device="cuda"):
    import torch
    size = accept_mbq_workspace_size(p) if isinstance(p, MbqParams) else accept_workspace_size(p)
    return torch.zeros((size + 3) // 4, dtype=torch.int32, device=device)
