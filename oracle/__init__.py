"""TEST INFRASTRUCTURE: ctypes access to the CPU oracle (``accept_oracle.c``).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package.  It
shares nothing with the CUDA library: its own C file, its own shared object, its own argument
lists.  ``build()`` compiles the C file with gcc (no fast-math, no FMA contraction).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "accept_oracle.c")
_LIB = os.path.join(_HERE, "libaccept_oracle.so")

RANGE_ABSMAX, RANGE_MINMAX = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
LAYOUT_INTERLEAVED, LAYOUT_BITPLANE = 0, 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if its shared object is missing or older than the source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    u64, u32, i32 = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int
    vp = ctypes.c_void_p
    lib.oracle_payload_offset.restype = u64
    lib.oracle_payload_offset.argtypes = [u64, u32]
    lib.oracle_payload_bytes.restype = u64
    lib.oracle_payload_bytes.argtypes = [u64, u32]
    lib.oracle_stream_bytes.restype = u64
    lib.oracle_stream_bytes.argtypes = [u64, u32, u32]
    lib.oracle_rng_hash.restype = u32
    lib.oracle_rng_hash.argtypes = [u64, u64]
    lib.oracle_rng_fill.restype = None
    lib.oracle_rng_fill.argtypes = [u64, u64, u64, vp]
    lib.oracle_rng_uniform.restype = ctypes.c_double
    lib.oracle_rng_uniform.argtypes = [u64, u64]
    lib.oracle_quantize.restype = i32
    lib.oracle_quantize.argtypes = [vp, u64, u32, u32, i32, i32, u64, u64, vp, vp]
    lib.oracle_pack.restype = None
    lib.oracle_pack.argtypes = [vp, u64, u32, u32, i32, vp]
    lib.oracle_unpack.restype = None
    lib.oracle_unpack.argtypes = [vp, u64, u32, u32, i32, vp]
    lib.oracle_dequantize.restype = None
    lib.oracle_dequantize.argtypes = [vp, vp, u64, u32, u32, i32, vp]
    lib.oracle_compress.restype = i32
    lib.oracle_compress.argtypes = [vp, u64, u32, u32, i32, i32, i32, u64, u64, vp]
    lib.oracle_decompress.restype = i32
    lib.oracle_decompress.argtypes = [vp, u64, u64, vp]
    lib.oracle_bitwidth_schedule.restype = i32
    lib.oracle_bitwidth_schedule.argtypes = [i32, i32]
    f32p = vp
    lib.oracle_mbq_payload_offset.restype = u64
    lib.oracle_mbq_payload_offset.argtypes = [u32]
    lib.oracle_mbq_stream_bytes.restype = u64
    lib.oracle_mbq_stream_bytes.argtypes = [u64, u32]
    lib.oracle_reciprocal_toward_zero.restype = ctypes.c_float
    lib.oracle_reciprocal_toward_zero.argtypes = [ctypes.c_float, ctypes.c_float]
    lib.oracle_exact_sum.restype = ctypes.c_double
    lib.oracle_exact_sum.argtypes = [vp, u64]
    lib.oracle_exact_abs_sum.restype = ctypes.c_double
    lib.oracle_exact_abs_sum.argtypes = [vp, u64]
    lib.oracle_exact_signed_sum.restype = ctypes.c_double
    lib.oracle_exact_signed_sum.argtypes = [vp, vp, u64, u32]
    lib.oracle_mbq_levels.restype = None
    lib.oracle_mbq_levels.argtypes = [f32p, u32, f32p]
    lib.oracle_mbq_assign_nearest.restype = None
    lib.oracle_mbq_assign_nearest.argtypes = [vp, u64, f32p, u32, vp]
    lib.oracle_mbq_assign_residue.restype = None
    lib.oracle_mbq_assign_residue.argtypes = [vp, u64, u32, vp, f32p]
    lib.oracle_mbq_update_alpha.restype = None
    lib.oracle_mbq_update_alpha.argtypes = [vp, vp, u64, u32, f32p, u32, f32p]
    lib.oracle_mbq_bias.restype = ctypes.c_float
    lib.oracle_mbq_bias.argtypes = [vp, vp, u64, u32, f32p]
    lib.oracle_mbq_compress.restype = None
    lib.oracle_mbq_compress.argtypes = [vp, u64, u32, u32, i32, f32p, vp, f32p]
    lib.oracle_mbq_decompress.restype = i32
    lib.oracle_mbq_decompress.argtypes = [vp, u64, u64, vp]
    lib.oracle_strided_payload_bytes.restype = u64
    lib.oracle_strided_payload_bytes.argtypes = [u64, u32, u32]
    lib.oracle_strided_stream_bytes.restype = u64
    lib.oracle_strided_stream_bytes.argtypes = [u64, u32, u32, u32]
    lib.oracle_compress_strided.restype = i32
    lib.oracle_compress_strided.argtypes = [vp, u64, u32, u32, i32, i32, i32, u64, u64, u32, vp]
    lib.oracle_decompress_strided.restype = i32
    lib.oracle_decompress_strided.argtypes = [vp, u64, u64, vp]
    _lib = lib
    return lib


def _f32(x) -> np.ndarray:
    a = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    return a


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def n_chunks(n: int, chunk: int) -> int:
    return (n + chunk - 1) // chunk


def payload_offset(n: int, chunk: int) -> int:
    return int(_load().oracle_payload_offset(n, chunk))


def payload_bytes(n: int, k: int) -> int:
    return int(_load().oracle_payload_bytes(n, k))


def stream_bytes(n: int, chunk: int, k: int) -> int:
    return int(_load().oracle_stream_bytes(n, chunk, k))


def rng_hash(seed: int, ctr: int) -> int:
    return int(_load().oracle_rng_hash(seed & (2**64 - 1), ctr & (2**64 - 1)))


def rng_words(seed: int, ctr0: int, n: int) -> np.ndarray:
    """The 32-bit words of counters ctr0 .. ctr0+n-1 (rng_hash in bulk)."""
    out = np.empty(n, dtype=np.uint32)
    _load().oracle_rng_fill(seed & (2**64 - 1), ctr0 & (2**64 - 1), n, _ptr(out))
    return out


def rng_uniform(seed: int, ctr: int) -> float:
    return float(_load().oracle_rng_uniform(seed & (2**64 - 1), ctr & (2**64 - 1)))


def quantize(x, chunk: int, k: int, range_: int = RANGE_ABSMAX, round_: int = ROUND_NEAREST,
             seed: int = 0, rng_offset: int = 0):
    """-> (codes uint8[n], meta float32[M,2], nonfinite flag)."""
    x = _f32(x)
    n = x.size
    codes = np.empty(n, dtype=np.uint8)
    meta = np.empty((n_chunks(n, chunk), 2), dtype=np.float32)
    flag = _load().oracle_quantize(_ptr(x), n, chunk, k, range_, round_, seed, rng_offset,
                                   _ptr(codes), _ptr(meta))
    return codes, meta, int(flag)


def pack(codes, chunk: int, k: int, layout: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    out = np.empty(payload_bytes(codes.size, k) // 4, dtype=np.uint32)
    _load().oracle_pack(_ptr(codes), codes.size, chunk, k, layout, _ptr(out))
    return out


def unpack(payload, n: int, chunk: int, k: int, layout: int) -> np.ndarray:
    payload = np.ascontiguousarray(payload, dtype=np.uint32).reshape(-1)
    assert payload.size * 4 >= payload_bytes(n, k)
    codes = np.empty(n, dtype=np.uint8)
    _load().oracle_unpack(_ptr(payload), n, chunk, k, layout, _ptr(codes))
    return codes


def dequantize(codes, meta, chunk: int, k: int, range_: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    meta = np.ascontiguousarray(meta, dtype=np.float32)
    xhat = np.empty(codes.size, dtype=np.float32)
    _load().oracle_dequantize(_ptr(codes), _ptr(meta), codes.size, chunk, k, range_, _ptr(xhat))
    return xhat


def compress(x, chunk: int, k: int, range_: int = RANGE_ABSMAX, round_: int = ROUND_NEAREST,
             layout: int = LAYOUT_INTERLEAVED, seed: int = 0, rng_offset: int = 0):
    """-> (stream uint8[stream_bytes], nonfinite flag)."""
    x = _f32(x)
    out = np.empty(stream_bytes(x.size, chunk, k), dtype=np.uint8)
    flag = _load().oracle_compress(_ptr(x), x.size, chunk, k, range_, round_, layout, seed,
                                   rng_offset, _ptr(out))
    return out, int(flag)


def decompress(stream, n: int) -> np.ndarray:
    stream = np.ascontiguousarray(stream, dtype=np.uint8).reshape(-1)
    xhat = np.empty(n, dtype=np.float32)
    rc = _load().oracle_decompress(_ptr(stream), stream.size, n, _ptr(xhat))
    if rc != 0:
        raise ValueError("oracle_decompress: invalid stream header")
    return xhat


def split_stream(stream, n: int, chunk: int):
    """Views of a stream: (header uint32[8], meta float32[M,2], payload uint32[...])."""
    stream = np.ascontiguousarray(stream, dtype=np.uint8).reshape(-1)
    m = n_chunks(n, chunk)
    header = stream[:32].view(np.uint32)
    meta = stream[32:32 + 8 * m].view(np.float32).reshape(m, 2)
    payload = stream[payload_offset(n, chunk):].view(np.uint32)
    return header, meta, payload


def bitwidth_schedule(is_backward: bool, n_lr_changes: int) -> int:
    return int(_load().oracle_bitwidth_schedule(int(is_backward), n_lr_changes))


# ---------------------------------------------------------------- multi-bit quantization (forward path)

def mbq_payload_offset(k: int) -> int:
    return int(_load().oracle_mbq_payload_offset(k))


def mbq_stream_bytes(n: int, k: int) -> int:
    return int(_load().oracle_mbq_stream_bytes(n, k))


def reciprocal_toward_zero(L: float, r: float) -> float:
    """The quantizer's reciprocal scale: L / r rounded toward zero in fp32."""
    return float(_load().oracle_reciprocal_toward_zero(L, r))


def exact_sum(x) -> float:
    """Sum of the fp32 values of x without rounding, rounded once to double (ties to even)."""
    x = _f32(x)
    return float(_load().oracle_exact_sum(_ptr(x), x.size))


def exact_abs_sum(x) -> float:
    x = _f32(x)
    return float(_load().oracle_exact_abs_sum(_ptr(x), x.size))


def exact_signed_sum(x, codes, p: int) -> float:
    """(B^T x)_p: +x where bit p of the code is set, -x elsewhere; exact, rounded once to double."""
    x = _f32(x)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    return float(_load().oracle_exact_signed_sum(_ptr(x), _ptr(codes), x.size, p))


def mbq_levels(alpha) -> np.ndarray:
    alpha = _f32(alpha)
    out = np.empty(1 << alpha.size, dtype=np.float32)
    _load().oracle_mbq_levels(_ptr(alpha), alpha.size, _ptr(out))
    return out


def mbq_assign_nearest(x, alpha) -> np.ndarray:
    x, alpha = _f32(x), _f32(alpha)
    codes = np.empty(x.size, dtype=np.uint8)
    _load().oracle_mbq_assign_nearest(_ptr(x), x.size, _ptr(alpha), alpha.size, _ptr(codes))
    return codes


def mbq_assign_residue(x, k: int):
    x = _f32(x)
    codes = np.empty(x.size, dtype=np.uint8)
    alpha0 = np.empty(k, dtype=np.float32)
    _load().oracle_mbq_assign_residue(_ptr(x), x.size, k, _ptr(codes), _ptr(alpha0))
    return codes, alpha0


def mbq_update_alpha(x, codes, alpha_prev, t: int) -> np.ndarray:
    x, alpha_prev = _f32(x), _f32(alpha_prev)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(alpha_prev.size, dtype=np.float32)
    _load().oracle_mbq_update_alpha(_ptr(x), _ptr(codes), x.size, alpha_prev.size, _ptr(alpha_prev), t, _ptr(out))
    return out


def mbq_bias(x, codes, alpha) -> float:
    x, alpha = _f32(x), _f32(alpha)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    return float(_load().oracle_mbq_bias(_ptr(x), _ptr(codes), x.size, alpha.size, _ptr(alpha)))


def mbq_compress(x, k: int, t: int, init: bool, alpha_prev=None):
    """-> (stream uint8[], alpha_next float32[k])."""
    x = _f32(x)
    alpha_prev = np.zeros(k, dtype=np.float32) if alpha_prev is None else _f32(alpha_prev)
    stream = np.empty(mbq_stream_bytes(x.size, k), dtype=np.uint8)
    alpha_next = np.empty(k, dtype=np.float32)
    _load().oracle_mbq_compress(_ptr(x), x.size, k, t, int(init), _ptr(alpha_prev), _ptr(stream), _ptr(alpha_next))
    return stream, alpha_next


def mbq_decompress(stream, n: int) -> np.ndarray:
    stream = np.ascontiguousarray(stream, dtype=np.uint8).reshape(-1)
    xhat = np.empty(n, dtype=np.float32)
    if _load().oracle_mbq_decompress(_ptr(stream), stream.size, n, _ptr(xhat)) != 0:
        raise ValueError("oracle_mbq_decompress: invalid stream header")
    return xhat


# ---------------------------------------------------------------- grouping along the batch dimension

def strided_stream_bytes(n: int, chunk: int, k: int, stride: int) -> int:
    return int(_load().oracle_strided_stream_bytes(n, chunk, k, stride))


def compress_strided(x, chunk: int, k: int, stride: int, range_: int = RANGE_ABSMAX, round_: int = ROUND_NEAREST,
                     layout: int = LAYOUT_INTERLEAVED, seed: int = 0, rng_offset: int = 0):
    """Pack groups = 32 batch neighbours of one feature; x is (n // stride) x stride.  -> (stream, flag)."""
    x = _f32(x)
    assert x.size % stride == 0
    out = np.empty(strided_stream_bytes(x.size, chunk, k, stride), dtype=np.uint8)
    flag = _load().oracle_compress_strided(_ptr(x), x.size, chunk, k, range_, round_, layout, seed, rng_offset,
                                           stride, _ptr(out))
    return out, int(flag)


def decompress_strided(stream, n: int) -> np.ndarray:
    stream = np.ascontiguousarray(stream, dtype=np.uint8).reshape(-1)
    xhat = np.empty(n, dtype=np.float32)
    if _load().oracle_decompress_strided(_ptr(stream), stream.size, n, _ptr(xhat)) != 0:
        raise ValueError("oracle_decompress_strided: invalid stream header")
    return xhat
