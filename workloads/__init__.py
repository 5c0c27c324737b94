"""Seeded synthetic boundary tensors shared by the tests, the oracle legs and the benchmark.

This module holds none of the codec's arithmetic: it only draws numbers.  Every tensor is
generated in independent blocks of ``BLOCK`` elements, block b of tensor T coming from
``numpy.random.default_rng([seed, tensor_id, b])``, so any slice can be produced without
generating what precedes it (used to check sampled chunks of the full-size tensors).

The tensors stand in for the boundary activations and gradients of the paper's MobileNetV2 /
simple-CNN pipelines (Sec. 4.3); their shapes and value distributions are the five workloads the
throughput metric is quoted on.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BLOCK = 1 << 20

RANGE_ABSMAX, RANGE_MINMAX = 0, 1
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
LAYOUT_INTERLEAVED, LAYOUT_BITPLANE = 0, 1


@dataclass(frozen=True)
class Mode:
    k: int
    range: int = RANGE_ABSMAX
    round: int = ROUND_NEAREST
    layout: int = LAYOUT_INTERLEAVED


@dataclass(frozen=True)
class Tensor:
    """One synthetic tensor: a name, a shape, a seed, a value recipe and the modes it is coded in."""
    name: str
    shape: tuple
    seed: int
    recipe: str               # key of _RECIPES
    chunk: int
    headline: tuple           # Modes that make the headline numbers
    also: tuple = ()          # Modes reported alongside
    tensor_id: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def n(self) -> int:
        return int(np.prod(self.shape))


def _relu_half_normal(rng, count, spec, start):
    """Exact zero with probability p_zero, else |N(0,1)|."""
    keep = rng.random(count) >= spec.extra.get("p_zero", 0.5)
    v = np.abs(rng.standard_normal(count, dtype=np.float32))
    return np.where(keep, v, np.float32(0)).astype(np.float32)


def _grad_outliers(rng, count, spec, start):
    """N(0, sigma) with a fraction p_out of positions replaced by +-50 sigma."""
    sigma = np.float32(spec.extra["sigma"])
    v = rng.standard_normal(count, dtype=np.float32) * sigma
    out = rng.random(count) < spec.extra.get("p_out", 0.001)
    sign = np.where(rng.random(count) < 0.5, np.float32(-1), np.float32(1))
    return np.where(out, sign * np.float32(50) * sigma, v).astype(np.float32)


def _relu_lognormal(rng, count, spec, start):
    """Exact zero with probability p_zero, else lognormal(mu=0, sigma=1)."""
    keep = rng.random(count) >= spec.extra.get("p_zero", 0.6)
    v = np.exp(rng.standard_normal(count, dtype=np.float32))
    return np.where(keep, v, np.float32(0)).astype(np.float32)


def _normal(rng, count, spec, start):
    return rng.standard_normal(count, dtype=np.float32) * np.float32(spec.extra["sigma"])


def _channel_scaled_normal(rng, count, spec, start):
    """N(0,1) times a per-hidden-channel scale U(lo,hi); the channel is the fastest dimension."""
    hidden = spec.shape[-1]
    srng = np.random.default_rng([spec.seed, spec.tensor_id, 0xC0FFEE])
    scale = srng.uniform(spec.extra.get("lo", 0.1), spec.extra.get("hi", 10.0), hidden)
    idx = (start + np.arange(count, dtype=np.int64)) % hidden
    return rng.standard_normal(count, dtype=np.float32) * scale.astype(np.float32)[idx]


_RECIPES = {
    "relu_half_normal": _relu_half_normal,
    "grad_outliers": _grad_outliers,
    "relu_lognormal": _relu_lognormal,
    "normal": _normal,
    "channel_scaled_normal": _channel_scaled_normal,
}

_ABS, _MM = RANGE_ABSMAX, RANGE_MINMAX
_NR, _SR = ROUND_NEAREST, ROUND_STOCHASTIC
_IL, _BP = LAYOUT_INTERLEAVED, LAYOUT_BITPLANE


def _sweep(name, nbytes, tid):
    return Tensor(name, (nbytes // 4,), 4, "relu_half_normal", 4096,
                  headline=(Mode(2, _ABS, _NR, _BP), Mode(4, _ABS, _NR, _BP), Mode(8, _ABS, _NR, _IL)),
                  also=(Mode(2, _ABS, _NR, _IL), Mode(4, _ABS, _NR, _IL), Mode(8, _ABS, _NR, _BP)),
                  tensor_id=tid)


TENSORS = {
    # 1: post-ReLU activation, 8 MB, 8-bit, chunk 4096
    "cfg1_act": Tensor("cfg1_act", (32, 64, 32, 32), 0, "relu_half_normal", 4096,
                       headline=(Mode(8, _ABS, _NR, _IL),),
                       also=(Mode(8, _MM, _NR, _IL), Mode(8, _ABS, _NR, _BP)), tensor_id=1),
    # 2: backward gradient with outliers, 4 MB, k in {2,4,8}, chunk 1024
    "cfg2_grad": Tensor("cfg2_grad", (32, 128, 16, 16), 1, "grad_outliers", 1024,
                        headline=tuple(Mode(k, _ABS, _SR, _IL) for k in (2, 4, 8)),
                        also=tuple(Mode(k, _ABS, _NR, _IL) for k in (2, 4, 8))
                        + tuple(Mode(k, _MM, _SR, _IL) for k in (2, 4, 8)),
                        tensor_id=2, extra={"sigma": 1e-3, "p_out": 0.001}),
    # 3: large CNN boundary: forward activation (compress) and same-shape gradient (decompress)
    "cfg3_act": Tensor("cfg3_act", (64, 256, 56, 56), 2, "relu_lognormal", 4096,
                       headline=(Mode(4, _ABS, _NR, _BP),), also=(Mode(4, _ABS, _NR, _IL),),
                       tensor_id=3, extra={"p_zero": 0.6}),
    "cfg3_grad": Tensor("cfg3_grad", (64, 256, 56, 56), 2, "normal", 4096,
                        headline=(Mode(4, _ABS, _SR, _IL),), also=(Mode(4, _ABS, _SR, _BP),),
                        tensor_id=4, extra={"sigma": 1e-2}),
    # 4: transformer hidden states, chunk = one hidden row
    "cfg4_hidden": Tensor("cfg4_hidden", (16, 1024, 4096), 3, "channel_scaled_normal", 4096,
                          headline=(Mode(8, _ABS, _NR, _IL),), also=(Mode(8, _MM, _NR, _IL),),
                          tensor_id=5, extra={"lo": 0.1, "hi": 10.0}),
    # 5: size sweep
    "cfg5_64KB": _sweep("cfg5_64KB", 64 << 10, 6),
    "cfg5_1MB": _sweep("cfg5_1MB", 1 << 20, 7),
    "cfg5_16MB": _sweep("cfg5_16MB", 16 << 20, 8),
    "cfg5_256MB": _sweep("cfg5_256MB", 256 << 20, 9),
    "cfg5_1GB": _sweep("cfg5_1GB", 1 << 30, 10),
}


def generate(name: str, start: int = 0, count: int | None = None) -> np.ndarray:
    """Elements [start, start+count) of tensor ``name`` as a flat float32 array."""
    spec = TENSORS[name]
    n = spec.n
    if count is None:
        count = n - start
    if start < 0 or count < 0 or start + count > n:
        raise ValueError("slice outside the tensor")
    out = np.empty(count, dtype=np.float32)
    fn = _RECIPES[spec.recipe]
    b = start // BLOCK
    pos = 0
    while pos < count:
        b0 = b * BLOCK
        blen = min(BLOCK, n - b0)
        rng = np.random.default_rng([spec.seed, spec.tensor_id, b])
        block = fn(rng, blen, spec, b0)
        lo = max(start, b0) - b0
        hi = min(start + count, b0 + blen) - b0
        out[pos:pos + hi - lo] = block[lo:hi]
        pos += hi - lo
        b += 1
    return out


def random_tensor(n: int, seed: int, kind: str = "normal") -> np.ndarray:
    """Small ad-hoc tensors for the property tests (no codec arithmetic here either)."""
    rng = np.random.default_rng([seed, n, 0xABCD])
    if kind == "normal":
        return rng.standard_normal(n, dtype=np.float32)
    if kind == "relu":
        v = np.abs(rng.standard_normal(n, dtype=np.float32))
        return np.where(rng.random(n) < 0.5, np.float32(0), v).astype(np.float32)
    if kind == "wide":  # values spread over many binades, both signs
        e = rng.uniform(-20, 20, n)
        return (np.exp2(e) * np.where(rng.random(n) < 0.5, -1.0, 1.0)).astype(np.float32)
    if kind == "uniform":
        return rng.uniform(-1, 1, n).astype(np.float32)
    raise ValueError(kind)
