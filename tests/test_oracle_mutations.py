"""The pins must be able to fail: each plausible mistake planted in a COPY of the oracle's source
(on the CPU, in a temporary directory) has to break at least one pin.  This guards the pins, not
the oracle: a pin that no mistake can break pins nothing."""
import ctypes
import os
import subprocess

import pytest

import oracle
from tests import test_oracle_mbq_pins as mbq_pins
from tests import test_oracle_pins as pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "accept_oracle.c")

MUTATIONS = [
    ("flipped comparison in Eq. 7", "q = (int)f + ((U < pr) ? 1 : 0);", "q = (int)f + ((U > pr) ? 1 : 0);"),
    ("wrong level count", "float L = (float)((1 << (k - 1)) - 1);", "float L = (float)((1 << (k - 1)));"),
    ("mirrored bit order", "words[pos / 32] |= bit << (pos % 32);", "words[pos / 32] |= bit << (31 - pos % 32);"),
    ("biased quantizer", "float t = d * inv;", "float t = d * inv + 0.5f;"),
    ("ties away from zero", "q = (int)rintf(t);", "q = (int)roundf(t);"),
    ("truncation instead of floor", "double f = floor((double)t);", "double f = trunc((double)t);"),
    ("dropped zero point", "u[i] = (uint8_t)(q + zero_point);", "u[i] = (uint8_t)(q);"),
    ("offset not subtracted", "float d = (range == RANGE_ABSMAX) ? x[i] : (x[i] - base);", "float d = x[i];"),
    ("transposed planes", "else pos = 32ull * ((uint64_t)(t / 32) * k + j) + (t % 32);",
     "else pos = 32ull * ((uint64_t)(t / 32) * k + (k - 1 - j)) + (t % 32);"),
    ("MBQ: wrong sign of a basis", "float term = ((c >> j) & 1u) ? alpha[j] : -alpha[j];",
     "float term = ((c >> j) & 1u) ? -alpha[j] : alpha[j];"),
    ("MBQ: moving average weights swapped", "(float)(beta * (double)alpha_prev[p] + (1.0 - beta) * cur[p]);",
     "(float)((1.0 - beta) * (double)alpha_prev[p] + beta * cur[p]);"),
    ("weak lane multiplier in the generator of Eq. 7", "{1u, 0x9E3779B1u, 0x85EBCA77u, 0xC2B2AE3Du}", "{1u, 0x00010001u, 0x85EBCA77u, 0xC2B2AE3Du}"),
    ("exact sum drops the part below 2^-149 * 2^64", "uint64_t lo = v << off, hi = off ? (v >> (64 - off)) : 0;", "uint64_t lo = v << off, hi = 0;"),
    ("exact sum rounds half up instead of to even", "if (guard && (sticky || (mant & 1u))) ++mant;", "if (guard) ++mant;"),
    ("MBQ: bias with the wrong sign", "return (float)((acc - sum_x) / (double)n);", "return (float)((sum_x - acc) / (double)n);"),
]

PIN_FUNCS = [getattr(pins, n) for n in dir(pins) if n.startswith("test_")] + \
            [getattr(mbq_pins, n) for n in dir(mbq_pins) if n.startswith("test_")]


def _run_all_pins():
    """1 as soon as a pin function fails (parametrized ones are run over their parameter sets), else 0."""
    failed = 0
    for fn in PIN_FUNCS:
        if failed:
            return failed
        marks = [m for m in getattr(fn, "pytestmark", []) if m.name == "parametrize"]
        cases = [{}]
        for m in marks:
            names = [s.strip() for s in m.args[0].split(",")]
            new = []
            for base in cases:
                for val in m.args[1]:
                    vals = val if len(names) > 1 else (val,)
                    new.append(dict(base, **dict(zip(names, vals))))
            cases = new
        for kw in cases:
            try:
                fn(**kw)
            except AssertionError:
                failed += 1
                break
            except Exception:
                failed += 1
                break
    return failed


@pytest.mark.parametrize("name,old,new", MUTATIONS, ids=[m[0] for m in MUTATIONS])
def test_planted_mistake_is_caught(tmp_path, name, old, new):
    text = open(SRC).read()
    assert text.count(old) >= 1, f"mutation target not found: {old}"
    src = tmp_path / "mutant.c"
    src.write_text(text.replace(old, new))
    lib = tmp_path / "libmutant.so"
    subprocess.run(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-o", str(lib), str(src), "-lm"],
                   check=True)
    real = oracle._load()
    mutant = ctypes.CDLL(str(lib))
    for attr in dir(real):
        if attr.startswith("oracle_"):
            f = getattr(mutant, attr)
            f.restype, f.argtypes = getattr(real, attr).restype, getattr(real, attr).argtypes
    oracle._lib = mutant
    try:
        assert _run_all_pins() >= 1, f"no pin noticed: {name}"
    finally:
        oracle._lib = real
