"""The cubic that replaces ex2.approx for part of the forward softmax, re-evaluated on the host in fp32.

The coefficients are read from the CUDA header (they live nowhere else); the steps are the kernel's: clamp at -126,
n = rint(x) through the 1.5 * 2^23 addition, f = x - n in [-1/2, 1/2], Horner in fp32, n added into the exponent field.
Pinned against numpy's exp2 in fp64: the relative error stays below 1e-4, a thirtieth of the bf16 rounding (2^-9) that
P goes through before it is used; the integer path is exact at integer arguments and masked scores give (almost) zero.
"""
import pathlib
import re

import numpy as np

HDR = pathlib.Path(__file__).resolve().parents[1] / "paper_2609_22755_b200" / "csrc" / "sm100_ptx.cuh"


def _coefficients():
    text = HDR.read_text()
    body = text[text.index("void ex2_poly2("):]
    body = body[:body.index("\n}\n")]
    vals = {m.group(1): np.float32(m.group(2)) for m in re.finditer(r"\b(c[0-3]) = ([0-9.eE+-]+)f", body)}
    assert sorted(vals) == ["c0", "c1", "c2", "c3"]
    magic = np.float32(re.search(r"kMagic = ([0-9.]+)f", body).group(1))
    assert magic == np.float32(1.5 * 2 ** 23)
    return vals, magic


def _ex2_poly(x):
    c, magic = _coefficients()
    x = np.maximum(np.asarray(x, dtype=np.float32), np.float32(-126.0))
    t = (x + magic).astype(np.float32)
    f = (x - (t - magic).astype(np.float32)).astype(np.float32)
    q = (f * c["c3"] + c["c2"]).astype(np.float32)
    q = (q * f + c["c1"]).astype(np.float32)
    q = (q * f + c["c0"]).astype(np.float32)
    bits = (q.view(np.uint32).astype(np.uint64) + (t.view(np.uint32).astype(np.uint64) << np.uint64(23))) & np.uint64(0xFFFFFFFF)
    return bits.astype(np.uint32).view(np.float32), f


def test_relative_error_is_far_below_the_bf16_rounding_of_p():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.uniform(-40.0, 8.0, 400000), np.linspace(-1.0, 1.0, 100001)]).astype(np.float32)
    got, f = _ex2_poly(x)
    assert np.all(np.abs(f) <= 0.5)
    rel = np.abs(got.astype(np.float64) / np.exp2(x.astype(np.float64)) - 1.0)
    assert rel.max() < 1e-4 < 2.0 ** -9 / 15


def test_integer_arguments_and_masked_scores():
    n = np.arange(-120, 100, dtype=np.float32)
    got, _ = _ex2_poly(n)
    c, _ = _coefficients()
    assert np.allclose(got.astype(np.float64), float(c["c0"]) * np.exp2(n.astype(np.float64)), rtol=1e-7)
    tiny, _ = _ex2_poly(np.array([-np.inf, -1e30, -500.0, -126.0], dtype=np.float32))
    assert np.all(tiny >= 0) and np.all(tiny < 2e-38)
