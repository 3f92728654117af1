"""Host-side check of the FMA-pipe exponential of the attention kernel (common.cuh, fma_exp2).

The device routine is a cubic for 2^f on [-0.5, 0.5] plus an exponent splice.  The test reads the four
coefficients and the two constants out of the source, repeats the routine's steps in float32 with numpy and
compares with 2^x in float64: a mistyped coefficient, a wrong magic number or a wrong clamp fails here
without a GPU."""
import os
import re

import numpy as np

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2604_08077_b200", "csrc", "common.cuh")


def _routine():
    text = open(SRC).read()
    body = text[text.index("float fma_exp2(float x)"):]
    body = body[:body.index("\n}\n")]
    coef = [np.float32(c) for c in re.search(r"fmaf\(fmaf\(fmaf\(([0-9.eE+-]+)f, f, ([0-9.eE+-]+)f\), f, ([0-9.eE+-]+)f\), f, ([0-9.eE+-]+)f\)", body).groups()]
    clamp = np.float32(re.search(r"fmaxf\(x, (-[0-9.]+)f\)", body).group(1))
    magic = np.float32(re.search(r"xc \+ ([0-9.]+)f", body).group(1))
    assert "<< 23" in body
    return coef, clamp, magic


def _fma_exp2(x, coef, clamp, magic):
    x = x.astype(np.float32)
    xc = np.maximum(x, clamp)
    xr = (xc + magic).astype(np.float32)
    f = (xc - (xr - magic)).astype(np.float32)
    # fmaf rounds once; float64 products of float32 values are exact, so rounding the float64 result is an fmaf
    p = np.float32(coef[0])
    for c in coef[1:]:
        p = (p.astype(np.float64) * f.astype(np.float64) + np.float64(c)).astype(np.float32)
    bits = p.view(np.uint32) + (xr.view(np.uint32) << np.uint32(23))
    return bits.view(np.float32)


def test_magic_number_and_clamp():
    coef, clamp, magic = _routine()
    assert magic == np.float32(1.5 * 2.0 ** 23)          # adding it rounds x to an integer held in the low mantissa bits
    assert clamp == np.float32(-125.0)                    # the spliced exponent stays that of a normal float


def test_relative_error_over_the_range_the_softmax_uses():
    coef, clamp, magic = _routine()
    x = np.concatenate([np.linspace(-125.0, 8.0, 400001), np.arange(-125, 9) + 0.5, np.arange(-125, 9) - 0.4999]).astype(np.float32)
    x = x[x >= -125.0]
    got = _fma_exp2(x, coef, clamp, magic).astype(np.float64)
    want = np.exp2(x.astype(np.float64))
    rel = np.abs(got / want - 1.0)
    assert rel.max() < 1e-4, rel.max()                    # bf16 rounding of the weights is 3.9e-3
    assert np.all(got > 0) and np.all(np.isfinite(got))


def test_masked_scores_give_a_vanishing_weight():
    coef, clamp, magic = _routine()
    x = np.array([-np.inf, -1e30, -126.0, -125.0], np.float32)
    got = _fma_exp2(x, coef, clamp, magic).astype(np.float64)
    assert np.all(np.isfinite(got)) and np.all(got > 0) and np.all(got < 2.0 ** -124)
