"""Pins for the oracle's quantiser (Section 2.2: INT8 KV cache, one scale per token per head)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2407_07304_b200 import workloads
from helpers import bf16_bits, bits_to_f64, exact_codes, mantissa_sweep_bits


def _rows(seed, n, **kw):
    x = workloads.random_rows(seed, n, **kw)
    return bf16_bits(x)


def test_exact_rational_brute_force():
    # ~10^4 values, with and without outlier channels, against exact Fraction arithmetic
    for seed, outlier in ((0, False), (1, True)):
        bits = _rows(seed, 40, outlier=outlier)
        codes, scales = so.quantize(bits)
        vals = bits_to_f64(bits)
        for r in range(bits.shape[0]):
            want, scale_fr = exact_codes(vals[r])
            assert codes[r].tolist() == want
            # fp32 nearest to the exact amax/127
            s = float(scales[r])
            lo, hi = np.nextafter(np.float32(s), np.float32(-np.inf)), np.nextafter(np.float32(s), np.float32(np.inf))
            err = abs(Fraction(s) - scale_fr)
            assert err <= abs(Fraction(float(lo)) - scale_fr) and err <= abs(Fraction(float(hi)) - scale_fr)


def test_significand_sweep_and_extreme_magnitudes_against_exact_rationals():
    # every significand of the largest element, element exponents 0..9 below it, magnitudes from subnormal
    # to 2^120: a sample of the rows against exact Fraction arithmetic, every scale against IEEE fp32 division
    bits = mantissa_sweep_bits([-126, -120, -61, -60, 0, 60, 61, 120])
    codes, scales = so.quantize(bits)
    vals = bits_to_f64(bits)
    picked = list(range(0, bits.shape[0], 37)) + list(range(bits.shape[0] - 5, bits.shape[0]))
    for r in picked:
        want, _ = exact_codes(vals[r])
        assert codes[r].tolist() == want, f"row {r}"
    amax = np.abs(vals).max(axis=1).astype(np.float32)
    with np.errstate(under="ignore"):
        want_scale = amax / np.float32(127.0)
    assert np.array_equal(scales.view(np.uint32), want_scale.view(np.uint32))


def test_scale_bits_match_fp32_division():
    bits = _rows(2, 4096, outlier=True)
    _, scales = so.quantize(bits)
    amax = np.abs(bits_to_f64(bits)).max(axis=1).astype(np.float32)
    want = amax / np.float32(127.0)          # IEEE fp32 division, correctly rounded
    assert np.array_equal(scales.view(np.uint32), want.view(np.uint32))


def test_fp32_evaluation_of_exact_ratio_agrees():
    # the GPU evaluates rint(fl32(127*x) / amax) in fp32; it must give the same codes
    bits = _rows(3, 20000, outlier=True)
    codes, _ = so.quantize(bits)
    x = bits_to_f64(bits).astype(np.float32)
    amax = np.abs(x).max(axis=1, keepdims=True)
    q32 = np.rint((np.float32(127.0) * x) / amax)
    assert np.array_equal(q32.astype(np.int8), codes)


def test_invariants():
    bits = _rows(4, 2000, outlier=True)
    codes, scales = so.quantize(bits)
    x = bits_to_f64(bits)
    c = codes.astype(np.int64)
    assert c.min() >= -127 and c.max() <= 127
    # the absmax element gets +-127
    idx = np.abs(x).argmax(axis=1)
    assert np.all(np.abs(c[np.arange(len(c)), idx]) == 127)
    # sign(code) == sign(x) or code == 0
    assert np.all((np.sign(c) == np.sign(x)) | (c == 0))
    # monotone in x within a row
    order = np.argsort(x, axis=1, kind="stable")
    cs = np.take_along_axis(c, order, axis=1)
    assert np.all(np.diff(cs, axis=1) >= 0)
    # dequantisation error <= scale/2 up to the rounding of the stored scale
    s = scales.astype(np.float64)[:, None]
    assert np.all(np.abs(x - c * s) <= 0.5 * s * (1 + 2.0 ** -16))


def test_zero_row_and_shapes():
    bits = _rows(5, 8, zero_rows=3)
    codes, scales = so.quantize(bits)
    assert np.all(codes[:3] == 0) and np.all(scales[:3] == 0.0)
    assert np.all(scales[3:] > 0)
    # leading dims are preserved
    c2, s2 = so.quantize(bits.reshape(2, 4, 128))
    assert c2.shape == (2, 4, 128) and s2.shape == (2, 4)
    assert np.array_equal(c2.reshape(8, 128), codes)


def test_power_of_two_scale_closed_form():
    # amax = 127 * 2^e  ->  scale = 2^e exactly and code = x / 2^e exactly when integral
    for e in (-9, -3, 0, 4):
        row = torch.zeros(128)
        row[0] = 127.0 * 2.0 ** e
        ints = torch.arange(-63, 64).float()          # 127 integers
        row[1:128] = ints * 2.0 ** e
        bits = bf16_bits(row.to(torch.bfloat16).view(1, 128))
        codes, scales = so.quantize(bits)
        assert float(scales[0]) == 2.0 ** e
        assert codes[0, 0] == 127
        assert codes[0, 1:].tolist() == list(range(-63, 64))


def test_ties_round_to_even():
    # amax = 127/64 -> quotient = 64*x; x = k/128 + ... gives exact .5 ties
    row = torch.zeros(128)
    row[0] = 127.0 / 64
    ties = [16.5, 17.5, -16.5, -17.5, 0.5, -0.5, 1.5, 63.5, -63.5, 62.5]
    for i, t in enumerate(ties):
        row[1 + i] = t / 64
    bits = bf16_bits(row.to(torch.bfloat16).view(1, 128))
    assert np.array_equal(bits_to_f64(bits)[0, 1:11] * 64, np.array(ties))   # exact in bf16
    codes, _ = so.quantize(bits)
    assert codes[0, 1:11].tolist() == [16, 18, -16, -18, 0, 0, 2, 64, -64, 62]


def test_eq1_kv_bytes():
    # Eq. (1) with the Section 2.2 example: Llama2-7B, b=256, 1024+1024 tokens
    assert so.kv_bytes(256, 1024, 1024, 32, 32, 128, 2) == 2 * 256 * 2048 * 32 * 32 * 128 * 2
    assert so.kv_bytes(256, 1024, 1024, 32, 32, 128, 1) == 128 * 2 ** 30   # the "128 GB" of the text
    # one layer, INT8: codes bytes of a decode step of workload 2
    assert so.kv_bytes(16, 2048, 1, 1, 32, 128, 1) == 2 * 16 * 2049 * 32 * 128
