"""Test-side helpers: dtype plumbing and independent reference arithmetic."""
import math
from fractions import Fraction

import numpy as np
import torch


def bf16_bits(t):
    """torch bf16 tensor -> numpy uint16 bit patterns (same shape)."""
    assert t.dtype == torch.bfloat16
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits):
    """numpy uint16 bf16 bit patterns -> float64 values."""
    w = bits.astype(np.uint32) << 16
    return w.view(np.float32).astype(np.float64)


def frac_to_bf16(fr):
    """Exact Fraction -> torch bf16 scalar; asserts it is representable."""
    x = torch.tensor(float(fr), dtype=torch.float32).to(torch.bfloat16)
    assert Fraction(float(x)) == Fraction(fr), f"{fr} is not exact in bf16"
    return x


def round_half_even(fr):
    """Exact round-half-to-even of a Fraction."""
    fl = math.floor(fr)
    rem = fr - fl
    if rem > Fraction(1, 2):
        return fl + 1
    if rem < Fraction(1, 2):
        return fl
    return fl if fl % 2 == 0 else fl + 1


def exact_codes(row_f64):
    """Exact rational quantiser of one row given as float64 values."""
    fr = [Fraction(float(x)) for x in row_f64]
    amax = max(abs(x) for x in fr)
    if amax == 0:
        return [0] * len(fr), Fraction(0)
    codes = [max(-127, min(127, round_half_even(127 * x / amax))) for x in fr]
    return codes, amax / 127


def dense_attention(q, k_hat, v_hat, kv_len, sm_scale):
    """Dense numpy fp64 softmax attention for one sequence.

    q [nq, Hq, D], k_hat/v_hat [L, Hkv, D] float64 (already dequantised).
    Builds the full masked score matrix per head and uses matrix products.
    """
    nq, Hq, D = q.shape
    Hkv = k_hat.shape[1]
    G = Hq // Hkv
    out = np.zeros((nq, Hq, D))
    jj = np.arange(kv_len)[None, :]
    tt = np.arange(nq)[:, None]
    visible = jj <= (kv_len - nq + tt)
    for h in range(Hq):
        g = h // G
        S = sm_scale * (q[:, h, :] @ k_hat[:kv_len, g, :].T)
        S = np.where(visible, S, -np.inf)
        S = S - S.max(axis=1, keepdims=True)
        P = np.exp(S)
        P = P / P.sum(axis=1, keepdims=True)
        out[:, h, :] = P @ v_hat[:kv_len, g, :]
    return out


def mantissa_sweep_bits(exponents, offsets=range(0, 10), subnormal_amax=(1, 2, 3, 64, 127)):
    """Rows of 128 bf16 bit patterns that sweep significands and magnitudes (inputs only, no quantiser arithmetic).

    For every unbiased exponent e in `exponents`, every one of the 128 bf16 significands of the row's
    largest element and every k in `offsets`: one row whose largest element is +-(1.m) * 2^e at position
    m, the other positions holding all 128 significands at exponent e - k (those that would exceed the
    largest element are set to zero), signs alternating.  Then, for the subnormal patterns given, rows
    whose largest element is that subnormal and whose other elements are the smaller subnormals."""
    rows = []
    mant = np.arange(128, dtype=np.uint32)
    sign = ((mant & 1) << 15).astype(np.uint32)
    for e in exponents:
        for m in range(128):
            for k in offsets:
                ex = e - k
                if ex < -126:
                    continue
                row = (np.uint32(ex + 127) << 7) | mant | sign
                if k == 0:
                    row = np.where(mant > m, 0, row)
                row[m] = (np.uint32(e + 127) << 7) | np.uint32(m) | (np.uint32((m >> 1) & 1) << 15)
                rows.append(row.astype(np.uint16))
    for m in subnormal_amax:
        row = np.where(mant <= m, mant, mant % (m + 1)).astype(np.uint32) | sign
        rows.append(row.astype(np.uint16))
    return np.stack(rows)


MAX_ABS = 2e-2     # output tolerance against the fp64 oracle: max-abs ...
MEAN_ABS = 2e-3    # ... and mean-abs


def output_bound(want_f64):
    """Per-element bound on |bf16 output - fp64 oracle value|.

    The flat 2e-2 wherever a bf16 output can meet it: below magnitude 8 the bf16 half-ulp is at most 2^-6 =
    1.56e-2.  From magnitude 8 on the half-ulp is 2^-5 or more, so the correctly rounded oracle value itself may
    miss 2e-2; there the bound is the bf16 half-ulp of the oracle value plus the arithmetic share that the flat
    bound leaves in the binade below, 2e-2 - 2^-6 = 4.4e-3."""
    a = np.abs(want_f64)
    half_ulp = 2.0 ** (np.floor(np.log2(np.maximum(a, 1.0))) - 8)   # bf16 has 8 significant bits
    return np.where(a >= 8.0, half_ulp + (MAX_ABS - 2.0 ** -6), MAX_ABS)
