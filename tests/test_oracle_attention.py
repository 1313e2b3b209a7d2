"""Pins for the oracle's attention (Section 2.1 SlimAttention = exact softmax attention,
row by row) and for the split/merge identity used by the decode path."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from helpers import bf16_bits, bits_to_f64, dense_attention, frac_to_bf16

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_example.txt")


def _rand_case(seed, nq, L, Hq, Hkv, D):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((nq, Hq, D), generator=g).to(torch.bfloat16)
    k = torch.randn((L, Hkv, D), generator=g).to(torch.bfloat16)
    v = torch.randn((L, Hkv, D), generator=g).to(torch.bfloat16)
    kc, ks = so.quantize(bf16_bits(k))
    vc, vs = so.quantize(bf16_bits(v))
    return bf16_bits(q), kc, ks, vc, vs


def _dequant(c, s):
    return c.astype(np.float64) * s.astype(np.float64)[..., None]


@pytest.mark.parametrize("nq,L,Hq,Hkv,D", [
    (8, 8, 1, 1, 4), (5, 8, 2, 1, 4), (1, 7, 4, 2, 128), (8, 8, 16, 1, 128), (3, 6, 2, 2, 128),
])
def test_matches_dense_numpy(nq, L, Hq, Hkv, D):
    q, kc, ks, vc, vs = _rand_case(nq * 100 + L + Hq, nq, L, Hq, Hkv, D)
    got = so.attention(q, kc, ks, vc, vs, L, D ** -0.5)
    want = dense_attention(bits_to_f64(q), _dequant(kc, ks), _dequant(vc, vs), L, D ** -0.5)
    assert np.max(np.abs(got - want)) < 1e-13


def test_kv_len_shorter_than_buffer_and_selection():
    q, kc, ks, vc, vs = _rand_case(7, 6, 12, 2, 1, 128)
    full = so.attention(q, kc, ks, vc, vs, 9, 0.1)
    want = dense_attention(bits_to_f64(q), _dequant(kc, ks), _dequant(vc, vs), 9, 0.1)
    assert np.max(np.abs(full - want)) < 1e-13
    sel = so.attention(q, kc, ks, vc, vs, 9, 0.1, sel=[4, 0, 5])
    assert np.array_equal(sel, full[[4, 0, 5]])


def test_rows_sum_to_one():
    # v^ == 1 in every channel -> output is sum_j p_j == 1
    q, kc, ks, _, _ = _rand_case(11, 6, 6, 2, 2, 128)
    vc = np.full_like(kc, 64)
    vs = np.full(ks.shape, 2.0 ** -6, dtype=np.float32)
    out = so.attention(q, kc, ks, vc, vs, 6, 128 ** -0.5)
    assert np.max(np.abs(out - 1.0)) < 1e-14


def test_first_causal_row_is_v0_and_causality():
    q, kc, ks, vc, vs = _rand_case(13, 8, 8, 2, 1, 128)
    out = so.attention(q, kc, ks, vc, vs, 8, 128 ** -0.5)
    v0 = _dequant(vc, vs)[0, 0]
    assert np.array_equal(out[0, 0], v0) and np.array_equal(out[0, 1], v0)
    # changing keys/values after position i leaves rows <= i bit-identical
    kc2, vc2, ks2, vs2 = kc.copy(), vc.copy(), ks.copy(), vs.copy()
    kc2[5:] = -kc2[5:]
    vc2[5:] = 7
    ks2[5:] *= 3
    vs2[5:] *= 0.5
    out2 = so.attention(q, kc2, ks2, vc2, vs2, 8, 128 ** -0.5)
    assert np.array_equal(out2[:5], out[:5])
    assert not np.array_equal(out2[5:], out[5:])


def test_equal_keys_give_mean_of_values_and_dominant_key():
    q, kc, ks, vc, vs = _rand_case(17, 1, 9, 2, 1, 128)
    kc[:] = kc[0]
    ks[:] = ks[0]
    out = so.attention(q, kc, ks, vc, vs, 9, 128 ** -0.5)
    mean_v = _dequant(vc, vs)[:, 0].mean(axis=0)
    assert np.max(np.abs(out[0, 0] - mean_v)) < 1e-14
    # one key aligned with q and scaled up dominates the softmax
    qv = bits_to_f64(q)[0, 0]
    big = np.clip(np.rint(qv / np.abs(qv).max() * 127), -127, 127).astype(np.int8)
    kc[:] = 0
    kc[4, 0] = big
    ks[:] = 1.0
    out = so.attention(q, kc, ks, vc, vs, 9, 1.0)
    assert np.max(np.abs(out[0, 0] - _dequant(vc, vs)[4, 0])) < 1e-12


def test_gqa_mapping():
    # consecutive q heads share a kv head: q head h reads kv head h // G
    nq, L, Hq, Hkv, D = 4, 6, 8, 2, 128
    q, kc, ks, vc, vs = _rand_case(19, nq, L, Hq, Hkv, D)
    q[:, 1] = q[:, 0]            # same group (G = 4): heads 0..3 -> kv 0
    q[:, 4] = q[:, 0]            # other group: head 4 -> kv 1
    out = so.attention(q, kc, ks, vc, vs, L, D ** -0.5)
    assert np.array_equal(out[:, 1], out[:, 0])
    assert not np.array_equal(out[:, 4], out[:, 0])
    # expanding K/V to one kv head per q head gives the same result
    rep = lambda a: np.repeat(a, Hq // Hkv, axis=1)
    out_mha = so.attention(q, rep(kc), rep(ks), rep(vc), rep(vs), L, D ** -0.5)
    assert np.array_equal(out_mha, out)


def test_decode_equals_last_prefill_row():
    q, kc, ks, vc, vs = _rand_case(23, 10, 10, 2, 1, 128)
    pre = so.attention(q, kc, ks, vc, vs, 10, 128 ** -0.5)
    dec = so.attention(q[9:10], kc, ks, vc, vs, 10, 128 ** -0.5)
    assert np.array_equal(dec[0], pre[9])
    # chunked prefill: the last 3 queries against 10 keys equal rows 7..9
    tail = so.attention(q[7:], kc, ks, vc, vs, 10, 128 ** -0.5)
    assert np.array_equal(tail, pre[7:])


@pytest.mark.parametrize("cuts", [[0, 37], [0, 1, 37], [0, 16, 32, 37], [0, 5, 6, 20, 36, 37]])
def test_split_merge_identity(cuts):
    q, kc, ks, vc, vs = _rand_case(29, 1, 37, 2, 2, 128)
    whole = so.attention(q, kc, ks, vc, vs, 37, 128 ** -0.5)
    for h in range(2):
        parts = [so.partial(q[0, h], kc, ks, vc, vs, a, b, h, 128 ** -0.5)
                 for a, b in zip(cuts[:-1], cuts[1:])]
        o = so.merge([p[0] for p in parts], [p[1] for p in parts], np.stack([p[2] for p in parts]))
        assert np.max(np.abs(o - whole[0, h])) < 1e-12


def test_partial_definition():
    # a partial over all keys, normalised, is the row itself; its m is the max score
    q, kc, ks, vc, vs = _rand_case(31, 1, 12, 1, 1, 128)
    m, l, O = so.partial(q[0, 0], kc, ks, vc, vs, 0, 12, 0, 0.05)
    whole = so.attention(q, kc, ks, vc, vs, 12, 0.05)
    assert np.max(np.abs(O / l - whole[0, 0])) < 1e-13
    s = 0.05 * (_dequant(kc, ks)[:, 0] @ bits_to_f64(q)[0, 0])
    assert abs(m - s.max()) < 1e-13 and abs(l - np.exp(s - s.max()).sum()) < 1e-12


# ---------------------------------------------------------------- hand-worked example

def _parse_golden():
    def num(tok):
        if tok.startswith("2^"):
            return 2.0 ** int(tok[2:])
        if tok.startswith("0x"):
            return float.fromhex(tok)
        return Fraction(tok)
    rows = {"k": {}, "v": {}, "q": {}, "o": {}}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            t = line.split()
            kind, tok = t[0], int(t[1])
            if kind in ("k", "v"):
                rows[kind][tok] = ([Fraction(x) for x in t[2:6]], [int(x) for x in t[6:10]], num(t[10]))
            elif kind == "q":
                rows[kind][tok] = [Fraction(x) for x in t[2:6]]
            else:
                rows[kind][tok] = [float(x) for x in t[2:6]]
    return rows


def _row128(fracs):
    r = torch.zeros(128, dtype=torch.bfloat16)
    for i, fr in enumerate(fracs):
        r[i] = frac_to_bf16(fr)
    return r


def test_hand_example():
    g = _parse_golden()
    K = torch.stack([_row128(g["k"][t][0]) for t in range(3)]).view(3, 1, 128)
    V = torch.stack([_row128(g["v"][t][0]) for t in range(3)]).view(3, 1, 128)
    Q = torch.stack([_row128(g["q"][t]) for t in range(3)]).view(3, 1, 128)
    kc, ks = so.quantize(bf16_bits(K))
    vc, vs = so.quantize(bf16_bits(V))
    for t in range(3):
        assert kc[t, 0, :4].tolist() == g["k"][t][1] and not kc[t, 0, 4:].any()
        assert vc[t, 0, :4].tolist() == g["v"][t][1] and not vc[t, 0, 4:].any()
        assert float(ks[t, 0]) == g["k"][t][2]
        assert float(vs[t, 0]) == g["v"][t][2]
    c = 128 ** -0.5
    pre = so.attention(bf16_bits(Q[:2]), kc, ks, vc, vs, 2, c)
    dec = so.attention(bf16_bits(Q[2:3]), kc, ks, vc, vs, 3, c)
    got = [pre[0, 0, :4], pre[1, 0, :4], dec[0, 0, :4]]
    for t in range(3):
        assert np.max(np.abs(got[t] - np.array(g["o"][t]))) < 5e-15
    assert not pre[:, :, 4:].any() and not dec[:, :, 4:].any()

    # the stored numbers themselves, re-derived by closed forms that do not use the oracle:
    # row 1 has two keys, so softmax = logistic of the score difference 0.484375/sqrt(128)
    p1 = 1.0 / (1.0 + math.exp(-0.484375 / math.sqrt(128.0)))
    v0 = np.array([0.9921875, -0.5, 0, 0])
    v1 = np.array([-1.984375, 1, 0.25, 0])
    assert np.max(np.abs((1 - p1) * v0 + p1 * v1 - np.array(g["o"][1]))) < 5e-15
    # row 2: scores (0.9921875, -3.34375, 1.6171875)/sqrt(128) from the dequantised keys
    s = np.array([0.5 * 1.984375 - 0.5 + 2 * 0.25,
                  -0.5 - 3.96875 + 2 * 0.5625,
                  0.375 + 0.25 + 0.9921875]) / math.sqrt(128.0)
    e = np.exp(s - s.max())
    p = e / e.sum()
    sv2 = float.fromhex("0x1.020408p-8")
    v2 = np.array([127 * sv2, 126 * sv2, 0, -64 * sv2])
    assert np.max(np.abs(p[0] * v0 + p[1] * v1 + p[2] * v2 - np.array(g["o"][2]))) < 5e-15
