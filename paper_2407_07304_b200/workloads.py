"""Seeded synthetic inputs for the five attention workloads.

This module only draws random tensors and lengths; it contains none of the
method's arithmetic (no quantiser, no attention) so that the CPU oracle and
the CUDA path can both be fed from it without sharing anything else.

The tensors stand in for the Llama-2-7B-shaped (32 heads x 128) and the
70B-class grouped-query attention layers the paper measures (Tables 2-4):
trained weights and prompts are not available, so Q/K/V are bf16 N(0, 1),
optionally with a few outlier channels per head scaled by 8 before the
rounding to bf16.

Every tensor is created on the CPU by one torch.Generator seeded with
SEED0 + workload index, in a fixed order, so the values do not depend on the
device or on which consumer asks for them.
"""
from dataclasses import dataclass, field
from typing import List, Optional

import torch

SEED0 = 240707304
HEAD_DIM = 128
PAGE_TOKENS = 128


@dataclass
class Workload:
    """One attention-layer workload.

    k, v        per sequence: bf16 [total_len_b, Hkv, 128], every K/V row the
                run ever appends, in position order
    q_prefill   per sequence: bf16 [prefill_len_b, Hq, 128] or None
    q_decode    bf16 [decode_steps, B, Hq, 128] or None
    prefill_len tokens appended and attended causally in the first phase
    bulk_len    tokens appended after the prefill with no attention
    decode_steps single-token append+decode steps after that
    """
    name: str
    index: int
    B: int
    Hq: int
    Hkv: int
    prefill_len: List[int]
    bulk_len: List[int]
    decode_steps: int
    k: List[torch.Tensor] = field(repr=False, default_factory=list)
    v: List[torch.Tensor] = field(repr=False, default_factory=list)
    q_prefill: Optional[List[torch.Tensor]] = field(repr=False, default=None)
    q_decode: Optional[torch.Tensor] = field(repr=False, default=None)
    sm_scale: float = HEAD_DIM ** -0.5

    @property
    def D(self):
        return HEAD_DIM

    def total_len(self, b):
        return self.prefill_len[b] + self.bulk_len[b] + self.decode_steps

    def pages_per_seq(self):
        return max((self.total_len(b) + PAGE_TOKENS - 1) // PAGE_TOKENS for b in range(self.B))


def _randn_bf16(gen, shape, outlier_channels=None):
    x = torch.randn(shape, generator=gen, dtype=torch.float32)
    if outlier_channels is not None:
        # outlier_channels: [Hkv, n_out] channel ids; x: [T, Hkv, D]
        for h in range(outlier_channels.shape[0]):
            x[:, h, outlier_channels[h]] *= 8.0
    return x.to(torch.bfloat16)


def _outliers(gen, Hkv, n_out=4):
    return torch.stack([torch.randperm(HEAD_DIM, generator=gen)[:n_out] for _ in range(Hkv)])


def make_workload(index, shrink=1):
    """Workload `index` (1..5).  shrink > 1 divides every token count by that
    factor (lengths stay >= 1) to give small cases with the same structure."""
    if index not in (1, 2, 3, 4, 5):
        raise ValueError("workload index must be 1..5")
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED0 + index)

    def sh(n):
        return max(1, n // shrink)

    if index == 1:
        w = Workload("c1_prefill256_decode16", 1, 1, 32, 32, [sh(256)], [0], 16)
        outl = False
    elif index == 2:
        w = Workload("c2_llama7b_decode_b16_ctx2048", 2, 16, 32, 32, [0] * 16, [sh(2048)] * 16, 1)
        outl = True
    elif index == 3:
        w = Workload("c3_prefill8192", 3, 1, 32, 32, [sh(8192)], [0], 0)
        outl = False
    elif index == 4:
        lo, hi = sh(1024), sh(4096)
        lens = torch.randint(lo, hi + 1, (32,), generator=gen).tolist()
        w = Workload("c4_gqa_decode_b32_ctx1024_4096", 4, 32, 64, 8, [0] * 32, lens, 1)
        outl = True
    else:
        w = Workload("c5_mqa_prefill16384_decode_to_32768", 5, 1, 32, 2,
                     [sh(16384)], [sh(16384) - 64 if sh(16384) > 64 else 0], 64)
        outl = False

    k_out = _outliers(gen, w.Hkv) if outl else None
    v_out = _outliers(gen, w.Hkv) if outl else None
    for b in range(w.B):
        T = w.total_len(b)
        w.k.append(_randn_bf16(gen, (T, w.Hkv, HEAD_DIM), k_out))
        w.v.append(_randn_bf16(gen, (T, w.Hkv, HEAD_DIM), v_out))
    if any(n > 0 for n in w.prefill_len):
        w.q_prefill = [_randn_bf16(gen, (n, w.Hq, HEAD_DIM)) for n in w.prefill_len]
    if w.decode_steps > 0:
        w.q_decode = _randn_bf16(gen, (w.decode_steps, w.B, w.Hq, HEAD_DIM))
    return w


def make_batched_prefill(shrink=1, B=16):
    """Batched variable-length prefill in the Llama-2-7B shape (32 q = 32 kv heads): B prompts of
    U{256..4096} tokens (integer, drawn from the seed), all attended causally in one call.  A serving-style
    case beside the five configured workloads; shrink divides the token counts."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED0 + 6)
    lo, hi = max(1, 256 // shrink), max(1, 4096 // shrink)
    lens = torch.randint(lo, hi + 1, (B,), generator=gen).tolist()
    w = Workload("batched_prefill_b16_len256_4096", 6, B, 32, 32, lens, [0] * B, 0)
    for b in range(B):
        w.k.append(_randn_bf16(gen, (lens[b], w.Hkv, HEAD_DIM)))
        w.v.append(_randn_bf16(gen, (lens[b], w.Hkv, HEAD_DIM)))
    w.q_prefill = [_randn_bf16(gen, (n, w.Hq, HEAD_DIM)) for n in lens]
    return w


def random_rows(seed, n_rows, outlier=False, zero_rows=0):
    """bf16 [n_rows, 128] rows for quantiser tests; the first zero_rows are all zero."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(SEED0 + 1000 + seed)
    x = torch.randn((n_rows, HEAD_DIM), generator=gen, dtype=torch.float32)
    if outlier:
        x[:, torch.randperm(HEAD_DIM, generator=gen)[:4]] *= 8.0
    x[:zero_rows] = 0.0
    return x.to(torch.bfloat16)
