"""The seeded input generator: shapes, determinism and structure of the five workloads."""
import torch

from paper_2407_07304_b200 import workloads


def test_shapes_small():
    for idx in range(1, 6):
        w = workloads.make_workload(idx, shrink=16)
        assert len(w.k) == w.B and len(w.v) == w.B
        for b in range(w.B):
            assert w.k[b].shape == (w.total_len(b), w.Hkv, 128) and w.k[b].dtype == torch.bfloat16
            assert w.v[b].shape == w.k[b].shape
        if w.q_prefill is not None:
            assert [t.shape[0] for t in w.q_prefill] == w.prefill_len
        if w.decode_steps:
            assert w.q_decode.shape == (w.decode_steps, w.B, w.Hq, 128)
        assert w.Hq % w.Hkv == 0


def test_deterministic():
    a = workloads.make_workload(4, shrink=32)
    b = workloads.make_workload(4, shrink=32)
    assert a.bulk_len == b.bulk_len
    assert all(torch.equal(x, y) for x, y in zip(a.k, b.k))
    assert torch.equal(a.q_decode, b.q_decode)


def test_structure():
    w1 = workloads.make_workload(1)
    assert (w1.B, w1.Hq, w1.Hkv, w1.prefill_len, w1.decode_steps) == (1, 32, 32, [256], 16)
    w4 = workloads.make_workload(4, shrink=8)
    assert min(w4.bulk_len) >= 128 and max(w4.bulk_len) <= 512 and len(set(w4.bulk_len)) > 8
    # outlier channels: 4 per kv head carry ~8x the spread of the others
    w2 = workloads.make_workload(2, shrink=8)
    std = torch.cat([k.float() for k in w2.k]).std(dim=0)      # [Hkv, 128]
    assert torch.all((std > 4).sum(dim=1) == 4)
    w5 = workloads.make_workload(5, shrink=64)
    assert w5.total_len(0) == 2 * 256 and w5.decode_steps == 64


def test_batched_prefill_workload_is_seeded_and_ragged():
    a, b = workloads.make_batched_prefill(shrink=16), workloads.make_batched_prefill(shrink=16)
    assert a.prefill_len == b.prefill_len and a.B == 16 and a.Hq == a.Hkv == 32
    assert all(16 <= n <= 256 for n in a.prefill_len) and len(set(a.prefill_len)) > 8
    assert all(torch.equal(x, y) for x, y in zip(a.k + a.v + a.q_prefill, b.k + b.v + b.q_prefill))
    assert [t.shape[0] for t in a.q_prefill] == a.prefill_len
