"""The plan that spreads one layer's decode attention over several GPUs (kv heads, and where there are fewer kv heads
than ranks the key range), checked on the CPU: every (sequence, kv head, token) has exactly one owner; the oracle
evaluated shard by shard and put together - concatenated over heads, merged by the log-sum-exp identity over key
ranges - equals the oracle on the whole problem; and two gloo ranks exchange their row partials the way the GPU path
does."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import slim_oracle as so
from paper_2407_07304_b200.shard import CHUNK_TOKENS, ShardPlan, exchange_partials
from helpers import bf16_bits

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("Hq,Hkv,world,lens", [
    (32, 32, 8, [2049] * 16),                 # Llama-2-7B shape: four kv heads per rank
    (64, 8, 8, [1024, 4096, 1777, 2500]),     # one kv head (eight query heads) per rank
    (64, 8, 4, [300, 1]),
    (64, 8, 3, [300, 1]),                     # uneven: 2 + 3 + 3 heads
    (32, 2, 8, [32768]),                      # fewer kv heads than ranks: four ranks per head divide the keys
    (32, 2, 4, [700, 255, 256, 257, 0]),
    (16, 1, 4, [5]),                          # shorter than a chunk: one rank holds all of it
    (4, 4, 1, [100, 200]),
])
def test_every_cached_token_has_exactly_one_owner(Hq, Hkv, world, lens):
    plan = ShardPlan(Hq, Hkv, lens, world)
    owners = [np.zeros((n, Hkv), dtype=np.int32) for n in lens]
    q_owner = np.zeros(Hq, dtype=np.int32)
    for s in plan.shards():
        assert list(s.q_heads) == [h * plan.G + i for h in s.kv_heads for i in range(plan.G)]
        assert s.group[s.part] == s.rank and len(s.group) == s.parts
        if s.part == 0:
            q_owner[list(s.q_heads)] += 1
        for b, (t0, t1) in enumerate(s.key_ranges):
            assert 0 <= t0 <= t1 <= lens[b]
            assert t0 % CHUNK_TOKENS == 0 or t0 == lens[b]      # ranges start on chunk boundaries
            owners[b][t0:t1, list(s.kv_heads)] += 1
    assert (q_owner == 1).all()
    for o in owners:
        assert (o == 1).all()
    # the bytes read per step add up to the unsharded problem's
    assert sum(plan.cache_bytes(r) for r in range(world)) == sum(lens) * Hkv * 264


def test_invalid_plans_are_rejected():
    with pytest.raises(ValueError):
        ShardPlan(32, 2, [100], 3)            # 3 ranks cannot divide 2 heads' keys evenly
    with pytest.raises(ValueError):
        ShardPlan(30, 4, [100], 2)


def _problem(Hq, Hkv, lens, seed):
    g = torch.Generator().manual_seed(seed)
    ks = [torch.randn((n, Hkv, 128), generator=g).to(torch.bfloat16) for n in lens]
    vs = [torch.randn((n, Hkv, 128), generator=g).to(torch.bfloat16) for n in lens]
    q = torch.randn((len(lens), Hq, 128), generator=g).to(torch.bfloat16)
    cache = []
    for k, v in zip(ks, vs):
        kc, ksc = so.quantize(bf16_bits(k))
        vc, vsc = so.quantize(bf16_bits(v))
        cache.append((kc, ksc, vc, vsc))
    return q, cache


def _unsharded(q, cache, lens, sm_scale):
    return np.concatenate([so.attention(bf16_bits(q[b:b + 1]), *cache[b], lens[b], sm_scale) for b in range(len(lens))])


def test_head_shards_concatenate_to_the_unsharded_oracle():
    Hq, Hkv, lens, sm = 16, 4, [300, 77], 128 ** -0.5
    q, cache = _problem(Hq, Hkv, lens, 1)
    want = _unsharded(q, cache, lens, sm)
    plan = ShardPlan(Hq, Hkv, lens, 4)
    got = np.zeros_like(want)
    for s in plan.shards():
        hk, hq = list(s.kv_heads), list(s.q_heads)
        for b in range(len(lens)):
            kc, ksc, vc, vsc = cache[b]
            got[b, hq] = so.attention(bf16_bits(q[b:b + 1, hq]), kc[:, hk], ksc[:, hk], vc[:, hk], vsc[:, hk], lens[b], sm)[0]
    assert np.array_equal(got, want)          # heads are independent: the same arithmetic, bit for bit


def _shard_partials(q, cache, lens, shard, G, sm):
    """Oracle partials (m, l, O) of a shard's key ranges: float64 [B, Hq_local, 132] in the layout of the GPU path
    (O[128], m, l, padding); a row without keys has m = -inf, l = 0."""
    B = len(lens)
    out = np.zeros((B, len(shard.q_heads), 132))
    out[:, :, 128] = -np.inf
    for b, (t0, t1) in enumerate(shard.key_ranges):
        if t1 <= t0:
            continue
        kc, ksc, vc, vsc = cache[b]
        for i, h in enumerate(shard.q_heads):
            m, l, O = so.partial(bf16_bits(q[b, h]), kc, ksc, vc, vsc, t0, t1, h // G, sm)
            out[b, i, :128], out[b, i, 128], out[b, i, 129] = O, m, l
    return out


def _merge_sets(sets):
    parts, B, H, _ = sets.shape
    out = np.zeros((B, H, 128))
    for b in range(B):
        for h in range(H):
            live = [r for r in range(parts) if sets[r, b, h, 128] != -np.inf]
            if live:
                out[b, h] = so.merge(sets[live, b, h, 128], sets[live, b, h, 129], sets[live, b, h, :128])
    return out


def test_key_range_shards_merge_to_the_unsharded_oracle():
    Hq, Hkv, lens, sm = 8, 2, [1300, 255, 513, 3], 128 ** -0.5
    q, cache = _problem(Hq, Hkv, lens, 2)
    want = _unsharded(q, cache, lens, sm)
    plan = ShardPlan(Hq, Hkv, lens, 8)        # four ranks per kv head
    got = np.zeros_like(want)
    for head in range(Hkv):
        group = [s for s in plan.shards() if list(s.kv_heads) == [head]]
        sets = np.stack([_shard_partials(q, cache, lens, s, plan.G, sm) for s in sorted(group, key=lambda s: s.part)])
        got[:, list(group[0].q_heads)] = _merge_sets(sets)
    assert np.abs(got - want).max() < 1e-12


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    Hq, Hkv, lens, sm = 4, 1, [700, 300, 1], 128 ** -0.5
    q, cache = _problem(Hq, Hkv, lens, 3)     # the same seeded problem on every rank
    plan = ShardPlan(Hq, Hkv, lens, world)    # one kv head, two ranks: each holds half of every sequence's chunks
    shard = plan.shard(rank)
    mine = torch.from_numpy(_shard_partials(q, cache, lens, shard, plan.G, sm))
    sets = exchange_partials(mine, shard)     # all-gather over gloo, as the GPU path does over NCCL
    got = _merge_sets(sets.numpy())
    want = _unsharded(q, cache, lens, sm)
    out[rank] = (float(np.abs(got - want).max()), [list(r) for r in shard.key_ranges], tuple(sets.shape))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_divide_the_keys_and_merge():
    world = 2
    port = 31500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    assert res[0][1] == [[0, 256], [0, 256], [0, 0]] and res[1][1] == [[256, 700], [256, 300], [0, 1]]
    for rank in range(world):
        err, _, shape = res[rank]
        assert shape == (2, 3, 4, 132)
        assert err < 1e-12                    # every rank ends with the unsharded result
