"""Decode attention of one layer spread over several GPUs, one process per GPU.

Every (sequence, kv head) of the cache is independent (in Eq. 1 the batch and the heads are plain factors), which is
how the paper's distributed runs divide the work (Section 2.3): a device owns a set of kv heads together with the
query heads they serve, holds cache pages for those heads only, and nothing crosses devices inside the attention (the
reduction belongs to the output projection behind it).  Only when there are fewer kv heads than devices is the key
range of a head divided as well: the devices of a head each attend over their part of the keys
(slim_attn_decode_partial), exchange one (O, M, l) row per (sequence, query head) with one all-gather and merge
locally (slim_attn_merge_partials).

This module holds the plan (who owns what; plain integer arithmetic, no attention arithmetic) and the per-rank call
sequence.  The exchange is torch.distributed's (NCCL on GPUs); the kernels only ever read the calling device's memory.
"""
from dataclasses import dataclass
from typing import List, Tuple

CHUNK_TOKENS = 256   # the key range of a head is divided at multiples of this (the decode kernel's chunk)


@dataclass
class Shard:
    """What one rank owns."""
    rank: int
    world: int
    kv_heads: range                      # global kv head ids (contiguous)
    q_heads: range                       # the query heads they serve
    key_ranges: List[Tuple[int, int]]    # per sequence: cached token positions [t0, t1) this rank holds
    part: int                            # index of this rank among the ranks that share its heads
    parts: int                           # how many ranks share its heads (1: nothing to merge)
    group: List[int]                     # those ranks, in part order


class ShardPlan:
    """Assignment of one layer's decode attention to `world` ranks.

    Hkv >= world: rank r owns kv heads [r * Hkv // world, (r + 1) * Hkv // world) and every token of them.
    Hkv <  world: world must be a multiple of Hkv; the world / Hkv ranks of a head divide every sequence's
                  256-token chunks among themselves in contiguous runs (the last run holds the newest tokens).
    """

    def __init__(self, Hq: int, Hkv: int, kv_len: List[int], world: int):
        if Hq % Hkv != 0:
            raise ValueError("Hq must be a multiple of Hkv")
        if world < 1:
            raise ValueError("world must be positive")
        if Hkv < world and world % Hkv != 0:
            raise ValueError("with fewer kv heads than ranks the rank count must be a multiple of the kv heads")
        self.Hq, self.Hkv, self.G, self.world = Hq, Hkv, Hq // Hkv, world
        self.kv_len = [max(0, int(n)) for n in kv_len]
        self.parts = 1 if Hkv >= world else world // Hkv
        self.mode = "heads" if self.parts == 1 else "keys"

    def shard(self, rank: int) -> Shard:
        if not 0 <= rank < self.world:
            raise ValueError("rank out of range")
        if self.parts == 1:
            h0, h1 = rank * self.Hkv // self.world, (rank + 1) * self.Hkv // self.world
            part, group = 0, [rank]
            ranges = [(0, n) for n in self.kv_len]
        else:
            h0 = rank // self.parts
            h1 = h0 + 1
            part = rank % self.parts
            group = [h0 * self.parts + i for i in range(self.parts)]
            ranges = []
            for n in self.kv_len:
                nc = (n + CHUNK_TOKENS - 1) // CHUNK_TOKENS
                c0, c1 = part * nc // self.parts, (part + 1) * nc // self.parts
                ranges.append((min(n, c0 * CHUNK_TOKENS), min(n, c1 * CHUNK_TOKENS)))
        return Shard(rank, self.world, range(h0, h1), range(h0 * self.G, h1 * self.G), ranges, part, self.parts, group)

    def shards(self) -> List[Shard]:
        return [self.shard(r) for r in range(self.world)]

    def cache_bytes(self, rank: int, row_bytes: int = 264) -> int:
        """Cache bytes the rank reads per decode step (264 B per token and kv head: codes + two scales)."""
        s = self.shard(rank)
        return sum(t1 - t0 for t0, t1 in s.key_ranges) * len(s.kv_heads) * row_bytes


def exchange_partials(partial, shard: Shard, group=None):
    """All-gather of the ranks' row partials within the group of ranks that share a head.

    partial: this rank's fp32 tensor [B, Hq_local, PARTIAL_FLOATS] (any device torch.distributed can move).  Returns
    the sets in part order as one tensor [parts, B, Hq_local, PARTIAL_FLOATS].  `group` is the torch.distributed
    process group of shard.group (None: the default group, when all ranks share the heads)."""
    import torch
    import torch.distributed as dist
    if shard.parts == 1:
        return partial.unsqueeze(0)
    sets = [torch.empty_like(partial) for _ in range(shard.parts)]
    dist.all_gather(sets, partial.contiguous(), group=group)
    return torch.stack(sets)


class ShardedLayer:
    """One rank's share of a workload's decode attention on its GPU: a cache holding only the rank's heads and
    key ranges, and the call sequence of a decode step."""

    def __init__(self, w, plan: ShardPlan, rank: int, device="cuda", group=None):
        import torch
        from . import binding as slim
        from .workloads import PAGE_TOKENS
        self.slim, self.torch = slim, torch
        self.w, self.plan, self.shard, self.group = w, plan, plan.shard(rank), group
        self.device = torch.device(device)
        s = self.shard
        self.Hkv, self.Hq = len(s.kv_heads), len(s.q_heads)
        self.local_len = [t1 - t0 for t0, t1 in s.key_ranges]
        pages = max(1, max((n + PAGE_TOKENS - 1) // PAGE_TOKENS for n in self.local_len))
        self.cache = slim.SlimCache(w.B, self.Hkv, pages, device=device)
        self.max_kv = max(self.local_len)
        self.ws = slim.workspace(slim.PHASE_DECODE, w.B, self.Hq, self.Hkv, 1, max(1, self.max_kv), device=device)
        self.kv_len = torch.tensor(self.local_len, dtype=torch.int32, device=self.device)
        self.partial = torch.empty((w.B, self.Hq, slim.PARTIAL_FLOATS), dtype=torch.float32, device=self.device)

    def fill(self):
        """Quantise-and-append the rank's part of every sequence (its heads, its key range) into its cache."""
        torch, slim, s, w = self.torch, self.slim, self.shard, self.w
        h0, h1 = s.kv_heads.start, s.kv_heads.stop
        ks = [w.k[b][t0:t1, h0:h1] for b, (t0, t1) in enumerate(s.key_ranges)]
        vs = [w.v[b][t0:t1, h0:h1] for b, (t0, t1) in enumerate(s.key_ranges)]
        if sum(self.local_len) == 0:
            return
        k_new = torch.cat(ks).to(self.device).contiguous()
        v_new = torch.cat(vs).to(self.device).contiguous()
        cu = [0]
        for n in self.local_len:
            cu.append(cu[-1] + n)
        cu_d = torch.tensor(cu, dtype=torch.int32, device=self.device)
        zero = torch.zeros(w.B, dtype=torch.int32, device=self.device)
        slim.slim_kv_append(self.cache, k_new, v_new, cu_d, zero, w.B, max(self.local_len))

    def decode(self, q_all, stream=None):
        """q_all: bf16 [B, Hq (all heads), 128] on this device.  Returns the rank's heads' output [B, Hq_local, 128]."""
        if self.shard.parts == 1:
            torch, slim, s = self.torch, self.slim, self.shard
            q = q_all[:, s.q_heads.start:s.q_heads.stop].contiguous()
            out = torch.empty_like(q)
            slim.slim_attn_decode(self.cache, q, out, self.kv_len, self.w.B, self.max_kv, self.Hq, self.w.sm_scale, self.ws, stream)
            return out
        return self.finish(exchange_partials(self.partial_step(q_all, stream), self.shard, self.group), stream)

    def partial_step(self, q_all, stream=None):
        """Key-range mode, first half: attention over this rank's part of the keys; returns its row partials."""
        s = self.shard
        q = q_all[:, s.q_heads.start:s.q_heads.stop].contiguous()
        self.slim.slim_attn_decode_partial(self.cache, q, self.partial, self.kv_len, self.w.B, self.max_kv, self.Hq,
                                           self.w.sm_scale, self.ws, stream)
        return self.partial

    def finish(self, sets, stream=None):
        """Key-range mode, second half: merge of the group's row partials [parts, B, Hq_local, PARTIAL_FLOATS]."""
        out = self.torch.empty((self.w.B, self.Hq, 128), dtype=self.torch.bfloat16, device=self.device)
        self.slim.slim_attn_merge_partials(sets.contiguous(), int(sets.shape[0]), out, self.w.B, self.Hq, stream)
        return out
