"""Drives a workload through the library on one GPU: buffers, call order, gathering results.

Plumbing only (uploads, index tensors, the append -> prefill -> append -> decode call
sequence of a workload); all arithmetic happens inside the library calls.
"""
import torch

from . import binding as slim
from .workloads import PAGE_TOKENS, Workload


class LayerRun:
    """One attention layer's cache and device copies of a workload's tensors."""

    def __init__(self, w: Workload, device="cuda", block_table=None, num_pages=None):
        self.w = w
        self.device = torch.device(device)
        self.cache = slim.SlimCache(w.B, w.Hkv, w.pages_per_seq(), device=device, block_table=block_table,
                                    num_pages=num_pages)
        self.k = [t.to(device) for t in w.k]
        self.v = [t.to(device) for t in w.v]
        self.pos = [0] * w.B          # tokens in the cache per sequence
        self.max_total = max(w.total_len(b) for b in range(w.B))
        self.ws_decode = slim.workspace(slim.PHASE_DECODE, w.B, w.Hq, w.Hkv, 1, self.max_total, device=device)
        self.ws_prefill = slim.workspace(slim.PHASE_PREFILL, w.B, w.Hq, w.Hkv, max(w.prefill_len + [1]),
                                         self.max_total, device=device)

    def _i32(self, values):
        return torch.tensor(values, dtype=torch.int32, device=self.device)

    # ------------------------------------------------------------------ append
    def append(self, counts):
        """Append the next counts[b] rows of sequence b's K/V to the cache."""
        w = self.w
        ks = [self.k[b][self.pos[b]:self.pos[b] + counts[b]] for b in range(w.B)]
        vs = [self.v[b][self.pos[b]:self.pos[b] + counts[b]] for b in range(w.B)]
        k_new = torch.cat(ks).contiguous()
        v_new = torch.cat(vs).contiguous()
        cu = [0]
        for c in counts:
            cu.append(cu[-1] + c)
        slim.slim_kv_append(self.cache, k_new, v_new, self._i32(cu), self._i32(self.pos), w.B, max(counts))
        for b in range(w.B):
            self.pos[b] += counts[b]

    # ------------------------------------------------------------------ attention
    def prefill(self, q_list, two_pass=False, full_row=False):
        """Causal attention of q_list[b] (bf16 [n_b, Hq, 128], the last n_b cached positions);
        two_pass selects slim_attn_prefill_two_pass (maxima first, then P.V, no corrections), full_row
        slim_attn_prefill_full_row (the whole score row on chip; caches of at most 256 tokens)."""
        w = self.w
        lens = [int(q.shape[0]) for q in q_list]
        q = torch.cat([t.to(self.device) for t in q_list]).contiguous()
        out = torch.empty_like(q)
        cu = [0]
        for n in lens:
            cu.append(cu[-1] + n)
        fn = slim.slim_attn_prefill_full_row if full_row else (slim.slim_attn_prefill_two_pass if two_pass else slim.slim_attn_prefill)
        fn(self.cache, q, out, self._i32(cu), self._i32(self.pos), w.B, max(lens), max(self.pos), w.Hq, w.sm_scale,
           self.ws_prefill)
        return [out[cu[b]:cu[b + 1]] for b in range(w.B)]

    def prefill_step(self, counts, q_list):
        """Append the next counts[b] rows of sequence b and attend q_list[b] (one query row per new token) over the
        lengthened cache, in one library call."""
        w = self.w
        k_new = torch.cat([self.k[b][self.pos[b]:self.pos[b] + counts[b]] for b in range(w.B)]).contiguous()
        v_new = torch.cat([self.v[b][self.pos[b]:self.pos[b] + counts[b]] for b in range(w.B)]).contiguous()
        q = torch.cat([t.to(self.device) for t in q_list]).contiguous()
        out = torch.empty_like(q)
        cu = [0]
        for c in counts:
            cu.append(cu[-1] + c)
        for b in range(w.B):
            self.pos[b] += counts[b]
        slim.slim_prefill_step(self.cache, q, k_new, v_new, out, self._i32(cu), self._i32(self.pos), w.B, max(counts),
                               max(self.pos), w.Hq, w.sm_scale, self.ws_prefill)
        return [out[cu[b]:cu[b + 1]] for b in range(w.B)]

    def decode(self, q):
        """One query token per sequence (bf16 [B, Hq, 128]) against the whole cache."""
        w = self.w
        q = q.to(self.device).contiguous()
        out = torch.empty_like(q)
        slim.slim_attn_decode(self.cache, q, out, self._i32(self.pos), w.B, max(self.pos), w.Hq, w.sm_scale,
                              self.ws_decode)
        return out

    def decode_step(self, q):
        """Append the next token of every sequence and attend over the lengthened cache in one library call."""
        w = self.w
        k_new = torch.stack([self.k[b][self.pos[b]] for b in range(w.B)]).contiguous()
        v_new = torch.stack([self.v[b][self.pos[b]] for b in range(w.B)]).contiguous()
        for b in range(w.B):
            self.pos[b] += 1
        q = q.to(self.device).contiguous()
        out = torch.empty_like(q)
        slim.slim_decode_step(self.cache, q, k_new, v_new, out, self._i32(self.pos), w.B, max(self.pos), w.Hq,
                              w.sm_scale, self.ws_decode)
        return out

    # ------------------------------------------------------------------ read-back
    def gather_cache(self, b):
        """Sequence b's cached rows in position order:
        (k_codes, k_scales, v_codes, v_scales) as CPU tensors [T, Hkv, 128] int8 / [T, Hkv] fp32."""
        T = self.pos[b]
        n_pages = (T + PAGE_TOKENS - 1) // PAGE_TOKENS
        pages = self.cache.block_table[b, :n_pages].long()
        codes = self.cache.codes_view()[pages]      # [n_pages, Hkv, 2, 128, 128]
        scales = self.cache.scales_view()[pages]    # [n_pages, Hkv, 2, 128]
        codes = codes.permute(2, 0, 3, 1, 4).reshape(2, n_pages * PAGE_TOKENS, self.w.Hkv, 128)[:, :T]
        scales = scales.permute(2, 0, 3, 1).reshape(2, n_pages * PAGE_TOKENS, self.w.Hkv)[:, :T]
        codes, scales = codes.cpu(), scales.cpu()
        return codes[0], scales[0], codes[1], scales[1]


def run_workload(w: Workload, device="cuda", decode_steps=None, block_table=None, num_pages=None, one_call_step=False):
    """The workload's full call sequence.  Returns (LayerRun, prefill outputs per sequence or None,
    {decode step: output [B, Hq, 128]}); decode_steps limits which steps' outputs are kept.  With one_call_step
    every decode step is one slim_decode_step call instead of slim_kv_append followed by slim_attn_decode."""
    run = LayerRun(w, device=device, block_table=block_table, num_pages=num_pages)
    out_prefill = None
    if any(n > 0 for n in w.prefill_len):
        run.append(w.prefill_len)
        out_prefill = run.prefill(w.q_prefill)
    if any(n > 0 for n in w.bulk_len):
        run.append(w.bulk_len)
    outs = {}
    for s in range(w.decode_steps):
        if one_call_step:
            o = run.decode_step(w.q_decode[s])
        else:
            run.append([1] * w.B)
            o = run.decode(w.q_decode[s])
        if decode_steps is None or s in decode_steps:
            outs[s] = o
    torch.cuda.synchronize()
    return run, out_prefill, outs
