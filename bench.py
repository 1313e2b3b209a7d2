#!/usr/bin/env python
"""Benchmark of the SlimAttention / INT8 KV cache hot path on B200.

One step = one pass of the decode hot path on the Llama-2-7B-shaped workload
(batch 16, 32 q = 32 kv heads, head_dim 128, 2048 cached tokens + 1 new token
per sequence): quantise-and-append the new K/V rows, then split + merge decode
attention over the 2049-token INT8 cache.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (under torchrun) every rank runs the same per-GPU workload on its own
GPU (sequences are independent; no collective on the data path; weak scaling)
and the line reports the aggregate over ranks with the max-over-ranks time.
`--impl reference` times the CPU oracle on the host cores instead.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode attention tokens/s (append + split/merge decode over the INT8 KV cache)"
UNIT = "tokens/s"
ROW_BYTES = 264            # per (token, kv head): 128 K codes + 128 V codes + 2 fp32 scales
N_ROT = 12                 # independent cache copies rotated between steps (12 x 277 MB = 3.3 GB).  Three copies are not
                           # enough: the stream is read with an evict-first L2 policy, under which part of every copy stayed
                           # L2-resident from one visit to the next (the step measured 2.5 us too fast); from 12 copies on the
                           # step time no longer depends on the count (12 and 40 copies measure the same)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops", 1590.0)), "measured"
    return 6650.0, 1590.0, "fallback"


def max_over_ranks(ms, world, device):
    """The slowest rank's time (every rank gets it); plain value when there is one rank."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step, steps, world, ms_max):
    """Aggregate units/s of `world` ranks that each did the same work, timed by the slowest rank."""
    return world * units_per_rank_per_step * steps / (ms_max * 1e-3)


class ClockSampler:
    """nvidia-smi clock/throttle sampling while the timed region runs (read-only queries)."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu_index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, sm_max, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                sm_max.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(sm_max) if sm_max else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# CPU oracle legs (the only places this file touches oracle/)
# ---------------------------------------------------------------------------------------------
def _bits(t):
    import numpy as np
    import torch
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


class OracleStep:
    """The decode step of the workload on the CPU oracle, on the first n_seq sequences."""

    def __init__(self, w, n_seq):
        from oracle import slim_oracle as so
        self.so, self.w, self.n_seq = so, w, n_seq
        self.ctx = w.bulk_len[0]
        self.cache = []
        for b in range(n_seq):
            kc, ks = so.quantize(_bits(w.k[b]))
            vc, vs = so.quantize(_bits(w.v[b]))
            self.cache.append([kc, ks, vc, vs])
        self.k_new = [_bits(w.k[b][self.ctx:self.ctx + 1]) for b in range(n_seq)]
        self.v_new = [_bits(w.v[b][self.ctx:self.ctx + 1]) for b in range(n_seq)]
        self.q = [_bits(w.q_decode[0, b:b + 1]) for b in range(n_seq)]

    def step(self):
        so, c = self.so, self.ctx
        for b in range(self.n_seq):
            kc, ks, vc, vs = self.cache[b]
            kc[c:c + 1], ks[c:c + 1] = so.quantize(self.k_new[b])
            vc[c:c + 1], vs[c:c + 1] = so.quantize(self.v_new[b])
            so.attention(self.q[b], kc, ks, vc, vs, c + 1, self.w.sm_scale)


def cpu_baseline(w, budget_s=12.0, max_reps=100):
    from oracle import slim_oracle as so
    st = OracleStep(w, w.B)
    st.step()
    reps, t0 = 0, time.perf_counter()
    while reps < max_reps and time.perf_counter() - t0 < budget_s:
        st.step()
        reps += 1
    dt = time.perf_counter() - t0
    return {"value": w.B * reps / dt, "unit": UNIT, "cores": so.threads(), "kind": "oracle",
            "sample": f"all {w.B} sequences of the workload, full step (quantise new rows + fp64 attention over "
                      f"{st.ctx + 1} tokens), {reps} repetitions in {dt:.1f} s"}


def run_reference(args, rank, world):
    if rank != 0:
        return
    from oracle import slim_oracle as so
    from paper_2407_07304_b200 import workloads
    w = workloads.make_workload(2)
    n_seq = 2                                    # bounded sample: 2 of the 16 sequences per step
    st = OracleStep(w, n_seq)
    for _ in range(args.warmup):
        st.step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        st.step()
    dt = time.perf_counter() - t0
    value = n_seq * args.steps / dt
    sample = f"{n_seq} of {w.B} sequences per step (all 32 heads, {st.ctx + 1} tokens), fp64 CPU oracle as it stands"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.B, "q_heads": w.Hq, "kv_heads": w.Hkv, "head_dim": 128,
                   "context": st.ctx + 1, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": so.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------
class CacheCopy:
    """One of the rotated cache copies: a cache and the decode workspace used with it."""

    def __init__(self, cache, ws_decode):
        self.cache, self.ws_decode = cache, ws_decode


def timed_blocks(fn, steps, min_ms, stream, barrier, world, dev):
    """Times blocks of exactly `steps` calls of fn, each block between two CUDA events on the launching stream and
    bracketed by a barrier + synchronize, until at least min_ms of device time are covered (at least one block).
    Returns the per-block times (each the max over ranks), in ms."""
    import torch
    blocks, total = [], 0.0
    while True:
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(steps):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        barrier()
        ms = max_over_ranks(ms, world, dev)     # every rank sees the same number, so every rank stops together
        blocks.append(ms)
        total += ms
        if total >= min_ms or len(blocks) >= 2000:
            return blocks


def stored_traffic():
    """DRAM bytes per launch of the step's kernel from the ncu capture summarised under profiles/, or None when the
    kernel's source has changed since that capture (the summary records the hash of the source it was taken on)."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", "decode_stream_workload2.md")
    src = os.path.join(ROOT, "paper_2407_07304_b200", "csrc", "slim_decode_stream.cu")
    try:
        text = open(path).read()
        digest = hashlib.sha1(open(src, "rb").read()).hexdigest()[:12]
    except OSError:
        return None
    m = re.search(r"traffic_bytes_per_launch:\s*([0-9.eE+]+)\s+kernel_source_sha1:\s*([0-9a-f]+)", text)
    if not m or m.group(2) != digest:
        return None
    return float(m.group(1))


def run_ours(args, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    from paper_2407_07304_b200 import binding as slim, workloads
    from paper_2407_07304_b200.harness import LayerRun

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the attention path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.shard:
        run_sharded(args, rank, world, dev, barrier)
        if world > 1:
            dist.destroy_process_group()
        return

    n_rot = max(1, args.copies)
    w = workloads.make_workload(2)
    B, Hq, Hkv, ctx = w.B, w.Hq, w.Hkv, w.bulk_len[0]
    kv_len_host = [ctx + 1] * B

    # n_rot independent caches, each pre-filled (untimed) with the 2048-token context
    first = LayerRun(w, device=dev)
    first.append(w.bulk_len)
    runs = [first]
    for _ in range(n_rot - 1):
        c = slim.SlimCache(B, Hkv, w.pages_per_seq(), device=dev)      # a copy of the filled cache in memory of its own
        c.codes.copy_(first.cache.codes)
        c.scales.copy_(first.cache.scales)
        runs.append(CacheCopy(c, first.ws_decode))
    torch.cuda.synchronize()
    k_new = torch.cat([w.k[b][ctx:ctx + 1] for b in range(B)]).to(dev).contiguous()    # [B, Hkv, 128]
    v_new = torch.cat([w.v[b][ctx:ctx + 1] for b in range(B)]).to(dev).contiguous()
    q = w.q_decode[0].to(dev).contiguous()
    out = torch.empty_like(q)
    kv_len = torch.full((B,), ctx + 1, dtype=torch.int32, device=dev)
    max_kv = ctx + 1
    ws = runs[0].ws_decode
    stream = torch.cuda.current_stream()

    def step(i):
        # one call, one kernel: it quantises the new token's K/V rows into the cache, attends over them from registers,
        # streams the rest of the cache once and merges its own partial results as its blocks finish
        slim.slim_decode_step(runs[i % n_rot].cache, q, k_new, v_new, out, kv_len, B, max_kv, Hq, w.sm_scale, ws, stream)

    for i in range(max(3, args.warmup)):
        step(i)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.1)
    # ---- headline: device-resident inputs, whole step.  Blocks of exactly --steps steps are repeated until MIN_TIMED_MS
    #      of device time are covered, and the median block is reported (a single block of 20 steps lasts 1 ms).
    blocks = timed_blocks(step, args.steps, args.min_ms, stream, barrier, world, dev)
    ms_total = statistics.median(blocks)
    # ---- per-kernel: events around every launch of the step's kernel (back to back in the loop above a launch's
    #      set-up overlaps the end of the one before it; here it does not)
    n_iso = max(args.steps, 100)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_iso)]
    barrier()
    for i in range(n_iso):
        evs[i][0].record(stream)
        step(i)
        evs[i][1].record(stream)
    torch.cuda.synchronize()
    split_ms = [a.elapsed_time(b) for a, b in evs]
    # ---- end to end: host (pinned) inputs and outputs through slim_decode_step_host
    # one pinned allocation holding q | k_new | v_new back to back: the step copies it with one transfer
    n_q, n_kv = q.numel(), k_new.numel()
    host_in = torch.empty(n_q + 2 * n_kv, dtype=torch.bfloat16).pin_memory()
    q_h, k_h, v_h = host_in[:n_q].view_as(q), host_in[n_q:n_q + n_kv].view_as(k_new), host_in[n_q + n_kv:].view_as(v_new)
    q_h.copy_(q.cpu()), k_h.copy_(k_new.cpu()), v_h.copy_(v_new.cpu())
    out_h = torch.empty_like(q_h).pin_memory()
    staging = torch.empty(slim.slim_step_staging_bytes(B, Hq, Hkv), dtype=torch.uint8, device=dev)

    def step_host(i):
        c = runs[i % n_rot].cache
        slim.slim_decode_step_host(c, q_h, k_h, v_h, out_h, staging, kv_len, B, max_kv, Hq, w.sm_scale, ws, stream)
        stream.synchronize()        # the caller needs the result before the next token

    for i in range(3):
        step_host(i)
    ms_e2e_eager = statistics.median(timed_blocks(step_host, args.steps, args.min_ms / 2, stream, barrier, world, dev))
    same = torch.equal(out_h, out.cpu())
    # The same call captured once per cache copy into a CUDA graph (one kernel that reads and writes the pinned buffers) and replayed:
    # what a serving loop does with a fixed-shape decode step.  The graph reads the pinned buffers at replay time.
    def graph_replay_ms():
        side = torch.cuda.Stream()
        graphs = []
        with torch.cuda.stream(side):
            for i in range(n_rot):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
                    slim.slim_decode_step_host(runs[i].cache, q_h, k_h, v_h, out_h, staging, kv_len, B, max_kv, Hq,
                                               w.sm_scale, ws, side)
                graphs.append(g)
            out_h.zero_()

            def step_graph(i):
                graphs[i % n_rot].replay()
                side.synchronize()      # the caller needs the result before the next token

            for i in range(3):
                step_graph(i)
            ok = torch.equal(out_h, out.cpu())
            ms = statistics.median(timed_blocks(step_graph, args.steps, args.min_ms / 2, side, barrier, world, dev))
        return ms, ok

    # For comparison, the classic form of the same step: one explicit copy in, the device entry point, one copy out.
    dev_in = torch.empty(n_q + 2 * n_kv, dtype=torch.bfloat16, device=dev)
    dq, dk, dv = dev_in[:n_q].view_as(q), dev_in[n_q:n_q + n_kv].view_as(k_new), dev_in[n_q + n_kv:].view_as(v_new)
    dev_out = torch.empty_like(q)

    def step_copies(i):
        dev_in.copy_(host_in, non_blocking=True)
        slim.slim_decode_step(runs[i % n_rot].cache, dq, dk, dv, dev_out, kv_len, B, max_kv, Hq, w.sm_scale, ws, stream)
        out_h.copy_(dev_out, non_blocking=True)
        stream.synchronize()

    for i in range(3):
        step_copies(i)
    ms_e2e_copies = statistics.median(timed_blocks(step_copies, args.steps, args.min_ms / 4, stream, barrier, world, dev))
    same = same and torch.equal(out_h, out.cpu())
    ms_e2e = ms_e2e_eager
    if not args.no_graph:
        ms_e2e, same_graph = graph_replay_ms()
        same = same and same_graph
    clocks = sampler.stop() if sampler else None

    # ---- the other workloads, single GPU only (context beside the headline, and the numbers the targets are set on)
    extra = {}
    if rank == 0 and world == 1 and not args.no_extra:
        extra = extra_numbers(slim, workloads, dev)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    hbm_peak, bf16_peak, peak_kind = _peaks()
    cache_bytes = sum(kv_len_host) * Hkv * ROW_BYTES
    # whole step: cache read once, Q in, O out, new K/V rows read as bf16 and written as codes + scales
    step_bytes = cache_bytes + 2 * B * Hq * 256 + B * Hkv * (2 * 256 + ROW_BYTES)
    split_bytes = step_bytes                     # the step is one kernel
    # The step is one kernel, so its average launch duration over the timed region is the step time: K launches
    # between two events on the launching stream.  Launched back to back a kernel's set-up overlaps the end of the
    # launch before it (programmatic dependent launch); with an event pair around every single launch it does
    # not, which is the `isolated_launch_ms` figure.
    split_avg_ms = ms_total / args.steps
    achieved = split_bytes / (split_avg_ms * 1e-3) / 1e9
    h2d = (B * Hq + 2 * B * Hkv) * 128 * 2
    d2h = B * Hq * 128 * 2
    line = {
        "metric": METRIC, "value": whole_job_rate(B, args.steps, world, ms_total), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_total / args.steps,
        "repeats": len(blocks), "block_ms": {"median": ms_total, "min": min(blocks), "max": max(blocks)},
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "s8 (tcgen05 kind::i8 MMA, s32 accumulate; fp32 softmax)",
        "data": "synthetic",
        "config": {"workload": w.name, "batch_per_gpu": B, "q_heads": Hq, "kv_heads": Hkv, "head_dim": 128,
                   "context": ctx + 1, "cache": "int8 codes + fp32 scale per (token, kv head), 128-token pages",
                   "l2": f"inputs larger than L2: {n_rot} cache copies of {cache_bytes / 1e6:.0f} MB rotated",
                   "parallelism": f"dp{world} (independent sequences per GPU, no collective)"},
        "hbm_gbs_step_per_gpu": step_bytes / (ms_total / args.steps * 1e-3) / 1e9,
        "pct_of_8tbs_step": 100.0 * step_bytes / (ms_total / args.steps * 1e-3) / 1e9 / 8000.0,
        "roofline": {"bound": "hbm", "kernel": "slim_decode_stream_kernel", "achieved": achieved, "peak": hbm_peak,
                     "unit": "GB/s", "frac": achieved / hbm_peak, "peak_kind": f"of {peak_kind}",
                     "frac_of_8tbs": achieved / 8000.0, "bytes_per_launch": split_bytes,
                     "avg_launch_ms": split_avg_ms, "isolated_launch_ms": statistics.mean(split_ms),
                     "isolated_min_launch_ms": min(split_ms), "traffic": stored_traffic()},
        "e2e": {"value": whole_job_rate(B, args.steps, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / args.steps, "matches_device_path": bool(same),
                "launch": ("slim_decode_step_host called and synchronised every step" if args.no_graph else
                           "slim_decode_step_host captured in a CUDA graph per cache copy, replayed and synchronised every step")
                          + "; inputs: read by the kernel from the pinned host buffers (every row crosses the bus once, no copy ahead"
                          " of the kernel), result: written by the kernel into the pinned host buffer",
                "ms_per_step_without_graph": ms_e2e_eager / args.steps,
                "ms_per_step_explicit_copies": ms_e2e_copies / args.steps},
        "gpu_launches": args.steps,
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu:
        line["cpu_baseline"] = cpu_baseline(w)
    if extra:
        line["targets"] = targets_summary(line, extra)
        line["extra"] = extra
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def targets_summary(line, extra):
    """The figures the targets are set on, side by side: decode attention as a fraction of 8 TB/s (target 0.70) and
    prefill attention as a fraction of the measured dense bf16 rate (target 0.50); append against the copy rate."""
    def dec(key):
        d = extra.get(key)
        return None if d is None else {"us": 1e3 * d["ms"], "frac_of_8tbs": d["gbs"] / 8000.0, "target": 0.70,
                                       "met": d["gbs"] / 8000.0 >= 0.70}

    def pre(key):
        d = extra.get(key)
        return None if d is None else {"ms": d["ms"], "tflops": d["tflops"], "frac_of_bf16_peak": d["frac_of_bf16_peak"],
                                       "kernel": "slim_attn_prefill (streamed form)", "target": 0.50,
                                       "met": d["frac_of_bf16_peak"] >= 0.50}
    t = {"decode_c2_step": {"us": 1e3 * line["ms_per_step"], "frac_of_8tbs": line["roofline"]["frac_of_8tbs"], "target": 0.70,
                            "met": line["roofline"]["frac_of_8tbs"] >= 0.70},
         "decode_c4": dec("decode_c4"), "decode_c4_step": dec("step_c4"),
         "prefill_c3": pre("prefill_c3"), "prefill_c5": pre("prefill_c5")}
    if "append_c3" in extra:
        t["append_c3"] = {"us": 1e3 * extra["append_c3"]["ms"], "frac_of_hbm_peak": extra["append_c3"]["frac_of_hbm_peak"]}
    return t


def run_sharded(args, rank, world, dev, barrier):
    """--shard: ONE workload's decode attention divided over the ranks (strong scaling): workload 4 by kv heads
    (64 query heads over 8 kv heads: one kv head per rank at 8 GPUs), workload 5 (2 kv heads) by key ranges with one
    all-gather of the row partials per step.  Every rank's kernels read its own GPU's memory only."""
    import torch
    import torch.distributed as dist
    from paper_2407_07304_b200 import workloads
    from paper_2407_07304_b200.shard import ShardPlan, ShardedLayer
    w = workloads.make_workload(args.shard_workload)
    lens = [w.total_len(b) - w.decode_steps + 1 for b in range(w.B)]
    plan = ShardPlan(w.Hq, w.Hkv, lens, world)
    shard = plan.shard(rank)
    group = None
    if plan.parts > 1 and plan.parts < world:
        # every rank creates every group (torch.distributed's rule); it keeps its own
        for h in range(w.Hkv):
            ranks = [h * plan.parts + i for i in range(plan.parts)]
            g = dist.new_group(ranks)
            if rank in ranks:
                group = g
    copies = max(1, min(12, int(2.5e9 // max(1, plan.cache_bytes(rank)))))   # rotated copies of this rank's cache
    layers = []
    for _ in range(copies):
        layer = ShardedLayer(w, plan, rank, device=dev, group=group)
        if layers:
            layer.cache.codes.copy_(layers[0].cache.codes)
            layer.cache.scales.copy_(layers[0].cache.scales)
        else:
            layer.fill()
        layers.append(layer)
    q = w.q_decode[0].to(dev).contiguous()
    stream = torch.cuda.current_stream()

    def step(i):
        layers[i % copies].decode(q, stream)

    for i in range(max(3, args.warmup)):
        step(i)
    sampler = ClockSampler(dev.index) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.1)
    blocks = timed_blocks(step, args.steps, args.min_ms, stream, barrier, world, dev)
    clocks = sampler.stop() if sampler else None
    if rank != 0:
        return
    ms_total = statistics.median(blocks)
    hbm_peak, _, peak_kind = _peaks()
    total_bytes = sum(lens) * w.Hkv * ROW_BYTES + 2 * w.B * w.Hq * 256
    achieved = total_bytes / world / (ms_total / args.steps * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": w.B * args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_total / args.steps, "repeats": len(blocks),
        "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
        "dtype": "s8 (tcgen05 kind::i8 MMA, s32 accumulate; fp32 softmax)", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.B, "q_heads": w.Hq, "kv_heads": w.Hkv, "head_dim": 128,
                   "parallelism": (f"tp{world} by kv heads, no collective" if plan.mode == "heads" else
                                   f"{w.Hkv} kv heads x {plan.parts} key ranges, one all-gather of "
                                   f"{w.B * len(shard.q_heads) * 528} B per rank and step"),
                   "l2": f"{copies} copies of each rank's {plan.cache_bytes(rank) / 1e6:.0f} MB cache share rotated"},
        "roofline": {"bound": "hbm", "kernel": "slim_decode_stream_kernel", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                     "frac": achieved / hbm_peak, "peak_kind": f"of {peak_kind}, per GPU", "traffic": None},
        "gpu_launches": args.steps * (2 if plan.mode == "heads" else 3), "clocks": clocks,
    }
    print(json.dumps(line), flush=True)


MIN_TIMED_MS = 200.0       # device time covered by the timed blocks of the headline number


def extra_numbers(slim, workloads, dev):
    """Prefill of workload 3 (S = 8192) timed alone: TFLOP/s against the bf16 dense peak."""
    import torch
    from paper_2407_07304_b200.harness import LayerRun
    _, bf16_peak, peak_kind = _peaks()
    w3 = workloads.make_workload(3)
    run = LayerRun(w3, device=dev)
    S = w3.prefill_len[0]
    k_new, v_new = run.k[0].contiguous(), run.v[0].contiguous()
    cu = torch.tensor([0, S], dtype=torch.int32, device=dev)
    zero = torch.zeros(1, dtype=torch.int32, device=dev)
    kvl = torch.tensor([S], dtype=torch.int32, device=dev)
    q = w3.q_prefill[0].to(dev).contiguous()
    out = torch.empty_like(q)
    stream = torch.cuda.current_stream()

    def append():
        slim.slim_kv_append(run.cache, k_new, v_new, cu, zero, 1, S, stream)

    def prefill():
        slim.slim_attn_prefill(run.cache, q, out, cu, kvl, 1, S, S, w3.Hq, w3.sm_scale, run.ws_prefill, stream)

    def time_it(fn, reps):
        """ms per call: the best of three blocks of `reps` calls (the matmul peak the prefill numbers are set against
        is itself a best-of-ten burst; a single block taken right after the decode loops runs under the power cap)."""
        fn()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(reps):
                fn()
            e1.record(stream)
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) / reps)
        return best

    def both():
        append()
        prefill()

    def step():
        slim.slim_prefill_step(run.cache, q, k_new, v_new, out, cu, kvl, 1, S, S, w3.Hq, w3.sm_scale, run.ws_prefill, stream)

    ms_append = time_it(append, 20)
    ms_prefill = time_it(prefill, 5)
    ms_both = time_it(both, 5)
    ms_step = time_it(step, 5)
    flops = 4 * 128 * w3.Hq * S * (S + 1) // 2
    append_bytes = S * w3.Hkv * (2 * 256 + ROW_BYTES)
    hbm_peak, _, _ = _peaks()
    del run, q, out, k_new, v_new

    def rotated_caches(w, ctx, copies):
        """`copies` caches filled with the first ctx[b] tokens of every sequence, each in memory of its own."""
        r = LayerRun(w, device=dev)
        r.append(ctx)
        caches = [r.cache]
        for _ in range(copies - 1):
            c = slim.SlimCache(w.B, w.Hkv, w.pages_per_seq(), device=dev)
            c.codes.copy_(r.cache.codes)
            c.scales.copy_(r.cache.scales)
            caches.append(c)
        return r, caches

    def decode_numbers(index, copies, label):
        """slim_attn_decode (split + merge) of workload `index` at its final context, cache pre-filled untimed."""
        w = workloads.make_workload(index)
        ctx = [w.total_len(b) - w.decode_steps + 1 for b in range(w.B)]
        r, caches = rotated_caches(w, ctx, copies)
        qd = w.q_decode[0].to(dev).contiguous()
        od = torch.empty_like(qd)
        kvl = torch.tensor(ctx, dtype=torch.int32, device=dev)
        mk = max(ctx)
        it = [0]

        def dec():
            c = caches[it[0] % copies]
            it[0] += 1
            slim.slim_attn_decode(c, qd, od, kvl, w.B, mk, w.Hq, w.sm_scale, r.ws_decode, stream)

        ms = time_it(dec, 10 * copies if copies > 1 else 50)
        nbytes = sum(ctx) * w.Hkv * ROW_BYTES + 2 * w.B * w.Hq * 256
        return {"workload": w.name, "ms": ms, "tokens_per_s": w.B / (ms * 1e-3), "gbs": nbytes / (ms * 1e-3) / 1e9,
                "frac_of_hbm_peak": nbytes / (ms * 1e-3) / 1e9 / hbm_peak, "frac_of_8tbs": nbytes / (ms * 1e-3) / 1e9 / 8000.0,
                "cache": label}

    def prefill_numbers(index, shrink=1, reps=3, two_pass=False, full_row=False):
        w = workloads.make_workload(index, shrink=shrink)
        r = LayerRun(w, device=dev)
        n = w.prefill_len[0]
        r.append(w.prefill_len)
        cu5 = torch.tensor([0, n], dtype=torch.int32, device=dev)
        kv5 = torch.tensor([n], dtype=torch.int32, device=dev)
        q5 = w.q_prefill[0].to(dev).contiguous()
        o5 = torch.empty_like(q5)

        call = slim.slim_attn_prefill_full_row if full_row else (slim.slim_attn_prefill_two_pass if two_pass else slim.slim_attn_prefill)

        def pf():
            call(r.cache, q5, o5, cu5, kv5, 1, n, n, w.Hq, w.sm_scale, r.ws_prefill, stream)

        ms = time_it(pf, reps)
        fl = 4 * 128 * w.Hq * n * (n + 1) // 2   # the attention's flops: the second Q.K^T of the two-pass form is not counted
        return {"workload": w.name, "tokens": n, "ms": ms, "tflops": fl / (ms * 1e-3) / 1e12,
                "frac_of_bf16_peak": fl / (ms * 1e-3) / 1e12 / bf16_peak}

    def batched_prefill_numbers():
        """One slim_attn_prefill call over sixteen prompts of 256..4096 tokens (variable-length batch)."""
        w = workloads.make_batched_prefill()
        r = LayerRun(w, device=dev)
        r.append(w.prefill_len)
        cu = [0]
        for n in w.prefill_len:
            cu.append(cu[-1] + n)
        cu_d = torch.tensor(cu, dtype=torch.int32, device=dev)
        kv_d = torch.tensor(w.prefill_len, dtype=torch.int32, device=dev)
        qb = torch.cat([t.to(dev) for t in w.q_prefill]).contiguous()
        ob = torch.empty_like(qb)
        mx = max(w.prefill_len)

        def pf():
            slim.slim_attn_prefill(r.cache, qb, ob, cu_d, kv_d, w.B, mx, mx, w.Hq, w.sm_scale, r.ws_prefill, stream)

        ms = time_it(pf, 5)
        fl = sum(4 * 128 * w.Hq * n * (n + 1) // 2 for n in w.prefill_len)
        return {"workload": w.name, "tokens": cu[-1], "lengths": w.prefill_len, "ms": ms,
                "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_bf16_peak": fl / (ms * 1e-3) / 1e12 / bf16_peak}

    def chunked_prefill_numbers(n=2048):
        """The last n tokens of workload 3 attend over its whole 8192-token cache (q_len < kv_len)."""
        w = workloads.make_workload(3)
        r = LayerRun(w, device=dev)
        r.append(w.prefill_len)
        S_ = w.prefill_len[0]
        cu_d = torch.tensor([0, n], dtype=torch.int32, device=dev)
        kv_d = torch.tensor([S_], dtype=torch.int32, device=dev)
        qc = w.q_prefill[0][S_ - n:].to(dev).contiguous()
        oc_ = torch.empty_like(qc)

        def pf():
            slim.slim_attn_prefill(r.cache, qc, oc_, cu_d, kv_d, 1, n, S_, w.Hq, w.sm_scale, r.ws_prefill, stream)

        ms = time_it(pf, 5)
        fl = 4 * 128 * w.Hq * (n * (S_ - n) + n * (n + 1) // 2)
        return {"workload": w.name + f"_last{n}", "q_tokens": n, "kv_tokens": S_, "ms": ms,
                "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_bf16_peak": fl / (ms * 1e-3) / 1e12 / bf16_peak}

    def step_numbers(index, label, copies=1):
        """slim_decode_step (append of one token per sequence + decode in one call) at the workload's final context."""
        w = workloads.make_workload(index)
        ctx = [w.total_len(b) - 1 for b in range(w.B)]
        r, caches = rotated_caches(w, ctx, copies)
        kn = torch.stack([r.k[b][ctx[b]] for b in range(w.B)]).contiguous()
        vn = torch.stack([r.v[b][ctx[b]] for b in range(w.B)]).contiguous()
        qd = w.q_decode[0].to(dev).contiguous()
        od = torch.empty_like(qd)
        kvl = torch.tensor([c + 1 for c in ctx], dtype=torch.int32, device=dev)
        it = [0]

        def st():
            c = caches[it[0] % copies]
            it[0] += 1
            slim.slim_decode_step(c, qd, kn, vn, od, kvl, w.B, max(ctx) + 1, w.Hq, w.sm_scale, r.ws_decode, stream)

        ms = time_it(st, 10 * copies if copies > 1 else 50)
        nbytes = (sum(ctx) + w.B) * w.Hkv * ROW_BYTES + 2 * w.B * w.Hq * 256 + w.B * w.Hkv * (2 * 256 + ROW_BYTES)
        res = {"workload": w.name, "ms": ms, "tokens_per_s": w.B / (ms * 1e-3), "gbs": nbytes / (ms * 1e-3) / 1e9,
               "frac_of_8tbs": nbytes / (ms * 1e-3) / 1e9 / 8000.0, "cache": label}
        if copies > 1:
            return res
        # the same step replayed from a CUDA graph of twenty calls: the device-side latency of a step without the
        # host's launch cost between steps (the same new row goes to the same slot every time: idempotent)
        side = torch.cuda.Stream()
        n_in_graph = 20
        c0 = caches[0]
        with torch.cuda.stream(side):
            slim.slim_decode_step(c0, qd, kn, vn, od, kvl, w.B, max(ctx) + 1, w.Hq, w.sm_scale, r.ws_decode, side)
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
                for _ in range(n_in_graph):
                    slim.slim_decode_step(c0, qd, kn, vn, od, kvl, w.B, max(ctx) + 1, w.Hq, w.sm_scale, r.ws_decode, side)
            g.replay()
            side.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(5):
                g.replay()
            e1.record(side)
            side.synchronize()
            res["ms_graph_replay"] = e0.elapsed_time(e1) / (5 * n_in_graph)
        return res

    more = {}
    if not os.environ.get("SLIM_BENCH_SHORT"):
        more = {"decode_c4": decode_numbers(4, 12, "twelve cache copies rotated (12 x 187 MB)"),
                "step_c4": step_numbers(4, "twelve cache copies rotated (12 x 187 MB)", copies=12),
                "decode_c5": decode_numbers(5, 1, "17 MB, L2-resident: a latency number, not an HBM number"),
                "decode_c1": decode_numbers(1, 1, "2 MB, L2-resident: a latency number, not an HBM number"),
                "prefill_c5": prefill_numbers(5),
                "prefill_c1": prefill_numbers(1),
                "step_c1": step_numbers(1, "2 MB, L2-resident: a latency number"),
                "step_c5": step_numbers(5, "17 MB, L2-resident: a latency number"),
                # the literal order (all scores of a row, then softmax, then .V): maxima first, no corrections
                "prefill_two_pass_c3": prefill_numbers(3, two_pass=True),
                "prefill_two_pass_sweep": [prefill_numbers(3, shrink=k, reps=10, two_pass=True) for k in (32, 16, 8, 4, 2)],
                # the other literal order: the whole score row of a 128-row block on chip, one softmax (caches up to 256 tokens)
                "prefill_full_row_256": prefill_numbers(3, shrink=32, reps=10, full_row=True),
                "prefill_batched": batched_prefill_numbers(),
                "prefill_chunked": chunked_prefill_numbers(),
                # one sequence, 32 heads, the sequence lengths of the paper's Table 3 (256 ... 4096 tokens)
                "prefill_sweep": [prefill_numbers(3, shrink=k, reps=10) for k in (32, 16, 8, 4, 2)]}
    return {**more, **{
        "prefill_c3": {"workload": w3.name, "ms": ms_prefill, "tflops": flops / (ms_prefill * 1e-3) / 1e12,
                       "frac_of_bf16_peak": flops / (ms_prefill * 1e-3) / 1e12 / bf16_peak,
                       "peak_tflops": bf16_peak, "peak_kind": f"of {peak_kind}",
                       "tokens_per_s_with_append": S / ((ms_prefill + ms_append) * 1e-3)},
        # append + prefill of workload 3 as two calls back to back, and as the one call slim_prefill_step
        "prefill_step_c3": {"workload": w3.name, "ms_two_calls": ms_both, "ms": ms_step, "tokens_per_s": S / (ms_step * 1e-3)},
        "append_c3": {"ms": ms_append, "gbs": append_bytes / (ms_append * 1e-3) / 1e9,
                      "frac_of_hbm_peak": append_bytes / (ms_append * 1e-3) / 1e9 / hbm_peak},
    }}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=30)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-extra", action="store_true", help="skip the prefill context numbers")
    ap.add_argument("--no-graph", action="store_true", help="end-to-end leg without CUDA-graph replay (plain calls)")
    ap.add_argument("--shard", action="store_true",
                    help="divide ONE workload's decode attention over the ranks (strong scaling) instead of replicating workload 2")
    ap.add_argument("--shard-workload", type=int, default=4, choices=[2, 4, 5],
                    help="workload divided by --shard: 4 (by kv heads) or 5 (2 kv heads: by key ranges beyond 2 ranks)")
    ap.add_argument("--min-ms", type=float, default=MIN_TIMED_MS,
                    help="device time the repeated timed blocks must cover (default 200; small values for profiler runs)")
    ap.add_argument("--copies", type=int, default=N_ROT,
                    help="cache copies rotated between steps (default 12; fewer only for profiler captures that must stay small)")
    ap.add_argument("--extra-only", action="store_true",
                    help="run only the workload-3 prefill/append timings (for profiling that kernel) and print them")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.extra_only:
        import torch
        from paper_2407_07304_b200 import binding as slim, workloads
        torch.cuda.set_device(local_rank)
        print(json.dumps({"extra": extra_numbers(slim, workloads, torch.device("cuda", local_rank))}), flush=True)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
