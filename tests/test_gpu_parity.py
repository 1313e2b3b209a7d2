"""CUDA path vs the CPU oracle, through the C ABI, on the five seeded workloads.

Codes and scale bits must be identical; attention outputs (bf16) must be within
max-abs 2e-2 and mean-abs 2e-3 of the fp64 oracle evaluated on the same codes.

The flat 2e-2 holds wherever a bf16 output can meet it: below magnitude 8 the bf16
half-ulp is at most 2^-6 = 1.56e-2.  From magnitude 8 on the half-ulp is 2^-5 or more,
so the correctly rounded oracle value itself may miss 2e-2 (the outlier channels of
workloads 2 and 4 produce a handful of such outputs).  There the bound is the bf16
half-ulp of the oracle value plus the arithmetic share the flat bound leaves in the
binade below, 2e-2 - 2^-6 = 4.4e-3.
"""
import numpy as np
import pytest
import torch

from oracle import slim_oracle as so
from paper_2407_07304_b200 import workloads
from helpers import MAX_ABS, MEAN_ABS, bf16_bits, mantissa_sweep_bits, output_bound

pytestmark = pytest.mark.gpu


def _oracle_cache(w):
    """Oracle codes/scales of every sequence's K and V (all rows the run appends)."""
    out = []
    for b in range(w.B):
        kc, ks = so.quantize(bf16_bits(w.k[b]))
        vc, vs = so.quantize(bf16_bits(w.v[b]))
        out.append((kc, ks, vc, vs))
    return out


def _assert_cache_bits(run, oc):
    for b in range(run.w.B):
        kc, ks, vc, vs = run.gather_cache(b)
        T = run.pos[b]
        assert np.array_equal(kc.numpy(), oc[b][0][:T]), f"K codes differ (seq {b})"
        assert np.array_equal(vc.numpy(), oc[b][2][:T]), f"V codes differ (seq {b})"
        assert np.array_equal(ks.numpy().view(np.uint32), oc[b][1][:T].view(np.uint32)), f"K scales differ (seq {b})"
        assert np.array_equal(vs.numpy().view(np.uint32), oc[b][3][:T].view(np.uint32)), f"V scales differ (seq {b})"


RELAXED = {"elements": 0, "worst_excess_over_flat": 0.0}   # how often the bound above magnitude 8 was needed


def _assert_close(got_bf16, want_f64, what):
    got = got_bf16.float().cpu().numpy().astype(np.float64)
    err = np.abs(got - want_f64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    bound = output_bound(want_f64)
    i = np.unravel_index((err - bound).argmax(), err.shape)
    assert (err <= bound).all(), f"{what}: abs error {err[i]:.3e} (bound {bound[i]:.3e}) at {i}: got {got[i]!r} want {want_f64[i]!r}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean-abs {err.mean():.3e}"
    over = err > MAX_ABS
    if over.any():
        RELAXED["elements"] += int(over.sum())
        RELAXED["worst_excess_over_flat"] = max(RELAXED["worst_excess_over_flat"], float((err - MAX_ABS).max()))
        print(f"{what}: {int(over.sum())} element(s) of magnitude >= 8 above the flat bound, worst {err[over].max():.3e}")
    return err.max(), err.mean()


def _sample_rows(n, extra, seed):
    base = [r for r in (0, 1, 63, 64, 65, 127, 128, 129, n - 2, n - 1) if 0 <= r < n]
    rng = np.random.default_rng(seed)
    more = rng.integers(0, n, size=extra).tolist() if n > len(base) else []
    return sorted(set(base + more))


def _check(w, prefill_rows=None, decode_steps=None, one_call_step=False):
    """Run the workload on the GPU and compare everything (or the given samples) with the oracle."""
    from paper_2407_07304_b200 import binding as slim, harness
    oc = _oracle_cache(w)
    run, out_prefill, outs = harness.run_workload(w, decode_steps=decode_steps, one_call_step=one_call_step)
    assert slim.slim_read_status(run.ws_decode) == slim.SLIM_OK
    _assert_cache_bits(run, oc)
    if out_prefill is not None:
        for b in range(w.B):
            n = w.prefill_len[b]
            sel = None if prefill_rows is None else _sample_rows(n, prefill_rows, 17 + b)
            want = so.attention(bf16_bits(w.q_prefill[b]), oc[b][0], oc[b][1], oc[b][2], oc[b][3], n, w.sm_scale, sel=sel)
            got = out_prefill[b] if sel is None else out_prefill[b][torch.tensor(sel, device=out_prefill[b].device)]
            _assert_close(got, want, f"{w.name} prefill seq {b}")
    for s, o in outs.items():
        for b in range(w.B):
            L = w.prefill_len[b] + w.bulk_len[b] + s + 1
            want = so.attention(bf16_bits(w.q_decode[s, b:b + 1]), oc[b][0], oc[b][1], oc[b][2], oc[b][3], L, w.sm_scale)
            _assert_close(o[b:b + 1], want, f"{w.name} decode step {s} seq {b}")


# ---------------------------------------------------------------- small versions: every output compared
@pytest.mark.parametrize("index,shrink", [(1, 1), (2, 8), (3, 16), (4, 8), (5, 32)])
def test_workload_small_all_outputs(index, shrink):
    _check(workloads.make_workload(index, shrink=shrink))


@pytest.mark.parametrize("index,shrink", [(1, 1), (2, 8), (4, 8), (5, 32)])
def test_workload_small_one_call_steps(index, shrink):
    # the decode steps through slim_decode_step: the new token is quantised inside the attention kernel
    _check(workloads.make_workload(index, shrink=shrink), one_call_step=True)


# ---------------------------------------------------------------- full sizes
def test_c2_full_all_rows():
    _check(workloads.make_workload(2))


def test_c4_full_all_rows():
    _check(workloads.make_workload(4))


@pytest.mark.parametrize("index", [2, 4])
def test_full_one_call_step(index):
    _check(workloads.make_workload(index), one_call_step=True)


def test_c5_full_one_call_steps_sampled():
    # 32 705 ... 32 768 cached tokens, 16 query heads per kv head: more partials per pair than the split kernel merges
    # itself, so the one-call step here is the split kernel (new rows written inside) followed by the merge kernel
    _check(workloads.make_workload(5), prefill_rows=8, decode_steps={0, 63}, one_call_step=True)


def test_c3_full_sampled_rows():
    _check(workloads.make_workload(3), prefill_rows=48)


def test_batched_ragged_prefill_full_size_sampled():
    # sixteen prompts of 256..4096 tokens attended in one call (the case the bench times as prefill_batched)
    _check(workloads.make_batched_prefill(), prefill_rows=6)


def test_chunked_prefill_full_size_sampled():
    # the last 2048 of workload 3's 8192 tokens attend over the whole cache (q_len < kv_len), as the bench's
    # prefill_chunked case does; sampled rows against the oracle's rows 6144.. of the full causal prefill
    from paper_2407_07304_b200 import harness
    w = workloads.make_workload(3)
    S, n = w.prefill_len[0], 2048
    oc = _oracle_cache(w)
    run = harness.LayerRun(w)
    run.append([S])
    _assert_cache_bits(run, oc)
    out = run.prefill([w.q_prefill[0][S - n:]])[0]
    sel = _sample_rows(n, 24, 5)
    want = so.attention(bf16_bits(w.q_prefill[0]), *oc[0], S, w.sm_scale, sel=[S - n + r for r in sel])
    _assert_close(out[torch.tensor(sel, device=out.device)], want, "chunked prefill of workload 3")


def _check_two_pass(w, prefill_rows=None):
    """slim_attn_prefill_two_pass (maxima first, then P.V) against the oracle, and against the one-pass kernel."""
    from paper_2407_07304_b200 import binding as slim, harness
    oc = _oracle_cache(w)
    run = harness.LayerRun(w)
    run.append(w.prefill_len)
    out = run.prefill(w.q_prefill, two_pass=True)
    ref = run.prefill(w.q_prefill)
    torch.cuda.synchronize()
    assert slim.slim_read_status(run.ws_prefill) == slim.SLIM_OK
    for b in range(w.B):
        n = w.prefill_len[b]
        sel = None if prefill_rows is None else _sample_rows(n, prefill_rows, 23 + b)
        want = so.attention(bf16_bits(w.q_prefill[b]), *oc[b], n, w.sm_scale, sel=sel)
        idx = slice(None) if sel is None else torch.tensor(sel, device=out[b].device)
        _assert_close(out[b][idx], want, f"{w.name} two-pass prefill seq {b}")
        # both kernels round the same exact result: they differ by a few bf16 ulps at most
        d = (out[b].float() - ref[b].float()).abs().max().item()
        assert d <= 2 * MAX_ABS, f"{w.name} seq {b}: two-pass and one-pass outputs differ by {d}"


@pytest.mark.parametrize("index,shrink", [(1, 1), (3, 16), (5, 32)])
def test_two_pass_prefill_small_all_outputs(index, shrink):
    _check_two_pass(workloads.make_workload(index, shrink=shrink))


@pytest.mark.parametrize("lens", [[1], [2, 127], [128, 129], [255, 256, 257], [1, 383, 640]])
def test_two_pass_prefill_ragged_lengths(lens):
    B = len(lens)
    _check_two_pass(_custom(B, 4, 2, lens, [0] * B, 0, 700 + lens[0]))


def test_two_pass_prefill_with_cached_prefix():
    # q_len < kv_len: the last 70 of 330 cached tokens attend
    from paper_2407_07304_b200 import harness
    w = _custom(1, 8, 2, [330], [0], 0, 900)
    oc = _oracle_cache(w)
    run = harness.LayerRun(w)
    run.append([330])
    out = run.prefill([w.q_prefill[0][260:]], two_pass=True)[0]
    want = so.attention(bf16_bits(w.q_prefill[0]), *oc[0], 330, w.sm_scale, sel=list(range(260, 330)))
    _assert_close(out, want, "two-pass prefill behind a cached prefix")


def test_two_pass_prefill_c3_full_sampled_rows():
    _check_two_pass(workloads.make_workload(3), prefill_rows=24)


def _check_full_row(w, tails=None, row_relative=False):
    """slim_attn_prefill_full_row (all scores of a row block on chip, one softmax, then .V) against the oracle;
    row_relative: error relative to each row's largest output (for inputs whose outputs span many binades)."""
    from paper_2407_07304_b200 import binding as slim, harness
    oc = _oracle_cache(w)
    run = harness.LayerRun(w)
    run.append(w.prefill_len)
    qs = w.q_prefill if tails is None else [w.q_prefill[b][w.prefill_len[b] - tails[b]:] for b in range(w.B)]
    out = run.prefill(qs, full_row=True)
    ref = run.prefill(qs)
    torch.cuda.synchronize()
    assert slim.slim_read_status(run.ws_prefill) == slim.SLIM_OK
    for b in range(w.B):
        n = w.prefill_len[b]
        sel = None if tails is None else list(range(n - tails[b], n))
        want = so.attention(bf16_bits(w.q_prefill[b]), *oc[b], n, w.sm_scale, sel=sel)
        if row_relative:
            got = out[b].float().cpu().numpy().astype(np.float64)
            denom = np.maximum(np.abs(want).max(axis=-1, keepdims=True), 1e-30)
            assert np.isfinite(got).all() and (np.abs(got - want) / denom).max() < 2e-2
            continue
        _assert_close(out[b], want, f"{w.name} full-row prefill seq {b}")
        if n > 0:
            d = (out[b].float() - ref[b].float()).abs().max().item()
            assert d <= 2 * MAX_ABS, f"{w.name} seq {b}: full-row and streamed outputs differ by {d}"


def test_full_row_prefill_c1_all_outputs():
    _check_full_row(workloads.make_workload(1))       # 256 tokens, 32 heads: every output


@pytest.mark.parametrize("lens", [[1], [2, 127], [128, 129], [255, 256, 31], [200, 1, 64, 130]])
def test_full_row_prefill_ragged_lengths(lens):
    B = len(lens)
    _check_full_row(_custom(B, 4, 2, lens, [0] * B, 0, 1700 + lens[0]))


def test_full_row_prefill_every_length_to_256():
    # every prompt length from 1 to 256 in batches of sixteen sequences, grouped-query heads (3 query heads per kv head)
    for first in range(1, 257, 16):
        lens = list(range(first, first + 16))
        _check_full_row(_custom(16, 3, 1, lens, [0] * 16, 0, 1800 + first))


def test_full_row_prefill_with_cached_prefix_and_scale_jump():
    # q_len < kv_len: the last 70 of 250 cached tokens attend ...
    _check_full_row(_custom(1, 8, 2, [250], [0], 0, 1900), tails=[70])
    # ... and with the second key tile's K 2^12 smaller and its V 2^9 larger than the first one's (each key tile is
    # normalised by its own power of two); the outputs span many binades, so the error is taken relative to the row
    w = _custom(1, 8, 2, [250], [0], 0, 1901)
    w.k[0][128:] *= 2.0 ** -12
    w.v[0][128:] *= 2.0 ** 9
    _check_full_row(w, tails=[70], row_relative=True)


def test_full_row_prefill_rejects_longer_caches():
    from paper_2407_07304_b200 import binding as slim, harness
    w = _custom(1, 2, 1, [300], [0], 0, 1950)
    run = harness.LayerRun(w)
    run.append([300])
    with pytest.raises(slim.SlimError) as e:
        run.prefill(w.q_prefill, full_row=True)
    assert e.value.code == slim.SLIM_ERR_UNSUPPORTED
    torch.cuda.synchronize()


def test_c5_full_sampled():
    _check(workloads.make_workload(5), prefill_rows=24, decode_steps={0, 31, 63})


# ---------------------------------------------------------------- decode spread over several ranks
@pytest.mark.parametrize("index,shrink,world", [(4, 8, 8), (4, 8, 2), (2, 8, 4), (5, 32, 8), (5, 32, 4), (5, 32, 2), (4, 1, 8), (5, 1, 8)])
def test_sharded_decode_every_rank_in_turn(index, shrink, world):
    # The ranks of a plan run one after the other on this GPU: every kernel reads only its own rank's cache (the rank's
    # kv heads, and in key-range mode its part of every sequence), and the exchange of the row partials, an all-gather
    # between GPUs, is a torch.stack here.  Workload 4: kv heads over ranks; workload 5 (2 kv heads): key ranges.
    from paper_2407_07304_b200.shard import ShardPlan, ShardedLayer
    w = workloads.make_workload(index, shrink=shrink)
    lens = [w.total_len(b) - w.decode_steps + 1 for b in range(w.B)]
    plan = ShardPlan(w.Hq, w.Hkv, lens, world)
    q = w.q_decode[0].cuda()
    out = torch.zeros_like(q)
    layers = [ShardedLayer(w, plan, r) for r in range(world)]
    for layer in layers:
        layer.fill()
    if plan.mode == "heads":
        for layer in layers:
            out[:, layer.shard.q_heads.start:layer.shard.q_heads.stop] = layer.decode(q)
    else:
        for head in range(w.Hkv):
            group = sorted((l for l in layers if layer_head(l) == head), key=lambda l: l.shard.part)
            sets = torch.stack([l.partial_step(q).clone() for l in group])
            res = group[0].finish(sets)
            out[:, group[0].shard.q_heads.start:group[0].shard.q_heads.stop] = res
    torch.cuda.synchronize()
    oc = _oracle_cache(w)
    rows = range(w.B) if shrink > 1 else range(min(w.B, 4))
    for b in rows:
        want = so.attention(bf16_bits(w.q_decode[0, b:b + 1]), *oc[b], lens[b], w.sm_scale)
        _assert_close(out[b:b + 1], want, f"{w.name} over {world} ranks, seq {b}")


def layer_head(layer):
    return layer.shard.kv_heads.start


# ---------------------------------------------------------------- edge cases
def _custom(B, Hq, Hkv, prefill, bulk, steps, seed):
    g = torch.Generator().manual_seed(seed)
    w = workloads.Workload(f"custom{seed}", 0, B, Hq, Hkv, prefill, bulk, steps)
    for b in range(B):
        T = w.total_len(b)
        w.k.append(torch.randn((T, Hkv, 128), generator=g).to(torch.bfloat16))
        w.v.append(torch.randn((T, Hkv, 128), generator=g).to(torch.bfloat16))
    if any(prefill):
        w.q_prefill = [torch.randn((n, Hq, 128), generator=g).to(torch.bfloat16) for n in prefill]
    if steps:
        w.q_decode = torch.randn((steps, B, Hq, 128), generator=g).to(torch.bfloat16)
    return w


@pytest.mark.parametrize("lens", [[1], [2, 127], [128, 129], [255, 256, 257], [1, 383, 640]])
def test_ragged_lengths_prefill_and_decode(lens):
    B = len(lens)
    _check(_custom(B, 4, 2, lens, [0] * B, 2, 100 + lens[0]))


@pytest.mark.parametrize("Hq,Hkv", [(1, 1), (8, 1), (16, 1), (12, 3), (6, 2), (4, 2), (10, 2), (7, 1), (9, 1), (13, 1), (30, 2)])
def test_group_sizes(Hq, Hkv):
    # 1, 2, 3, 4, 5, 7, 8 query heads per kv head (the eight-head kernel, some of its operand rows empty) and
    # 9, 13, 15, 16 (the sixteen-head kernel)
    _check(_custom(2, Hq, Hkv, [70, 200], [37, 0], 2, 200 + Hq))


def test_random_shapes_against_the_oracle():
    # sixty seeded random problems: batch 1..5, 1..8 kv heads, 1..16 query heads per kv head, prompt lengths at and
    # around the 128-token page and 256-token chunk boundaries, a bulk append, up to three decode steps (as
    # append + decode or as one call); every code, scale and output is compared
    import random
    rng = random.Random(20240707)
    for _ in range(60):
        B = rng.randint(1, 5)
        Hkv = rng.choice([1, 2, 3, 4, 8])
        G = rng.choice([1, 1, 2, 4, 8, 16])
        pre = [rng.choice([1, 2, 127, 128, 129, 255, 256, 257, 300, 511, 513, rng.randint(1, 1200)]) for _ in range(B)]
        bulk = [rng.choice([0, 0, 1, 130, rng.randint(0, 600)]) for _ in range(B)]
        steps = rng.choice([0, 1, 2, 3])
        one = steps > 0 and rng.random() < 0.5
        _check(_custom(B, Hkv * G, Hkv, pre, bulk, steps, rng.randint(0, 10 ** 6)), one_call_step=one)


@pytest.mark.parametrize("factor", [8.0, 64.0, 512.0])
@pytest.mark.parametrize("n_channels", [1, 4])
@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 1)])
def test_query_outlier_channels(factor, n_channels, Hq, Hkv):
    # Query rows with a few channels far above the rest (as trained models have): the other channels must keep
    # their precision.  The same channels of K are divided by the factor, so the scores stay of order one and the
    # softmax does not saturate (a saturated softmax would hide an inaccurate score).  Prefill of 299 and 2048
    # tokens, then decode steps at 300 / 2049 and 301 / 2050 cached tokens, and a batch of very short contexts
    # (1..6 tokens) where two or three keys share the weight and a score error shows undiluted.
    for lens, seed in (([299, 2048], 4100), ([1, 2, 3, 5], 4200)):
        B = len(lens)
        w = _custom(B, Hq, Hkv, lens, [0] * B, 2, seed + int(factor) + n_channels)
        ch = torch.randperm(128, generator=torch.Generator().manual_seed(seed))[:n_channels]
        for b in range(B):
            w.q_prefill[b][:, :, ch] = (w.q_prefill[b][:, :, ch].float() * factor).to(torch.bfloat16)
            w.k[b][:, :, ch] = (w.k[b][:, :, ch].float() / factor).to(torch.bfloat16)
        w.q_decode[:, :, :, ch] = (w.q_decode[:, :, :, ch].float() * factor).to(torch.bfloat16)
        _check(w)


@pytest.mark.parametrize("length", [8200, 12345, 20000, 40001, 66000])
def test_decode_long_rows_every_merge_kernel(length):
    # one sequence, two query heads on one kv head: 33 / 49 / 79 / 157 / 258 chunks per row, i.e. the block-per-row
    # merge with 4, 4, 8 and 16 warps and, past 256 chunks, the four-group kernel
    _check(_custom(1, 2, 1, [0], [length - 1], 1, 3000 + length))


def test_scale_extremes_and_zero_rows():
    # rows scaled far apart, zero K and V rows, and large-magnitude queries
    w = _custom(1, 2, 1, [150], [0], 2, 300)
    w.k[0][5] = 0
    w.v[0][7] = 0
    w.v[0][20:40] *= 2.0 ** -5
    w.v[0][60:70] *= 2.0 ** 6
    w.k[0][80:90] *= 2.0 ** -9
    w.q_prefill[0][100:110] *= 8.0
    w.q_decode[0] *= 2.0 ** -8
    oc = _oracle_cache(w)
    from paper_2407_07304_b200 import harness
    run, out_prefill, outs = harness.run_workload(w)
    _assert_cache_bits(run, oc)
    want = so.attention(bf16_bits(w.q_prefill[0]), *oc[0], 150, w.sm_scale)
    got = out_prefill[0].float().cpu().numpy().astype(np.float64)
    # outputs span 2^11: compare relative to each row's magnitude
    denom = np.maximum(np.abs(want).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - want) / denom).max() < 2e-2
    for s, o in outs.items():
        want = so.attention(bf16_bits(w.q_decode[s]), *oc[0], 151 + s, w.sm_scale)
        denom = np.maximum(np.abs(want).max(axis=-1, keepdims=True), 1e-30)
        assert (np.abs(o.float().cpu().numpy() - want) / denom).max() < 2e-2


def test_quantiser_significand_sweep_and_extreme_magnitudes():
    # codes and scales, bit for bit, on rows that sweep every significand of the largest element against every
    # significand of the others, 0..9 binades below it, at magnitudes from subnormal to 2^120 (the kernel rescales
    # rows outside [2^-60, 2^60]); three kv heads, so that a thread's rows change token in the middle of a block
    bits = mantissa_sweep_bits([-126, -120, -61, -60, 0, 60, 61, 120])
    n = bits.shape[0] // 3 * 3
    k = torch.from_numpy(bits[:n].view(np.int16).copy()).view(torch.bfloat16).reshape(n // 3, 3, 128)
    v = torch.flip(k, dims=[0]).contiguous()
    w = workloads.Workload("sweep", 0, 1, 3, 3, [0], [n // 3], 0)
    w.k.append(k)
    w.v.append(v)
    from paper_2407_07304_b200 import harness
    run = harness.LayerRun(w)
    run.append([n // 3])
    _assert_cache_bits(run, _oracle_cache(w))


def test_chunked_prefill_offset_and_shuffled_pages():
    # q_len < kv_len (the last 50 of 300 cached tokens attend) through a permuted block table
    from paper_2407_07304_b200 import harness
    w = _custom(2, 4, 2, [300, 140], [0, 0], 0, 400)
    pages = w.pages_per_seq()
    perm = torch.randperm(2 * pages + 3, generator=torch.Generator().manual_seed(1))[:2 * pages]
    bt = perm.to(torch.int32).view(2, pages)
    run = harness.LayerRun(w, block_table=bt, num_pages=2 * pages + 3)
    run.append(w.prefill_len)
    oc = _oracle_cache(w)
    _assert_cache_bits(run, oc)
    tails = [50, 140]
    outs = run.prefill([w.q_prefill[b][-tails[b]:] for b in range(2)])
    torch.cuda.synchronize()
    for b in range(2):
        want = so.attention(bf16_bits(w.q_prefill[b][-tails[b]:]), *oc[b], w.prefill_len[b], w.sm_scale)
        _assert_close(outs[b], want, f"chunked prefill seq {b}")


def test_prefill_step_fresh_prompts_and_behind_a_cached_prefix():
    # slim_prefill_step = slim_kv_append + slim_attn_prefill in one call: ragged prompts written and attended at once,
    # then a second call whose new tokens sit behind the first call's (chunked prefill through a permuted block table)
    from paper_2407_07304_b200 import binding as slim, harness
    w = _custom(3, 8, 2, [333, 70, 258], [0, 0, 0], 0, 4242)
    pages = w.pages_per_seq()
    perm = torch.randperm(3 * pages + 2, generator=torch.Generator().manual_seed(5))[:3 * pages]
    run = harness.LayerRun(w, block_table=perm.to(torch.int32).view(3, pages), num_pages=3 * pages + 2)
    oc = _oracle_cache(w)
    first = [200, 70, 129]
    outs = run.prefill_step(first, [w.q_prefill[b][:first[b]] for b in range(3)])
    torch.cuda.synchronize()
    _assert_cache_bits(run, oc)
    for b in range(3):
        want = so.attention(bf16_bits(w.q_prefill[b][:first[b]]), *oc[b], first[b], w.sm_scale)
        _assert_close(outs[b], want, f"prefill step, fresh prompt, seq {b}")
    rest = [w.prefill_len[b] - first[b] for b in range(3)]   # 133, 0, 129: the second sequence adds nothing
    outs = run.prefill_step(rest, [w.q_prefill[b][first[b]:] for b in range(3)])
    torch.cuda.synchronize()
    _assert_cache_bits(run, oc)
    for b in range(3):
        if rest[b] == 0:
            continue
        want = so.attention(bf16_bits(w.q_prefill[b][first[b]:]), *oc[b], w.prefill_len[b], w.sm_scale)
        _assert_close(outs[b], want, f"prefill step behind a prefix, seq {b}")
    assert slim.slim_read_status(run.ws_prefill) == slim.SLIM_OK


def test_prefill_step_random_prompts_in_two_parts_through_permuted_pages():
    # forty seeded random batches: every prompt is written and attended in two calls (either part may be empty, so a call
    # mixes fresh prompts, continued ones and sequences without new tokens), pages in a random order
    import random
    from paper_2407_07304_b200 import binding as slim, harness
    rng = random.Random(2407)
    for it in range(40):
        B = rng.choice([1, 2, 3, 4, 7])
        Hkv = rng.choice([1, 2, 4, 8])
        G = rng.choice([1, 2, 4, 8, 16])
        lens = [rng.choice([1, 2, 127, 128, 129, 255, 256, 257, 300, 511, 513, rng.randint(1, 1500)]) for _ in range(B)]
        w = _custom(B, Hkv * G, Hkv, lens, [0] * B, 0, rng.randint(0, 10 ** 6))
        pages = w.pages_per_seq()
        extra = rng.randint(0, 5)
        perm = torch.randperm(B * pages + extra, generator=torch.Generator().manual_seed(rng.randint(0, 10 ** 6)))[:B * pages]
        run = harness.LayerRun(w, block_table=perm.to(torch.int32).view(B, pages), num_pages=B * pages + extra)
        oc = _oracle_cache(w)
        first = [rng.choice([0, n, rng.randint(0, n)]) for n in lens]
        if sum(first) == 0:
            first[0] = lens[0]
        done = [0] * B
        for part in (first, [lens[b] - first[b] for b in range(B)]):
            if sum(part) == 0:
                continue
            outs = run.prefill_step(part, [w.q_prefill[b][done[b]:done[b] + part[b]] for b in range(B)])
            torch.cuda.synchronize()
            for b in range(B):
                if part[b] > 0:
                    want = so.attention(bf16_bits(w.q_prefill[b][done[b]:done[b] + part[b]]), *oc[b], done[b] + part[b], w.sm_scale)
                    _assert_close(outs[b], want, f"problem {it} seq {b}")
                    done[b] += part[b]
        _assert_cache_bits(run, oc)
        assert slim.slim_read_status(run.ws_prefill) == slim.SLIM_OK


def test_prefill_step_equals_append_then_prefill_bit_for_bit():
    from paper_2407_07304_b200 import harness
    w = workloads.make_workload(3, shrink=8)   # 1024 tokens, 32 heads
    a, b_ = harness.LayerRun(w), harness.LayerRun(w)
    a.append(w.prefill_len)
    want = a.prefill(w.q_prefill)
    got = b_.prefill_step(w.prefill_len, w.q_prefill)
    torch.cuda.synchronize()
    assert torch.equal(a.cache.codes, b_.cache.codes) and torch.equal(a.cache.scales, b_.cache.scales)
    for x, y in zip(got, want):
        assert torch.equal(x, y)


def test_prefill_step_c1_all_outputs():
    from paper_2407_07304_b200 import harness
    w = workloads.make_workload(1)
    run = harness.LayerRun(w)
    oc = _oracle_cache(w)
    outs = run.prefill_step(w.prefill_len, w.q_prefill)
    torch.cuda.synchronize()
    _assert_cache_bits(run, oc)
    for b in range(w.B):
        want = so.attention(bf16_bits(w.q_prefill[b]), *oc[b], w.prefill_len[b], w.sm_scale)
        _assert_close(outs[b], want, f"prefill step workload 1 seq {b}")


def test_empty_and_zero_length():
    from paper_2407_07304_b200 import binding as slim, harness
    w = _custom(2, 2, 1, [0, 0], [0, 5], 0, 500)
    run = harness.LayerRun(w)
    run.append([0, 5])
    q = torch.randn((2, 2, 128)).to(torch.bfloat16)
    out = run.decode(q)
    torch.cuda.synchronize()
    assert not out[0].any()            # kv_len 0 -> zeros
    oc = _oracle_cache(w)
    want = so.attention(bf16_bits(q[1:2]), *oc[1], 5, w.sm_scale)
    _assert_close(out[1:2], want, "short decode")
    # B == 0 and max_new == 0 are no-ops
    slim.slim_kv_append(run.cache, None, None, None, None, 0, 0)
    slim.slim_attn_decode(run.cache, None, None, None, 0, 0, 2, 1.0, run.ws_decode)


def test_bad_arguments_are_rejected_on_the_host():
    from paper_2407_07304_b200 import binding as slim, harness
    w = _custom(1, 4, 2, [0], [10], 0, 600)
    run = harness.LayerRun(w)
    q = torch.zeros((1, 4, 128), dtype=torch.bfloat16, device="cuda")
    kvl = torch.tensor([10], dtype=torch.int32, device="cuda")
    with pytest.raises(slim.SlimError) as e:
        slim.slim_attn_decode(run.cache, q, q.clone(), kvl, 1, 10, 3, 1.0, run.ws_decode)   # 3 % 2 != 0
    assert e.value.code == slim.SLIM_ERR_UNSUPPORTED
    with pytest.raises(slim.SlimError) as e:
        slim.slim_attn_decode(run.cache, q, q.clone(), kvl, 1, 10, 4, 1.0, None)
    assert e.value.code == slim.SLIM_ERR_WORKSPACE
    with pytest.raises(slim.SlimError) as e:
        slim.slim_attn_decode(run.cache, None, q, kvl, 1, 10, 4, 1.0, run.ws_decode)
    assert e.value.code == slim.SLIM_ERR_INVALID_ARG
    with pytest.raises(slim.SlimError) as e:
        slim.slim_attn_decode(run.cache, q, q.clone(), kvl, 1, 100000, 4, 1.0, run.ws_decode)  # beyond the page table
    assert e.value.code == slim.SLIM_ERR_INVALID_ARG
    # rows are read 16 bytes at a time: inputs that are only 8-byte aligned are refused, not read
    kn = torch.zeros((1 * 2 * 128 + 4,), dtype=torch.bfloat16, device="cuda")
    cu = torch.tensor([0, 1], dtype=torch.int32, device="cuda")
    pos = torch.tensor([10], dtype=torch.int32, device="cuda")
    with pytest.raises(slim.SlimError) as e:
        slim.slim_kv_append(run.cache, kn[4:], kn[:256], cu, pos, 1, 1)
    assert e.value.code == slim.SLIM_ERR_INVALID_ARG
    with pytest.raises(slim.SlimError) as e:
        slim.slim_prefill_step(run.cache, q, None, kn[:256], q.clone(), cu, kvl, 1, 1, 10, 4, 1.0, run.ws_prefill)
    assert e.value.code == slim.SLIM_ERR_INVALID_ARG
    with pytest.raises(slim.SlimError) as e:
        slim.slim_prefill_step(run.cache, q, kn[4:], kn[:256], q.clone(), cu, kvl, 1, 1, 10, 4, 1.0, run.ws_prefill)
    assert e.value.code == slim.SLIM_ERR_INVALID_ARG
    torch.cuda.synchronize()


# ---------------------------------------------------------------- more decode shapes and the host-step entry point
@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (16, 1)])
def test_decode_tail_lengths(Hq, Hkv):
    # lengths around every boundary of the streaming kernel: the 16-row boxes of a ragged tile, the
    # 128-token tile, the 256-token chunk; one and sixteen query heads per kv head (both consumer layouts)
    lens = [1, 15, 16, 17, 31, 127, 128, 129, 144, 255, 256, 257, 272, 383, 511, 513]
    B = len(lens)
    _check(_custom(B, Hq, Hkv, [0] * B, [n - 1 for n in lens], 1, 700 + Hq))


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (16, 1), (8, 2)])
def test_one_call_step_tail_lengths(Hq, Hkv):
    # the same boundaries with the new token written by the attention kernel itself; at length 1 and 2 the new
    # token carries most of the softmax weight, so a stale or missing row could not pass
    lens = [1, 2, 15, 16, 17, 31, 127, 128, 129, 144, 255, 256, 257, 272, 383, 511, 513]
    B = len(lens)
    w = _custom(B, Hq, Hkv, [0] * B, [n - 1 for n in lens], 3, 900 + Hq)
    _check(w, one_call_step=True)


def test_one_call_step_equals_append_then_decode_bit_for_bit():
    from paper_2407_07304_b200 import harness
    w = workloads.make_workload(4, shrink=8)
    a, _, outs_a = harness.run_workload(w)
    b, _, outs_b = harness.run_workload(w, one_call_step=True)
    for s_ in outs_a:
        assert torch.equal(outs_a[s_], outs_b[s_])
    assert torch.equal(a.cache.codes, b.cache.codes) and torch.equal(a.cache.scales, b.cache.scales)


def test_one_workspace_serves_calls_of_different_shapes():
    # the decode workspace's header (status word + the in-kernel merge's counters) is zeroed once; every call
    # leaves it at zero, so calls of other shapes can follow in the same workspace without zeroing it again
    from paper_2407_07304_b200 import binding as slim, harness
    shapes = [_custom(5, 4, 4, [0] * 5, [300, 511, 40, 700, 256], 2, 960),       # in-kernel merge, pairs shared between blocks
              _custom(2, 16, 1, [0] * 2, [9000, 100], 1, 961),                    # too many partials per pair: merge kernel
              _custom(40, 2, 2, [0] * 40, [(13 * i) % 90 + 1 for i in range(40)], 2, 962)]
    big = max(slim.slim_workspace_bytes(slim.PHASE_DECODE, w.B, w.Hq, w.Hkv, 1, max(w.total_len(b) for b in range(w.B)))
              for w in shapes)
    ws = torch.zeros(big, dtype=torch.uint8, device="cuda")
    for rounds in range(2):
        for w in shapes:
            run = harness.LayerRun(w)
            run.ws_decode = ws
            run.append(w.bulk_len)
            oc = _oracle_cache(w)
            for s_ in range(w.decode_steps):
                o = run.decode_step(w.q_decode[s_])
                for b in range(w.B):
                    want = so.attention(bf16_bits(w.q_decode[s_, b:b + 1]), *oc[b], w.bulk_len[b] + s_ + 1, w.sm_scale)
                    _assert_close(o[b:b + 1], want, f"{w.name} step {s_} seq {b}")
            torch.cuda.synchronize()
            assert not ws[:slim.WORKSPACE_HEADER_BYTES].any(), "the header is not back at zero"


def test_one_call_step_many_short_sequences():
    # more (sequence, kv head) pairs than thread blocks: every block quantises several new rows
    B = 300
    lens = [(7 * i) % 40 + 1 for i in range(B)]
    _check(_custom(B, 4, 2, [0] * B, [n - 1 for n in lens], 2, 950), one_call_step=True)


def test_more_pairs_than_the_split_kernel_counts():
    # 2100 sequences x 8 kv heads = 16800 (sequence, kv head) pairs: more than the 16384 counters of the split kernel's
    # own merge, so the merge kernel follows; lengths 1..40, two one-call steps
    B = 2100
    lens = [(11 * i) % 40 + 1 for i in range(B)]
    _check(_custom(B, 8, 8, [0] * B, [n - 1 for n in lens], 2, 951), one_call_step=True)


def test_status_words_stay_clear():
    from paper_2407_07304_b200 import binding as slim, harness
    w = workloads.make_workload(1, shrink=2)
    run, _, _ = harness.run_workload(w, decode_steps={0})
    assert slim.slim_read_status(run.ws_decode) == slim.SLIM_OK
    assert slim.slim_read_status(run.ws_prefill) == slim.SLIM_OK


@pytest.mark.parametrize("pinned_in,pinned_out", [(True, True), (True, False), (False, True), (False, False)])
def test_decode_step_from_host_buffers(pinned_in, pinned_out):
    # slim_decode_step_host: pinned inputs are read by the kernel where they are, ordinary host memory is copied into
    # the staging buffer first; the result is either written by the kernel into the pinned host buffer or, for
    # ordinary host memory, copied back through the staging buffer
    from paper_2407_07304_b200 import binding as slim, harness
    w = workloads.make_workload(4, shrink=16)
    run = harness.LayerRun(w)
    run.append(w.bulk_len)
    dev = run.device
    B, Hq, Hkv = w.B, w.Hq, w.Hkv
    ctx = list(run.pos)
    pin = (lambda t: t.pin_memory()) if pinned_in else (lambda t: t.clone())
    k_new = pin(torch.stack([w.k[b][ctx[b]] for b in range(B)]).contiguous())
    v_new = pin(torch.stack([w.v[b][ctx[b]] for b in range(B)]).contiguous())
    q = pin(w.q_decode[0].contiguous())
    out = torch.zeros_like(q).pin_memory() if pinned_out else torch.zeros(q.shape, dtype=q.dtype)
    staging = torch.empty(slim.slim_step_staging_bytes(B, Hq, Hkv), dtype=torch.uint8, device=dev)
    kv_len = torch.tensor(ctx, dtype=torch.int32, device=dev) + 1
    slim.slim_decode_step_host(run.cache, q, k_new, v_new, out, staging, kv_len, B, max(ctx) + 1, Hq,
                               w.sm_scale, run.ws_decode)
    torch.cuda.synchronize()
    run.pos = [c + 1 for c in ctx]
    oc = _oracle_cache(w)
    _assert_cache_bits(run, oc)
    for b in range(B):
        want = so.attention(bf16_bits(w.q_decode[0, b:b + 1]), *oc[b], ctx[b] + 1, w.sm_scale)
        _assert_close(out[b:b + 1], want, f"host step seq {b}")


def test_decode_step_replayed_from_a_graph():
    # the host-buffer step recorded by stream capture after one ordinary call; each replay reads the pinned
    # buffers as they are then, so a replay with the next token's inputs must equal the ordinary call on them
    from paper_2407_07304_b200 import binding as slim, harness
    w = workloads.make_workload(1)
    run = harness.LayerRun(w)
    run.append([w.total_len(b) - w.decode_steps for b in range(w.B)])
    dev = run.device
    B, Hq, Hkv = w.B, w.Hq, w.Hkv
    ctx = list(run.pos)
    k_new = torch.stack([w.k[b][ctx[b]] for b in range(B)]).contiguous().pin_memory()
    v_new = torch.stack([w.v[b][ctx[b]] for b in range(B)]).contiguous().pin_memory()
    q = w.q_decode[0].contiguous().pin_memory()
    out = torch.empty_like(q).pin_memory()
    staging = torch.empty(slim.slim_step_staging_bytes(B, Hq, Hkv), dtype=torch.uint8, device=dev)
    kv_len = torch.tensor(ctx, dtype=torch.int32, device=dev) + 1
    side = torch.cuda.Stream()

    def call():
        slim.slim_decode_step_host(run.cache, q, k_new, v_new, out, staging, kv_len, B, max(ctx) + 1,
                                   Hq, w.sm_scale, run.ws_decode, side)

    with torch.cuda.stream(side):
        call()
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
            call()
        # other inputs for the same cache slot: the replay must pick them up
        q.copy_(w.q_decode[1])
        k_new.mul_(-0.5), v_new.mul_(2.0)
        out.zero_()
        graph.replay()
        side.synchronize()
        replayed = out.clone()
        out.zero_()
        call()
        side.synchronize()
    assert torch.equal(replayed, out)
    assert replayed.float().abs().max() > 0
    assert slim.slim_read_status(run.ws_decode) == 0


def test_prefill_scale_jumps_between_key_tiles():
    # K and V magnitudes that differ by 2^18 from one 128-key tile to the next, in both directions: every key tile
    # is normalised by its own power of two, so none of them may overflow or vanish in the fp16 operands
    w = _custom(1, 2, 1, [512], [0], 0, 800)
    w.v[0][0:128] *= 2.0 ** -12
    w.v[0][128:256] *= 2.0 ** 6
    w.v[0][384:512] *= 2.0 ** -3
    w.k[0][256:384] *= 2.0 ** -10
    w.k[0][384:512] *= 2.0 ** 3
    oc = _oracle_cache(w)
    from paper_2407_07304_b200 import harness
    run, out_prefill, _ = harness.run_workload(w)
    _assert_cache_bits(run, oc)
    want = so.attention(bf16_bits(w.q_prefill[0]), *oc[0], 512, w.sm_scale)
    got = out_prefill[0].float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    denom = np.maximum(np.abs(want).max(axis=-1, keepdims=True), 1e-30)
    assert (np.abs(got - want) / denom).max() < 2e-2


def test_a_wait_that_runs_out_is_reported_not_hung():
    # the failure path of the bounded waits, exercised without any failure: a barrier nothing arrives on
    from paper_2407_07304_b200 import binding as slim, harness
    ws = torch.zeros(16, dtype=torch.uint8, device="cuda")
    assert slim.slim_read_status(ws) == slim.SLIM_OK
    slim.slim_selftest_timeout(ws)
    assert slim.slim_read_status(ws) == slim.SLIM_ERR_TIMEOUT
    ws.zero_()
    assert slim.slim_read_status(ws) == slim.SLIM_OK
    # the context is intact: a normal run still matches the oracle
    _check(_custom(1, 2, 1, [40], [0], 1, 900))
