"""slim_attn_decode_static: the decode entry point for callers that cannot allocate.

A caller inside a stream capture, or one living in a runtime that owns all device memory,
has no way to provide the workspace slim_attn_decode asks for.  The static variant keeps the
split pass's partials in an 8 MiB array built into the library.  These tests call it through
the C ABI twice in a row (the array keeps the first call's contents, so the second call shows
that stale partials do no harm) and compare each result with slim_attn_decode's and with the
CPU oracle, on a shape the split kernel merges itself and on one that takes the separate merge
kernel.  The file runs last so that a failure here cannot hide the other GPU tests.
"""
import numpy as np
import pytest
import torch

from helpers import MAX_ABS, MEAN_ABS, output_bound

pytestmark = pytest.mark.gpu


def _bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _oracle_rows(w, lens, q):
    """fp64 oracle decode outputs [B, Hq, 128] for query rows q (bf16 [B, Hq, 128]) at the given lengths."""
    from oracle import slim_oracle as so
    rows = []
    for b in range(w.B):
        kc, ks = so.quantize(_bits(w.k[b]))
        vc, vs = so.quantize(_bits(w.v[b]))
        rows.append(so.attention(_bits(q[b:b + 1]), kc, ks, vc, vs, int(lens[b]), w.sm_scale))
    return np.concatenate(rows)


def _close(got, want, what):
    err = np.abs(got.float().cpu().numpy().astype(np.float64) - want)
    assert torch.isfinite(got.float()).all(), what
    assert (err <= output_bound(want)).all() and err.mean() <= MEAN_ABS, f"{what}: {err.max():.3e} / {err.mean():.3e}"


def _setup(w):
    from paper_2407_07304_b200 import harness
    run = harness.LayerRun(w)
    run.append(w.bulk_len)
    run.append([1] * w.B)
    return run


def _custom(B, Hq, Hkv, bulk, seed):
    from paper_2407_07304_b200 import workloads
    g = torch.Generator().manual_seed(seed)
    w = workloads.Workload(f"static{seed}", 0, B, Hq, Hkv, [0] * B, bulk, 1)
    for b in range(B):
        w.k.append(torch.randn((bulk[b] + 1, Hkv, 128), generator=g).to(torch.bfloat16))
        w.v.append(torch.randn((bulk[b] + 1, Hkv, 128), generator=g).to(torch.bfloat16))
    w.q_decode = torch.randn((1, B, Hq, 128), generator=g).to(torch.bfloat16)
    return w


def _two_calls(w, what):
    """A long call, then a shorter one with other queries: fewer partial slots are written the second time than
    the array still holds.  Each result against slim_attn_decode and against the oracle."""
    from paper_2407_07304_b200 import binding as slim
    run = _setup(w)
    dev = run.device
    kv_len = torch.tensor(run.pos, dtype=torch.int32, device=dev)
    cases = [(w.q_decode[0], kv_len), (-w.q_decode[0], torch.clamp(kv_len // 2, min=1))]
    for n, (q_cpu, lens) in enumerate(cases):
        q = q_cpu.to(dev).contiguous()
        max_kv = int(lens.max().item())
        want, got = torch.empty_like(q), torch.empty_like(q)
        slim.slim_attn_decode(run.cache, q, want, lens, w.B, max_kv, w.Hq, w.sm_scale, run.ws_decode)
        slim.slim_attn_decode_static(run.cache, q, got, lens, w.B, max_kv, w.Hq, w.sm_scale)
        torch.cuda.synchronize()
        assert slim.slim_static_status() == slim.SLIM_OK
        # the two entry points run the same kernels on the same inputs
        assert torch.equal(got, want), f"{what} call {n}: differs from slim_attn_decode"
        _close(got, _oracle_rows(w, lens.cpu().tolist(), q_cpu), f"{what} call {n} vs oracle")


def test_static_scratch_matches_workspace_variant_and_oracle_twice():
    # grouped-query shape with ragged lengths 128..512: the split kernel merges its own partials
    from paper_2407_07304_b200 import workloads
    _two_calls(workloads.make_workload(4, shrink=8), "in-kernel merge")


def test_static_scratch_through_the_merge_kernel():
    # sixteen query heads on one kv head, 9001 and 101 tokens: too many partials per (sequence, kv head) for the
    # split kernel's own merge, so the merge kernel reads the partials back from the built-in array (0.6 MB of it)
    _two_calls(_custom(2, 16, 1, [9000, 100], 77), "merge kernel")


def test_static_scratch_rejects_oversized_problem():
    from paper_2407_07304_b200 import binding as slim, workloads
    w = workloads.make_workload(4, shrink=8)
    run = _setup(w)
    dev = run.device
    # a shape whose partials exceed the built-in array: 512 sequences x 64 heads x many chunks
    B, Hq, Hkv, max_kv = 512, 64, 8, 4096
    assert slim.slim_workspace_bytes(slim.PHASE_DECODE, B, Hq, Hkv, 1, max_kv) > slim.STATIC_SCRATCH_BYTES
    big = slim.SlimCacheStruct(run.cache.codes.data_ptr(), run.cache.scales.data_ptr(),
                               run.cache.block_table.data_ptr(), run.cache.num_pages, 128, Hkv, 128, 32)

    class Fake:
        struct = big
    q = torch.zeros((B, Hq, 128), dtype=torch.bfloat16, device=dev)
    kvl = torch.zeros((B,), dtype=torch.int32, device=dev)
    with pytest.raises(slim.SlimError) as e:
        slim.slim_attn_decode_static(Fake, q, torch.empty_like(q), kvl, B, max_kv, Hq, 1.0)
    assert e.value.code == slim.SLIM_ERR_WORKSPACE
    torch.cuda.synchronize()


def test_static_scratch_status_and_reset():
    # the failure path of the bounded waits on the built-in array, exercised without any failure: a wait that
    # nothing answers raises the array's status word; the reset clears the header; decode is correct again
    from paper_2407_07304_b200 import binding as slim, workloads
    assert slim.slim_static_status() == slim.SLIM_OK
    slim.slim_static_selftest_timeout()
    assert slim.slim_static_status() == slim.SLIM_ERR_TIMEOUT
    slim.slim_static_reset()
    assert slim.slim_static_status() == slim.SLIM_OK
    _two_calls(workloads.make_workload(4, shrink=16), "after reset")
