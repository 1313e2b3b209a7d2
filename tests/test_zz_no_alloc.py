"""slim_attn_decode_static: the decode entry point for callers that cannot allocate.

A caller inside a stream capture, or one living in a runtime that owns all device memory,
has no way to provide the workspace slim_attn_decode asks for.  The static variant keeps the
split pass's partials in an 8 MiB array built into the library.  This test calls it through
the C ABI twice in a row (the array keeps the first call's contents, so the second call shows
that stale partials do no harm) and compares each result with slim_attn_decode's.
It runs last so that a failure here cannot hide the other GPU tests.
"""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _setup():
    from paper_2407_07304_b200 import harness, workloads
    w = workloads.make_workload(4, shrink=8)        # GQA, ragged lengths 128..512, 32 sequences
    run = harness.LayerRun(w)
    run.append(w.bulk_len)
    run.append([1] * w.B)
    return w, run


def test_static_scratch_matches_workspace_variant_twice():
    from paper_2407_07304_b200 import binding as slim
    w, run = _setup()
    dev = run.device
    kv_len = torch.tensor(run.pos, dtype=torch.int32, device=dev)
    max_kv = max(run.pos)
    # first call: all sequences at full length
    q1 = w.q_decode[0].to(dev).contiguous()
    want1 = torch.empty_like(q1)
    got1 = torch.empty_like(q1)
    slim.slim_attn_decode(run.cache, q1, want1, kv_len, w.B, max_kv, w.Hq, w.sm_scale, run.ws_decode)
    slim.slim_attn_decode_static(run.cache, q1, got1, kv_len, w.B, max_kv, w.Hq, w.sm_scale)
    # second call: other queries and shorter lengths, so fewer partial slots are written than the array still holds
    q2 = (-w.q_decode[0]).to(dev).contiguous()
    kv_len2 = torch.clamp(kv_len // 2, min=1)
    max_kv2 = int(kv_len2.max().item())
    want2 = torch.empty_like(q2)
    got2 = torch.empty_like(q2)
    slim.slim_attn_decode(run.cache, q2, want2, kv_len2, w.B, max_kv2, w.Hq, w.sm_scale, run.ws_decode)
    slim.slim_attn_decode_static(run.cache, q2, got2, kv_len2, w.B, max_kv2, w.Hq, w.sm_scale)
    torch.cuda.synchronize()
    for got, want in ((got1, want1), (got2, want2)):
        err = (got.float() - want.float()).abs()
        assert torch.isfinite(got.float()).all()
        assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3


def test_static_scratch_rejects_oversized_problem():
    from paper_2407_07304_b200 import binding as slim
    w, run = _setup()
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
