"""The C-ABI library loads on a machine without a GPU and exports everything include/slim.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "slim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slim_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2407_07304_b200 import build as slim_build, binding
    path = slim_build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"slim_kv_append", "slim_attn_prefill", "slim_attn_decode"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in slim.h but not exported"
    assert set(binding.EXPORTS) <= set(names)


def test_host_only_entry_points():
    from paper_2407_07304_b200 import binding as slim
    assert slim.slim_version() >= 100
    L = slim.lib()
    assert L.slim_strerror(0) == b"ok" and L.slim_strerror(-3).startswith(b"workspace")
    # pool sizes: Eq. (1) with s_d = 1 for one layer, plus two fp32 scales per token and head
    assert L.slim_cache_code_bytes(17 * 16, 32) == 2 * 17 * 16 * 128 * 32 * 128
    assert L.slim_cache_scale_bytes(17 * 16, 32) == 2 * 17 * 16 * 128 * 32 * 4
    assert slim.slim_workspace_bytes(slim.PHASE_DECODE, 16, 32, 32, 1, 2049) > 0
    assert slim.slim_workspace_bytes(slim.PHASE_DECODE, 0, 32, 32, 1, 2049) == 0


def test_invalid_cache_is_rejected_before_any_launch():
    from paper_2407_07304_b200 import binding as slim
    st = slim.SlimCacheStruct(None, None, None, 1, 128, 1, 128, 1)
    rc = slim.lib().slim_kv_append(ctypes.byref(st), None, None, None, None, 1, 1, None)
    assert rc == slim.SLIM_ERR_INVALID_ARG
    st = slim.SlimCacheStruct(16, 16, 16, 1, 64, 1, 128, 1)      # page_tokens 64 is not supported
    rc = slim.lib().slim_kv_append(ctypes.byref(st), None, None, None, None, 1, 1, None)
    assert rc == slim.SLIM_ERR_UNSUPPORTED
