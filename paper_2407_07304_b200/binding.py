"""ctypes binding of libslim.so: the same entry points as include/slim.h.

Argument marshalling only.  torch supplies device memory and streams; every
step of the attention path runs in the library's CUDA kernels.  There is no
fallback: if the library has not been built the first call raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libslim.so")

SLIM_OK = 0
SLIM_ERR_INVALID_ARG = -1
SLIM_ERR_UNSUPPORTED = -2
SLIM_ERR_WORKSPACE = -3
SLIM_ERR_CUDA = -4
SLIM_ERR_TIMEOUT = -5
PHASE_PREFILL = 0
PHASE_DECODE = 1
HEAD_DIM = 128
PAGE_TOKENS = 128

EXPORTS = (
    "slim_kv_append", "slim_attn_prefill", "slim_prefill_step", "slim_attn_prefill_two_pass", "slim_attn_prefill_full_row", "slim_attn_decode", "slim_attn_decode_split",
    "slim_attn_decode_merge", "slim_attn_decode_static", "slim_static_status", "slim_static_reset",
    "slim_static_selftest_timeout", "slim_attn_decode_partial", "slim_attn_merge_partials", "slim_decode_step", "slim_decode_step_host", "slim_step_staging_bytes", "slim_read_status", "slim_selftest_timeout", "slim_workspace_bytes",
    "slim_cache_code_bytes", "slim_cache_scale_bytes", "slim_strerror", "slim_last_cuda_error",
    "slim_version",
)


class SlimCacheStruct(ctypes.Structure):
    """Mirror of slim_cache_t."""
    _fields_ = [
        ("codes", ctypes.c_void_p),
        ("scales", ctypes.c_void_p),
        ("block_table", ctypes.c_void_p),
        ("num_pages", ctypes.c_int32),
        ("page_tokens", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("max_pages_per_seq", ctypes.c_int32),
    ]


class SlimError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = lib().slim_strerror(code).decode()
        if code == SLIM_ERR_CUDA:
            msg += f" (cudaError {lib().slim_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")


_lib = None


def lib():
    """The loaded library; raises if libslim.so has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2407_07304_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        P, I, F, Z = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float, ctypes.c_size_t
        CP = ctypes.POINTER(SlimCacheStruct)
        L.slim_kv_append.argtypes = [CP, P, P, P, P, I, I, P]
        L.slim_kv_append.restype = ctypes.c_int
        L.slim_attn_prefill.argtypes = [CP, P, P, P, P, I, I, I, I, F, P, Z, P]
        L.slim_attn_prefill.restype = ctypes.c_int
        L.slim_prefill_step.argtypes = [CP, P, P, P, P, P, P, I, I, I, I, F, P, Z, P]
        L.slim_prefill_step.restype = ctypes.c_int
        L.slim_attn_prefill_two_pass.argtypes = [CP, P, P, P, P, I, I, I, I, F, P, Z, P]
        L.slim_attn_prefill_two_pass.restype = ctypes.c_int
        L.slim_attn_prefill_full_row.argtypes = [CP, P, P, P, P, I, I, I, I, F, P, Z, P]
        L.slim_attn_prefill_full_row.restype = ctypes.c_int
        L.slim_attn_decode.argtypes = [CP, P, P, P, I, I, I, F, P, Z, P]
        L.slim_attn_decode.restype = ctypes.c_int
        L.slim_attn_decode_split.argtypes = [CP, P, P, P, P, I, I, I, F, P, Z, P]
        L.slim_attn_decode_split.restype = ctypes.c_int
        L.slim_attn_decode_merge.argtypes = [CP, P, P, I, I, I, P, Z, P]
        L.slim_attn_decode_merge.restype = ctypes.c_int
        L.slim_attn_decode_static.argtypes = [CP, P, P, P, I, I, I, F, P]
        L.slim_attn_decode_static.restype = ctypes.c_int
        for name in ("slim_static_status", "slim_static_reset", "slim_static_selftest_timeout"):
            getattr(L, name).argtypes = [P]
            getattr(L, name).restype = ctypes.c_int
        L.slim_attn_decode_partial.argtypes = [CP, P, P, P, I, I, I, F, P, Z, P]
        L.slim_attn_decode_partial.restype = ctypes.c_int
        L.slim_attn_merge_partials.argtypes = [P, I, P, I, I, P]
        L.slim_attn_merge_partials.restype = ctypes.c_int
        L.slim_decode_step.argtypes = [CP, P, P, P, P, P, I, I, I, F, P, Z, P]
        L.slim_decode_step.restype = ctypes.c_int
        L.slim_decode_step_host.argtypes = [CP, P, P, P, P, P, Z, P, I, I, I, F, P, Z, P]
        L.slim_decode_step_host.restype = ctypes.c_int
        L.slim_step_staging_bytes.argtypes = [I, I, I]
        L.slim_step_staging_bytes.restype = Z
        L.slim_read_status.argtypes = [P, P]
        L.slim_read_status.restype = ctypes.c_int
        L.slim_selftest_timeout.argtypes = [P, P]
        L.slim_selftest_timeout.restype = ctypes.c_int
        L.slim_workspace_bytes.argtypes = [I, I, I, I, I, I]
        L.slim_workspace_bytes.restype = Z
        L.slim_cache_code_bytes.argtypes = [I, I]
        L.slim_cache_code_bytes.restype = Z
        L.slim_cache_scale_bytes.argtypes = [I, I]
        L.slim_cache_scale_bytes.restype = Z
        L.slim_strerror.argtypes = [ctypes.c_int]
        L.slim_strerror.restype = ctypes.c_char_p
        L.slim_last_cuda_error.argtypes = []
        L.slim_last_cuda_error.restype = ctypes.c_int
        L.slim_version.argtypes = []
        L.slim_version.restype = ctypes.c_int
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _nbytes(t):
    return 0 if t is None else t.numel() * t.element_size()


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(rc, where):
    if rc != SLIM_OK:
        raise SlimError(rc, where)


class SlimCache:
    """Device memory of one layer's paged INT8 KV cache plus its slim_cache_t.

    Pages are handed to sequences in order: sequence b owns pages
    [b * max_pages_per_seq, (b + 1) * max_pages_per_seq) unless a block table is given.
    """

    def __init__(self, B, num_kv_heads, max_pages_per_seq, device="cuda", block_table=None, num_pages=None):
        self.B, self.Hkv, self.max_pages_per_seq = B, num_kv_heads, max_pages_per_seq
        self.num_pages = num_pages if num_pages is not None else B * max_pages_per_seq
        L = lib()
        self.codes = torch.zeros(L.slim_cache_code_bytes(self.num_pages, num_kv_heads), dtype=torch.int8, device=device)
        self.scales = torch.zeros(L.slim_cache_scale_bytes(self.num_pages, num_kv_heads) // 4, dtype=torch.float32,
                                  device=device)
        if block_table is None:
            block_table = torch.arange(B * max_pages_per_seq, dtype=torch.int32).view(B, max_pages_per_seq)
        self.block_table = block_table.to(device=device, dtype=torch.int32).contiguous()
        self.struct = SlimCacheStruct(self.codes.data_ptr(), self.scales.data_ptr(), self.block_table.data_ptr(),
                                      self.num_pages, PAGE_TOKENS, num_kv_heads, HEAD_DIM, max_pages_per_seq)

    def codes_view(self):
        """int8 [num_pages, Hkv, 2, 128, 128]"""
        return self.codes.view(self.num_pages, self.Hkv, 2, PAGE_TOKENS, HEAD_DIM)

    def scales_view(self):
        """fp32 [num_pages, Hkv, 2, 128]"""
        return self.scales.view(self.num_pages, self.Hkv, 2, PAGE_TOKENS)


def slim_kv_append(cache, k_new, v_new, cu_new, start_pos, B, max_new, stream=None):
    rc = lib().slim_kv_append(ctypes.byref(cache.struct), _ptr(k_new), _ptr(v_new), _ptr(cu_new), _ptr(start_pos),
                              B, max_new, _stream(stream))
    _check(rc, "slim_kv_append")


def slim_attn_prefill(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, sm_scale, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().slim_attn_prefill(ctypes.byref(cache.struct), _ptr(q), _ptr(out), _ptr(cu_q), _ptr(kv_len),
                                 B, max_q, max_kv, Hq, sm_scale, _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "slim_attn_prefill")


def slim_prefill_step(cache, q, k_new, v_new, out, cu_q, kv_len, B, max_q, max_kv, Hq, sm_scale, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().slim_prefill_step(ctypes.byref(cache.struct), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(cu_q), _ptr(kv_len),
                                 B, max_q, max_kv, Hq, sm_scale, _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "slim_prefill_step")


def slim_attn_prefill_two_pass(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, sm_scale, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().slim_attn_prefill_two_pass(ctypes.byref(cache.struct), _ptr(q), _ptr(out), _ptr(cu_q), _ptr(kv_len),
                                          B, max_q, max_kv, Hq, sm_scale, _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "slim_attn_prefill_two_pass")


FULL_ROW_MAX_KEYS = 256


def slim_attn_prefill_full_row(cache, q, out, cu_q, kv_len, B, max_q, max_kv, Hq, sm_scale, workspace=None, stream=None):
    """Prefill with the whole score row on chip (caches of at most FULL_ROW_MAX_KEYS tokens)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().slim_attn_prefill_full_row(ctypes.byref(cache.struct), _ptr(q), _ptr(out), _ptr(cu_q), _ptr(kv_len),
                                          B, max_q, max_kv, Hq, sm_scale, _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "slim_attn_prefill_full_row")


def slim_attn_decode(cache, q, out, kv_len, B, max_kv, Hq, sm_scale, workspace, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().slim_attn_decode(ctypes.byref(cache.struct), _ptr(q), _ptr(out), _ptr(kv_len), B, max_kv, Hq,
                                sm_scale, _ptr(workspace), ws_bytes, _stream(stream))
    _check(rc, "slim_attn_decode")


def slim_attn_decode_split(cache, q, kv_len, B, max_kv, Hq, sm_scale, workspace, stream=None, k_new=None, v_new=None):
    rc = lib().slim_attn_decode_split(ctypes.byref(cache.struct), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(kv_len), B, max_kv,
                                      Hq, sm_scale, _ptr(workspace), _nbytes(workspace), _stream(stream))
    _check(rc, "slim_attn_decode_split")


def slim_attn_decode_merge(cache, out, kv_len, B, max_kv, Hq, workspace, stream=None):
    rc = lib().slim_attn_decode_merge(ctypes.byref(cache.struct), _ptr(out), _ptr(kv_len), B, max_kv, Hq,
                                      _ptr(workspace), _nbytes(workspace), _stream(stream))
    _check(rc, "slim_attn_decode_merge")


STATIC_SCRATCH_BYTES = 8 * 1024 * 1024
WORKSPACE_HEADER_BYTES = 16 + 16384 * 4   # zero at first use (SLIM_WORKSPACE_HEADER_BYTES)


def slim_attn_decode_static(cache, q, out, kv_len, B, max_kv, Hq, sm_scale, stream=None):
    """slim_attn_decode without a workspace argument: partials go to the library's built-in
    8 MiB device array, for callers that may not allocate.  Calls sharing a device must not
    overlap on the GPU."""
    rc = lib().slim_attn_decode_static(ctypes.byref(cache.struct), _ptr(q), _ptr(out), _ptr(kv_len), B, max_kv, Hq,
                                       sm_scale, _stream(stream))
    _check(rc, "slim_attn_decode_static")


PARTIAL_FLOATS = 132   # fp32 per (sequence, query head) row of slim_attn_decode_partial: O[128], M, l, padding


def slim_attn_decode_partial(cache, q, partial, kv_len, B, max_kv, Hq, sm_scale, workspace, stream=None):
    """slim_attn_decode over the part of the keys this device holds, without the final normalisation:
    partial fp32 [B, Hq, PARTIAL_FLOATS] receives every row's merged (O, M, l)."""
    rc = lib().slim_attn_decode_partial(ctypes.byref(cache.struct), _ptr(q), _ptr(partial), _ptr(kv_len), B, max_kv, Hq,
                                        sm_scale, _ptr(workspace), _nbytes(workspace), _stream(stream))
    _check(rc, "slim_attn_decode_partial")


def slim_attn_merge_partials(partials, n_sets, out, B, Hq, stream=None):
    """Final merge of n_sets sets of row partials (fp32 [n_sets, B, Hq, PARTIAL_FLOATS]) into bf16 out [B, Hq, 128]."""
    _check(lib().slim_attn_merge_partials(_ptr(partials), n_sets, _ptr(out), B, Hq, _stream(stream)), "slim_attn_merge_partials")


def slim_static_status(stream=None):
    """slim_read_status for the built-in array of slim_attn_decode_static."""
    return lib().slim_static_status(_stream(stream))


def slim_static_reset(stream=None):
    """Clears the built-in array's header (needed after a SLIM_ERR_TIMEOUT); allocates nothing."""
    _check(lib().slim_static_reset(_stream(stream)), "slim_static_reset")


def slim_static_selftest_timeout(stream=None):
    """slim_selftest_timeout aimed at the built-in array's status word."""
    _check(lib().slim_static_selftest_timeout(_stream(stream)), "slim_static_selftest_timeout")


def slim_decode_step(cache, q, k_new, v_new, out, kv_len, B, max_kv, Hq, sm_scale, workspace, stream=None):
    """Appends one token per sequence at position kv_len - 1 and attends over kv_len tokens, in one kernel."""
    rc = lib().slim_decode_step(ctypes.byref(cache.struct), _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(kv_len),
                                B, max_kv, Hq, sm_scale, _ptr(workspace), _nbytes(workspace), _stream(stream))
    _check(rc, "slim_decode_step")


def slim_decode_step_host(cache, q_host, k_new_host, v_new_host, out_host, staging, kv_len, B, max_kv, Hq, sm_scale,
                          workspace, stream=None):
    """q_host / k_new_host / v_new_host / out_host are CPU (pinned) bf16 tensors."""
    rc = lib().slim_decode_step_host(ctypes.byref(cache.struct), _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host),
                                     _ptr(out_host), _ptr(staging), _nbytes(staging), _ptr(kv_len), B, max_kv, Hq,
                                     sm_scale, _ptr(workspace), _nbytes(workspace), _stream(stream))
    _check(rc, "slim_decode_step_host")


def slim_read_status(workspace, stream=None):
    """Synchronises the stream and returns SLIM_OK or SLIM_ERR_TIMEOUT (a bounded device-side wait ran out)."""
    return lib().slim_read_status(_ptr(workspace), _stream(stream))


def slim_selftest_timeout(workspace, stream=None):
    """Makes a bounded device-side wait run out on purpose (nothing faults); the status word of `workspace` is set."""
    _check(lib().slim_selftest_timeout(_ptr(workspace), _stream(stream)), "slim_selftest_timeout")


def slim_step_staging_bytes(B, Hq, Hkv):
    return lib().slim_step_staging_bytes(B, Hq, Hkv)


def slim_workspace_bytes(phase, B, Hq, Hkv, max_q, max_kv):
    return lib().slim_workspace_bytes(phase, B, Hq, Hkv, max_q, max_kv)


def slim_version():
    return lib().slim_version()


def workspace(phase, B, Hq, Hkv, max_q, max_kv, device="cuda"):
    """A torch uint8 buffer of the size the phase needs (at least 16 bytes)."""
    n = max(16, slim_workspace_bytes(phase, B, Hq, Hkv, max_q, max_kv))
    return torch.zeros(n, dtype=torch.uint8, device=device)
