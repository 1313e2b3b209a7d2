"""numpy front end of the CPU oracle (oracle/slim_oracle.c).  TEST INFRASTRUCTURE ONLY.

Nothing in the product imports this module; it is used by the tests, by the
smoke check and by the CPU-baseline leg of the benchmark.  It holds no
arithmetic of its own: every function marshals numpy arrays into the C
functions, which are the plain fp64 statement of the paper's method
(Section 2.1 SlimAttention, Section 2.2 INT8 KV cache, Eq. 1).

bf16 tensors cross this boundary as uint16 bit patterns.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slim_oracle.c")
_LIB = os.path.join(_HERE, "libslim_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with gcc (no fast-math, no contraction)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
           "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        P = ctypes.c_void_p
        lib.slim_oracle_quantize.argtypes = [P, ctypes.c_int64, ctypes.c_int32, P, P]
        lib.slim_oracle_quantize.restype = None
        lib.slim_oracle_attention.argtypes = [P, P, P, P, P] + [ctypes.c_int32] * 5 + \
            [ctypes.c_double, P, ctypes.c_int32, P]
        lib.slim_oracle_attention.restype = None
        lib.slim_oracle_partial.argtypes = [P, P, P, P, P] + [ctypes.c_int32] * 5 + \
            [ctypes.c_double, P, P, P]
        lib.slim_oracle_partial.restype = None
        lib.slim_oracle_merge.argtypes = [P, P, P, ctypes.c_int32, ctypes.c_int32, P]
        lib.slim_oracle_merge.restype = None
        lib.slim_oracle_kv_bytes.argtypes = [ctypes.c_double] * 7
        lib.slim_oracle_kv_bytes.restype = ctypes.c_double
        _lib = lib
    return _lib


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def quantize(x_bf16_bits):
    """x: uint16 [..., D] bf16 bit patterns -> (codes int8 [..., D], scales float32 [...])."""
    x = _c(x_bf16_bits, np.uint16)
    D = x.shape[-1]
    n = x.size // D if D else 0
    codes = np.empty(x.shape, dtype=np.int8)
    scales = np.empty(x.shape[:-1], dtype=np.float32)
    _load().slim_oracle_quantize(_ptr(x), n, D, _ptr(codes), _ptr(scales))
    return codes, scales


def attention(q_bits, k_codes, k_scales, v_codes, v_scales, kv_len, sm_scale, sel=None):
    """One sequence.  q uint16 [nq, Hq, D]; codes int8 [L, Hkv, D]; scales f32 [L, Hkv].

    Query t sees keys j <= kv_len - nq + t.  Returns float64 [n_sel or nq, Hq, D].
    """
    q = _c(q_bits, np.uint16)
    kc, vc = _c(k_codes, np.int8), _c(v_codes, np.int8)
    ks, vs = _c(k_scales, np.float32), _c(v_scales, np.float32)
    nq, Hq, D = q.shape
    L, Hkv, D2 = kc.shape
    assert D2 == D and vc.shape == kc.shape and ks.shape == (L, Hkv) and vs.shape == (L, Hkv)
    assert kv_len <= L and Hq % Hkv == 0
    if sel is None:
        sel_arr, n_sel, sel_p = None, nq, None
    else:
        sel_arr = _c(sel, np.int32)
        n_sel, sel_p = sel_arr.size, _ptr(sel_arr)
    out = np.empty((n_sel, Hq, D), dtype=np.float64)
    _load().slim_oracle_attention(_ptr(q), _ptr(kc), _ptr(ks), _ptr(vc), _ptr(vs),
                                  nq, int(kv_len), Hq, Hkv, D, float(sm_scale),
                                  sel_p, n_sel, _ptr(out))
    return out


def partial(q_row_bits, k_codes, k_scales, v_codes, v_scales, j0, j1, g, sm_scale):
    """(m, l, O[D]) of keys [j0, j1) of kv head g for one query row (uint16 [D])."""
    qr = _c(q_row_bits, np.uint16)
    kc, vc = _c(k_codes, np.int8), _c(v_codes, np.int8)
    ks, vs = _c(k_scales, np.float32), _c(v_scales, np.float32)
    L, Hkv, D = kc.shape
    m = ctypes.c_double()
    l = ctypes.c_double()
    O = np.empty(D, dtype=np.float64)
    _load().slim_oracle_partial(_ptr(qr), _ptr(kc), _ptr(ks), _ptr(vc), _ptr(vs),
                                int(j0), int(j1), int(g), Hkv, D, float(sm_scale),
                                ctypes.byref(m), ctypes.byref(l), _ptr(O))
    return m.value, l.value, O


def merge(m, l, O):
    """Log-sum-exp merge of n pieces: m [n], l [n], O [n, D] -> o [D]."""
    m, l, O = _c(m, np.float64), _c(l, np.float64), _c(O, np.float64)
    n, D = O.shape
    o = np.empty(D, dtype=np.float64)
    _load().slim_oracle_merge(_ptr(m), _ptr(l), _ptr(O), n, D, _ptr(o))
    return o


def kv_bytes(b, L_in, L_out, layers, n_head, s_head, s_d):
    """Eq. (1)."""
    return _load().slim_oracle_kv_bytes(b, L_in, L_out, layers, n_head, s_head, s_d)


def threads():
    """Number of OpenMP threads the C oracle will use."""
    n = os.environ.get("OMP_NUM_THREADS")
    return int(n) if n else (os.cpu_count() or 1)
