"""TEST INFRASTRUCTURE -- not part of the product path.

Python face of the fp64 CPU oracle for the decode-attention hot path of multi-query
attention (arXiv 1911.02150).  Two independent restatements live here:

* ``attention_oracle.c`` -- the bf16-boundary step functions (multi-query step of
  Section 3, multi-head step of Section 2.4, the cache append, the single-query
  attention of Section 2.1, and the attention lines of the batched multi-query function
  of Section 3 under the autoregressive mask of Section 2.3), loaded through ``ctypes``;
* ``paper_functions.py`` -- the paper's five layer functions *with* their projections,
  in numpy fp64, used by the pins that need the projections (incremental == causal).

Only ``tests/``, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` / reference legs of
``bench.py`` may import this package.  It imports nothing from the CUDA package.
Every function is pinned in ``tests/test_oracle_pins.py``; nothing is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "attention_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``attention_oracle.c`` with gcc (OpenMP) into ``liboracle.so`` beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        i32p = ctypes.POINTER(ctypes.c_int32)
        f64p = ctypes.POINTER(ctypes.c_double)
        I = ctypes.c_int
        lib.oracle_dot_product_attention.argtypes = [f64p, f64p, f64p, f64p, I, I, I]
        lib.oracle_dot_product_attention.restype = I
        for name in ("oracle_mqa_decode_step", "oracle_mha_decode_step"):
            fn = getattr(lib, name)
            fn.argtypes = [u16p, u16p, u16p, i32p, f64p, I, I, I, I, I]
            fn.restype = I
        lib.oracle_mqa_batched_attention.argtypes = [u16p, u16p, u16p, i32p, f64p, I, I, I, I, I, I]
        lib.oracle_mqa_batched_attention.restype = I
        lib.oracle_kv_cache_append.argtypes = [u16p, u16p, u16p, u16p, i32p, I, I, I, I, I, I]
        lib.oracle_kv_cache_append.restype = I
        lib.oracle_num_threads.restype = I
        lib.oracle_set_num_threads.argtypes = [I]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _u16(a, shape) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 tensors are passed to the oracle as uint16 bit patterns")
    if tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {tuple(shape)}, got {tuple(a.shape)}")
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def dot_product_attention(q, K, V) -> np.ndarray:
    """Section 2.1: one query ``q[k]`` over ``K[m,k]``, ``V[m,v]`` -> ``y[v]`` (fp64)."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    m, k = K.shape
    v = V.shape[1]
    assert q.shape == (k,) and V.shape[0] == m and m >= 1
    y = np.empty(v, dtype=np.float64)
    rc = _load().oracle_dot_product_attention(
        _ptr(q, ctypes.c_double), _ptr(K, ctypes.c_double), _ptr(V, ctypes.c_double),
        _ptr(y, ctypes.c_double), m, k, v)
    if rc:
        raise MemoryError("oracle scratch allocation failed")
    return y


def _decode(fn_name, q, K, V, lens, kv_heads_of):
    q = np.ascontiguousarray(q)
    b, h, k = q.shape
    kvh = kv_heads_of(h)
    K = np.ascontiguousarray(K)
    V = np.ascontiguousarray(V)
    m_max = K.shape[-2]
    v = V.shape[-1]
    kshape = (b, m_max, k) if kvh == 1 and K.ndim == 3 else (b, kvh, m_max, k)
    vshape = kshape[:-1] + (v,)
    q = _u16(q, (b, h, k))
    K = _u16(K, kshape)
    V = _u16(V, vshape)
    lens = np.ascontiguousarray(lens, dtype=np.int32)
    assert lens.shape == (b,)
    o = np.empty((b, h, v), dtype=np.float64)
    rc = getattr(_load(), fn_name)(
        _ptr(q, ctypes.c_uint16), _ptr(K, ctypes.c_uint16), _ptr(V, ctypes.c_uint16),
        _ptr(lens, ctypes.c_int32), _ptr(o, ctypes.c_double), b, h, m_max, k, v)
    if rc:
        raise MemoryError("oracle scratch allocation failed")
    return o


def mqa_decode_step(q, K, V, lens) -> np.ndarray:
    """Section 3 step: ``q[b,h,k]``, shared ``K[b,m_max,k]``, ``V[b,m_max,v]`` (uint16 bf16
    bits), ``lens[b]`` valid rows -> ``o[b,h,v]`` fp64."""
    if np.ndim(K) != 3:
        raise ValueError("the multi-query cache has no heads axis: K is [b, m_max, k]")
    return _decode("oracle_mqa_decode_step", q, K, V, lens, lambda h: 1)


def mha_decode_step(q, K, V, lens) -> np.ndarray:
    """Section 2.4 step: ``q[b,h,k]``, per-head ``K[b,h,m_max,k]``, ``V[b,h,m_max,v]``
    (uint16 bf16 bits), ``lens[b]`` -> ``o[b,h,v]`` fp64."""
    if np.ndim(K) != 4:
        raise ValueError("the multi-head cache is [b, h, m_max, k]")
    return _decode("oracle_mha_decode_step", q, K, V, lens, lambda h: h)


def mqa_batched_attention(Q, K, V, start=None) -> np.ndarray:
    """Section 3, the attention lines of the batched multi-query function under the autoregressive mask of
    Section 2.3: ``Q[b,h,n,k]``, shared ``K[b,m_max,k]``, ``V[b,m_max,v]`` (uint16 bf16 bits) -> ``O[b,h,n,v]`` fp64.
    Query position t of sequence b is memory position ``start[b] + t`` and may look at positions up to its own
    (``start`` None: zeros, the memory is the n positions of the queries themselves)."""
    Q = np.ascontiguousarray(Q)
    b, h, n, k = Q.shape
    K = np.ascontiguousarray(K)
    V = np.ascontiguousarray(V)
    m_max, v = K.shape[-2], V.shape[-1]
    Q = _u16(Q, (b, h, n, k))
    K = _u16(K, (b, m_max, k))
    V = _u16(V, (b, m_max, v))
    st = None
    if start is not None:
        st = np.ascontiguousarray(start, dtype=np.int32)
        assert st.shape == (b,)
    O = np.empty((b, h, n, v), dtype=np.float64)
    rc = _load().oracle_mqa_batched_attention(
        _ptr(Q, ctypes.c_uint16), _ptr(K, ctypes.c_uint16), _ptr(V, ctypes.c_uint16),
        None if st is None else _ptr(st, ctypes.c_int32), _ptr(O, ctypes.c_double), b, h, n, m_max, k, v)
    if rc == 2:
        raise ValueError("start[b] + n must lie within [n, m_max]")
    if rc:
        raise MemoryError("oracle scratch allocation failed")
    return O


def kv_cache_append(K, V, k_new, v_new, lens, advance: bool = True) -> int:
    """In-place append of one row per (sequence, cache head) at row ``lens[b]``.

    ``K``/``V`` are writable C-contiguous uint16 arrays ``[b,m_max,k]`` (multi-query) or
    ``[b,kv_heads,m_max,k]`` (multi-head); ``k_new``/``v_new`` are ``[b,k]`` or
    ``[b,kv_heads,k]``; ``lens`` is a writable int32 array.  Returns how many sequences
    were skipped because ``lens[b]`` was outside ``[0, m_max)``."""
    for a in (K, V, lens):
        if not (isinstance(a, np.ndarray) and a.flags.c_contiguous and a.flags.writeable):
            raise TypeError("K, V and lens must be writable C-contiguous numpy arrays")
    if K.dtype != np.uint16 or V.dtype != np.uint16 or lens.dtype != np.int32:
        raise TypeError("K, V are uint16 bf16 bit patterns and lens is int32")
    if K.ndim == 3:
        b, m_max, k = K.shape
        kvh = 1
    else:
        b, kvh, m_max, k = K.shape
    v = V.shape[-1]
    k_new = _u16(np.asarray(k_new).reshape(b, kvh, k), (b, kvh, k))
    v_new = _u16(np.asarray(v_new).reshape(b, kvh, v), (b, kvh, v))
    return int(_load().oracle_kv_cache_append(
        _ptr(K, ctypes.c_uint16), _ptr(V, ctypes.c_uint16),
        _ptr(k_new, ctypes.c_uint16), _ptr(v_new, ctypes.c_uint16),
        _ptr(lens, ctypes.c_int32), int(bool(advance)), b, kvh, m_max, k, v))
