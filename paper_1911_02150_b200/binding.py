"""ctypes binding of ``libmqa_decode.so`` (the C ABI of ``include/mqa_decode.h``).

Argument marshalling only: every function here checks tensor dtypes/shapes, takes device
pointers and the current CUDA stream from PyTorch and calls the C entry point of the same
name.  All arithmetic of the decode step runs inside the library's CUDA kernels.  There is
no fallback: if the library is missing or was not built, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmqa_decode.so")

MQA_OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_STATIC_SCRATCH_TOO_SMALL = 1, 2, 3, 4, 5
NOALLOC_SCRATCH_BYTES = 8 * 1024 * 1024
STATUS_APPEND_CACHE_FULL, STATUS_APPEND_NEGATIVE_LEN, STATUS_LEN_CLAMPED, STATUS_PIPELINE_TIMEOUT = 1, 2, 4, 8

EXPORTS = (
    "kv_cache_append", "mqa_decode_step", "mha_decode_step",
    "mqa_decode_step_split", "mqa_decode_step_combine",
    "mha_decode_step_split", "mha_decode_step_combine",
    "mqa_workspace_bytes", "mqa_plan_splits", "mqa_plan_kernel_name", "mqa_set_wait_limit_cycles", "mqa_set_test_withhold_copy", "mqa_prefill_attention", "mqa_prefill_workspace_bytes", "mqa_status_string", "mqa_decode_step_noalloc",
    "mqa_decode_append_step", "mqa_append_step_launches",
    "mqa_layer_decode_step", "mqa_layer_workspace_bytes", "mqa_decode_local_step",
    "mqa_decode_append_step_host", "mqa_host_staging_bytes",
)

_lib = None


class MqaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (code {code})")


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1911_02150_b200.build` "
                "(the decode step has no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, I, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.kv_cache_append.argtypes = [vp, vp, vp, vp, vp, I, vp, I, I, I, I, I, vp]
        L.kv_cache_append.restype = I
        for n in ("mqa_decode_step", "mha_decode_step", "mqa_decode_step_split", "mha_decode_step_split"):
            f = getattr(L, n)
            f.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp, I, I, I, I, I, vp]
            f.restype = I
        for n in ("mqa_decode_step_combine", "mha_decode_step_combine"):
            f = getattr(L, n)
            f.argtypes = [vp, vp, vp, sz, I, I, I, I, I, vp]
            f.restype = I
        L.mqa_decode_step_noalloc.argtypes = [vp, vp, vp, vp, vp, vp, I, I, I, I, I, vp]
        L.mqa_decode_step_noalloc.restype = I
        L.mqa_decode_append_step.argtypes = [vp, vp, vp, vp, vp, vp, I, vp, vp, sz, vp, I, I, I, I, I, vp]
        L.mqa_decode_append_step.restype = I
        L.mqa_append_step_launches.argtypes = [I, I, I, I, I]
        L.mqa_append_step_launches.restype = I
        L.mqa_layer_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, I, vp, vp, sz, vp, I, I, I, I, I, I, vp]
        L.mqa_layer_decode_step.restype = I
        L.mqa_decode_local_step.argtypes = [vp, vp, vp, vp, vp, vp, I, vp, vp, I, I, I, I, I, vp]
        L.mqa_decode_local_step.restype = I
        L.mqa_decode_append_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, I, vp, sz, vp, sz, vp, I, I, I, I, I, vp]
        L.mqa_decode_append_step_host.restype = I
        L.mqa_host_staging_bytes.argtypes = [I, I, I, I]
        L.mqa_host_staging_bytes.restype = sz
        L.mqa_layer_workspace_bytes.argtypes = [I, I, I, I, I, I]
        L.mqa_layer_workspace_bytes.restype = sz
        L.mqa_workspace_bytes.argtypes = [I, I, I, I, I]
        L.mqa_workspace_bytes.restype = sz
        L.mqa_plan_splits.argtypes = [I, I, I, I, I, I, ctypes.POINTER(I)]
        L.mqa_plan_splits.restype = I
        L.mqa_plan_kernel_name.argtypes = [I, I, I, I, I, I, I]
        L.mqa_plan_kernel_name.restype = ctypes.c_char_p
        L.mqa_prefill_attention.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp, I, I, I, I, I, I, vp]
        L.mqa_prefill_attention.restype = I
        L.mqa_prefill_workspace_bytes.argtypes = [I, I, I, I, I, I]
        L.mqa_prefill_workspace_bytes.restype = sz
        L.mqa_set_wait_limit_cycles.argtypes = [ctypes.c_longlong]
        L.mqa_set_wait_limit_cycles.restype = I
        L.mqa_set_test_withhold_copy.argtypes = [I]
        L.mqa_set_test_withhold_copy.restype = I
        L.mqa_status_string.argtypes = [I]
        L.mqa_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().mqa_status_string(int(code)).decode()


def workspace_bytes(b: int, h: int, m_max: int, k: int = 128, v: int = 128) -> int:
    return int(lib().mqa_workspace_bytes(b, h, m_max, k, v))


def append_step_launches(b: int, h: int, m_max: int, k: int = 128, v: int = 128) -> int:
    """Kernel launches of one :func:`mqa_decode_append_step` call at these sizes ."""
    return int(lib().mqa_append_step_launches(b, h, m_max, k, v))


def plan_splits(multi_query: bool, b: int, h: int, m_max: int, k: int = 128, v: int = 128):
    """(n_splits, chunk_rows) the library will use for these sizes on the current device."""
    chunk = ctypes.c_int(0)
    n = lib().mqa_plan_splits(int(bool(multi_query)), b, h, m_max, k, v, ctypes.byref(chunk))
    return int(n), int(chunk.value)


def plan_kernel_name(multi_query: bool, whole_step: bool, b: int, h: int, m_max: int, k: int = 128, v: int = 128) -> str:
    """Name of the kernel that passes over the cache for these sizes (informational)."""
    return lib().mqa_plan_kernel_name(int(bool(multi_query)), int(bool(whole_step)), b, h, m_max, k, v).decode()


def alloc_workspace(b: int, h: int, m_max: int, device, k: int = 128, v: int = 128) -> torch.Tensor:
    """A byte tensor large enough for both step variants at these sizes (at least 16 bytes)."""
    with torch.cuda.device(device):
        n = workspace_bytes(b, h, m_max, k, v)
    return torch.empty(max(n, 16), dtype=torch.uint8, device=device)


class _OnDevice:
    """`with` block that makes a tensor's device current only when it is not already (the common case costs nothing)."""
    __slots__ = ("ctx",)

    def __init__(self, device):
        idx = device.index if device.index is not None else torch.cuda.current_device()
        self.ctx = None if idx == torch.cuda.current_device() else torch.cuda.device(idx)

    def __enter__(self):
        if self.ctx is not None:
            self.ctx.__enter__()

    def __exit__(self, *exc):
        if self.ctx is not None:
            self.ctx.__exit__(*exc)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _need(t: torch.Tensor, dtype, shape, name: str):
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must have shape {tuple(shape)}, got {tuple(t.shape)}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")


STEP_ADVANCE, STEP_CHAINED, STEP_TEST_WRONG_GUESS, STEP_TEST_WITHHOLD_COPY = 1, 2, 4, 8


def _step_flags(advance, chained, withhold_copy=False) -> int:
    """``chained``: False, True, or "wrong-guess" (the testing form of True); ``withhold_copy``: the testing flag that
    makes one bounded wait run out."""
    return ((STEP_ADVANCE if advance else 0) | (STEP_CHAINED if chained else 0) |
            (STEP_TEST_WRONG_GUESS if chained == "wrong-guess" else 0) | (STEP_TEST_WITHHOLD_COPY if withhold_copy else 0))


def set_test_withhold_copy(on: bool) -> None:
    """For tests: the batched form's kernel leaves one copy of its first CTA unstarted while this is on."""
    _check(lib().mqa_set_test_withhold_copy(1 if on else 0), "mqa_set_test_withhold_copy")


def set_wait_limit_cycles(cycles: int) -> None:
    """How long a kernel waits for one of its own on-chip copies before it flags PIPELINE_TIMEOUT and returns
    (SM clock cycles; <= 0 restores the default of about a second).  Synchronous."""
    _check(lib().mqa_set_wait_limit_cycles(int(cycles)), "mqa_set_wait_limit_cycles")


def _check(rc: int, where: str):
    if rc != MQA_OK:
        raise MqaError(rc, where)


def kv_cache_append(K, V, k_new, v_new, lens, advance: bool = True, status=None, stream=None) -> None:
    """Write the new token's rows into row ``lens[b]`` of the cache, in place.

    ``K``/``V``: ``[b,m_max,128]`` (multi-query) or ``[b,kv_heads,m_max,128]`` (multi-head) bf16;
    ``k_new``/``v_new``: ``[b,128]`` or ``[b,kv_heads,128]``; ``lens``: int32 ``[b]``, advanced by one
    on the device when ``advance``."""
    if K.dim() == 3:
        b, m_max, k = K.shape
        kvh = 1
        new_shape = (b, k)
    else:
        b, kvh, m_max, k = K.shape
        new_shape = (b, kvh, k)
    v = V.shape[-1]
    _need(K, torch.bfloat16, K.shape, "K")
    _need(V, torch.bfloat16, tuple(K.shape[:-1]) + (v,), "V")
    _need(k_new, torch.bfloat16, new_shape, "k_new")
    _need(v_new, torch.bfloat16, new_shape[:-1] + (v,), "v_new")
    _need(lens, torch.int32, (b,), "lens")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    with _OnDevice(K.device):
        rc = lib().kv_cache_append(_ptr(K), _ptr(V), _ptr(k_new), _ptr(v_new), _ptr(lens), int(bool(advance)),
                                   _ptr(status), b, kvh, m_max, k, v, _stream(stream))
    _check(rc, "kv_cache_append")


def _step(name: str, multi_query: bool, q, K, V, lens, o, workspace, status, stream, phase: str):
    b, h, k = q.shape
    m_max, v = K.shape[-2], V.shape[-1]
    cache = (b, m_max) if multi_query else (b, h, m_max)
    _need(q, torch.bfloat16, (b, h, k), "q")
    _need(K, torch.bfloat16, cache + (k,), "K")
    _need(V, torch.bfloat16, cache + (v,), "V")
    _need(lens, torch.int32, (b,), "lens")
    _need(o, torch.float32, (b, h, v), "o")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (_ptr(workspace), workspace.numel() * workspace.element_size())
    with _OnDevice(q.device):
        if phase == "combine":
            rc = getattr(lib(), name)(_ptr(lens), _ptr(o), ws_ptr, ws_bytes, b, h, m_max, k, v, _stream(stream))
        else:
            rc = getattr(lib(), name)(_ptr(q), _ptr(K), _ptr(V), _ptr(lens), _ptr(o), ws_ptr, ws_bytes,
                                      _ptr(status), b, h, m_max, k, v, _stream(stream))
    _check(rc, name)
    return o


def mqa_decode_step(q, K, V, lens, o, workspace=None, status=None, stream=None):
    """Multi-query step: ``q[b,h,128]`` over the shared ``K[b,m_max,128]``, ``V[b,m_max,128]`` (bf16),
    first ``lens[b]`` rows -> ``o[b,h,128]`` fp32 (written in place and returned)."""
    return _step("mqa_decode_step", True, q, K, V, lens, o, workspace, status, stream, "step")


def mha_decode_step(q, K, V, lens, o, workspace=None, status=None, stream=None):
    """Multi-head step: as above with per-head caches ``K[b,h,m_max,128]``, ``V[b,h,m_max,128]``."""
    return _step("mha_decode_step", False, q, K, V, lens, o, workspace, status, stream, "step")


def mqa_decode_step_split(q, K, V, lens, o, workspace=None, status=None, stream=None):
    return _step("mqa_decode_step_split", True, q, K, V, lens, o, workspace, status, stream, "split")


def mha_decode_step_split(q, K, V, lens, o, workspace=None, status=None, stream=None):
    return _step("mha_decode_step_split", False, q, K, V, lens, o, workspace, status, stream, "split")


def mqa_decode_step_combine(q, K, V, lens, o, workspace=None, status=None, stream=None):
    return _step("mqa_decode_step_combine", True, q, K, V, lens, o, workspace, status, stream, "combine")


def mha_decode_step_combine(q, K, V, lens, o, workspace=None, status=None, stream=None):
    return _step("mha_decode_step_combine", False, q, K, V, lens, o, workspace, status, stream, "combine")


def mqa_decode_step_noalloc(q, K, V, lens, o, status=None, stream=None):
    """The multi-query step for callers that cannot allocate a workspace (a plugin inside a host
    framework that planned and reserved all device memory up front): same arguments as
    :func:`mqa_decode_step` minus the workspace; the scratch is a fixed array inside the library.

    Make the first call on each device during set-up (it looks up the array's address).  All
    calls on a device share that one array, so calls whose kernels could overlap on the GPU must
    not be issued concurrently.  Raises ``MqaError`` with ``ERR_STATIC_SCRATCH_TOO_SMALL`` when the
    sizes need more than ``NOALLOC_SCRATCH_BYTES`` of scratch."""
    b, h, k = q.shape
    m_max, v = K.shape[-2], V.shape[-1]
    _need(q, torch.bfloat16, (b, h, k), "q")
    _need(K, torch.bfloat16, (b, m_max, k), "K")
    _need(V, torch.bfloat16, (b, m_max, v), "V")
    _need(lens, torch.int32, (b,), "lens")
    _need(o, torch.float32, (b, h, v), "o")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    with _OnDevice(q.device):
        rc = lib().mqa_decode_step_noalloc(_ptr(q), _ptr(K), _ptr(V), _ptr(lens), _ptr(o), _ptr(status),
                                           b, h, m_max, k, v, _stream(stream))
    _check(rc, "mqa_decode_step_noalloc")
    return o


def _append_step_args(q, K, V, k_new, v_new, lens, o, workspace, status, advance, stream, chained, withhold_copy=False):
    """Checks the tensors of the append-and-attend step and returns the C call's argument tuple (plain integers)."""
    b, h, k = q.shape
    m_max, v = K.shape[-2], V.shape[-1]
    _need(q, torch.bfloat16, (b, h, k), "q")
    _need(K, torch.bfloat16, (b, m_max, k), "K")
    _need(V, torch.bfloat16, (b, m_max, v), "V")
    _need(k_new, torch.bfloat16, (b, k), "k_new")
    _need(v_new, torch.bfloat16, (b, v), "v_new")
    _need(lens, torch.int32, (b,), "lens")
    _need(o, torch.float32, (b, h, v), "o")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    s = torch.cuda.current_stream(q.device) if stream is None else stream
    return (q.data_ptr(), K.data_ptr(), V.data_ptr(), k_new.data_ptr(), v_new.data_ptr(), lens.data_ptr(),
            _step_flags(advance, chained, withhold_copy), o.data_ptr(), None if workspace is None else workspace.data_ptr(),
            0 if workspace is None else workspace.numel() * workspace.element_size(),
            None if status is None else status.data_ptr(), b, h, m_max, k, v, s.cuda_stream)


def mqa_decode_append_step(q, K, V, k_new, v_new, lens, o, workspace=None, status=None, advance: bool = True, stream=None,
                           chained: bool = False, withhold_copy: bool = False):
    """One whole multi-query decoding step in one call: append ``k_new``/``v_new`` at row ``lens[b]`` of the
    shared cache, then attend over ``lens[b] + 1`` rows; ``lens`` is advanced on the device when ``advance``.
    For batches the persistent kernel serves (h <= 64) the whole step is one kernel launch.  ``chained``: the
    caller's promise that nothing enqueued on the stream since this library's last step on this cache writes
    the cache, ``lens`` or the workspace (a decoding loop); the kernel then starts on the cache before the
    kernel ahead of it has finished."""
    args = _append_step_args(q, K, V, k_new, v_new, lens, o, workspace, status, advance, stream, chained, withhold_copy)
    with _OnDevice(q.device):
        rc = lib().mqa_decode_append_step(*args)
    _check(rc, "mqa_decode_append_step")
    return o


def _as_c_args(fn, args):
    """The argument tuple as instances of the function's declared ctypes types, made once: a call then converts nothing
    (about a microsecond for the twenty arguments of a step)."""
    return tuple(t(a) for t, a in zip(fn.argtypes, args))


class AppendStep:
    """:func:`mqa_decode_append_step` bound once to its tensors: a decoding loop refills the same q, k_new and v_new
    buffers for every token, so the checks and the pointer marshalling (about 20 us of Python per call, several times
    a short step) are done here and each call is the C call alone.  The tensors are kept alive by this object; the
    stream is the one current (or given) at construction, and the cache's device must be current when it is called."""
    __slots__ = ("fn", "args", "keep", "o")

    def __init__(self, q, K, V, k_new, v_new, lens, o, workspace=None, status=None, advance: bool = True, stream=None,
                 chained: bool = False):
        self.args = _append_step_args(q, K, V, k_new, v_new, lens, o, workspace, status, advance, stream, chained)
        self.keep = (q, K, V, k_new, v_new, lens, o, workspace, status, stream)
        self.fn = lib().mqa_decode_append_step
        self.args = _as_c_args(self.fn, self.args)
        self.o = o

    def __call__(self, stream=None):
        """``stream``: another stream than the bound one for this call (a stream that is capturing a graph, say)."""
        rc = self.fn(*self.args) if stream is None else self.fn(*self.args[:-1], stream.cuda_stream)
        if rc != MQA_OK:
            raise MqaError(rc, "mqa_decode_append_step")
        return self.o


def layer_workspace_bytes(b: int, h: int, d: int, m_max: int, k: int = 128, v: int = 128) -> int:
    return int(lib().mqa_layer_workspace_bytes(b, h, d, m_max, k, v))


def alloc_layer_workspace(b: int, h: int, d: int, m_max: int, device) -> torch.Tensor:
    return torch.empty(max(16, layer_workspace_bytes(b, h, d, m_max)), dtype=torch.uint8, device=device)


def mqa_layer_decode_step(x, P_q, P_k, P_v, P_o, K, V, lens, y, workspace, status=None, advance: bool = True, stream=None):
    """The whole incremental multi-query layer step: projections of ``x[b,d]`` to q, k_new, v_new, append +
    attention over the shared cache, output projection to ``y[b,d]`` (fp32)."""
    b, d = x.shape
    h, _, k = P_q.shape
    m_max, v = K.shape[-2], V.shape[-1]
    _need(x, torch.bfloat16, (b, d), "x")
    _need(P_q, torch.bfloat16, (h, d, k), "P_q")
    _need(P_k, torch.bfloat16, (d, k), "P_k")
    _need(P_v, torch.bfloat16, (d, v), "P_v")
    _need(P_o, torch.bfloat16, (h, d, v), "P_o")
    _need(K, torch.bfloat16, (b, m_max, k), "K")
    _need(V, torch.bfloat16, (b, m_max, v), "V")
    _need(lens, torch.int32, (b,), "lens")
    _need(y, torch.float32, (b, d), "y")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    with _OnDevice(x.device):
        rc = lib().mqa_layer_decode_step(_ptr(x), _ptr(P_q), _ptr(P_k), _ptr(P_v), _ptr(P_o), _ptr(K), _ptr(V), _ptr(lens),
                                         int(bool(advance)), _ptr(y), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _ptr(status),
                                         b, h, d, m_max, k, v, _stream(stream))
    _check(rc, "mqa_layer_decode_step")
    return y


def mqa_decode_local_step(q, K, V, k_new, v_new, pos, o, status=None, advance: bool = True, stream=None):
    """One decoding step of local multi-query attention: ``K``/``V`` ``[b, window, 128]`` are rings of the last
    ``window`` positions, ``pos[b]`` counts the tokens so far; the new row goes to row ``pos % window``."""
    b, h, k = q.shape
    window, v = K.shape[-2], V.shape[-1]
    _need(q, torch.bfloat16, (b, h, k), "q")
    _need(K, torch.bfloat16, (b, window, k), "K")
    _need(V, torch.bfloat16, (b, window, v), "V")
    _need(k_new, torch.bfloat16, (b, k), "k_new")
    _need(v_new, torch.bfloat16, (b, v), "v_new")
    _need(pos, torch.int32, (b,), "pos")
    _need(o, torch.float32, (b, h, v), "o")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    with _OnDevice(q.device):
        rc = lib().mqa_decode_local_step(_ptr(q), _ptr(K), _ptr(V), _ptr(k_new), _ptr(v_new), _ptr(pos), int(bool(advance)),
                                         _ptr(o), _ptr(status), b, h, window, k, v, _stream(stream))
    _check(rc, "mqa_decode_local_step")
    return o


def prefill_workspace_bytes(b: int, h: int, n: int, m_max: int, k: int = 128, v: int = 128) -> int:
    return int(lib().mqa_prefill_workspace_bytes(b, h, n, m_max, k, v))


def mqa_prefill_attention(Q, K, V, O, workspace, start=None, status=None, stream=None):
    """The attention lines of the batched multi-query function under the autoregressive mask: ``Q[b,h,n,k]`` bf16 over
    the shared ``K[b,m_max,k]``, ``V[b,m_max,v]``; query t of sequence b is memory position ``start[b] + t`` (``start``
    None: zeros) and attends over the rows up to its own; ``O[b,h,n,v]`` fp32 is written."""
    b, h, n, k = Q.shape
    m_max, v = K.shape[-2], V.shape[-1]
    _need(Q, torch.bfloat16, (b, h, n, k), "Q")
    _need(K, torch.bfloat16, (b, m_max, k), "K")
    _need(V, torch.bfloat16, (b, m_max, v), "V")
    _need(O, torch.float32, (b, h, n, v), "O")
    if start is not None:
        _need(start, torch.int32, (b,), "start")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    s = torch.cuda.current_stream(Q.device) if stream is None else stream
    with _OnDevice(Q.device):
        rc = lib().mqa_prefill_attention(Q.data_ptr(), K.data_ptr(), V.data_ptr(), None if start is None else start.data_ptr(),
                                         O.data_ptr(), workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                         None if status is None else status.data_ptr(), b, h, n, m_max, k, v, s.cuda_stream)
    _check(rc, "mqa_prefill_attention")
    return O


def host_staging_bytes(b: int, h: int, k: int = 128, v: int = 128) -> int:
    return int(lib().mqa_host_staging_bytes(b, h, k, v))


def _host_step_args(q_host, k_new_host, v_new_host, o_host, K, V, lens, staging, workspace, status, advance, stream, chained=False):
    """Checks the tensors of the host-buffer step and returns the C call's argument tuple (plain integers)."""
    b, h, k = q_host.shape
    m_max, v = K.shape[-2], V.shape[-1]
    for t, dt, shape, name in ((q_host, torch.bfloat16, (b, h, k), "q_host"), (k_new_host, torch.bfloat16, (b, k), "k_new_host"),
                               (v_new_host, torch.bfloat16, (b, v), "v_new_host"), (o_host, torch.float32, (b, h, v), "o_host")):
        if t.is_cuda or t.dtype != dt or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError(f"{name}: want a contiguous CPU tensor {dt} {shape}")
    _need(K, torch.bfloat16, (b, m_max, k), "K")
    _need(V, torch.bfloat16, (b, m_max, v), "V")
    _need(lens, torch.int32, (b,), "lens")
    if status is not None:
        _need(status, torch.int32, (1,), "status")
    s = torch.cuda.current_stream(K.device) if stream is None else stream
    return (q_host.data_ptr(), k_new_host.data_ptr(), v_new_host.data_ptr(), o_host.data_ptr(), K.data_ptr(), V.data_ptr(),
            lens.data_ptr(), _step_flags(advance, chained), staging.data_ptr(), staging.numel() * staging.element_size(),
            None if workspace is None else workspace.data_ptr(), 0 if workspace is None else workspace.numel() * workspace.element_size(),
            None if status is None else status.data_ptr(), b, h, m_max, k, v, s.cuda_stream)


def mqa_decode_append_step_host(q_host, k_new_host, v_new_host, o_host, K, V, lens, staging, workspace=None, status=None,
                                advance: bool = True, stream=None, chained: bool = False):
    """:func:`mqa_decode_append_step` with the per-token inputs and the result in host memory (CPU tensors, pinned for
    asynchronous copies); ``staging`` is a device uint8 tensor of ``host_staging_bytes(b, h)`` bytes.  Nothing is
    synchronised: wait on the stream before reading ``o_host``."""
    args = _host_step_args(q_host, k_new_host, v_new_host, o_host, K, V, lens, staging, workspace, status, advance, stream, chained)
    with _OnDevice(K.device):
        rc = lib().mqa_decode_append_step_host(*args)
    _check(rc, "mqa_decode_append_step_host")
    return o_host


class HostStep:
    """The host-buffer decoding step bound once to its buffers: a decoding loop refills the same pinned tensors for
    every token, so the checks and the pointer marshalling are done here and each call is the C call alone.  The
    tensors are kept alive by this object; the stream is the one current (or given) at construction, and the cache's
    device must be current when the step is called."""
    __slots__ = ("fn", "args", "keep", "o_host")

    def __init__(self, q_host, k_new_host, v_new_host, o_host, K, V, lens, staging, workspace=None, status=None,
                 advance: bool = True, stream=None, chained: bool = False):
        self.args = _host_step_args(q_host, k_new_host, v_new_host, o_host, K, V, lens, staging, workspace, status, advance, stream,
                                    chained)
        self.keep = (q_host, k_new_host, v_new_host, o_host, K, V, lens, staging, workspace, status, stream)
        self.fn = lib().mqa_decode_append_step_host
        self.args = _as_c_args(self.fn, self.args)
        self.o_host = o_host

    def __call__(self, stream=None):
        """``stream``: another stream than the bound one for this call."""
        rc = self.fn(*self.args) if stream is None else self.fn(*self.args[:-1], stream.cuda_stream)
        if rc != MQA_OK:
            raise MqaError(rc, "mqa_decode_append_step_host")
        return self.o_host
