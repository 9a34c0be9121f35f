"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, answers its host-only calls, and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

from paper_1911_02150_b200 import binding
from paper_1911_02150_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build_library()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mqa_decode.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"^\s*#.*$", "", text, flags=re.M)          # preprocessor lines
    return sorted(set(re.findall(r"\b(\w+)\s*\([^;{}]*\)\s*;", text)))


def test_header_and_binding_agree(L):
    names = declared_functions()
    assert "mqa_decode_step" in names and "mha_decode_step" in names and "kv_cache_append" in names
    assert sorted(binding.EXPORTS) == names
    for n in names:
        assert hasattr(L, n), f"{n} is declared in include/mqa_decode.h but not exported"


def test_header_constants_and_binding_agree():
    text = open(os.path.join(ROOT, "include", "mqa_decode.h")).read()
    defines = {m.group(1): int(m.group(2), 0) for m in re.finditer(r"^#define\s+(MQA_\w+)\s+\(?(\d+|0x[0-9a-fA-F]+)u?\)?\s*$", text, flags=re.M)}
    assert defines["MQA_STEP_ADVANCE"] == binding.STEP_ADVANCE == 1
    assert defines["MQA_STEP_CHAINED"] == binding.STEP_CHAINED == 2
    assert defines["MQA_STEP_TEST_WRONG_GUESS"] == binding.STEP_TEST_WRONG_GUESS == 4
    assert binding._step_flags(True, False) == 1 and binding._step_flags(False, True) == 2
    assert binding._step_flags(True, "wrong-guess") == 7
    assert defines["MQA_STEP_TEST_WITHHOLD_COPY"] == binding.STEP_TEST_WITHHOLD_COPY == 8
    assert binding._step_flags(False, False, True) == 8


def test_step_flags_are_checked_before_any_launch(L):
    vp = ctypes.c_void_p
    a = vp(0x1000)
    # an unknown flag bit: refused on the host, nothing dereferenced
    rc = L.mqa_decode_append_step(a, a, a, a, a, a, 16, a, a, 1 << 30, None, 4, 8, 256, 128, 128, None)
    assert rc == binding.ERR_INVALID_ARG


def test_status_strings(L):
    seen = {binding.status_string(c) for c in range(0, 5)}
    assert len(seen) == 5
    assert "unknown" in binding.status_string(99)


def test_plan_and_workspace_are_consistent(L):
    for mq in (True, False):
        for (b, h, m) in [(1, 8, 128), (128, 8, 128), (32, 32, 8192), (256, 16, 2048), (1, 16, 32768), (256, 16, 32768)]:
            n, chunk = binding.plan_splits(mq, b, h, m)
            assert n >= 1 and chunk >= 1
            need = binding.workspace_bytes(b, h, m)
            if n > 1:
                assert need >= h * n * (128 + 2) * 4
    assert binding.workspace_bytes(0, 8, 128) == 0
    assert binding.workspace_bytes(1, 8, 128, k=64, v=64) == 0
    assert binding.plan_splits(True, 1, 8, 0) == (0, 0)


def test_bad_arguments_are_rejected_before_any_launch(L):
    vp = ctypes.c_void_p
    a = vp(0x1000)          # plausible, 16-byte aligned, never dereferenced on the host
    odd = vp(0x1004)
    step = L.mqa_decode_step
    ok_tail = (1, 8, 128, 128, 128, None)
    assert step(None, a, a, a, a, None, 0, None, *ok_tail) == binding.ERR_INVALID_ARG
    assert step(a, a, a, a, None, None, 0, None, *ok_tail) == binding.ERR_INVALID_ARG
    assert step(odd, a, a, a, a, None, 0, None, *ok_tail) == binding.ERR_INVALID_ARG
    assert step(a, a, odd, a, a, None, 0, None, *ok_tail) == binding.ERR_INVALID_ARG
    assert step(a, a, a, a, a, None, 0, None, 0, 8, 128, 128, 128, None) == binding.ERR_INVALID_ARG
    assert step(a, a, a, a, a, None, 0, None, 1, 8, -5, 128, 128, None) == binding.ERR_INVALID_ARG
    assert step(a, a, a, a, a, None, 0, None, 1, 8, 128, 64, 128, None) == binding.ERR_UNSUPPORTED
    assert L.mha_decode_step(a, a, a, a, a, None, 0, None, 1, 8, 128, 128, 96, None) == binding.ERR_UNSUPPORTED
    # a plan with several splits needs a workspace of the advertised size
    n, _ = binding.plan_splits(True, 1, 16, 32768)
    assert n > 1
    need = binding.workspace_bytes(1, 16, 32768)
    big = (1, 16, 32768, 128, 128, None)
    assert step(a, a, a, a, a, None, 0, None, *big) == binding.ERR_INVALID_ARG
    assert step(a, a, a, a, a, a, need - 1, None, *big) == binding.ERR_WORKSPACE_TOO_SMALL
    assert L.mqa_decode_step_combine(a, a, a, need - 1, 1, 16, 32768, 128, 128, None) == binding.ERR_WORKSPACE_TOO_SMALL
    app = L.kv_cache_append
    assert app(None, a, a, a, a, 1, None, 1, 1, 128, 128, 128, None) == binding.ERR_INVALID_ARG
    assert app(a, a, a, odd, a, 1, None, 1, 1, 128, 128, 128, None) == binding.ERR_INVALID_ARG
    assert app(a, a, a, a, a, 1, None, 1, 0, 128, 128, 128, None) == binding.ERR_INVALID_ARG
    assert app(a, a, a, a, a, 1, None, 1, 1, 128, 32, 128, None) == binding.ERR_UNSUPPORTED


def test_binding_type_checks():
    import torch
    q = torch.zeros(1, 8, 128, dtype=torch.bfloat16)
    with pytest.raises(TypeError):
        binding.mqa_decode_step(q, q, q, torch.zeros(1, dtype=torch.int32), torch.zeros(1, 8, 128))


def test_plans_of_many_query_rows_and_of_the_batched_form(L):
    """More than 32 query rows per sequence are planned on the kernel with the query rows as tile rows, and the batched
    form's workspace and refusals are answered on the host (the plan assumes the 148 SMs of a B200 without a GPU)."""
    assert binding.plan_kernel_name(True, False, 32, 128, 8192) == "mqa_decode_wide_kernel"       # 65 .. 128 rows: rows as tile rows
    assert binding.plan_kernel_name(True, False, 32, 192, 8192) == "mqa_decode_wide_kernel"       # beyond: tiles of 128 rows
    assert binding.plan_kernel_name(True, True, 32, 32, 8192) == "mqa_decode_stream_umma_kernel<32, fused, guess>"
    assert binding.plan_kernel_name(False, False, 32, 32, 8192) == "decode_split_simt_kernel"
    assert binding.plan_kernel_name(True, False, 0, 32, 8192) == ""
    assert binding.append_step_launches(32, 128, 8192) == 2
    assert binding.append_step_launches(256, 128, 8192) == 1
    assert binding.append_step_launches(32, 192, 8192) == 2
    assert binding.workspace_bytes(32, 128, 8192) >= binding.workspace_bytes(32, 64, 8192)
    need = binding.prefill_workspace_bytes(2, 8, 128, 256)
    assert need > 0
    assert binding.prefill_workspace_bytes(2, 8, 100, 256) > 0           # any number of positions
    assert binding.prefill_workspace_bytes(2, 8, 512, 256) == 0          # the queries' positions must fit the memory
    assert binding.prefill_workspace_bytes(2, 8, 128, 256, k=64) == 0
    a = ctypes.c_void_p(0x1000)
    pf = L.mqa_prefill_attention
    assert pf(a, a, a, None, a, a, need, None, 2, 8, 512, 256, 128, 128, None) == binding.ERR_UNSUPPORTED
    assert pf(a, a, a, None, a, a, need - 1, None, 2, 8, 128, 256, 128, 128, None) == binding.ERR_WORKSPACE_TOO_SMALL
    assert pf(None, a, a, None, a, a, need, None, 2, 8, 128, 256, 128, 128, None) == binding.ERR_INVALID_ARG
    assert pf(a, a, a, ctypes.c_void_p(0x1002), a, a, need, None, 2, 8, 128, 256, 128, 128, None) == binding.ERR_INVALID_ARG
