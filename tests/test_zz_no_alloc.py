"""mqa_decode_step_noalloc: the entry point for callers that cannot allocate a workspace (a
plugin inside a host framework that planned and reserved the device memory ahead of time).

It must give what mqa_decode_step gives, on calls in a row that share its built-in scratch
array, and refuse sizes whose scratch would not fit.  This file is collected last so that a
run that stops at the first failure has already run every other test."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_1911_02150_b200 as mqa
from paper_1911_02150_b200 import binding, workloads as wl
from paper_1911_02150_b200.build import build_library

ABS_TOL = 4e-3          # the tolerances of tests/test_parity_gpu.py
REL_TOL = 1e-2


def _close(a: torch.Tensor, ref):
    a = a.double().cpu().numpy()
    ref = ref if isinstance(ref, np.ndarray) else ref.double().cpu().numpy()
    err = np.abs(a - ref)
    assert np.all(np.isfinite(a))
    assert err.max() <= ABS_TOL
    assert np.all(err.max(-1) <= REL_TOL * np.abs(ref).max(-1))


@pytest.mark.gpu
def test_noalloc_matches_the_workspace_entry_point_on_two_calls_in_a_row():
    dev = "cuda:0"
    # two different problems, both cut into several pieces so that the scratch is really used;
    # the second call finds the first call's partial results still lying in the array
    cases = [(24, 32, 4096, 41), (70, 16, 1500, 42)]
    for b, h, m_max, seed in cases:
        assert 0 < mqa.workspace_bytes(b, h, m_max) <= binding.NOALLOC_SCRATCH_BYTES
        assert mqa.plan_splits(True, b, h, m_max)[0] > 1
        inp = wl.make_inputs(b, h, m_max, "mqa", seed=seed, device=dev)
        lens_np = np.random.default_rng(seed).integers(1, m_max + 1, size=b).astype(np.int32)
        lens_np[0] = m_max
        wl.poison_tail(inp["K"], lens_np)
        wl.poison_tail(inp["V"], lens_np)
        lens = torch.from_numpy(lens_np).to(dev)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        want = torch.empty(b, h, 128, dtype=torch.float32, device=dev)
        mqa.mqa_decode_step(inp["q"], inp["K"], inp["V"], lens, want, mqa.alloc_workspace(b, h, m_max, dev), status)
        got = torch.full_like(want, float("nan"))
        mqa.mqa_decode_step_noalloc(inp["q"], inp["K"], inp["V"], lens, got, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        _close(got, want)
        # same kernels, same plan: in fact the very same bits
        assert torch.equal(got.view(torch.int32), want.view(torch.int32))
        # and, directly, what the paper's step defines (the fp64 oracle on the same bits)
        _close(got, oracle.mqa_decode_step(wl.bits(inp["q"]), wl.bits(inp["K"]), wl.bits(inp["V"]), lens_np))


def test_noalloc_refuses_sizes_beyond_its_scratch_without_launching():
    build_library()
    L = binding.lib()
    b, h, m_max = 1024, 32, 4096                       # needs far more than 8 MiB of partials
    assert binding.workspace_bytes(b, h, m_max) > binding.NOALLOC_SCRATCH_BYTES
    a = ctypes.c_void_p(0x1000)                         # never dereferenced: the size check comes first
    rc = L.mqa_decode_step_noalloc(a, a, a, a, a, None, b, h, m_max, 128, 128, None)
    assert rc == binding.ERR_STATIC_SCRATCH_TOO_SMALL
    assert "scratch" in binding.status_string(rc)
    # bad arguments get the ordinary answers
    assert L.mqa_decode_step_noalloc(None, a, a, a, a, None, 1, 8, 128, 128, 128, None) in (
        binding.ERR_INVALID_ARG, binding.ERR_CUDA)
