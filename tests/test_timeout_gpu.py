"""A bounded wait that runs out.  No kernel of the library waits without a limit: when a copy it waits for does not
arrive, the kernel flags MQA_STATUS_PIPELINE_TIMEOUT, lets its other copies land, frees its tensor memory and
returns by itself.  Here the limit is shortened to about a millisecond and a testing flag keeps one copy of the
first CTA from ever being started; afterwards the limit is restored and an ordinary call on the same workspace and
the same GPU must be correct again (nothing was left behind: no held tensor memory, no stale bookkeeping)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1911_02150_b200 as mqa
from paper_1911_02150_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ABS_TOL, REL_TOL = 4e-3, 1e-2
SHORT_LIMIT = 2_000_000          # SM clock cycles: about a millisecond


def check_close(got, ref, what):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = np.abs(got.astype(np.float64) - ref)
    assert err.max() <= ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert np.all(err.max(-1) <= REL_TOL * np.abs(ref).max(-1)), f"{what}: row-relative error"


@pytest.mark.parametrize("b,h,m_max,chained", [
    (40, 16, 2048, False),      # persistent kernel, pieces merged through global memory
    (32, 32, 2048, True),       # persistent kernel launched as clusters, copies started on a guess
    (6, 8, 300, False),         # fixed-split kernel, one CTA per sequence
    (20, 96, 2048, False),      # many query rows: the kernel with the query rows as tile rows, pieces and a second pass
    (160, 40, 700, False),      # the same kernel, one split per sequence
])
def test_a_wait_that_runs_out_is_reported_and_leaves_nothing_behind(b, h, m_max, chained):
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=77, device=DEV)
    lens0 = np.full(b, m_max - 1, np.int32)
    lens0[1::3] = np.random.default_rng(7).integers(m_max // 2, m_max - 1, size=len(lens0[1::3]))
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    oracle.kv_cache_append(Kh, Vh, wl.bits(inp["k_new"]), wl.bits(inp["v_new"]), lens_h, True)
    ref = oracle.mqa_decode_step(wl.bits(inp["q"]), Kh, Vh, lens_h)
    lens = torch.from_numpy(lens0).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    o = torch.zeros(b, h, 128, dtype=torch.float32, device=DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    try:
        mqa.set_wait_limit_cycles(SHORT_LIMIT)
        mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens, o, ws, status,
                                   advance=False, chained=chained, withhold_copy=True)
        torch.cuda.synchronize()                     # the kernel came back by itself
    finally:
        mqa.set_wait_limit_cycles(0)
    assert int(status.item()) & binding.STATUS_PIPELINE_TIMEOUT
    assert np.array_equal(lens.cpu().numpy(), lens0)
    # the same step again, as it should be: same workspace, nothing cleared
    for rnd in range(2):
        status.zero_()
        o.fill_(float("nan"))
        lens.copy_(torch.from_numpy(lens0))
        mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens, o, ws, status,
                                   advance=True, chained=chained and rnd > 0)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(lens.cpu().numpy(), lens_h)
        check_close(o.cpu().numpy(), ref, f"call {rnd} after the timed-out one")
    assert np.array_equal(wl.bits(inp["K"]), Kh) and np.array_equal(wl.bits(inp["V"]), Vh)


def test_the_batched_form_reports_a_wait_that_runs_out_and_is_correct_again_afterwards():
    b, h, n, m_max = 3, 4, 512, 600
    gen = torch.Generator(device=DEV).manual_seed(4)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    st = np.array([88, 0, 31], np.int32)
    start = torch.from_numpy(st).to(DEV)
    O = torch.zeros(b, h, n, 128, dtype=torch.float32, device=DEV)
    ws = torch.empty(max(16, mqa.prefill_workspace_bytes(b, h, n, m_max)), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    try:
        mqa.set_wait_limit_cycles(SHORT_LIMIT)
        mqa.set_test_withhold_copy(True)
        mqa.mqa_prefill_attention(Q, K, V, O, ws, start, status)
        torch.cuda.synchronize()                     # the kernel came back by itself
    finally:
        mqa.set_test_withhold_copy(False)
        mqa.set_wait_limit_cycles(0)
    assert int(status.item()) & binding.STATUS_PIPELINE_TIMEOUT
    status.zero_()
    O.fill_(float("nan"))
    mqa.mqa_prefill_attention(Q, K, V, O, ws, start, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.mqa_batched_attention(wl.bits(Q), wl.bits(K), wl.bits(V), st)
    check_close(O.cpu().numpy(), ref, "the call after the timed-out one")
