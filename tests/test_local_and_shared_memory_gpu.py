"""Two variants the paper evaluates around the same step (Section 4): local attention (the current position and
the previous 31, the cache a ring of the window's size) and several query rows per sequence over one shared
memory (beam search over the encoder memory: beam x heads query rows, no append)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1911_02150_b200 as mqa
from paper_1911_02150_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ABS_TOL, REL_TOL = 4e-3, 1e-2


def check_close(got, ref, what):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = np.abs(got.astype(np.float64) - ref)
    assert err.max() <= ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert np.all(err.max(-1) <= REL_TOL * np.abs(ref).max(-1)), f"{what}: row-relative error"


@pytest.mark.parametrize("b,h,window,steps", [
    (128, 8, 32, 80), (16, 32, 32, 70), (5, 16, 96, 200),
    (1024, 8, 32, 40),        # a thousand sequences: one wave of eight-sequence CTAs
    (61, 64, 32, 40),         # 64 heads: four passes of 16 over the window; a last CTA with five sequences
    (20, 40, 96, 120),        # a head count that is no multiple of 16, a window of three tiles
    (3, 16, 512, 530),        # a window of sixteen tiles
])
def test_local_attention_ring_equals_attention_over_the_last_window_rows(b, h, window, steps):
    gen = torch.Generator(device=DEV).manual_seed(window + b)
    K = torch.zeros(b, window, 128, dtype=torch.bfloat16, device=DEV)
    V = torch.zeros_like(K)
    nan = torch.tensor(wl.NAN_BITS, dtype=torch.int16, device=DEV)
    K.view(torch.int16).fill_(nan); V.view(torch.int16).fill_(nan)          # rows never written must not be read
    pos = torch.zeros(b, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    hist_k = np.zeros((b, steps, 128), np.uint16); hist_v = np.zeros_like(hist_k)
    outs, qs = [], []
    for t in range(steps):
        q = wl.bf16_normal((b, h, 128), 128 ** -0.5, gen, DEV)
        k_new = wl.bf16_normal((b, 128), 1.0, gen, DEV); v_new = wl.bf16_normal((b, 128), 1.0, gen, DEV)
        hist_k[:, t], hist_v[:, t] = wl.bits(k_new), wl.bits(v_new)
        o = torch.empty(b, h, 128, dtype=torch.float32, device=DEV)
        mqa.mqa_decode_local_step(q, K, V, k_new, v_new, pos, o, status)
        outs.append(o); qs.append(q)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(pos.cpu().numpy(), np.full(b, steps))
    for t in (0, 1, window - 2, window - 1, window, window + 1, steps - 1):
        lo = max(0, t + 1 - window)
        n = t + 1 - lo
        Kw = np.zeros((b, window, 128), np.uint16); Vw = np.zeros_like(Kw)
        Kw[:, :n], Vw[:, :n] = hist_k[:, lo : t + 1], hist_v[:, lo : t + 1]      # the last n positions, oldest first
        ref = oracle.mqa_decode_step(wl.bits(qs[t]), Kw, Vw, np.full(b, n, np.int32))
        check_close(outs[t].cpu().numpy(), ref, f"step {t}")
    # the ring holds exactly the last `window` rows, each at position % window
    Kg, Vg = wl.bits(K), wl.bits(V)
    for t in range(steps - window, steps):
        assert np.array_equal(Kg[:, t % window], hist_k[:, t]) and np.array_equal(Vg[:, t % window], hist_v[:, t])


def test_local_step_without_advance_and_negative_position():
    b, h, window = 6, 8, 32
    inp = wl.make_inputs(b, h, window, "mqa", seed=2, device=DEV)
    pos0 = np.array([0, 5, 31, 32, 100, -3], np.int32)
    pos = torch.from_numpy(pos0).to(DEV)
    Kh, Vh = wl.bits(inp["K"]).copy(), wl.bits(inp["V"]).copy()
    o = torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mqa.mqa_decode_local_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], pos, o, status, advance=False)
    torch.cuda.synchronize()
    assert np.array_equal(pos.cpu().numpy(), pos0)
    assert int(status.item()) == (binding.STATUS_APPEND_NEGATIVE_LEN | binding.STATUS_LEN_CLAMPED)
    kn, vn = wl.bits(inp["k_new"]), wl.bits(inp["v_new"])
    lens = np.zeros(b, np.int32)
    for s in range(b - 1):
        Kh[s, pos0[s] % window], Vh[s, pos0[s] % window] = kn[s], vn[s]
        lens[s] = min(pos0[s] + 1, window)
    assert np.array_equal(wl.bits(inp["K"]), Kh) and np.array_equal(wl.bits(inp["V"]), Vh)
    ref = oracle.mqa_decode_step(wl.bits(inp["q"]), Kh, Vh, lens)          # rows 0 .. lens-1 of the ring hold tokens
    check_close(o.cpu().numpy(), ref, "local step")
    assert float(o[-1].abs().max()) == 0.0                                   # negative position: no row, zeros


def test_local_step_refuses_windows_one_cta_cannot_cover():
    b, h, window = 4, 8, 8192
    inp = wl.make_inputs(b, h, window, "mqa", seed=3, device=DEV)
    o = torch.zeros(b, h, 128, dtype=torch.float32, device=DEV)
    with pytest.raises(mqa.MqaError) as e:
        mqa.mqa_decode_local_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"],
                                  torch.zeros(b, dtype=torch.int32, device=DEV), o)
    assert e.value.code == binding.ERR_UNSUPPORTED


@pytest.mark.parametrize("b,beam,h,m", [(32, 4, 8, 2048), (24, 4, 16, 1536), (128, 4, 8, 128)])
def test_beams_share_one_memory_as_more_query_rows(b, beam, h, m):
    """Beam search over the encoder memory (Section 4.3, beam 4): the beams of a sentence attend over the same keys and
    values, so they are beam x h query rows of one multi-query step; each beam's rows equal its own step."""
    inp = wl.make_inputs(b, beam * h, m, "mqa", seed=beam + h, device=DEV)
    lens = np.random.default_rng(b).integers(1, m + 1, size=b).astype(np.int32)
    wl.poison_tail(inp["K"], lens); wl.poison_tail(inp["V"], lens)
    o = torch.empty(b, beam * h, 128, dtype=torch.float32, device=DEV)
    mqa.mqa_decode_step(inp["q"], inp["K"], inp["V"], torch.from_numpy(lens).to(DEV), o, mqa.alloc_workspace(b, beam * h, m, DEV))
    torch.cuda.synchronize()
    qb, Kb, Vb = wl.bits(inp["q"]), wl.bits(inp["K"]), wl.bits(inp["V"])
    got = o.cpu().numpy().reshape(b, beam, h, 128)
    for j in range(beam):
        ref = oracle.mqa_decode_step(np.ascontiguousarray(qb.reshape(b, beam, h, 128)[:, j]), Kb, Vb, lens)
        check_close(got[:, j], ref, f"beam {j}")
