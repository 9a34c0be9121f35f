"""mqa_decode_append_step (append + attention + merge in one call, one kernel launch for large
batches) against the oracle: oracle append, then oracle multi-query step on the grown cache."""
import numpy as np
import pytest
import torch

import oracle
import paper_1911_02150_b200 as mqa
from guards import Guarded
from paper_1911_02150_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ABS_TOL, REL_TOL = 4e-3, 1e-2


def check_close(got, ref, what):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = np.abs(got.astype(np.float64) - ref)
    assert err.max() <= ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert np.all(err.max(-1) <= REL_TOL * np.abs(ref).max(-1)), f"{what}: row-relative error"


def run(b, h, m_max, lens0, advance, seed, chained=False):
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=seed, device=DEV)
    lens0 = np.asarray(lens0, np.int32)
    wl.poison_tail(inp["K"], np.clip(lens0, 0, m_max))
    wl.poison_tail(inp["V"], np.clip(lens0, 0, m_max))
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    skipped = oracle.kv_cache_append(Kh, Vh, wl.bits(inp["k_new"]), wl.bits(inp["v_new"]), lens_h, True)
    ref = oracle.mqa_decode_step(wl.bits(inp["q"]), Kh, Vh, lens_h)
    # everything small that the step reads or writes sits between guard regions, checked after the kernels have run
    lens_g = Guarded((b,), torch.int32, DEV, like=torch.from_numpy(lens0).to(DEV))
    lens_t = lens_g.t
    o_g = Guarded((b, h, 128), torch.float32, DEV)
    o = o_g.t
    o.fill_(float("nan"))
    ws_g = Guarded((max(16, mqa.workspace_bytes(b, h, m_max)),), torch.uint8, DEV)
    ws = ws_g.t
    ws.fill_(0xFF)
    status_g = Guarded((1,), torch.int32, DEV)
    status = status_g.t
    status.zero_()
    q_g, kn_g, vn_g = (Guarded(tuple(inp[n].shape), torch.bfloat16, DEV, like=inp[n]) for n in ("q", "k_new", "v_new"))
    mqa.mqa_decode_append_step(q_g.t, inp["K"], inp["V"], kn_g.t, vn_g.t, lens_t, o, ws, status,
                               advance=advance, chained=chained)
    torch.cuda.synchronize()
    for g, name in ((lens_g, "lens"), (o_g, "o"), (ws_g, "workspace"), (status_g, "status"), (q_g, "q"), (kn_g, "k_new"), (vn_g, "v_new")):
        g.check(f"append_step b={b} h={h} m_max={m_max}: {name}")
    assert torch.equal(q_g.t, inp["q"]) and torch.equal(kn_g.t, inp["k_new"]) and torch.equal(vn_g.t, inp["v_new"])
    check_close(o.cpu().numpy(), ref, f"append_step b={b} h={h} m_max={m_max}")
    assert np.array_equal(wl.bits(inp["K"]), Kh) and np.array_equal(wl.bits(inp["V"]), Vh)   # the append, bit for bit
    assert np.array_equal(lens_t.cpu().numpy(), lens_h if advance else lens0)
    want_status = 0
    if (lens0 >= m_max).any():
        want_status |= binding.STATUS_APPEND_CACHE_FULL
    if (lens0 < 0).any():
        want_status |= binding.STATUS_APPEND_NEGATIVE_LEN | binding.STATUS_LEN_CLAMPED
    assert int(status.item()) == want_status, (int(status.item()), want_status, skipped)
    return inp, o


def lens_mix(b, m_max, seed):
    r = np.random.default_rng(seed)
    lens = r.integers(0, m_max, size=b).astype(np.int32)
    lens[r.integers(0, b, size=max(1, b // 8))] = 0          # first token of a sequence
    lens[r.integers(0, b, size=max(1, b // 8))] = m_max - 1  # fills the cache
    return lens


CASES = [
    # b, h, m_max: plans with the append inside the pass (persistent kernels) ...
    (40, 16, 1500), (160, 32, 333), (300, 8, 200), (37, 32, 4000), (64, 5, 777),
    # ... 33 .. 128 query rows per sequence: the kernel with the query rows as tile rows (fixed splits; the CTA whose rows
    # hold the new one stores it; one split per sequence moves lens on itself, else the second pass does) ...
    (40, 48, 1500), (33, 64, 2100), (24, 128, 2048), (20, 96, 1500), (150, 33, 700), (1, 127, 20000), (5, 65, 129),
    # ... more query rows than that: row tiles of 128 over the same cache rows, each CTA of the row's split storing the
    # new row; with one split per sequence lens is moved on by a kernel of its own ...
    (6, 200, 3000), (80, 160, 600), (2, 129, 5000), (3, 300, 1500),
    # ... and plans that run as separate launches (small batches)
    (4, 8, 300), (1, 16, 20000), (2, 40, 600),
]


@pytest.mark.parametrize("advance", [True, False])
@pytest.mark.parametrize("b,h,m_max", CASES)
def test_append_step_matches_oracle(b, h, m_max, advance):
    run(b, h, m_max, lens_mix(b, m_max, seed=b + h), advance, seed=b * 7 + h)


@pytest.mark.parametrize("chained", [True, "wrong-guess"])
@pytest.mark.parametrize("b,h,m_max", CASES + [(300, 16, 1500), (1024, 8, 1024)])
def test_append_step_with_the_chained_promise_matches_oracle(b, h, m_max, chained):
    """Every plan accepts the promise (most ignore it); nothing but the set-up copies precedes the step here, so it holds."""
    run(b, h, m_max, lens_mix(b, m_max, seed=b + h + 1), True, seed=b * 5 + h, chained=chained)


def test_append_step_full_and_negative_sequences_take_no_row():
    b, h, m_max = 48, 16, 1024
    lens = lens_mix(b, m_max, seed=5)
    lens[3] = m_max          # full: no row, attends over m_max rows
    lens[7] = -2             # negative: no row, empty prefix -> zeros
    run(b, h, m_max, lens, True, seed=77)


def test_incremental_decoding_with_append_steps():
    """A decoding loop of 40 steps on a batch large enough for the persistent kernel (append inside the pass): every step's
    output against the oracle on the cache as it then stands, and two runs bit-identical."""
    b, h, m_max, steps = 96, 16, 512, 40
    gen = torch.Generator(device=DEV)
    outs = []
    for rep in range(2):
        gen.manual_seed(321)
        K = torch.zeros(b, m_max, 128, dtype=torch.bfloat16, device=DEV)
        V = torch.zeros_like(K)
        nan = torch.tensor(wl.NAN_BITS, dtype=torch.int16, device=DEV)
        K.view(torch.int16).fill_(nan); V.view(torch.int16).fill_(nan)
        start = np.random.default_rng(3).integers(380, 470, size=b).astype(np.int32)     # prefill of different lengths
        for s in range(b):
            K[s, : start[s]] = wl.bf16_normal((int(start[s]), 128), 1.0, gen, DEV)
            V[s, : start[s]] = wl.bf16_normal((int(start[s]), 128), 1.0, gen, DEV)
        lens_t = torch.from_numpy(start.copy()).to(DEV)
        ws = mqa.alloc_workspace(b, h, m_max, DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        run_outs, qs = [], []
        for t in range(steps):
            q = wl.bf16_normal((b, h, 128), 128 ** -0.5, gen, DEV)
            k_new = wl.bf16_normal((b, 128), 1.0, gen, DEV)
            v_new = wl.bf16_normal((b, 128), 1.0, gen, DEV)
            o = torch.empty(b, h, 128, dtype=torch.float32, device=DEV)
            mqa.mqa_decode_append_step(q, K, V, k_new, v_new, lens_t, o, ws, status)
            run_outs.append(o); qs.append(q)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(lens_t.cpu().numpy(), start + steps)
        outs.append(run_outs)
        if rep == 0:
            Kb, Vb = wl.bits(K), wl.bits(V)
            for t in (0, 1, 17, steps - 1):
                ref = oracle.mqa_decode_step(wl.bits(qs[t]), Kb, Vb, (start + t + 1).astype(np.int32))
                check_close(run_outs[t].cpu().numpy(), ref, f"step {t}")
    for a, c in zip(*outs):
        assert torch.equal(a.view(torch.int32), c.view(torch.int32))


def test_host_buffer_entry_point_matches_the_device_one():
    b, h, m_max = 40, 16, 1500
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=21, device=DEV)
    lens0 = lens_mix(b, m_max, seed=21)
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    K2, V2 = inp["K"].clone(), inp["V"].clone()
    lens_a, lens_b = torch.from_numpy(lens0).to(DEV), torch.from_numpy(lens0.copy()).to(DEV)
    o_dev = torch.empty(b, h, 128, dtype=torch.float32, device=DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens_a, o_dev, ws)
    # host side: once as three separate pinned tensors, once packed back to back (one copy)
    for packed in (False, True):
        Kc, Vc, lens_c = K2.clone(), V2.clone(), lens_b.clone()
        if packed:
            parts = [inp[n].cpu().contiguous() for n in ("q", "k_new", "v_new")]
            buf = torch.empty(sum(t.numel() * 2 for t in parts), dtype=torch.uint8).pin_memory()
            views, at = [], 0
            for t in parts:
                n = t.numel() * 2
                buf[at : at + n].copy_(t.view(torch.uint8).view(-1))
                views.append(buf[at : at + n].view(torch.bfloat16).view(t.shape))
                at += n
            qh, kh, vh = views
        else:
            qh, kh, vh = (inp[n].cpu().pin_memory() for n in ("q", "k_new", "v_new"))
        o_host = torch.full((b, h, 128), float("nan"), dtype=torch.float32).pin_memory()
        staging = torch.empty(mqa.host_staging_bytes(b, h), dtype=torch.uint8, device=DEV)
        if packed:
            mqa.HostStep(qh, kh, vh, o_host, Kc, Vc, lens_c, staging, ws)()      # bound once, then the bare C call
        else:
            mqa.mqa_decode_append_step_host(qh, kh, vh, o_host, Kc, Vc, lens_c, staging, ws)
        torch.cuda.synchronize()
        assert torch.equal(o_host, o_dev.cpu())
        assert torch.equal(Kc.view(torch.int16), inp["K"].view(torch.int16)) and torch.equal(lens_c, lens_a)


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("b,h,m_max", [(32, 32, 2048), (40, 16, 1500), (6, 48, 700), (4, 8, 100), (3, 130, 300), (150, 8, 1100)])
def test_host_buffer_steps_in_a_loop_against_the_oracle(b, h, m_max, pinned):
    """Five consecutive steps through the host-buffer entry point, bound once, the same host buffers refilled before each
    step (pinned: the inputs are fetched by a kernel and o is stored to the host by the kernels; pageable: copies either
    side): every step is the oracle's append and step on the grown cache, lens moves on, the cache holds the new rows."""
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=31, device=DEV)
    lens0 = np.minimum(lens_mix(b, m_max, seed=31), m_max - 5).clip(0).astype(np.int32)
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    lens_t = torch.from_numpy(lens0).to(DEV)
    hold = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    qh, kh, vh = (hold(torch.empty(tuple(inp[n].shape), dtype=torch.bfloat16)) for n in ("q", "k_new", "v_new"))
    o_host = hold(torch.empty(b, h, 128, dtype=torch.float32))
    staging = torch.empty(mqa.host_staging_bytes(b, h), dtype=torch.uint8, device=DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    step = mqa.HostStep(qh, kh, vh, o_host, inp["K"], inp["V"], lens_t, staging, ws, status)
    for t in range(5):
        new = wl.make_inputs(b, h, 1, "mqa", seed=100 + t, device="cpu")
        qh.copy_(new["q"]); kh.copy_(new["k_new"]); vh.copy_(new["v_new"])
        o_host.fill_(float("nan"))
        step()
        torch.cuda.synchronize()
        oracle.kv_cache_append(Kh, Vh, wl.bits(kh), wl.bits(vh), lens_h, True)
        check_close(o_host.numpy(), oracle.mqa_decode_step(wl.bits(qh), Kh, Vh, lens_h), f"host step {t}")
        assert np.array_equal(lens_t.cpu().numpy(), lens_h)
    assert int(status.item()) == 0
    assert np.array_equal(wl.bits(inp["K"]), Kh) and np.array_equal(wl.bits(inp["V"]), Vh)


def test_bound_step_gives_what_the_call_gives():
    b, h, m_max = 40, 16, 1500
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=22, device=DEV)
    lens0 = lens_mix(b, m_max, seed=22)
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    K2, V2 = inp["K"].clone(), inp["V"].clone()
    lens_a, lens_b = torch.from_numpy(lens0).to(DEV), torch.from_numpy(lens0.copy()).to(DEV)
    o_a, o_b = (torch.empty(b, h, 128, dtype=torch.float32, device=DEV) for _ in range(2))
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    for _ in range(3):                                        # three tokens each way (the same q and rows: only lens moves)
        mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens_a, o_a, ws)
    step = mqa.AppendStep(inp["q"], K2, V2, inp["k_new"], inp["v_new"], lens_b, o_b, ws)
    for _ in range(3):
        assert step() is o_b
    torch.cuda.synchronize()
    assert torch.equal(o_a.view(torch.int32), o_b.view(torch.int32)) and torch.equal(lens_a, lens_b)
    assert torch.equal(inp["K"].view(torch.int16), K2.view(torch.int16)) and torch.equal(inp["V"].view(torch.int16), V2.view(torch.int16))
    with pytest.raises(TypeError):
        mqa.AppendStep(inp["q"].float(), K2, V2, inp["k_new"], inp["v_new"], lens_b, o_b, ws)
