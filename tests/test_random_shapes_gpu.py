"""Seeded random shapes through the C ABI against the oracle: the dispatch picks whatever kernel each shape falls to
(streaming, query rows as tile rows with one or several row tiles and splits, fixed splits, CUDA cores), the lengths
mix empty, full and arbitrary prefixes, and the append-and-attend step is checked with and without the lens advance."""
import numpy as np
import pytest
import torch

import oracle
import paper_1911_02150_b200 as mqa
from paper_1911_02150_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ABS_TOL, REL_TOL = 4e-3, 1e-2


def check_close(got, ref, what):
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    err = np.abs(got.astype(np.float64) - ref)
    assert err.max() <= ABS_TOL, f"{what}: max abs err {err.max():.3e}"
    assert np.all(err.max(-1) <= REL_TOL * np.maximum(np.abs(ref).max(-1), 1e-30)), f"{what}: row-relative error"


def shapes(n, seed):
    r = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        h = int(r.choice([1, 7, 16, 24, 32, 33, 47, 64, 65, 100, 128, 129, 200, 257]))
        m_max = int(r.choice([1, 31, 64, 127, 128, 129, 300, 777, 1024, 1500, 2049, 4100]))
        b = int(r.choice([1, 2, 3, 5, 9, 17, 40, 150]))
        if b * h * m_max > 40_000_000:            # keeps the oracle to a second or so per case
            b = max(1, 40_000_000 // (h * m_max))
        out.append((b, h, m_max, int(r.integers(1 << 30))))
    return out


@pytest.mark.parametrize("b,h,m_max,seed", shapes(36, 2024))
def test_random_shape_step_and_append_step(b, h, m_max, seed):
    r = np.random.default_rng(seed)
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=seed % 1000, device=DEV)
    lens0 = r.integers(0, m_max + 1, size=b).astype(np.int32)
    lens0[r.integers(0, b)] = 0
    lens0[r.integers(0, b)] = m_max
    if b > 2:
        lens0[r.integers(0, b)] = max(0, m_max - 1)
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    # the step over the prefix as it stands
    o = torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV)
    lens_t = torch.from_numpy(lens0).to(DEV)
    mqa.mqa_decode_step(inp["q"], inp["K"], inp["V"], lens_t, o, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_close(o.cpu().numpy(), oracle.mqa_decode_step(wl.bits(inp["q"]), wl.bits(inp["K"]), wl.bits(inp["V"]), lens0), f"step b={b} h={h} m={m_max}")
    # append + attend, lens advanced; full sequences take no row and are flagged
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    oracle.kv_cache_append(Kh, Vh, wl.bits(inp["k_new"]), wl.bits(inp["v_new"]), lens_h, True)
    ref = oracle.mqa_decode_step(wl.bits(inp["q"]), Kh, Vh, lens_h)
    o.fill_(float("nan"))
    status.zero_()
    mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens_t, o, ws, status, advance=True)
    torch.cuda.synchronize()
    expect = mqa.binding.STATUS_APPEND_CACHE_FULL if (lens0 >= m_max).any() else 0
    assert int(status.item()) == expect
    assert np.array_equal(lens_t.cpu().numpy(), lens_h)
    assert np.array_equal(wl.bits(inp["K"]), Kh) and np.array_equal(wl.bits(inp["V"]), Vh)
    check_close(o.cpu().numpy(), ref, f"append step b={b} h={h} m={m_max}")


def prefill_shapes(n, seed):
    r = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        h = int(r.choice([1, 2, 3, 8, 17, 32]))
        nq = int(r.choice([1, 5, 64, 127, 128, 129, 200, 384, 640, 1100]))
        b = int(r.choice([1, 2, 3, 6]))
        extra = int(r.choice([0, 1, 100, 1000]))
        if b * h * nq * (nq + extra) > 30_000_000:
            b, h = 1, min(h, 2)
        out.append((b, h, nq, nq + extra, int(r.integers(1 << 30))))
    return out


@pytest.mark.parametrize("b,h,n,m_max,seed", prefill_shapes(24, 77))
def test_random_shape_batched_form(b, h, n, m_max, seed):
    r = np.random.default_rng(seed)
    gen = torch.Generator(device=DEV).manual_seed(seed % 1000)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    st = r.integers(0, m_max - n + 1, size=b).astype(np.int32)
    st[r.integers(0, b)] = m_max - n
    wl.poison_tail(K, st + n); wl.poison_tail(V, st + n)
    O = torch.full((b, h, n, 128), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(max(16, mqa.prefill_workspace_bytes(b, h, n, m_max)), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mqa.mqa_prefill_attention(Q, K, V, O, ws, torch.from_numpy(st).to(DEV), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.mqa_batched_attention(wl.bits(Q), wl.bits(K), wl.bits(V), st)
    check_close(O.cpu().numpy(), ref, f"batched b={b} h={h} n={n} m={m_max}")


def test_mixed_back_to_back_launches_stay_bit_identical():
    """The three kernels that take all of an SM's tensor memory (the streaming step, the many-rows step, the batched form),
    launched back to back on one stream 200 times in turn (each may begin while the one before is finishing): every result
    is bit for bit what the first round gave, and no wait ran out."""
    b, h, m = 32, 32, 2048
    a = wl.make_inputs(b, h, m, "mqa", seed=1, device=DEV)
    c = wl.make_inputs(16, 96, 1100, "mqa", seed=2, device=DEV)
    lens_a = torch.full((b,), m - 1, dtype=torch.int32, device=DEV)
    lens_c = torch.from_numpy(np.random.default_rng(3).integers(0, 1100, size=16).astype(np.int32)).to(DEV)
    ws_a, ws_c = mqa.alloc_workspace(b, h, m, DEV), mqa.alloc_workspace(16, 96, 1100, DEV)
    o_a = torch.empty(b, h, 128, dtype=torch.float32, device=DEV)
    o_c = torch.empty(16, 96, 128, dtype=torch.float32, device=DEV)
    gen = torch.Generator(device=DEV).manual_seed(9)
    Q = wl.bf16_normal((2, 5, 333, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((2, 400, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((2, 400, 128), 1.0, gen, DEV)
    O = torch.empty(2, 5, 333, 128, dtype=torch.float32, device=DEV)
    ws_p = torch.empty(64, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert mqa.plan_kernel_name(True, True, b, h, m).startswith("mqa_decode_stream_umma_kernel")
    assert mqa.plan_kernel_name(True, True, 16, 96, 1100) == "mqa_decode_wide_kernel"
    first = None
    for it in range(200):
        mqa.mqa_decode_append_step(a["q"], a["K"], a["V"], a["k_new"], a["v_new"], lens_a, o_a, ws_a, status, advance=False, chained=it > 0)
        mqa.mqa_prefill_attention(Q, K, V, O, ws_p, None, status)
        mqa.mqa_decode_append_step(c["q"], c["K"], c["V"], c["k_new"], c["v_new"], lens_c, o_c, ws_c, status, advance=False)
        if it % 40 == 0 or it == 199:
            torch.cuda.synchronize()
            cur = [t.clone().view(torch.int32) for t in (o_a, O, o_c)]
            first = first or cur
            assert all(torch.equal(x, y) for x, y in zip(first, cur)), f"round {it}"
    assert int(status.item()) == 0
