"""mqa_layer_decode_step (Section 3, the incremental multi-query layer: projections either side of the attention step)
against the layer oracle, in both of its forms: the one that rounds to bf16 where the path stores or feeds bf16 (q, the
new cache rows, o), and the paper's function itself with q and o left unrounded (only the cache, which has no other
type, takes bf16 rows).

Tolerance against the unrounded form.  Two roundings separate it from the path: q (an input of the logits) and o (an
operand of the output product), each at most 2^-8 relative per element, about 1.6e-3 rms.  A rounding of q moves a
logit by the sum of 128 independent terms, 1.6e-3 rms in all for q ~ N(0, 1/k) and keys ~ N(0, 1), which moves every
weight by that relative amount and o by about 1.6e-3 of its scale; the rounding of o adds as much again.  Through the
output product (P_o ~ N(0, 1/(h v)), independent signs) y is off by about 1.6e-3 * sqrt(2) = 2.3e-3 of its rms, the
largest of a row's d errors by about 3.5 times that, and a row's largest |y| is about 3.3 rms: 2.5e-3 of the row's
scale expected (3.6e-3 is the most the two oracle forms differ on these shapes, computed on the CPU).  The gate is
1e-2 of each row's scale, the relative tolerance of the step itself; the absolute 4e-3 gate is applied to the rounded
form only, since y here is not small (rows of scale 2 to 4 where a sequence attends over one row)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1911_02150_b200 as mqa
from oracle import layer_step as ls
from paper_1911_02150_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ABS_TOL, REL_TOL = 4e-3, 1e-2


def layer_inputs(b, h, d, m_max, seed):
    """x ~ N(0,1); P_q ~ N(0, 1/(d k)) so that q ~ N(0, 1/k) as in the step's workloads; P_k, P_v ~ N(0, 1/d) so that
    the new rows are ~ N(0,1) like the cache; P_o ~ N(0, 1/(h v)); cache ~ N(0,1).  Drawn on the device, seeded."""
    gen = torch.Generator(device=DEV).manual_seed(seed)
    n = lambda shape, std: wl.bf16_normal(shape, std, gen, DEV)
    return dict(x=n((b, d), 1.0), P_q=n((h, d, 128), (d * 128) ** -0.5), P_k=n((d, 128), d ** -0.5), P_v=n((d, 128), d ** -0.5),
                P_o=n((h, d, 128), (h * 128) ** -0.5), K=n((b, m_max, 128), 1.0), V=n((b, m_max, 128), 1.0))


def one_ulp_apart_at_most(a_bits, b_bits):
    """bf16 bit patterns that are equal or neighbours (same sign), NaN nowhere."""
    a, c = a_bits.astype(np.int32), b_bits.astype(np.int32)
    return np.abs(a - c) <= 1


def run(b, h, d, m_max, lens0, seed, advance=True):
    inp = layer_inputs(b, h, d, m_max, seed)
    lens0 = np.asarray(lens0, np.int32)
    wl.poison_tail(inp["K"], np.clip(lens0, 0, m_max)); wl.poison_tail(inp["V"], np.clip(lens0, 0, m_max))
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    weights = [wl.bits(inp[n]) for n in ("x", "P_q", "P_k", "P_v", "P_o")]
    # the paper's function, nothing rounded but the rows the cache stores
    y_paper = ls.multiquery_layer_decode_step(*weights, Kh.copy(), Vh.copy(), lens0.copy(), round_interfaces=False)[0]
    y_ref, q_ref, k_ref, v_ref = ls.multiquery_layer_decode_step(*weights, Kh, Vh, lens_h)
    lens_t = torch.from_numpy(lens0).to(DEV)
    y = torch.full((b, d), float("nan"), dtype=torch.float32, device=DEV)
    ws = mqa.alloc_layer_workspace(b, h, d, m_max, DEV)
    ws.fill_(0xFF)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mqa.mqa_layer_decode_step(inp["x"], inp["P_q"], inp["P_k"], inp["P_v"], inp["P_o"], inp["K"], inp["V"], lens_t, y, ws, status,
                              advance=advance)
    torch.cuda.synchronize()
    got = y.cpu().numpy()
    assert np.all(np.isfinite(got))
    err = np.abs(got.astype(np.float64) - y_ref)
    assert err.max() <= ABS_TOL, f"max abs err {err.max():.3e}"
    assert np.all(err.max(-1) <= REL_TOL * np.abs(y_ref).max(-1)), "row-relative error"
    err_paper = np.abs(got.astype(np.float64) - y_paper)
    assert np.all(err_paper.max(-1) <= REL_TOL * np.abs(y_paper).max(-1)), \
        f"against the unrounded function: {np.max(err_paper.max(-1) / np.abs(y_paper).max(-1)):.3e} of a row's scale"
    # the appended rows: the oracle's bf16 rows up to the last bit (fp32 against fp64 accumulation before the rounding)
    Kg, Vg = wl.bits(inp["K"]), wl.bits(inp["V"])
    took = (lens0 >= 0) & (lens0 < m_max)
    for s in np.nonzero(took)[0]:
        r = lens0[s]
        assert one_ulp_apart_at_most(Kg[s, r], Kh[s, r]).all() and one_ulp_apart_at_most(Vg[s, r], Vh[s, r]).all()
        assert (Kg[s, r] == Kh[s, r]).mean() > 0.97 and (Vg[s, r] == Vh[s, r]).mean() > 0.97
        Kg[s, r], Vg[s, r] = Kh[s, r], Vh[s, r]
    assert np.array_equal(Kg, Kh) and np.array_equal(Vg, Vh)                     # nothing else in the cache moved
    assert np.array_equal(lens_t.cpu().numpy(), lens_h if advance else lens0)
    return got


CASES = [
    # b, h, d, m_max
    (32, 32, 1024, 2048),     # the headline shapes: persistent kernel, one launch for the step
    (40, 16, 512, 1500),
    (8, 8, 256, 300),         # small: fixed-split kernel
    (130, 8, 384, 1100),      # two batch tiles of 128 (the second nearly empty)
    (64, 33, 512, 1200),      # an odd head count: the last head group of the output projection holds one head
]


@pytest.mark.parametrize("b,h,d,m_max", CASES)
def test_layer_step_matches_oracle(b, h, d, m_max):
    r = np.random.default_rng(b + h)
    lens0 = r.integers(0, m_max, size=b).astype(np.int32)
    lens0[0], lens0[-1] = 0, m_max - 1
    run(b, h, d, m_max, lens0, seed=b * 3 + h)


def test_layer_step_full_cache_and_no_advance():
    b, h, d, m_max = 24, 16, 256, 1536
    lens0 = np.random.default_rng(5).integers(1, m_max, size=b).astype(np.int32)
    lens0[2] = m_max                                       # takes no row, attends over its m_max rows
    inp_status = run(b, h, d, m_max, lens0, seed=9, advance=False)
    assert inp_status.shape == (b, d)


def test_layer_step_twice_is_bit_identical():
    b, h, d, m_max = 32, 32, 1024, 2048
    lens0 = np.full(b, 1999, np.int32)
    a = run(b, h, d, m_max, lens0, seed=3)
    c = run(b, h, d, m_max, lens0, seed=3)
    assert np.array_equal(a.view(np.int32), c.view(np.int32))


def test_layer_step_rejects_what_it_does_not_support():
    b, h, d, m_max = 4, 8, 200, 300                        # d not a multiple of 128
    assert mqa.layer_workspace_bytes(b, h, d, m_max) == 0
    inp = layer_inputs(b, h, d, m_max, 1)
    y = torch.zeros(b, d, dtype=torch.float32, device=DEV)
    with pytest.raises(mqa.MqaError):
        mqa.mqa_layer_decode_step(inp["x"], inp["P_q"], inp["P_k"], inp["P_v"], inp["P_o"], inp["K"], inp["V"],
                                  torch.zeros(b, dtype=torch.int32, device=DEV), y, torch.empty(1 << 20, dtype=torch.uint8, device=DEV))
    assert float(y.abs().max()) == 0.0
