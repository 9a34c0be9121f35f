"""mqa_prefill_attention (Section 3, the attention lines of the batched multi-query function under the autoregressive
mask of Section 2.3) against the fp64 oracle on the same bf16 bits.  Tolerance as for the decode step: every element
within 4e-3, every (sequence, head, position) row within 1e-2 of its own scale."""
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
    bad = err.max(-1) > REL_TOL * np.abs(ref).max(-1)
    assert not bad.any(), f"{what}: {bad.sum()} rows over the relative tolerance"


def run(b, h, n, m_max, start=None, seed=0, sample=None):
    gen = torch.Generator(device=DEV).manual_seed(seed)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    st = np.zeros(b, np.int32) if start is None else np.asarray(start, np.int32)
    wl.poison_tail(K, st + n)                              # rows after a sequence's last query position are never read
    wl.poison_tail(V, st + n)
    Og = Guarded((b, h, n, 128), torch.float32, DEV)
    Og.t.fill_(float("nan"))
    wsg = Guarded((max(16, mqa.prefill_workspace_bytes(b, h, n, m_max)),), torch.uint8, DEV)
    wsg.t.fill_(0xFF)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    start_t = None if start is None else torch.from_numpy(st).to(DEV)
    mqa.mqa_prefill_attention(Q, K, V, Og.t, wsg.t, start_t, status)
    torch.cuda.synchronize()
    Og.check("O"); wsg.check("workspace")
    assert int(status.item()) == 0
    O = Og.t
    assert bool(torch.isfinite(O).all())                   # every row was written, sampled or not
    if sample is None:
        ref = oracle.mqa_batched_attention(wl.bits(Q), wl.bits(K), wl.bits(V), st)
        check_close(O.cpu().numpy(), ref, f"b={b} h={h} n={n}")
    else:
        for s, heads in sample:
            hs = torch.as_tensor(heads, device=DEV)
            ref = oracle.mqa_batched_attention(wl.bits(Q[s:s + 1, hs]), wl.bits(K[s:s + 1]), wl.bits(V[s:s + 1]), st[s:s + 1])
            check_close(O[s:s + 1, hs].cpu().numpy(), ref, f"b={b} h={h} n={n} sequence {s} heads {heads}")
    return O


SMALL = [
    # b, h, n, m_max, start
    (1, 1, 64, 64, None),                       # one group: every column has its own last row
    (2, 8, 128, 128, None),
    (3, 4, 192, 512, [0, 100, 320]),            # a chunk of a longer prompt: queries begin at start[b]
    (2, 3, 256, 300, [44, 0]),                  # a head count that does not divide 64
    (1, 32, 128, 1100, [900]),                  # long memory in front of few queries
    (5, 16, 64, 2048, [1984, 0, 63, 64, 1000]),
    (2, 5, 100, 260, [160, 0]),                 # n is no multiple of anything: the last tile of a head is partly filled
    (3, 2, 1, 700, [0, 699, 350]),              # one position: a decoding step
    (1, 3, 129, 129, None),                     # one position in a tile of its own
    (2, 4, 333, 1200, [867, 5]),
]


@pytest.mark.parametrize("b,h,n,m_max,start", SMALL)
def test_small_cases_match_oracle(b, h, n, m_max, start):
    run(b, h, n, m_max, start, seed=b * 100 + h)


@pytest.mark.parametrize("b,h", [(128, 8), (32, 32)])
@pytest.mark.parametrize("n", [128, 1024, 4096])
def test_prompt_lengths_of_the_decode_configurations(b, h, n):
    """n = m in {128, 1024, 4096} for the batch and head counts of the paper-shaped and the long-context
    configurations.  The oracle is the plain fp64 definition (n^2 / 2 pairs per head): checked in full at n = 128, on
    seeded (sequence, heads) samples beyond (all positions of those heads)."""
    r = np.random.default_rng(n + b)
    if n == 128:
        sample = None
    else:
        seqs = sorted({0, b - 1, *r.integers(0, b, size=2).tolist()})
        per = 4 if n == 1024 else 1
        sample = [(s, sorted(set(r.integers(0, h, size=per).tolist()) | ({0} if s == 0 else {h - 1}))) for s in seqs]
    run(b, h, n, n, None, seed=n + h, sample=sample)


def test_rows_are_the_decode_steps():
    """Position t of the batched form is the incremental step over start + t + 1 rows (Section 2.4: up to and
    including its own position): the two entry points agree to within the two paths' rounding."""
    b, h, n, m_max = 2, 16, 128, 1300
    start = np.array([1000, 1172], np.int32)
    O = run(b, h, n, m_max, start, seed=5)
    gen = torch.Generator(device=DEV).manual_seed(5)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    for t in (0, 1, 63, 64, 127):
        o = torch.empty(b, h, 128, dtype=torch.float32, device=DEV)
        mqa.mqa_decode_step(Q[:, :, t].contiguous(), K, V, torch.from_numpy(start + t + 1).to(DEV), o, ws)
        torch.cuda.synchronize()
        assert float((o - O[:, :, t]).abs().max()) <= 2e-3


WHOLE_TILES = [
    # b, h, n, m_max, start: n a multiple of 128 (the kernel of the batched form: two heads per CTA)
    (2, 5, 384, 700, [300, 17]),                # an odd head count: the last CTA of a position tile holds one head
    (1, 2, 1152, 1300, [100]),                  # memories on both sides of 1024 rows (two roundings of the weights below it)
    (3, 7, 256, 1000, [744, 0, 511]),           # start + n = m_max exactly; a stage that ends inside the next sequence's rows
    (2, 1, 128, 128, None),                     # a single head
    (1, 4, 512, 2049, [1537]),                  # one row of the memory in a stage of its own
]


@pytest.mark.parametrize("b,h,n,m_max,start", WHOLE_TILES)
def test_whole_tiles_match_oracle(b, h, n, m_max, start):
    run(b, h, n, m_max, start, seed=7 * b + h)


def test_a_logit_far_above_every_earlier_one_in_a_long_memory():
    """A key row 300 times larger than the others, deep in a memory of more than 1024 rows, makes logits hundreds of
    units above (and below) everything before it: the rows' reference maxima move late and by a lot, and their
    accumulated outputs are rescaled by factors that underflow."""
    b, h, n, m_max = 2, 3, 256, 1536
    gen = torch.Generator(device=DEV).manual_seed(21)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    st = np.array([1280, 1100], np.int32)
    K[0, 1400] *= 300
    K[1, 1290] *= 300
    K[1, 5] *= 40                                           # (and one in the first stage, for comparison)
    O = torch.full((b, h, n, 128), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(max(16, mqa.prefill_workspace_bytes(b, h, n, m_max)), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mqa.mqa_prefill_attention(Q, K, V, O, ws, torch.from_numpy(st).to(DEV), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.mqa_batched_attention(wl.bits(Q), wl.bits(K), wl.bits(V), st)
    check_close(O.cpu().numpy(), ref, "a dominant key row late in the memory")


def test_a_negative_start_gives_zeros_and_a_flag():
    """start[b] < 0 is an empty memory for that sequence (zeros, LEN_CLAMPED); the other sequences are not affected."""
    b, h, n, m_max = 3, 4, 256, 512
    gen = torch.Generator(device=DEV).manual_seed(11)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    st = np.array([5, -1, 100], np.int32)
    O = torch.full((b, h, n, 128), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(max(16, mqa.prefill_workspace_bytes(b, h, n, m_max)), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mqa.mqa_prefill_attention(Q, K, V, O, ws, torch.from_numpy(st).to(DEV), status)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.STATUS_LEN_CLAMPED
    assert bool((O[1] == 0).all())
    keep = [0, 2]
    ref = oracle.mqa_batched_attention(wl.bits(Q[keep]), wl.bits(K[keep]), wl.bits(V[keep]), st[keep])
    check_close(O[keep].cpu().numpy(), ref, "sequences beside a bad start")


def test_two_runs_are_bit_identical():
    a = run(4, 8, 256, 700, [0, 400, 444, 13], seed=9)
    c = run(4, 8, 256, 700, [0, 400, 444, 13], seed=9)
    assert torch.equal(a.view(torch.int32), c.view(torch.int32))


def test_what_is_not_supported_is_refused_before_any_launch():
    b, h, n, m_max = 2, 4, 300, 256                        # more positions than the memory holds
    assert mqa.prefill_workspace_bytes(b, h, n, m_max) == 0
    Q = torch.zeros(b, h, n, 128, dtype=torch.bfloat16, device=DEV)
    K = torch.zeros(b, m_max, 128, dtype=torch.bfloat16, device=DEV)
    O = torch.full((b, h, n, 128), 7.0, dtype=torch.float32, device=DEV)
    with pytest.raises(mqa.MqaError) as e:
        mqa.mqa_prefill_attention(Q, K, K, O, torch.empty(1 << 20, dtype=torch.uint8, device=DEV))
    assert e.value.code == binding.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((O == 7.0).all())


def test_a_memory_that_would_pass_m_max_is_cut_there_and_flagged():
    """start[b] + n > m_max: the positions past the end of the memory attend over all m_max rows (there is no row of
    their own to add), LEN_CLAMPED is flagged, nothing outside K and V is read; the other sequences are not affected.
    Checked row by row against the decoding step's oracle over min(start + t + 1, m_max) rows."""
    b, h, n, m_max = 2, 4, 256, 600
    gen = torch.Generator(device=DEV).manual_seed(31)
    Q = wl.bf16_normal((b, h, n, 128), 128 ** -0.5, gen, DEV)
    K = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    V = wl.bf16_normal((b, m_max, 128), 1.0, gen, DEV)
    st = np.array([m_max - n + 70, 100], np.int32)          # the first sequence's last 70 positions have no row
    O = torch.full((b, h, n, 128), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(max(16, mqa.prefill_workspace_bytes(b, h, n, m_max)), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mqa.mqa_prefill_attention(Q, K, V, O, ws, torch.from_numpy(st).to(DEV), status)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.STATUS_LEN_CLAMPED
    Oh = O.cpu().numpy()
    assert np.all(np.isfinite(Oh))
    for t in (0, 100, 185, 186, 200, 255):
        lens = np.minimum(st + t + 1, m_max).astype(np.int32)
        ref = oracle.mqa_decode_step(wl.bits(Q[:, :, t].contiguous()), wl.bits(K), wl.bits(V), lens)
        check_close(Oh[:, :, t], ref, f"position {t}")
