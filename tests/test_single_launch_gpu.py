"""The single-launch decoding step of the persistent tcgen05 kernel: the pieces of a sequence that was cut over
several CTAs are merged inside the kernel, under an epoch kept in the caller's workspace.  What is checked here is
what that adds: the workspace may hold anything (other shapes' leftovers included), every call works under a new
epoch (CUDA-graph replays too), lens is advanced exactly once, and the shared reference maximum of the softmax
moves when a large logit turns up late in a long cache."""
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
    assert np.all(err.max(-1) <= REL_TOL * np.abs(ref).max(-1)), f"{what}: row-relative error"


def lens_for(b, m_max, seed):
    r = np.random.default_rng(seed)
    lens = r.integers(1, m_max + 1, size=b).astype(np.int32)
    lens[0], lens[-1] = m_max, 1
    return lens


def test_launch_counts():
    assert mqa.append_step_launches(32, 32, 8192) == 1        # cut into a few pieces per sequence: merged in the kernel
    assert mqa.append_step_launches(256, 16, 2048) == 1
    assert mqa.append_step_launches(1, 16, 32768) == 2        # one sequence over every SM: second-pass kernel
    assert mqa.append_step_launches(4, 8, 300) == 2           # small, fixed splits: pass with the append inside, second pass


def test_workspace_contents_do_not_matter():
    shapes = [(40, 32, 2048, 1), (64, 16, 1500, 2), (33, 64, 2100, 3), (40, 32, 2048, 4)]
    nbytes = max(mqa.workspace_bytes(b, h, m) for b, h, m, _ in shapes)
    gen = torch.Generator(device=DEV).manual_seed(0)
    ws = torch.randint(0, 256, (nbytes,), dtype=torch.uint8, device=DEV, generator=gen)   # garbage to begin with
    for rnd in range(2):
        for b, h, m_max, seed in shapes:                      # each shape finds what the shape before left behind
            inp = wl.make_inputs(b, h, m_max, "mqa", seed=seed, device=DEV)
            lens = lens_for(b, m_max, seed)
            wl.poison_tail(inp["K"], lens); wl.poison_tail(inp["V"], lens)
            o = torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV)
            status = torch.zeros(1, dtype=torch.int32, device=DEV)
            mqa.mqa_decode_step(inp["q"], inp["K"], inp["V"], torch.from_numpy(lens).to(DEV), o, ws, status)
            torch.cuda.synchronize()
            ref = oracle.mqa_decode_step(wl.bits(inp["q"]), wl.bits(inp["K"]), wl.bits(inp["V"]), lens)
            check_close(o.cpu().numpy(), ref, f"round {rnd} b={b} h={h} m_max={m_max}")
            assert int(status.item()) == 0
        ws[: nbytes // 2].fill_(0xFF)                         # and a partly overwritten workspace


@pytest.mark.parametrize("noalloc", [False, True])
def test_two_shapes_whose_counters_overlap_share_one_epoch(noalloc):
    """Batches of 601 and 602 sequences (h = 8, 1024 rows) take the same grid, cut most sequences in two and count the
    delivered pieces in the same words of the control block.  The second shape's first call must not take the first
    shape's counts for its own: the epoch is one per workspace, not one per shape.  Also through the entry point that
    brings its own scratch."""
    h, m_max = 8, 1024
    sizes = (601, 602, 601)
    ws = None if noalloc else mqa.alloc_workspace(max(sizes), h, m_max, DEV)
    for rnd, b in enumerate(sizes):
        assert mqa.append_step_launches(b, h, m_max) == 1
        inp = wl.make_inputs(b, h, m_max, "mqa", seed=50 + rnd, device=DEV)
        lens = np.full(b, m_max, np.int32)
        lens[::7] = np.random.default_rng(rnd).integers(1, m_max, size=len(lens[::7]))
        wl.poison_tail(inp["K"], lens); wl.poison_tail(inp["V"], lens)
        o = torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        if noalloc:
            mqa.mqa_decode_step_noalloc(inp["q"], inp["K"], inp["V"], torch.from_numpy(lens).to(DEV), o, status)
        else:
            mqa.mqa_decode_step(inp["q"], inp["K"], inp["V"], torch.from_numpy(lens).to(DEV), o, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = oracle.mqa_decode_step(wl.bits(inp["q"]), wl.bits(inp["K"]), wl.bits(inp["V"]), lens)
        check_close(o.cpu().numpy(), ref, f"call {rnd}: b={b}")


@pytest.mark.parametrize("b,h,m_max,rows", [(32, 16, 1024, 300), (64, 8, 1024, 100), (32, 32, 2048, 2048), (16, 32, 4096, 4000)])
def test_equal_sequences_in_clusters(b, h, m_max, rows):
    """A batch that divides the grid is launched as clusters, and with sequences of equal length a cluster holds one
    sequence: its CTAs take the stages in turn and merge through the cluster's shared memory.  Short sequences leave
    CTAs of a cluster without a stage (300 rows are three stages for four CTAs): their empty pieces must be skipped."""
    assert mqa.append_step_launches(b, h, m_max) == 1
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=b + rows, device=DEV)
    lens0 = np.full(b, rows - 1, np.int32)
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    oracle.kv_cache_append(Kh, Vh, wl.bits(inp["k_new"]), wl.bits(inp["v_new"]), lens_h, True)
    ref = oracle.mqa_decode_step(wl.bits(inp["q"]), Kh, Vh, lens_h)
    lens_t = torch.from_numpy(lens0).to(DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    ws.fill_(0xFF)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for chained in (False, True):
        lens_t.copy_(torch.from_numpy(lens0))
        o = torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV)
        mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens_t, o, ws, status,
                                   advance=True, chained=chained)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert np.array_equal(lens_t.cpu().numpy(), lens_h)
        check_close(o.cpu().numpy(), ref, f"b={b} rows={rows} chained={chained}")


def test_many_calls_on_one_workspace_are_bit_identical():
    b, h, m_max = 48, 32, 3000
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=11, device=DEV)
    lens_t = torch.from_numpy(lens_for(b, m_max, 11)).to(DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    outs = []
    for _ in range(6):
        o = torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV)
        mqa.mqa_decode_step(inp["q"], inp["K"], inp["V"], lens_t, o, ws)
        outs.append(o)
    torch.cuda.synchronize()
    for o in outs[1:]:
        assert torch.equal(o, outs[0])                        # whichever CTA merged: pieces in a fixed order


def test_graph_replays_of_append_steps_advance_lens_once_each():
    b, h, m_max, per_graph, replays = 40, 16, 2048, 3, 2
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=12, device=DEV)
    lens0 = np.random.default_rng(12).integers(900, 2000, size=b).astype(np.int32)
    lens0[3] = m_max - 2                                      # fills up on the way: later steps take no row
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    lens_t = torch.from_numpy(lens0).to(DEV)
    o = torch.zeros(b, h, 128, dtype=torch.float32, device=DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    side = torch.cuda.Stream(device=DEV)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens_t, o, ws, status,
                                   advance=True)              # set-up call outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    steps = 1
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(per_graph):
            mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens_t, o, ws, status,
                                       advance=True)
    for _ in range(replays):
        graph.replay()
        steps += per_graph
    torch.cuda.synchronize()
    k_new, v_new = wl.bits(inp["k_new"]), wl.bits(inp["v_new"])
    for _ in range(steps):
        oracle.kv_cache_append(Kh, Vh, k_new, v_new, lens_h, True)
    ref = oracle.mqa_decode_step(wl.bits(inp["q"]), Kh, Vh, lens_h)
    assert np.array_equal(lens_t.cpu().numpy(), lens_h)
    assert np.array_equal(wl.bits(inp["K"]), Kh) and np.array_equal(wl.bits(inp["V"]), Vh)
    check_close(o.cpu().numpy(), ref, "last step of the replayed graph")


def test_reference_maximum_moves_late_in_a_long_cache():
    b, h, m_max = 40, 32, 4096
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=13, device=DEV)
    q = torch.zeros_like(inp["q"]); q[..., 0] = 1.0
    K = torch.zeros_like(inp["K"])
    K[:, 700, 0] = 30.0                                       # a first jump of the maximum, in a later stage ...
    K[:, 3001, 0] = 200.0                                     # ... and a dominant logit still later
    K[5, 3001, 0] = 0.0; K[5, 40, 0] = 200.0                  # one sequence has it in its very first stage
    lens_t = torch.full((b,), m_max, dtype=torch.int32, device=DEV)
    o = torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV)
    mqa.mqa_decode_step(q, K, inp["V"], lens_t, o, mqa.alloc_workspace(b, h, m_max, DEV))
    torch.cuda.synchronize()
    star = torch.full((b,), 3001, device=DEV); star[5] = 40
    want = inp["V"][torch.arange(b, device=DEV), star].float()[:, None, :].expand(b, h, 128)
    assert torch.equal(o, want.contiguous())                  # weight exactly 1 on that row, 0 elsewhere


@pytest.mark.parametrize("chained", [True, "wrong-guess"])
@pytest.mark.parametrize("b,h,m_max", [(40, 16, 2048), (32, 32, 4096), (33, 64, 2100), (256, 8, 1100)])
def test_chained_steps_in_a_loop_match_unchained_ones_and_the_oracle(b, h, m_max, chained):
    """A decoding loop whose steps carry the promise that lets the kernel fetch the cache before the step ahead of it
    has finished.  lens moves under every early guess (each step advances it), prefixes cross tile and stage
    boundaries on the way, one sequence fills up; with "wrong-guess" every early fetch is the wrong one and is redone."""
    steps = 70
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=31, device=DEV)
    r = np.random.default_rng(31)
    lens0 = r.integers(m_max // 2, m_max - steps - 1, size=b).astype(np.int32)
    lens0[0] = 4 * 128 - 3                                    # crosses a stage boundary after three steps
    lens0[1] = m_max - 5                                      # fills up
    lens0[2] = 1                                              # a short prefix: nothing to fetch early
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    gen = torch.Generator(device=DEV).manual_seed(32)
    qs = [wl.bf16_normal((b, h, 128), 128 ** -0.5, gen, DEV) for _ in range(steps)]
    ks = [wl.bf16_normal((b, 128), 1.0, gen, DEV) for _ in range(steps)]
    vs = [wl.bf16_normal((b, 128), 1.0, gen, DEV) for _ in range(steps)]
    results = {}
    for mode in (False, chained):
        K, V = inp["K"].clone(), inp["V"].clone()
        lens_t = torch.from_numpy(lens0.copy()).to(DEV)
        ws = mqa.alloc_workspace(b, h, m_max, DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        outs = [torch.empty(b, h, 128, dtype=torch.float32, device=DEV) for _ in range(steps)]
        torch.cuda.synchronize()
        for t in range(steps):                                # back to back: each kernel starts under the one before
            mqa.mqa_decode_append_step(qs[t], K, V, ks[t], vs[t], lens_t, outs[t], ws, status, advance=True,
                                       chained=mode if t > 0 else False)    # the first step follows the set-up copies
        torch.cuda.synchronize()
        results[mode] = (K, V, lens_t, outs, int(status.item()))
    Ka, Va, la, oa, sa = results[False]
    Kc, Vc, lc, oc, sc = results[chained]
    assert sa == sc and torch.equal(la, lc)
    assert torch.equal(Ka.view(torch.int16), Kc.view(torch.int16)) and torch.equal(Va.view(torch.int16), Vc.view(torch.int16))
    for t in range(steps):
        assert torch.equal(oa[t].view(torch.int32), oc[t].view(torch.int32)), f"step {t}"
    # and the loop itself against the oracle, at a few steps
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    for t in range(steps):
        oracle.kv_cache_append(Kh, Vh, wl.bits(ks[t]), wl.bits(vs[t]), lens_h, True)
        if t in (0, 3, 4, steps - 1):
            ref = oracle.mqa_decode_step(wl.bits(qs[t]), Kh, Vh, lens_h)
            check_close(oc[t].cpu().numpy(), ref, f"chained step {t}")
    assert np.array_equal(lc.cpu().numpy(), lens_h)
    assert np.array_equal(wl.bits(Kc), Kh) and np.array_equal(wl.bits(Vc), Vh)


def test_chained_steps_replayed_from_a_graph():
    b, h, m_max, per_graph, replays = 32, 32, 4096, 4, 3
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=41, device=DEV)
    lens0 = np.full(b, 3 * 128 - 5, np.int32)                 # every sequence crosses a stage boundary together
    lens0[5] = m_max - 3
    wl.poison_tail(inp["K"], lens0); wl.poison_tail(inp["V"], lens0)
    Kh, Vh, lens_h = wl.bits(inp["K"]), wl.bits(inp["V"]), lens0.copy()
    lens_t = torch.from_numpy(lens0).to(DEV)
    o = torch.zeros(b, h, 128, dtype=torch.float32, device=DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    step = lambda chained: mqa.mqa_decode_append_step(inp["q"], inp["K"], inp["V"], inp["k_new"], inp["v_new"], lens_t, o, ws,
                                                      status, advance=True, chained=chained)
    side = torch.cuda.Stream(device=DEV)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(False)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(per_graph):
            step(True)                                        # in a replay the step before is the previous replay's last
    for _ in range(replays):
        graph.replay()
    torch.cuda.synchronize()
    k_new, v_new = wl.bits(inp["k_new"]), wl.bits(inp["v_new"])
    for _ in range(1 + per_graph * replays):
        oracle.kv_cache_append(Kh, Vh, k_new, v_new, lens_h, True)
    assert np.array_equal(lens_t.cpu().numpy(), lens_h)
    assert np.array_equal(wl.bits(inp["K"]), Kh) and np.array_equal(wl.bits(inp["V"]), Vh)
    check_close(o.cpu().numpy(), oracle.mqa_decode_step(wl.bits(inp["q"]), Kh, Vh, lens_h), "last chained step of the replayed graph")


def test_unknown_step_flags_are_refused():
    b, h, m_max = 8, 8, 256
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=1, device=DEV)
    lens_t = torch.full((b,), 7, dtype=torch.int32, device=DEV)
    o = torch.zeros(b, h, 128, dtype=torch.float32, device=DEV)
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    from paper_1911_02150_b200 import binding
    rc = binding.lib().mqa_decode_append_step(inp["q"].data_ptr(), inp["K"].data_ptr(), inp["V"].data_ptr(), inp["k_new"].data_ptr(),
                                              inp["v_new"].data_ptr(), lens_t.data_ptr(), 16, o.data_ptr(), ws.data_ptr(), ws.numel(),
                                              None, b, h, m_max, 128, 128, None)
    assert rc == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(lens_t[0]) == 7 and float(o.abs().max()) == 0.0


def test_chained_steps_of_the_paper_shaped_loop():
    """128 sequences, 8 heads, a cache growing from nothing to 128 rows (Section 4.1), every step after the first
    carrying the promise: the one-CTA-per-sequence kernel fetches its lower tiles ahead of the wait."""
    b, h, m_max, steps = 128, 8, 128, 128
    inp = wl.make_inputs(b, h, m_max, "mqa", seed=51, device=DEV)
    gen = torch.Generator(device=DEV).manual_seed(52)
    qs = [wl.bf16_normal((b, h, 128), 128 ** -0.5, gen, DEV) for _ in range(steps)]
    ks = [wl.bf16_normal((b, 128), 1.0, gen, DEV) for _ in range(steps)]
    vs = [wl.bf16_normal((b, 128), 1.0, gen, DEV) for _ in range(steps)]
    nan = torch.tensor(wl.NAN_BITS, dtype=torch.int16, device=DEV)
    runs = {}
    for chained in (False, True):
        K, V = torch.empty_like(inp["K"]), torch.empty_like(inp["V"])
        K.view(torch.int16).fill_(nan); V.view(torch.int16).fill_(nan)
        lens_t = torch.zeros(b, dtype=torch.int32, device=DEV)
        lens_t[3] = 100                                       # one sequence starts with a prefix (of NaN rows it never reads: replaced below)
        K[3, :100] = wl.bf16_normal((100, 128), 1.0, gen, DEV) if not runs else runs[False][3][3, :100]
        V[3, :100] = wl.bf16_normal((100, 128), 1.0, gen, DEV) if not runs else runs[False][4][3, :100]
        K0, V0 = K.clone(), V.clone()
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        ws = mqa.alloc_workspace(b, h, m_max, DEV)
        outs = [torch.empty(b, h, 128, dtype=torch.float32, device=DEV) for _ in range(steps)]
        torch.cuda.synchronize()
        for t in range(steps):
            mqa.mqa_decode_append_step(qs[t], K, V, ks[t], vs[t], lens_t, outs[t], ws, status, advance=True,
                                       chained=chained and t > 0)
        torch.cuda.synchronize()
        runs[chained] = (outs, K, lens_t, K0, V0, V, int(status.item()))
    for t in range(steps):
        assert torch.equal(runs[False][0][t].view(torch.int32), runs[True][0][t].view(torch.int32)), f"step {t}"
    assert torch.equal(runs[False][1].view(torch.int16), runs[True][1].view(torch.int16))
    assert torch.equal(runs[False][2], runs[True][2]) and runs[False][6] == runs[True][6]
    # the chained loop against the oracle at a few steps (sequence 3 fills up after 28 steps and takes no more rows)
    Kh, Vh = wl.bits(runs[True][3]), wl.bits(runs[True][4])
    lens_h = np.zeros(b, np.int32); lens_h[3] = 100
    for t in range(steps):
        oracle.kv_cache_append(Kh, Vh, wl.bits(ks[t]), wl.bits(vs[t]), lens_h, True)
        if t in (0, 1, 31, 32, 33, 64, steps - 1):
            ref = oracle.mqa_decode_step(wl.bits(qs[t]), Kh, Vh, lens_h)
            check_close(runs[True][0][t].cpu().numpy(), ref, f"paper-shaped chained step {t}")
    assert np.array_equal(runs[True][2].cpu().numpy(), lens_h)
    assert runs[True][6] == mqa.binding.STATUS_APPEND_CACHE_FULL


def test_the_configuration_the_bench_times_at_full_size():
    """Long-context workload at full size (b=32, h=32, 8192-row caches), launched as the bench launches it: steps bound
    once per cache set (AppendStep), chained, lens not advanced, two cache sets in rotation, replayed from a CUDA graph.
    Every step's output for its set against the oracle (all sequences, all heads), and the appended rows bit for bit."""
    w = wl.WORKLOADS["long_context"]
    b, h, m_max = w.b, w.h, w.m_max
    lens0 = wl.initial_lens(w, seed=0)
    sets = [wl.make_inputs(b, h, m_max, "mqa", seed=60 + i, device=DEV) for i in range(2)]
    before = [(wl.bits(s["K"]), wl.bits(s["V"])) for s in sets]
    lens_t = torch.from_numpy(lens0).to(DEV)
    outs = [torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV) for _ in sets]
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert mqa.append_step_launches(b, h, m_max) == 1
    steps = [mqa.AppendStep(s["q"], s["K"], s["V"], s["k_new"], s["v_new"], lens_t, o, ws, status, advance=False, chained=True)
             for s, o in zip(sets, outs)]
    side = torch.cuda.Stream(device=DEV)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(4):
            steps[i % 2](side)                                # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for o in outs:
        o.fill_(float("nan"))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(6):
            steps[i % 2](torch.cuda.current_stream())
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and np.array_equal(lens_t.cpu().numpy(), lens0)
    for s, o, (Kb, Vb) in zip(sets, outs, before):
        Kh, Vh, lens_h = Kb.copy(), Vb.copy(), lens0.copy()
        oracle.kv_cache_append(Kh, Vh, wl.bits(s["k_new"]), wl.bits(s["v_new"]), lens_h, True)
        assert np.array_equal(wl.bits(s["K"]), Kh) and np.array_equal(wl.bits(s["V"]), Vh)
        check_close(o.cpu().numpy(), oracle.mqa_decode_step(wl.bits(s["q"]), Kh, Vh, lens_h), "bench configuration")


@pytest.mark.parametrize("rows", [64, 128])
def test_the_many_rows_step_the_bench_times_at_full_size(rows):
    """4 beams x 32 heads (and 64 rows) over the long-context workload's caches, as the bench's many-rows block launches
    it: the append-and-attend step, lens not advanced, replayed from a CUDA graph over two cache sets.  Every output
    against the oracle (all sequences, all rows), and the appended rows bit for bit."""
    w = wl.WORKLOADS["long_context"]
    b, h, m_max = w.b, rows, w.m_max
    lens0 = wl.initial_lens(w, seed=0)
    sets = [wl.make_inputs(b, h, m_max, "mqa", seed=80 + i, device=DEV) for i in range(2)]
    before = [(wl.bits(s["K"]), wl.bits(s["V"])) for s in sets]
    lens_t = torch.from_numpy(lens0).to(DEV)
    outs = [torch.full((b, h, 128), float("nan"), dtype=torch.float32, device=DEV) for _ in sets]
    ws = mqa.alloc_workspace(b, h, m_max, DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    assert mqa.plan_kernel_name(True, True, b, h, m_max) == "mqa_decode_wide_kernel"
    steps = [mqa.AppendStep(s["q"], s["K"], s["V"], s["k_new"], s["v_new"], lens_t, o, ws, status, advance=False, chained=True)
             for s, o in zip(sets, outs)]
    side = torch.cuda.Stream(device=DEV)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(4):
            steps[i % 2](side)                                # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for o in outs:
        o.fill_(float("nan"))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(6):
            steps[i % 2](torch.cuda.current_stream())
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and np.array_equal(lens_t.cpu().numpy(), lens0)
    for s, o, (Kb, Vb) in zip(sets, outs, before):
        Kh, Vh, lens_h = Kb.copy(), Vb.copy(), lens0.copy()
        oracle.kv_cache_append(Kh, Vh, wl.bits(s["k_new"]), wl.bits(s["v_new"]), lens_h, True)
        assert np.array_equal(wl.bits(s["K"]), Kh) and np.array_equal(wl.bits(s["V"]), Vh)
        check_close(o.cpu().numpy(), oracle.mqa_decode_step(wl.bits(s["q"]), Kh, Vh, lens_h), f"many rows ({rows}) at the bench's size")
