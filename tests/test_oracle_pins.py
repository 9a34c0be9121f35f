"""Pins for the CPU oracle: each test ties an oracle function to something fixed by the
paper or by mathematics, not to the oracle itself.

  brute-force einsum (Section 2.1's definition of einsum)   every contraction and index order
  closed forms                                             softmax normalisation, exp, sign
  reductions (one head == Section 2.1; MQA == MHA with
  shared K,V, Section 3; incremental == causal batched,
  Sections 2.3/2.4/3)                                      head/cache indexing, append order
  a library routine (torch SDPA, fp64, scale 1)            the whole step
  invariants                                               shift, permutation, convexity, mask
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import paper_functions as pf

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- helpers
def bf16_bits(x):
    """fp64 array -> (uint16 bf16 bit patterns, the fp64 values those patterns hold)."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float64)).to(torch.bfloat16)
    b = t.contiguous().view(torch.int16).numpy().view(np.uint16).copy()
    return b, t.to(torch.float64).numpy()


def brute_einsum(eq, *ops):
    """einsum exactly as the paper words it: broadcast every operand to the union of all
    index letters, multiply component-wise, sum over the letters absent from the output.
    Pure Python loops over the full index space; tiny shapes only."""
    lhs, out = eq.split("->")
    terms = lhs.split(",")
    size = {}
    for t, a in zip(terms, ops):
        assert len(t) == np.ndim(a)
        for ax, letter in enumerate(t):
            assert size.setdefault(letter, a.shape[ax]) == a.shape[ax]
    letters = sorted(size)
    res = np.zeros([size[c] for c in out], dtype=np.float64)
    for idx in itertools.product(*[range(size[c]) for c in letters]):
        at = dict(zip(letters, idx))
        prod = 1.0
        for t, a in zip(terms, ops):
            prod *= float(a[tuple(at[c] for c in t)])
        res[tuple(at[c] for c in out)] += prod
    return res


def brute_softmax_last(x):
    e = np.exp(x)                       # plain definition, no max shift (tiny logits only)
    return e / e.sum(axis=-1, keepdims=True)


def rng(seed):
    return np.random.default_rng(seed)


def step_inputs(b, h, m_max, k, v, variant, seed, scale_q=None):
    r = rng(seed)
    sq = (k ** -0.5) if scale_q is None else scale_q
    cache = (b, m_max) if variant == "mqa" else (b, h, m_max)
    qb, qf = bf16_bits(r.normal(size=(b, h, k)) * sq)
    Kb, Kf = bf16_bits(r.normal(size=cache + (k,)))
    Vb, Vf = bf16_bits(r.normal(size=cache + (v,)))
    return (qb, Kb, Vb), (qf, Kf, Vf)


# ------------------------------------------------------------ closed forms (golden file)
def read_golden_cases():
    """tests/golden/closed_form_cases.txt: hand-derived cases, one per block."""
    cases, cur = [], {}
    with open(os.path.join(GOLDEN, "closed_form_cases.txt")) as f:
        for line in f:
            if line.lstrip().startswith("#"):
                continue
            line = line.split("#", 1)[0].strip()
            if not line:
                if cur:
                    cases.append(cur)
                    cur = {}
                continue
            key, val = line.split(":", 1)
            cur[key.strip()] = val.strip()
    if cur:
        cases.append(cur)
    return cases


def _expr(s):
    return eval(s, {"__builtins__": {}}, {"ln": math.log, "e": math.e, "exp": math.exp})


@pytest.mark.parametrize("case", read_golden_cases(), ids=lambda c: c["name"])
def test_closed_form_cases(case):
    q = np.array(_expr(case["q"]), dtype=np.float64)
    K = np.array(_expr(case["K"]), dtype=np.float64)
    V = np.array(_expr(case["V"]), dtype=np.float64)
    want = np.array(_expr(case["y"]), dtype=np.float64)
    got = oracle.dot_product_attention(q, K, V)
    np.testing.assert_allclose(got, want, rtol=1e-14, atol=1e-14)
    np.testing.assert_allclose(pf.attend(q, K, V), want, rtol=1e-14, atol=1e-14)
    # the same case through the bf16 step functions when every number is bf16-exact
    if case.get("bf16_exact", "no") == "yes":
        qb, _ = bf16_bits(q[None, None, :])
        Kb, _ = bf16_bits(K[None])
        Vb, _ = bf16_bits(V[None])
        lens = np.array([K.shape[0]], dtype=np.int32)
        np.testing.assert_allclose(oracle.mqa_decode_step(qb, Kb, Vb, lens)[0, 0], want, rtol=1e-14, atol=1e-14)
        np.testing.assert_allclose(oracle.mha_decode_step(qb, Kb[:, None], Vb[:, None], lens)[0, 0], want,
                                   rtol=1e-14, atol=1e-14)


# ---------------------------------------------------------------- brute force, tiny shapes
@pytest.mark.parametrize("m,k,v", [(1, 1, 1), (2, 3, 1), (3, 2, 4), (4, 3, 2)])
def test_single_query_vs_brute_einsum(m, k, v):
    r = rng(10 + m)
    q, K, V = r.normal(size=k), r.normal(size=(m, k)), r.normal(size=(m, v))
    logits = brute_einsum("k,mk->m", q, K)
    y = brute_einsum("m,mv->v", brute_softmax_last(logits), V)
    np.testing.assert_allclose(oracle.dot_product_attention(q, K, V), y, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(pf.attend(q, K, V), y, rtol=1e-13, atol=1e-14)


@pytest.mark.parametrize("b,h,m,k,v", [(1, 1, 1, 1, 1), (2, 3, 4, 2, 3), (3, 2, 3, 3, 2)])
def test_mqa_step_vs_brute_einsum(b, h, m, k, v):
    (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, "mqa", seed=20 + b, scale_q=1.0)
    logits = brute_einsum("bhk,bmk->bhm", q, K)
    o = brute_einsum("bhm,bmv->bhv", brute_softmax_last(logits), V)
    got = oracle.mqa_decode_step(qb, Kb, Vb, np.full(b, m, np.int32))
    np.testing.assert_allclose(got, o, rtol=1e-13, atol=1e-14)


@pytest.mark.parametrize("b,h,m,k,v", [(1, 1, 1, 1, 1), (2, 3, 4, 2, 3), (3, 2, 3, 3, 2)])
def test_mha_step_vs_brute_einsum(b, h, m, k, v):
    (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, "mha", seed=30 + b, scale_q=1.0)
    logits = brute_einsum("bhk,bhmk->bhm", q, K)
    o = brute_einsum("bhm,bhmv->bhv", brute_softmax_last(logits), V)
    got = oracle.mha_decode_step(qb, Kb, Vb, np.full(b, m, np.int32))
    np.testing.assert_allclose(got, o, rtol=1e-13, atol=1e-14)


def test_ragged_prefix_vs_brute_einsum_with_additive_mask():
    """The valid-prefix rule is the additive -inf mask of Section 2.3 with the illegal
    positions being j >= lens[b]."""
    b, h, m, k, v = 3, 2, 4, 2, 3
    (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, "mqa", seed=41, scale_q=1.0)
    lens = np.array([1, 4, 2], dtype=np.int32)
    logits = brute_einsum("bhk,bmk->bhm", q, K)
    mask = np.where(np.arange(m)[None, None, :] < lens[:, None, None], 0.0, -np.inf)
    with np.errstate(over="ignore"):
        w = brute_softmax_last(logits + mask)
    o = brute_einsum("bhm,bmv->bhv", w, V)
    np.testing.assert_allclose(oracle.mqa_decode_step(qb, Kb, Vb, lens), o, rtol=1e-13, atol=1e-14)


def test_multihead_attention_with_projections_vs_brute_einsum():
    r = rng(50)
    h, d, k, v, m = 2, 3, 2, 3, 4
    x, M = r.normal(size=d), r.normal(size=(m, d))
    P_q, P_k = r.normal(size=(h, d, k)), r.normal(size=(h, d, k))
    P_v, P_o = r.normal(size=(h, d, v)), r.normal(size=(h, d, v))
    q = brute_einsum("d,hdk->hk", x, P_q)
    K = brute_einsum("md,hdk->hmk", M, P_k)
    V = brute_einsum("md,hdv->hmv", M, P_v)
    w = brute_softmax_last(brute_einsum("hk,hmk->hm", q, K))
    y = brute_einsum("hv,hdv->d", brute_einsum("hm,hmv->hv", w, V), P_o)
    np.testing.assert_allclose(pf.multihead_attention(x, M, P_q, P_k, P_v, P_o), y, rtol=1e-12, atol=1e-13)


def test_batched_functions_vs_brute_einsum():
    r = rng(51)
    b, n, m, h, d, k, v = 2, 2, 3, 2, 3, 2, 2
    X, M = r.normal(size=(b, n, d)), r.normal(size=(b, m, d))
    mask = np.zeros((b, h, n, m))
    mask[0, :, 0, 2] = -np.inf
    mask[1, 1, 1, 0] = -np.inf
    P_q, P_o = r.normal(size=(h, d, k)), r.normal(size=(h, d, v))
    # multi-head
    P_k, P_v = r.normal(size=(h, d, k)), r.normal(size=(h, d, v))
    Q = brute_einsum("bnd,hdk->bhnk", X, P_q)
    K = brute_einsum("bmd,hdk->bhmk", M, P_k)
    V = brute_einsum("bmd,hdv->bhmv", M, P_v)
    w = brute_softmax_last(brute_einsum("bhnk,bhmk->bhnm", Q, K) + mask)
    Y = brute_einsum("bhnv,hdv->bnd", brute_einsum("bhnm,bhmv->bhnv", w, V), P_o)
    np.testing.assert_allclose(pf.multihead_attention_batched(X, M, mask, P_q, P_k, P_v, P_o), Y,
                               rtol=1e-12, atol=1e-13)
    # multi-query: P_k, P_v lose the heads axis
    P_k1, P_v1 = r.normal(size=(d, k)), r.normal(size=(d, v))
    K1 = brute_einsum("bmd,dk->bmk", M, P_k1)
    V1 = brute_einsum("bmd,dv->bmv", M, P_v1)
    w1 = brute_softmax_last(brute_einsum("bhnk,bmk->bhnm", Q, K1) + mask)
    Y1 = brute_einsum("bhnv,hdv->bnd", brute_einsum("bhnm,bmv->bhnv", w1, V1), P_o)
    np.testing.assert_allclose(pf.multiquery_attention_batched(X, M, mask, P_q, P_k1, P_v1, P_o), Y1,
                               rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------------- reductions
def test_one_head_is_single_query_attention():
    b, h, m, k, v = 3, 4, 37, 128, 128
    for variant in ("mqa", "mha"):
        (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, variant, seed=60)
        lens = np.array([37, 1, 20], dtype=np.int32)
        fn = oracle.mqa_decode_step if variant == "mqa" else oracle.mha_decode_step
        o = fn(qb, Kb, Vb, lens)
        for s in range(b):
            for i in range(h):
                Ks = K[s] if variant == "mqa" else K[s, i]
                Vs = V[s] if variant == "mqa" else V[s, i]
                ref = oracle.dot_product_attention(q[s, i], Ks[: lens[s]], Vs[: lens[s]])
                np.testing.assert_allclose(o[s, i], ref, rtol=1e-13, atol=1e-15)
                np.testing.assert_allclose(o[s, i], pf.attend(q[s, i], Ks[: lens[s]], Vs[: lens[s]]),
                                           rtol=1e-12, atol=1e-15)


def test_mqa_equals_mha_with_replicated_cache():
    b, h, m, k, v = 2, 8, 50, 128, 128
    (qb, Kb, Vb), _ = step_inputs(b, h, m, k, v, "mqa", seed=61)
    lens = np.array([50, 13], dtype=np.int32)
    Krep = np.ascontiguousarray(np.broadcast_to(Kb[:, None], (b, h, m, k)))
    Vrep = np.ascontiguousarray(np.broadcast_to(Vb[:, None], (b, h, m, v)))
    a = oracle.mqa_decode_step(qb, Kb, Vb, lens)
    c = oracle.mha_decode_step(qb, Krep, Vrep, lens)
    assert np.array_equal(a, c)


def test_mha_heads_use_their_own_cache():
    """Swapping two heads' caches and queries swaps their outputs and nothing else."""
    b, h, m, k, v = 1, 3, 9, 128, 128
    (qb, Kb, Vb), _ = step_inputs(b, h, m, k, v, "mha", seed=62)
    lens = np.array([9], dtype=np.int32)
    o = oracle.mha_decode_step(qb, Kb, Vb, lens)
    perm = [2, 1, 0]
    o2 = oracle.mha_decode_step(qb[:, perm], Kb[:, perm], Vb[:, perm], lens)
    assert np.array_equal(o2, o[:, perm])
    assert not np.allclose(o[0, 0], o[0, 2])


def test_library_sdpa_fp64():
    """torch's scaled_dot_product_attention (CPU, fp64, scale 1) is the same function."""
    b, h, m, k, v = 2, 4, 33, 128, 128
    (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, "mha", seed=63)
    lens = np.full(b, m, np.int32)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[:, :, None, :], torch.from_numpy(K), torch.from_numpy(V), scale=1.0)[:, :, 0].numpy()
    np.testing.assert_allclose(oracle.mha_decode_step(qb, Kb, Vb, lens), ref, rtol=1e-12, atol=1e-14)
    (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, "mqa", seed=64)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[:, :, None, :], torch.from_numpy(K)[:, None].expand(b, h, m, k),
        torch.from_numpy(V)[:, None].expand(b, h, m, v), scale=1.0)[:, :, 0].numpy()
    np.testing.assert_allclose(oracle.mqa_decode_step(qb, Kb, Vb, lens), ref, rtol=1e-12, atol=1e-14)


def _causal_mask(b, h, n):
    allowed = np.arange(n)[None, :] <= np.arange(n)[:, None]       # position t sees j <= t
    return np.broadcast_to(np.where(allowed, 0.0, -np.inf), (b, h, n, n)).copy()


def test_incremental_equals_causal_batched_multihead():
    r = rng(70)
    b, n, h, d, k, v = 2, 6, 3, 5, 4, 3
    X = r.normal(size=(b, n, d))
    P_q, P_k = r.normal(size=(h, d, k)), r.normal(size=(h, d, k))
    P_v, P_o = r.normal(size=(h, d, v)), r.normal(size=(h, d, v))
    Y = pf.multihead_attention_batched(X, X, _causal_mask(b, h, n), P_q, P_k, P_v, P_o)
    K = np.zeros((b, h, 0, k))
    V = np.zeros((b, h, 0, v))
    for t in range(n):
        y, K, V = pf.multihead_self_attention_incremental(X[:, t], K, V, P_q, P_k, P_v, P_o)
        assert K.shape == (b, h, t + 1, k) and V.shape == (b, h, t + 1, v)
        np.testing.assert_allclose(y, Y[:, t], rtol=1e-12, atol=1e-13)


def test_incremental_equals_causal_batched_multiquery():
    r = rng(71)
    b, n, h, d, k, v = 2, 6, 3, 5, 4, 3
    X = r.normal(size=(b, n, d))
    P_q, P_o = r.normal(size=(h, d, k)), r.normal(size=(h, d, v))
    P_k, P_v = r.normal(size=(d, k)), r.normal(size=(d, v))
    Y = pf.multiquery_attention_batched(X, X, _causal_mask(b, h, n), P_q, P_k, P_v, P_o)
    K = np.zeros((b, 0, k))
    V = np.zeros((b, 0, v))
    for t in range(n):
        y, K, V = pf.multiquery_self_attention_incremental(X[:, t], K, V, P_q, P_k, P_v, P_o)
        assert K.shape == (b, t + 1, k) and V.shape == (b, t + 1, v)
        np.testing.assert_allclose(y, Y[:, t], rtol=1e-12, atol=1e-13)


def test_multiquery_is_multihead_with_one_shared_projection():
    r = rng(72)
    b, n, m, h, d, k, v = 2, 3, 4, 3, 5, 4, 2
    X, M = r.normal(size=(b, n, d)), r.normal(size=(b, m, d))
    mask = np.zeros((b, h, n, m))
    P_q, P_o = r.normal(size=(h, d, k)), r.normal(size=(h, d, v))
    P_k, P_v = r.normal(size=(d, k)), r.normal(size=(d, v))
    a = pf.multiquery_attention_batched(X, M, mask, P_q, P_k, P_v, P_o)
    c = pf.multihead_attention_batched(X, M, mask, P_q, np.stack([P_k] * h), np.stack([P_v] * h), P_o)
    np.testing.assert_allclose(a, c, rtol=1e-13, atol=1e-14)


def test_incremental_step_through_the_bf16_boundary():
    """A decoding loop in the hot path's own terms -- append the new row into a padded
    cache at lens[b], then attend over lens[b]+1 rows -- reproduces the paper's incremental
    function (with identity-like projections so that q, k_new, v_new are the inputs)."""
    b, h, k, v, steps, m_max = 2, 3, 128, 128, 5, 8
    r = rng(73)
    Kc = np.full((b, m_max, k), 0x7FC0, np.uint16)      # unwritten rows are NaN
    Vc = np.full((b, m_max, v), 0x7FC0, np.uint16)
    lens = np.zeros(b, np.int32)
    Kp = np.zeros((b, 0, k))
    Vp = np.zeros((b, 0, v))
    for t in range(steps):
        qb, qf = bf16_bits(r.normal(size=(b, h, k)) * k ** -0.5)
        knb, knf = bf16_bits(r.normal(size=(b, k)))
        vnb, vnf = bf16_bits(r.normal(size=(b, v)))
        assert oracle.kv_cache_append(Kc, Vc, knb, vnb, lens, advance=True) == 0
        assert np.all(lens == t + 1)
        o = oracle.mqa_decode_step(qb, Kc, Vc, lens)
        Kp = np.concatenate([Kp, knf[:, None]], axis=1)
        Vp = np.concatenate([Vp, vnf[:, None]], axis=1)
        for s in range(b):
            for i in range(h):
                np.testing.assert_allclose(o[s, i], pf.attend(qf[s, i], Kp[s], Vp[s]), rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------- closed-form behaviour
def test_identical_keys_give_mean_of_values():
    b, h, m, k, v = 2, 3, 11, 128, 128
    (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, "mqa", seed=80)
    Kb[:] = Kb[:, :1]                                   # every row equal to row 0
    lens = np.array([11, 7], np.int32)
    o = oracle.mqa_decode_step(qb, Kb, Vb, lens)
    for s in range(b):
        want = V[s, : lens[s]].mean(axis=0)
        for i in range(h):
            np.testing.assert_allclose(o[s, i], want, rtol=1e-13, atol=1e-15)


def test_dominant_logit_returns_that_value_row():
    m, k, v, star = 9, 128, 128, 5
    q = np.zeros((1, 1, k))
    q[0, 0, 0] = 1.0
    K = np.zeros((1, m, k))
    K[0, star, 0] = 200.0                               # logit 200 against zeros: e^-200 ~ 1e-87
    V = rng(81).normal(size=(1, m, v))
    qb, _ = bf16_bits(q)
    Kb, _ = bf16_bits(K)
    Vb, Vf = bf16_bits(V)
    o = oracle.mqa_decode_step(qb, Kb, Vb, np.array([m], np.int32))
    np.testing.assert_allclose(o[0, 0], Vf[0, star], rtol=0, atol=1e-80)
    # sign check: a dominant NEGATIVE logit must be ignored, not selected
    Kb2, _ = bf16_bits(-K)
    o2 = oracle.mqa_decode_step(qb, Kb2, Vb, np.array([m], np.int32))
    others = np.delete(Vf[0], star, axis=0).mean(axis=0)
    np.testing.assert_allclose(o2[0, 0], others, rtol=1e-13, atol=1e-15)


def test_two_row_sigmoid_closed_form():
    """Two rows whose logits differ by delta get weights sigmoid(-+delta)."""
    k = v = 128
    for delta in (0.0, 0.5, -3.0, 10.0):
        q = np.zeros((1, 1, k)); q[0, 0, 3] = 1.0
        K = np.zeros((1, 2, k)); K[0, 1, 3] = delta
        V = np.zeros((1, 2, v)); V[0, 0, :] = 1.0; V[0, 1, :] = -2.0
        qb, _ = bf16_bits(q); Kb, Kf = bf16_bits(K); Vb, _ = bf16_bits(V)
        dl = Kf[0, 1, 3]
        w1 = 1.0 / (1.0 + math.exp(-dl))
        want = (1 - w1) * 1.0 + w1 * (-2.0)
        o = oracle.mha_decode_step(qb, Kb[:, None], Vb[:, None], np.array([2], np.int32))
        np.testing.assert_allclose(o[0, 0], np.full(v, want), rtol=1e-14)


# --------------------------------------------------------------------------- invariants
def test_shift_permutation_and_convexity():
    b, h, m, k, v = 1, 4, 29, 128, 128
    (qb, Kb, Vb), (q, K, V) = step_inputs(b, h, m, k, v, "mqa", seed=90)
    lens = np.array([m], np.int32)
    o = oracle.mqa_decode_step(qb, Kb, Vb, lens)
    # convexity: each output coordinate lies between the extreme values of that column
    assert np.all(o[0] <= V[0].max(axis=0)[None] + 1e-15)
    assert np.all(o[0] >= V[0].min(axis=0)[None] - 1e-15)
    # joint permutation of the K and V rows leaves o unchanged (up to summation order)
    p = rng(91).permutation(m)
    o_p = oracle.mqa_decode_step(qb, np.ascontiguousarray(Kb[:, p]), np.ascontiguousarray(Vb[:, p]), lens)
    np.testing.assert_allclose(o_p, o, rtol=1e-12, atol=1e-15)
    # all V rows equal -> that row, whatever the weights
    Vc = np.ascontiguousarray(np.broadcast_to(Vb[:, :1], Vb.shape))
    o_c = oracle.mqa_decode_step(qb, Kb, Vc, lens)
    np.testing.assert_allclose(o_c[0], np.broadcast_to(V[0, 0], (h, v)), rtol=1e-13, atol=1e-15)
    # shift invariance: adding u to every key adds the constant q.u to every logit of a head
    qf = q[0, 0]
    u = np.zeros(k); u[7] = 4.0                         # bf16-exact shift on one coordinate
    Kshift = K[0] + u[None]
    y0 = oracle.dot_product_attention(qf, K[0], V[0])
    y1 = oracle.dot_product_attention(qf, Kshift, V[0])
    np.testing.assert_allclose(y1, y0, rtol=1e-11, atol=1e-14)


def test_rows_beyond_lens_are_never_read():
    b, h, m_max, k, v = 3, 2, 16, 128, 128
    (qb, Kb, Vb), _ = step_inputs(b, h, m_max, k, v, "mqa", seed=92)
    lens = np.array([5, 16, 0], np.int32)
    base = oracle.mqa_decode_step(qb, Kb, Vb, lens)
    Kn, Vn, Kz, Vz = Kb.copy(), Vb.copy(), Kb.copy(), Vb.copy()
    for s in range(b):
        Kn[s, lens[s]:] = 0x7FC0; Vn[s, lens[s]:] = 0x7FC0          # NaN
        Kz[s, lens[s]:] = 0x7F80; Vz[s, lens[s]:] = 0xFF80          # +inf / -inf
    assert np.array_equal(oracle.mqa_decode_step(qb, Kn, Vn, lens), base)
    assert np.array_equal(oracle.mqa_decode_step(qb, Kz, Vz, lens), base)
    assert np.all(np.isfinite(base))
    assert np.all(base[2] == 0.0)                                   # empty prefix -> zeros
    # truncating the cache to the longest prefix changes nothing either
    (qb1, Kb1, Vb1) = qb[:1], Kb[:1, :5], Vb[:1, :5]
    assert np.array_equal(oracle.mqa_decode_step(qb1, np.ascontiguousarray(Kb1), np.ascontiguousarray(Vb1),
                                                 np.array([5], np.int32)), base[:1])
    # multi-head form
    (qb, Kb, Vb), _ = step_inputs(b, h, m_max, k, v, "mha", seed=93)
    base = oracle.mha_decode_step(qb, Kb, Vb, lens)
    Kn, Vn = Kb.copy(), Vb.copy()
    for s in range(b):
        Kn[s, :, lens[s]:] = 0x7FC0; Vn[s, :, lens[s]:] = 0x7FC0
    assert np.array_equal(oracle.mha_decode_step(qb, Kn, Vn, lens), base)


def test_split_and_recombine_is_exact():
    r = rng(94)
    m, k, v = 53, 16, 8
    q, K, V = r.normal(size=k), r.normal(size=(m, k)) * 2, r.normal(size=(m, v))
    whole = oracle.dot_product_attention(q, K, V)
    for cuts in ([0, 53], [0, 1, 53], [0, 7, 8, 30, 53], list(range(54))):
        parts = []
        for a, z in zip(cuts[:-1], cuts[1:]):
            lg = K[a:z] @ q
            top = lg.max()
            w = np.exp(lg - top)
            parts.append((top, w.sum(), w @ V[a:z]))
        np.testing.assert_allclose(pf.combine_partials(parts), whole, rtol=1e-13, atol=1e-15)


# ------------------------------------------------------------------------------ append
@pytest.mark.parametrize("kvh", [1, 3])
def test_append_writes_exactly_one_row_bit_exact(kvh):
    b, m_max, k, v = 4, 6, 128, 128
    r = rng(95)
    shape = (b, m_max) if kvh == 1 else (b, kvh, m_max)
    K = r.integers(0, 1 << 16, size=shape + (k,), dtype=np.uint16)
    V = r.integers(0, 1 << 16, size=shape + (v,), dtype=np.uint16)
    new_shape = (b,) if kvh == 1 else (b, kvh)
    k_new = r.integers(0, 1 << 16, size=new_shape + (k,), dtype=np.uint16)
    v_new = r.integers(0, 1 << 16, size=new_shape + (v,), dtype=np.uint16)
    # awkward bit patterns must survive: -0.0, a subnormal, NaNs with payloads, infinities
    k_new[..., :6] = np.array([0x8000, 0x0001, 0x7FC1, 0xFFFF, 0x7F80, 0xFF80], np.uint16)
    lens = np.array([0, 5, 6, 3], np.int32)             # sequence 2 is full -> skipped
    K0, V0, lens0 = K.copy(), V.copy(), lens.copy()
    skipped = oracle.kv_cache_append(K, V, k_new, v_new, lens, advance=True)
    assert skipped == 1
    assert np.array_equal(lens, np.array([1, 6, 6, 4], np.int32))
    K4, V4 = K.reshape(b, kvh, m_max, k), V.reshape(b, kvh, m_max, v)
    K04, V04 = K0.reshape(b, kvh, m_max, k), V0.reshape(b, kvh, m_max, v)
    kn, vn = k_new.reshape(b, kvh, k), v_new.reshape(b, kvh, v)
    for s in range(b):
        for g in range(kvh):
            for row in range(m_max):
                if s != 2 and row == lens0[s]:
                    assert np.array_equal(K4[s, g, row], kn[s, g])
                    assert np.array_equal(V4[s, g, row], vn[s, g])
                else:
                    assert np.array_equal(K4[s, g, row], K04[s, g, row])
                    assert np.array_equal(V4[s, g, row], V04[s, g, row])
    # advance = False leaves lens alone; negative lens is skipped too
    lens2 = np.array([0, -1, 2, 2], np.int32)
    keep = lens2.copy()
    assert oracle.kv_cache_append(K, V, k_new, v_new, lens2, advance=False) == 1
    assert np.array_equal(lens2, keep)


def test_threads_are_reported_and_do_not_change_results():
    (qb, Kb, Vb), _ = step_inputs(4, 4, 40, 128, 128, "mqa", seed=96)
    lens = np.array([40, 3, 17, 29], np.int32)
    n = oracle.num_threads()
    assert n >= 1
    a = oracle.mqa_decode_step(qb, Kb, Vb, lens)
    oracle.set_num_threads(1)
    c = oracle.mqa_decode_step(qb, Kb, Vb, lens)
    oracle.set_num_threads(n)
    assert np.array_equal(a, c)


# ---------------------------------------------------------------------------------------------
# The whole-layer oracle (projections either side of the step), Section 3
# ---------------------------------------------------------------------------------------------
def _layer_case(seed, b=3, h=4, d=24, k=8, v=8, m=5):
    from oracle import layer_step as ls
    r = np.random.default_rng(seed)
    def bf(shape, std):
        return ls.f64_to_bf16_bits(r.normal(0.0, std, size=shape))
    x, Pq, Pk, Pv, Po = bf((b, d), 1.0), bf((h, d, k), d ** -0.5), bf((d, k), d ** -0.5), bf((d, v), d ** -0.5), bf((h, d, v), (h * v) ** -0.5)
    K, V = bf((b, m + 1, k), 1.0), bf((b, m + 1, v), 1.0)
    return ls, x, Pq, Pk, Pv, Po, K, V, m


def test_layer_oracle_without_interface_roundings_is_the_papers_incremental_function():
    ls, x, Pq, Pk, Pv, Po, K, V, m = _layer_case(11)
    b = x.shape[0]
    lens = np.full(b, m, np.int32)
    Kc, Vc = K.copy(), V.copy()
    y, qb, kb, vb = ls.multiquery_layer_decode_step(x, Pq, Pk, Pv, Po, Kc, Vc, lens, round_interfaces=False)
    f = ls.bf16_to_f64
    # the paper's function keeps the new row unrounded; give it the row as the bf16 cache holds it by projecting
    # with the same inputs and checking the two agree to bf16 precision on the row, exactly on everything else
    y_ref, K_ref, V_ref = pf.multiquery_self_attention_incremental(f(x), f(K[:, :m]), f(V[:, :m]), f(Pq), f(Pk), f(Pv), f(Po))
    assert np.array_equal(lens, np.full(b, m + 1))
    assert np.array_equal(Kc[:, :m], K[:, :m]) and np.array_equal(Vc[:, :m], V[:, :m])
    np.testing.assert_allclose(f(Kc[:, m]), K_ref[:, m], rtol=2 ** -8, atol=1e-30)       # one bf16 rounding of the new row
    np.testing.assert_allclose(f(Vc[:, m]), V_ref[:, m], rtol=2 ** -8, atol=1e-30)
    # attending, head by head with the paper's single-query function, over the cache as stored (rounded row): y to fp64
    Kf, Vf = f(Kc), f(Vc)
    y_chk = np.zeros_like(y)
    for s in range(b):
        for i in range(Pq.shape[0]):
            y_chk[s] += f(Po)[i] @ pf.attend(f(x)[s] @ f(Pq)[i], Kf[s], Vf[s])
    np.testing.assert_allclose(y, y_chk, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(y, y_ref, rtol=0, atol=2e-2)                             # the row's rounding moves y only slightly


def test_layer_oracle_interface_roundings_are_small_and_where_stated():
    ls, x, Pq, Pk, Pv, Po, K, V, m = _layer_case(12)
    b = x.shape[0]
    y0, qb0, kb0, vb0 = ls.multiquery_layer_decode_step(x, Pq, Pk, Pv, Po, K.copy(), V.copy(), np.full(b, m, np.int32), round_interfaces=False)
    y1, qb1, kb1, vb1 = ls.multiquery_layer_decode_step(x, Pq, Pk, Pv, Po, K.copy(), V.copy(), np.full(b, m, np.int32), round_interfaces=True)
    assert np.array_equal(qb0, qb1) and np.array_equal(kb0, kb1) and np.array_equal(vb0, vb1)
    assert 0 < np.abs(y0 - y1).max() < 2e-2
    f = ls.bf16_to_f64
    assert np.array_equal(ls.f64_to_bf16_bits(f(qb1)), qb1)                              # rounding is idempotent
    # ties to even, and exactness of the widening
    assert ls.f64_to_bf16_bits(np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8]))[0] == 0x3F80 and ls.f64_to_bf16_bits(np.array([1.0 + 3 * 2 ** -8]))[0] == 0x3F82
    assert f(np.array([0x3F80, 0xC000], np.uint16)).tolist() == [1.0, -2.0]


def test_layer_oracle_empty_and_full_sequences():
    ls, x, Pq, Pk, Pv, Po, K, V, m = _layer_case(13)
    b = x.shape[0]
    lens = np.array([0, m, m + 1], np.int32)                                            # first token; normal; cache full
    Kc, Vc = K.copy(), V.copy()
    y, _, kb, vb = ls.multiquery_layer_decode_step(x, Pq, Pk, Pv, Po, Kc, Vc, lens)
    assert lens.tolist() == [1, m + 1, m + 1]
    assert np.array_equal(Kc[0, 0], kb[0]) and np.array_equal(Kc[2], K[2])              # row 0 written; full cache untouched
    f = ls.bf16_to_f64
    # a single row: the output is that value row, whatever the query
    o_single = f(ls.f64_to_bf16_bits(f(vb[0])))
    np.testing.assert_allclose(y[0], np.einsum("hv,hdv->d", np.tile(o_single, (Pq.shape[0], 1)), f(Po)), rtol=1e-12, atol=1e-13)


# ------------------------------------------- the batched multi-query attention lines (Section 3) under the causal mask
def _batched_inputs(b, h, n, m_max, k, v, seed):
    r = rng(seed)
    Qb, Qf = bf16_bits(r.normal(size=(b, h, n, k)) * k ** -0.5)
    Kb, Kf = bf16_bits(r.normal(size=(b, m_max, k)))
    Vb, Vf = bf16_bits(r.normal(size=(b, m_max, v)))
    return (Qb, Kb, Vb), (Qf, Kf, Vf)


def test_batched_attention_vs_brute_einsum_with_the_additive_mask():
    """logits = einsum(bhnk,bmk->bhnm), softmax(logits + mask), einsum(bhnm,bmv->bhnv), written out index by
    index, with the -inf mask of Section 2.3 built here from its definition (a later position is illegal)."""
    b, h, n, k, v = 2, 3, 4, 3, 2
    start = np.array([0, 2], np.int32)
    m_max = 7
    (Qb, Kb, Vb), (Q, K, V) = _batched_inputs(b, h, n, m_max, k, v, seed=301)
    got = oracle.mqa_batched_attention(Qb, Kb, Vb, start)
    for s in range(b):
        m = int(start[s]) + n
        mask = np.zeros((1, h, n, m))
        for t in range(n):
            for j in range(m):
                if j > start[s] + t:
                    mask[0, :, t, j] = -np.inf
        w = brute_softmax_last(brute_einsum("bhnk,bmk->bhnm", Q[s:s + 1], K[s:s + 1, :m]) + mask)
        ref = brute_einsum("bhnm,bmv->bhnv", w, V[s:s + 1, :m])
        np.testing.assert_allclose(got[s:s + 1], ref, rtol=1e-12, atol=1e-14)
    # start = None means zeros
    np.testing.assert_array_equal(oracle.mqa_batched_attention(Qb, Kb, Vb), oracle.mqa_batched_attention(Qb, Kb, Vb, np.zeros(b, np.int32)))


def test_batched_attention_rows_are_the_incremental_steps():
    """Section 2.4's reading of autoregressive decoding: query position t attends up to and including its own
    position, so row t of the batched function under the causal mask is the incremental step over start + t + 1 rows."""
    b, h, n, m_max, k, v = 3, 4, 9, 40, 128, 128
    start = np.array([0, 5, 31], np.int32)
    (Qb, Kb, Vb), _ = _batched_inputs(b, h, n, m_max, k, v, seed=302)
    got = oracle.mqa_batched_attention(Qb, Kb, Vb, start)
    for t in range(n):
        step = oracle.mqa_decode_step(np.ascontiguousarray(Qb[:, :, t]), Kb, Vb, (start + t + 1).astype(np.int32))
        np.testing.assert_allclose(got[:, :, t], step, rtol=1e-13, atol=1e-15)


def test_batched_attention_is_the_papers_function_between_its_projections():
    """With projections chosen so that they pass their input through (d = k = v, one-hot P_q, P_k, P_v, P_o), the
    paper's MultiqueryAttentionBatched is the attention lines alone: Y[b,n,:] = sum over heads of O[b,h,n,:]."""
    b, h, n, d = 2, 3, 5, 4
    r = rng(303)
    Xb, X = bf16_bits(r.normal(size=(b, n, d)))
    eye = np.eye(d)
    P_q = np.stack([eye * 2.0 ** i for i in range(h)])      # head i scales the queries by 2^i (exact in bf16)
    P_k, P_v = eye, eye
    P_o = np.stack([eye for _ in range(h)])
    Y = pf.multiquery_attention_batched(X, X, _causal_mask(b, h, n), P_q, P_k, P_v, P_o)
    Qb, _ = bf16_bits(np.einsum("bnd,hdk->bhnk", X, P_q))
    O = oracle.mqa_batched_attention(Qb, Xb, Xb)
    np.testing.assert_allclose(O.sum(axis=1), Y, rtol=1e-12, atol=1e-13)


def test_batched_attention_library_sdpa_causal_fp64():
    b, h, n, k, v = 2, 3, 37, 128, 128
    (Qb, Kb, Vb), (Q, K, V) = _batched_inputs(b, h, n, n, k, v, seed=304)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q), torch.from_numpy(K)[:, None].expand(b, h, n, k), torch.from_numpy(V)[:, None].expand(b, h, n, v),
        is_causal=True, scale=1.0).numpy()
    np.testing.assert_allclose(oracle.mqa_batched_attention(Qb, Kb, Vb), ref, rtol=1e-12, atol=1e-14)


def test_batched_attention_never_reads_beyond_a_sequences_memory_and_refuses_what_does_not_fit():
    b, h, n, m_max, k, v = 2, 2, 6, 20, 8, 8
    start = np.array([3, 14], np.int32)
    (Qb, Kb, Vb), _ = _batched_inputs(b, h, n, m_max, k, v, seed=305)
    ref = oracle.mqa_batched_attention(Qb, Kb, Vb, start)
    Kp, Vp = Kb.copy(), Vb.copy()
    for s in range(b):
        Kp[s, start[s] + n:] = 0x7FC0                       # NaN beyond the memory
        Vp[s, start[s] + n:] = 0x7FC0
    np.testing.assert_array_equal(oracle.mqa_batched_attention(Qb, Kp, Vp, start), ref)
    with pytest.raises(ValueError):
        oracle.mqa_batched_attention(Qb, Kb, Vb, np.array([3, 15], np.int32))
