"""TEST INFRASTRUCTURE -- not part of the product path.

fp64 numpy restatement of the paper's layer functions *including* the learned
projections (arXiv 1911.02150).  The hot path itself never sees a projection; these
exist so that the pins can check what the paper fixes about the step as a whole:
that the incremental functions reproduce the batched ones under a causal mask, that
multi-query is multi-head with one shared key/value projection, and that one head is
the single-query attention of Section 2.1.

Everything is built from one primitive, ``attend`` (a single query over a memory), and
plain matrix-vector products, with explicit loops over sequences, positions and heads:
slow and meant to be read next to the paper.

  attend                                     Section 2.1 (+ the additive mask of 2.3)
  multihead_attention                        Section 2.2
  multihead_attention_batched                Section 2.3
  multihead_self_attention_incremental       Section 2.4
  multiquery_attention_batched               Section 3 (batched form)
  multiquery_self_attention_incremental      Section 3 (one step)

Readings: in the two incremental functions the new key/value row is projected from the
current input ``x`` (the printed code names another variable there, but the text says
each position attends up to and including itself); the new row is concatenated on the
memory axis m, so the caches grow from m to m+1 rows; no 1/sqrt(k) factor.
"""
from __future__ import annotations

import numpy as np

F = np.float64


def attend(q, K, V, mask_row=None):
    """One query ``q[k]`` over ``K[m,k]``, ``V[m,v]``; ``mask_row[m]`` (0 or -inf) is added
    to the logits before the softmax."""
    q, K, V = np.asarray(q, F), np.asarray(K, F), np.asarray(V, F)
    logits = K @ q
    if mask_row is not None:
        logits = logits + np.asarray(mask_row, F)
    top = logits.max()
    if not np.isfinite(top):
        raise ValueError("every position is masked: softmax is undefined")
    w = np.exp(logits - top)
    w = w / w.sum()
    return w @ V


def multihead_attention(x, M, P_q, P_k, P_v, P_o):
    """Section 2.2: ``x[d]``, ``M[m,d]``, ``P_q,P_k[h,d,k]``, ``P_v,P_o[h,d,v]`` -> ``y[d]``."""
    x, M = np.asarray(x, F), np.asarray(M, F)
    h, d, _ = P_q.shape
    y = np.zeros(d, F)
    for i in range(h):
        q = x @ P_q[i]            # [k]
        K = M @ P_k[i]            # [m,k]
        V = M @ P_v[i]            # [m,v]
        o = attend(q, K, V)       # [v]
        y += P_o[i] @ o           # [d,v] @ [v]
    return y


def multihead_attention_batched(X, M, mask, P_q, P_k, P_v, P_o):
    """Section 2.3: ``X[b,n,d]``, ``M[b,m,d]``, ``mask[b,h,n,m]`` -> ``Y[b,n,d]``."""
    X, M = np.asarray(X, F), np.asarray(M, F)
    b, n, d = X.shape
    h = P_q.shape[0]
    Y = np.zeros((b, n, d), F)
    for s in range(b):
        for i in range(h):
            K = M[s] @ P_k[i]
            V = M[s] @ P_v[i]
            for t in range(n):
                q = X[s, t] @ P_q[i]
                Y[s, t] += P_o[i] @ attend(q, K, V, mask[s, i, t])
    return Y


def multihead_self_attention_incremental(x, prev_K, prev_V, P_q, P_k, P_v, P_o):
    """Section 2.4: ``x[b,d]``, ``prev_K[b,h,m,k]``, ``prev_V[b,h,m,v]`` ->
    ``y[b,d]``, ``new_K[b,h,m+1,k]``, ``new_V[b,h,m+1,v]``."""
    x = np.asarray(x, F)
    b, d = x.shape
    h, _, k = P_q.shape
    v = P_v.shape[2]
    m = prev_K.shape[2]
    new_K = np.empty((b, h, m + 1, k), F)
    new_V = np.empty((b, h, m + 1, v), F)
    y = np.zeros((b, d), F)
    for s in range(b):
        for i in range(h):
            new_K[s, i, :m] = prev_K[s, i]
            new_V[s, i, :m] = prev_V[s, i]
            new_K[s, i, m] = x[s] @ P_k[i]
            new_V[s, i, m] = x[s] @ P_v[i]
            q = x[s] @ P_q[i]
            y[s] += P_o[i] @ attend(q, new_K[s, i], new_V[s, i])
    return y, new_K, new_V


def multiquery_attention_batched(X, M, mask, P_q, P_k, P_v, P_o):
    """Section 3: as the batched multi-head function but ``P_k[d,k]``, ``P_v[d,v]`` carry no
    heads axis, so all heads of a sequence see the same K and V."""
    X, M = np.asarray(X, F), np.asarray(M, F)
    b, n, d = X.shape
    h = P_q.shape[0]
    Y = np.zeros((b, n, d), F)
    for s in range(b):
        K = M[s] @ P_k
        V = M[s] @ P_v
        for i in range(h):
            for t in range(n):
                q = X[s, t] @ P_q[i]
                Y[s, t] += P_o[i] @ attend(q, K, V, mask[s, i, t])
    return Y


def multiquery_self_attention_incremental(x, prev_K, prev_V, P_q, P_k, P_v, P_o):
    """Section 3, one step: ``x[b,d]``, ``prev_K[b,m,k]``, ``prev_V[b,m,v]`` ->
    ``y[b,d]``, ``K[b,m+1,k]``, ``V[b,m+1,v]``."""
    x = np.asarray(x, F)
    b, d = x.shape
    h = P_q.shape[0]
    k, v = P_k.shape[1], P_v.shape[1]
    m = prev_K.shape[1]
    K = np.empty((b, m + 1, k), F)
    V = np.empty((b, m + 1, v), F)
    y = np.zeros((b, d), F)
    for s in range(b):
        K[s, :m] = prev_K[s]
        V[s, :m] = prev_V[s]
        K[s, m] = x[s] @ P_k
        V[s, m] = x[s] @ P_v
        for i in range(h):
            q = x[s] @ P_q[i]
            y[s] += P_o[i] @ attend(q, K[s], V[s])
    return y, K, V


def combine_partials(parts):
    """Exact re-association of one softmax over a partition of the memory axis.

    ``parts`` is a list of ``(M_s, l_s, acc_s)`` with ``M_s`` the largest logit of part s,
    ``l_s = sum_j exp(logit_j - M_s)`` and ``acc_s[v] = sum_j exp(logit_j - M_s) V[j]``.
    Returns ``sum_s e^{M_s-M} acc_s / sum_s e^{M_s-M} l_s`` with ``M = max_s M_s`` -- the
    identity a split-m implementation relies on; it is not in the paper and is pinned
    against ``attend`` on the unsplit memory."""
    top = max(p[0] for p in parts)
    num = sum(np.exp(p[0] - top) * np.asarray(p[2], F) for p in parts)
    den = sum(np.exp(p[0] - top) * p[1] for p in parts)
    return num / den
