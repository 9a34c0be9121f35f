"""TEST INFRASTRUCTURE -- not part of the product path.

fp64 oracle of one whole incremental multi-query layer step (Section 3, the function
``MultiquerySelfAttentionIncremental``) at the bf16 boundaries the decode path has:

    q     = einsum("bd,hdk->bhk", x, P_q)          rounded to bf16 (the step takes bf16 queries)
    k_new = einsum("bd,dk->bk",  x, P_k)           rounded to bf16 (the cache is bf16)
    v_new = einsum("bd,dv->bv",  x, P_v)           rounded to bf16
    K[b, lens[b]] = k_new[b], V likewise, lens[b] += 1              (concatenation on the memory axis)
    o     = softmax(einsum("bhk,bmk->bhm", q, K)) applied to V      (the multi-query step, fp64)
    y     = einsum("bhv,hdv->bd", bf16(o), P_o)    o rounded to bf16 (an operand of the output product)

Every contraction is a plain numpy einsum in fp64 on the exactly widened bf16 inputs; the three
roundings are the points where the path stores or feeds bf16 (``round_interfaces=False`` leaves
them out: then this is the paper's function itself, which a pin checks against
``paper_functions.multiquery_self_attention_incremental``).  Readings as there: the new row comes
from the current input x, it is appended before attending, no 1/sqrt(k) factor.
"""
from __future__ import annotations

import numpy as np

from . import kv_cache_append, mqa_decode_step


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round to the nearest bf16 (ties to even), from float64 through float32."""
    f = np.ascontiguousarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> 16) & np.uint32(1))) >> 16
    return rounded.astype(np.uint16)


def multiquery_layer_decode_step(x, P_q, P_k, P_v, P_o, K, V, lens, round_interfaces: bool = True):
    """``x[b,d]``, ``P_q[h,d,k]``, ``P_k[d,k]``, ``P_v[d,v]``, ``P_o[h,d,v]`` as bf16 bit patterns;
    ``K[b,m_max,k]``, ``V[b,m_max,v]`` writable bf16 bit patterns, ``lens[b]`` writable int32 (rows valid
    before the step).  Appends in place, advances ``lens``, returns ``(y[b,d] float64, q_bits, k_new_bits,
    v_new_bits)``.  With ``round_interfaces=False`` the projected rows are still stored as bf16 in the cache
    (it has no other type) but q and o are used unrounded."""
    xf, Pq, Pk, Pv, Po = (bf16_to_f64(a) for a in (x, P_q, P_k, P_v, P_o))
    q = np.einsum("bd,hdk->bhk", xf, Pq)
    k_new = np.einsum("bd,dk->bk", xf, Pk)
    v_new = np.einsum("bd,dv->bv", xf, Pv)
    q_bits, k_bits, v_bits = f64_to_bf16_bits(q), f64_to_bf16_bits(k_new), f64_to_bf16_bits(v_new)
    kv_cache_append(K, V, k_bits, v_bits, lens, True)
    if round_interfaces:
        o = mqa_decode_step(q_bits, K, V, lens)
        o = bf16_to_f64(f64_to_bf16_bits(o))
    else:
        b, h, _ = q.shape
        o = np.zeros((b, h, V.shape[-1]))
        Kf, Vf = bf16_to_f64(K), bf16_to_f64(V)
        for s in range(b):
            L = int(lens[s])
            if L <= 0:
                continue
            logits = q[s] @ Kf[s, :L].T
            w = np.exp(logits - logits.max(axis=1, keepdims=True))
            o[s] = (w / w.sum(axis=1, keepdims=True)) @ Vf[s, :L]
    y = np.einsum("bhv,hdv->bd", o, Po)
    return y, q_bits, k_bits, v_bits
