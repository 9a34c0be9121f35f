"""Seeded synthetic inputs for the decode-attention step, shared by the tests, the
bench and the smoke check.  This module holds no attention arithmetic: it only draws
random tensors, rounds them to bf16, and names the workload shapes.

Shapes follow the paper's experimental setup (Section 4.1: h = 8, d_k = d_v = 128,
d_model = 1024; Section 4.3: 128 sequences per core, 128 target positions) and the
longer-context variants this build is measured on.  Value distributions: ``q ~ N(0, 1/k)``
(the omitted 1/sqrt(k) logit scale folded into the query, as the note closing Section 2.2
allows) and ``K, V, k_new, v_new ~ N(0, 1)``, drawn in fp32 and rounded to bf16.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

import numpy as np
import torch

K_DIM = 128
V_DIM = 128
NAN_BITS = 0x7FC0  # a bf16 quiet NaN, used to poison rows that must never be read


@dataclass(frozen=True)
class Workload:
    name: str
    b: int
    h: int
    m_max: int
    lens: str          # "full" | "full_minus_one" | "ragged" | "grow"
    steps: int = 1     # decode steps in the workload ("grow": the cache grows by one per step)
    k: int = K_DIM
    v: int = V_DIM


WORKLOADS = {
    # one step over a full 128-row cache
    "single_step": Workload("single_step", b=1, h=8, m_max=128, lens="full"),
    # the paper's timed decoding shape: cache grows 1 -> 128 over 128 steps
    "paper_incremental": Workload("paper_incremental", b=128, h=8, m_max=128, lens="grow", steps=128),
    # long context: 8191 rows resident, the step appends row 8191 and attends over 8192
    "long_context": Workload("long_context", b=32, h=32, m_max=8192, lens="full_minus_one"),
    # ragged batch: valid lengths uniform on [1, 2048]
    "ragged": Workload("ragged", b=256, h=16, m_max=2048, lens="ragged"),
}
SWEEP_B = (1, 8, 64, 256)
SWEEP_M = (512, 4096, 32768)
for _b in SWEEP_B:
    for _m in SWEEP_M:
        WORKLOADS[f"sweep_b{_b}_m{_m}"] = Workload(f"sweep_b{_b}_m{_m}", b=_b, h=16, m_max=_m, lens="full")


def ragged_lens(b: int, m_max: int, seed: int = 0) -> np.ndarray:
    """Valid lengths uniform on [1, m_max], drawn on the host so that they do not depend on
    the device the tensors are generated on."""
    return np.random.default_rng(seed).integers(1, m_max + 1, size=b).astype(np.int32)


def initial_lens(w: Workload, seed: int = 0) -> np.ndarray:
    """``lens`` BEFORE the step's append (the step attends over ``lens + 1`` rows)."""
    if w.lens == "full":
        return np.full(w.b, w.m_max - 1, dtype=np.int32)
    if w.lens == "full_minus_one":
        return np.full(w.b, w.m_max - 1, dtype=np.int32)
    if w.lens == "ragged":
        return (ragged_lens(w.b, w.m_max, seed) - 1).astype(np.int32)
    if w.lens == "grow":
        return np.zeros(w.b, dtype=np.int32)
    raise ValueError(w.lens)


def bf16_normal(shape, std: float, gen: torch.Generator, device, chunk_elems: int = 1 << 26) -> torch.Tensor:
    """``N(0, std^2)`` drawn in fp32 and rounded to bf16 (round-to-nearest-even), generated in
    slices along the first axis so that the fp32 temporary stays small."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    if out.numel() == 0:
        return out
    flat = out.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        r = torch.randn(e - s, generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            r.mul_(std)
        flat[s:e] = r.to(torch.bfloat16)
    return out


def make_inputs(b: int, h: int, m_max: int, variant: str, seed: int = 0, device="cpu",
                k: int = K_DIM, v: int = V_DIM) -> dict:
    """Draw ``q, K, V, k_new, v_new`` for one step.

    ``variant`` is ``"mqa"`` (cache ``[b,m_max,k]``) or ``"mha"`` (cache ``[b,h,m_max,k]``).
    The draw order is fixed (q, K, V, k_new, v_new) and the two variants use different
    streams (seed and seed + 1000), so a tensor never depends on which variants were built."""
    if variant not in ("mqa", "mha"):
        raise ValueError(variant)
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed + (1000 if variant == "mha" else 0))
    kvh = 1 if variant == "mqa" else h
    cache = (b, m_max) if variant == "mqa" else (b, h, m_max)
    new = (b,) if variant == "mqa" else (b, h)
    return {
        "variant": variant, "b": b, "h": h, "m_max": m_max, "k": k, "v": v, "kv_heads": kvh,
        "q": bf16_normal((b, h, k), k ** -0.5, gen, dev),
        "K": bf16_normal(cache + (k,), 1.0, gen, dev),
        "V": bf16_normal(cache + (v,), 1.0, gen, dev),
        "k_new": bf16_normal(new + (k,), 1.0, gen, dev),
        "v_new": bf16_normal(new + (v,), 1.0, gen, dev),
    }


def poison_tail(cache: torch.Tensor, lens, bits: int = NAN_BITS) -> None:
    """Overwrite, in place, every cache row at or beyond ``lens[b]`` with the given 16-bit
    pattern (NaN by default).  ``cache`` is ``[b,m_max,*]`` or ``[b,h,m_max,*]``."""
    m_max = cache.shape[-2]
    lens_t = torch.as_tensor(np.asarray(lens), device=cache.device).to(torch.int64)
    rows = torch.arange(m_max, device=cache.device)
    dead = rows[None, :] >= lens_t[:, None]                      # [b, m_max]
    if cache.dim() == 4:
        dead = dead[:, None, :].expand(cache.shape[0], cache.shape[1], m_max)
    fill = torch.tensor(bits if bits < 0x8000 else bits - 0x10000, dtype=torch.int16, device=cache.device)
    cache.view(torch.int16)[dead] = fill


def bits(t: torch.Tensor) -> np.ndarray:
    """A bf16 tensor's bit patterns as a host uint16 array (what the oracle takes)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def from_bits(a: np.ndarray, device="cpu") -> torch.Tensor:
    """Inverse of :func:`bits`."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16).to(device)


def algorithmic_bytes(sum_lens: int, b: int, h: int, kv_heads: int, k: int = K_DIM, v: int = V_DIM) -> int:
    """Bytes one decode step must move: every valid K and V row once (bf16), q once (bf16),
    o once (fp32).  Split partials and the append are overhead and are not counted."""
    return kv_heads * sum_lens * (k + v) * 2 + b * h * k * 2 + b * h * v * 4
