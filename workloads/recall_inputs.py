"""Seeded synthetic inputs for the ILRe token-recall path.

This module only *makes inputs*: a RoPE'd bf16 key cache [L, n_kv_heads, d], a bf16 query
block [q_len, n_q_heads, d], planted "needle" spans, and the budget / pooling spec of each
workload.  It contains none of the recall method's arithmetic (no logits, softmax, pooling or
selection); both the CUDA library's tests and the CPU oracle's tests receive the identical
bytes produced here.

Recipe (all draws from one CPU ``torch.Generator`` seeded with the workload's seed, in this
fixed order; all math in fp32 with one final round-to-nearest-even to bf16):

1. query  ~ N(0,1), shape [q_len, n_q_heads, d]  (taken as already rotated);
2. per-workload key parameters (outlier channel ids, low-rank bases / mixture means);
3. span offsets, then span lengths;
4. background keys, drawn in blocks of ``KEY_BLOCK`` positions (the block size is part of the
   recipe: the stream of normal variates depends on it), each block rotated by RoPE
   (rotate-half pairing i <-> i + d/2, inv_freq_i = theta^(-2i/d), theta = 500000, position =
   index in the cache; Eq. 3 of the paper) and rounded to bf16;
5. needle noise: for every span, every kv head g: key = gain*sqrt(d)*u_g + 0.5*N(0,I)
   (gain 3 unless the workload says otherwise), where
   u_g is the unit vector along the mean of the 4*q_len bf16 query vectors of group g.  The
   needles overwrite the cache after RoPE (they live in cache space).

Spans never overlap: the cache is cut into n_spans equal segments and each span is placed
uniformly at random inside its own segment.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Tuple

import torch

KEY_BLOCK = 16384          # positions per generator draw (part of the recipe)
ROPE_THETA = 500000.0


@dataclass
class RecallWorkload:
    name: str
    seed: int
    L: int
    q_len: int
    n_kv_heads: int = 8
    n_q_heads: int = 32
    d: int = 128
    key_kind: str = "gauss"          # gauss | lowrank | outlier
    n_spans: int = 0
    span_len: Tuple[int, int] = (32, 32)     # inclusive range of span lengths
    budget: int = 512
    max_sizes: Tuple[int, ...] = (1,)        # strided max-pool sizes m_i (Algorithm 1)
    win_sizes: Tuple[int, ...] = (1,)        # stride-1 window sizes n_j (Algorithm 1)
    win_op: int = 1                          # 0 = average (Algorithm 1), 1 = max
    n_sink: int = 0
    needle_gain: float = 3.0                 # needle key = gain * sqrt(d) * u_g + noise
    span_seed: int = -1                      # >= 0: span offsets/lengths from a generator of
                                             # their own (same spans for workloads that differ
                                             # in seed, e.g. the layers of one context)


@dataclass
class RecallInputs:
    workload: RecallWorkload
    K: torch.Tensor                  # bf16 [L, n_kv_heads, d], CPU, contiguous
    Q: torch.Tensor                  # bf16 [q_len, n_q_heads, d], CPU, contiguous
    spans: List[Tuple[int, int]] = field(default_factory=list)   # (offset, length)

    def planted_positions(self) -> torch.Tensor:
        if not self.spans:
            return torch.empty(0, dtype=torch.int64)
        return torch.cat([torch.arange(o, o + n) for o, n in self.spans])


# The five benchmark configurations (head layout of Llama-3.1-8B; budget 4K as in the
# paper's RULER setup; q_len 64 as in its LongBench setup; lengths 32K..1M as in Table 1).
CONFIGS = {
    "cfg1_L4k": RecallWorkload("cfg1_L4k", seed=0, L=4096, q_len=16, n_spans=4,
                               span_len=(32, 32), budget=512, win_sizes=(1, 7, 15)),
    "cfg2_L32k": RecallWorkload("cfg2_L32k", seed=1, L=32768, q_len=64, n_spans=16,
                                span_len=(64, 64), budget=4096, win_sizes=(1, 7, 15, 31)),
    "cfg3_L128k": RecallWorkload("cfg3_L128k", seed=2, L=131072, q_len=64, key_kind="lowrank",
                                 n_spans=32, span_len=(16, 128), budget=4096,
                                 win_sizes=(1, 7, 15, 31)),
    "cfg4_L512k": RecallWorkload("cfg4_L512k", seed=3, L=524288, q_len=128, key_kind="outlier",
                                 n_spans=64, span_len=(32, 32), budget=4096,
                                 win_sizes=(1, 7, 15, 31, 63)),
    "cfg5_L1m": RecallWorkload("cfg5_L1m", seed=4, L=1048576, q_len=256, n_spans=128,
                               span_len=(8, 256), budget=4096, win_sizes=(1, 7, 15, 31, 63)),
}

# Algorithm 1's default pooling spec: max sizes {2,4,8} x average sizes 1..16 (48 combinations).
PAPER_DEFAULT_MAX_SIZES = (2, 4, 8)
PAPER_DEFAULT_WIN_SIZES = tuple(range(1, 17))

# Supplementary timing rows on the L = 1M cache (not benchmark configurations):
#   a short query (4 * q_len = 64 rows per kv head: 64 flop per key byte, below the ridge, so
#   the key scan is HBM-bound), and the benchmark configuration under Algorithm 1's default
#   pooling spec.
CONFIGS["probe_L1m_q16"] = RecallWorkload(
    "probe_L1m_q16", seed=5, L=1048576, q_len=16, n_spans=128, span_len=(8, 256), budget=4096,
    win_sizes=(1, 7, 15, 31, 63))
CONFIGS["cfg5_L1m_paper_pool"] = RecallWorkload(
    "cfg5_L1m_paper_pool", seed=4, L=1048576, q_len=256, n_spans=128, span_len=(8, 256),
    budget=4096, max_sizes=PAPER_DEFAULT_MAX_SIZES, win_sizes=PAPER_DEFAULT_WIN_SIZES, win_op=0,
    n_sink=4)


def _rope_inplace(x: torch.Tensor, pos0: int) -> torch.Tensor:
    """Rotate x [n, H, d] (fp32) by RoPE at positions pos0 .. pos0+n-1 (rotate-half form)."""
    n, _, d = x.shape
    half = d // 2
    idx = torch.arange(half, dtype=torch.float64)
    inv_freq = ROPE_THETA ** (-2.0 * idx / d)
    pos = torch.arange(pos0, pos0 + n, dtype=torch.float64)
    ang = pos[:, None] * inv_freq[None, :]
    cos = torch.cos(ang).to(torch.float32)[:, None, :]
    sin = torch.sin(ang).to(torch.float32)[:, None, :]
    x1 = x[..., :half]
    x2 = x[..., half:]
    out = torch.empty_like(x)
    out[..., :half] = x1 * cos - x2 * sin
    out[..., half:] = x2 * cos + x1 * sin
    return out


def make_inputs(w: RecallWorkload) -> RecallInputs:
    g = torch.Generator().manual_seed(w.seed)
    H, d, L = w.n_kv_heads, w.d, w.L
    group = w.n_q_heads // H

    # 1. query
    Q = torch.randn(w.q_len, w.n_q_heads, d, generator=g, dtype=torch.float32).to(torch.bfloat16)

    # 2. key-distribution parameters
    outlier_dims = None
    lowrank = None
    if w.key_kind == "outlier":
        outlier_dims = torch.stack([torch.randperm(d, generator=g)[:4] for _ in range(H)])
    elif w.key_kind == "lowrank":
        U = torch.randn(H, 16, d, generator=g)                 # rank-16 basis per kv head
        mu = torch.randn(H, 8, 16, generator=g)                # 8 mixture means in R^16
        lowrank = (U, mu)

    # 3. spans
    spans: List[Tuple[int, int]] = []
    if w.n_spans > 0:
        seg = L // w.n_spans
        lo, hi = w.span_len
        gs = g if w.span_seed < 0 else torch.Generator().manual_seed(w.span_seed)
        u_off = torch.rand(w.n_spans, generator=gs, dtype=torch.float64)
        lens = torch.randint(lo, hi + 1, (w.n_spans,), generator=gs)
        for s in range(w.n_spans):
            n = int(lens[s])
            if n > seg:
                raise ValueError("span longer than its segment")
            off = s * seg + int(u_off[s].item() * (seg - n + 1))
            spans.append((off, n))

    # 4. background keys
    K = torch.empty(L, H, d, dtype=torch.bfloat16)
    for p0 in range(0, L, KEY_BLOCK):
        n = min(KEY_BLOCK, L - p0)
        if w.key_kind == "lowrank":
            U, mu = lowrank
            comp = torch.randint(0, 8, (n, H), generator=g)
            z = torch.randn(n, H, 16, generator=g) * 0.5
            z = z + mu[torch.arange(H)[None, :], comp]              # [n, H, 16]
            x = torch.einsum("nhr,hrd->nhd", z, U) / math.sqrt(16 * 1.25)
            x = x + 0.3 * torch.randn(n, H, d, generator=g)
        else:
            x = torch.randn(n, H, d, generator=g)
            if w.key_kind == "outlier":
                for h in range(H):
                    x[:, h, outlier_dims[h]] *= 8.0
        K[p0:p0 + n] = _rope_inplace(x, p0).to(torch.bfloat16)

    # 5. needles (cache space, after RoPE)
    if spans:
        Qg = Q.to(torch.float32).view(w.q_len, H, group, d)
        mean_dir = Qg.mean(dim=(0, 2))                              # [H, d]
        u = mean_dir / mean_dir.norm(dim=-1, keepdim=True)
        for off, n in spans:
            noise = torch.randn(n, H, d, generator=g)
            K[off:off + n] = (w.needle_gain * math.sqrt(d) * u[None] + 0.5 * noise).to(torch.bfloat16)

    return RecallInputs(w, K.contiguous(), Q.contiguous(), spans)


def small_workload(L: int, q_len: int, seed: int = 7, n_kv_heads: int = 8, n_q_heads: int = 32,
                   n_spans: int = 2, span_len: Tuple[int, int] = (8, 24), budget: int = 64,
                   max_sizes=(1,), win_sizes=(1, 7), win_op: int = 1, n_sink: int = 0,
                   key_kind: str = "gauss") -> RecallWorkload:
    """Free-form workload for parity tests at odd sizes (ragged L, q_len, sinks...)."""
    return RecallWorkload(f"small_L{L}_q{q_len}_s{seed}", seed=seed, L=L, q_len=q_len,
                          n_kv_heads=n_kv_heads, n_q_heads=n_q_heads, key_kind=key_kind,
                          n_spans=n_spans, span_len=span_len, budget=budget,
                          max_sizes=tuple(max_sizes), win_sizes=tuple(win_sizes), win_op=win_op,
                          n_sink=n_sink)


def layer_sweep_workloads(base: RecallWorkload, gains) -> List[RecallWorkload]:
    """One workload per candidate layer of the same context: the same planted spans
    (span_seed), a different query and key cache per layer (seed), and a per-layer needle
    gain that makes the phrases easier or harder to recall, as layers differ in the paper's
    retrieval task."""
    import dataclasses
    return [dataclasses.replace(base, name=f"{base.name}_layer{l}", seed=base.seed + 1000 * (l + 1),
                                span_seed=base.seed, needle_gain=float(gain))
            for l, gain in enumerate(gains)]
