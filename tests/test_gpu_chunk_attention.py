"""GPU parity of the streaming chunked prefill attention against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


CASES = [
    # c, n_prefix, n_q, n_kv
    (128, 0, 4, 1),            # one tile, purely causal
    (1, 0, 4, 4),              # a single token sees itself
    (100, 37, 8, 2),           # ragged query tile, ragged prefix
    (256, 128, 4, 2),          # prefix of exactly one tile
    (1024, 516, 32, 8),        # the paper's defaults: chunk 1024, sink 4 + window 512
    (300, 1000, 4, 4),         # long prefix, no grouping
    (200, 130, 28, 4),         # seven query heads per kv head: one head per CTA
    (2048, 516, 8, 2),         # 16 query tiles, up to 21 key tiles: the K/V ring wraps many times
    # more widths of the visible part of the last key tile (40, 60 and 90 keys here)
    (128, 40, 4, 2),
    (256, 60, 2, 1),
    (384, 90, 4, 4),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"c{c[0]}_p{c[1]}_h{c[2]}_kv{c[3]}")
def test_chunk_attention_matches_oracle(case):
    from paper_2508_17892_b200 import IlreRecall
    c, n_prefix, n_q, n_kv = case
    Q = _rand((c, n_q, 128), c + 1)
    K = _rand((n_prefix + c, n_kv, 128), n_prefix + 2)
    V = _rand((n_prefix + c, n_kv, 128), 3)
    want = oracle.chunk_attention(Q, K, V, n_prefix)
    eng = IlreRecall(max_L=4096, max_q_len=16, max_budget=64, n_kv_heads=n_kv, n_q_heads=n_q)
    out = eng.chunk_attention(Q.cuda(), K.cuda(), V.cuda(), n_prefix)
    torch.cuda.synchronize()
    eng.check_status()
    got = out.cpu().to(torch.float64).numpy()
    # Probabilities are rounded to bf16 before they multiply the values: each carries a relative
    # error of at most 2^-9, so the output is off by at most 2^-9 * sum_k p_k |v_k| <= 2^-9 max|v|;
    # the bf16 output adds 2^-8 of its own value.  (The exponentials' 2^-22 does not show.)
    vmax = float(V.to(torch.float32).abs().max())
    bound = 2.0 ** -8 * np.abs(want) + 2.0 ** -9 * vmax * 1.05
    err = np.abs(got - want)
    assert np.all(err <= bound), float((err / bound).max())
    # on average the two roundings are far smaller than their bounds
    assert err.mean() < 2e-3 * vmax
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()
