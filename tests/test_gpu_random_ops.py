"""Seeded random shapes of the entry points around the recall (chunk attention, Eq. 7
re-rotation, key fill) through the C ABI against their oracles."""
import random

import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


@pytest.mark.parametrize("seed", range(12))
def test_random_shapes(seed):
    from paper_2508_17892_b200 import IlreRecall
    rng = random.Random(100 + seed)
    n_kv = rng.choice([1, 2, 4, 8])
    n_q = n_kv * rng.choice([1, 2, 3, 4, 7])
    eng = IlreRecall(max_L=70000, max_q_len=16, max_budget=64, n_kv_heads=n_kv, n_q_heads=n_q)

    # chunk attention: within the bf16 rounding of P and of the output
    c = rng.choice([1, 17, 128, 129, 300, 777])
    n_pre = rng.choice([0, 1, 4, 127, 128, 516, 900])
    Q, K, V = (_rand((c, n_q, 128), seed), _rand((n_pre + c, n_kv, 128), seed + 1),
               _rand((n_pre + c, n_kv, 128), seed + 2))
    got = eng.chunk_attention(Q.cuda(), K.cuda(), V.cuda(), n_pre).cpu().to(torch.float64).numpy()
    eng.check_status()
    ref = oracle.chunk_attention(Q, K, V, n_pre)
    vmax = np.abs(V.to(torch.float64).numpy()).max()
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -9 * vmax + 1e-6)

    # Eq. 7: one bf16 rounding of an fp32 rotation
    L = rng.randint(1, 3000)
    chunk = rng.choice([1, 7, 64, 100, 1024])
    n_sink = min(rng.choice([0, 3, 4]), L)
    if (L - n_sink + chunk - 1) // chunk - 2 <= 8192:
        Kc = _rand((L, n_kv, 128), seed + 3, 3.0)
        got = eng.rerope_keys(Kc.cuda(), chunk, n_sink).cpu().to(torch.float64).numpy()
        ref = oracle.dca_rerope(Kc, chunk, n_sink)
        assert np.all(np.abs(got - ref) <= 2.0 ** -8 * (1 + 1e-3) * np.abs(ref) + 4e-6)

    # key fill: one bf16 rounding of an fp32 dot product and rotation; rows outside untouched
    n_tok = rng.choice([1, 5, 128, 200, 515])
    d_model = rng.choice([64, 128, 512, 1024])
    pos0 = rng.randint(0, 60000)
    X, W = _rand((n_tok, d_model), seed + 4), _rand((n_kv * 128, d_model), seed + 5, 1.0 / 16)
    cache = torch.zeros(pos0 + n_tok + 3, n_kv, 128, dtype=torch.bfloat16, device="cuda")
    eng.fill_keys(X.cuda(), W.cuda(), cache, pos0)
    torch.cuda.synchronize()
    eng.check_status()
    ref = oracle.key_fill(X, W, pos0)
    got = cache[pos0:pos0 + n_tok].cpu().to(torch.float64).numpy()
    mag = (np.abs(X.to(torch.float64).numpy()) @ np.abs(W.to(torch.float64).numpy()).T)
    mag = mag.reshape(n_tok, n_kv, 128)
    pair = np.maximum(mag[..., :64], mag[..., 64:])
    pair = 2.0 * np.concatenate([pair, pair], axis=-1)
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * (1 + 1e-3) * np.abs(ref) + 1e-6 * pair + 1e-7)
    assert float(cache[pos0 + n_tok:].abs().max()) == 0.0
    assert pos0 == 0 or float(cache[:pos0].abs().max()) == 0.0
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()
