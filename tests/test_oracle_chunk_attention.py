"""Pins of the oracle's streaming chunked prefill attention (Eq. 2 with the Lambda mask)."""
import numpy as np
import torch
from scipy.special import softmax

import oracle


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


def test_against_library_softmax_and_explicit_mask():
    c, n_prefix, n_q, n_kv, d = 9, 5, 4, 2, 16
    Q, K, V = _rand((c, n_q, d), 0), _rand((n_prefix + c, n_kv, d), 1), _rand((n_prefix + c, n_kv, d), 2)
    out = oracle.chunk_attention(Q, K, V, n_prefix)
    q, k, v = (t.to(torch.float64).numpy() for t in (Q, K, V))
    mask = np.full((c, n_prefix + c), -np.inf)
    for j in range(c):
        mask[j, : n_prefix + j + 1] = 0.0                      # prefix fully visible, chunk causal
    for h in range(n_q):
        g = h // 2
        p = softmax(np.einsum("jd,kd->jk", q[:, h], k[:, g]) / 4.0 + mask, axis=1)
        np.testing.assert_allclose(out[:, h], p @ v[:, g], rtol=1e-12, atol=1e-14)


def test_constant_values_come_back_and_future_tokens_do_not_matter():
    c, n_prefix = 12, 7
    Q, K = _rand((c, 2, 8), 3), _rand((n_prefix + c, 1, 8), 4)
    V = torch.ones(n_prefix + c, 1, 8).to(torch.bfloat16) * 3
    np.testing.assert_allclose(oracle.chunk_attention(Q, K, V, n_prefix), 3.0, rtol=1e-13)
    V = _rand((n_prefix + c, 1, 8), 5)
    base = oracle.chunk_attention(Q, K, V, n_prefix)
    K2, V2 = K.clone(), V.clone()
    K2[n_prefix + 6:], V2[n_prefix + 6:] = 9.0, -9.0          # change the keys after chunk token 5
    again = oracle.chunk_attention(Q, K2, V2, n_prefix)
    np.testing.assert_array_equal(again[:6], base[:6])        # queries 0..5 never see them
    assert np.abs(again[6:] - base[6:]).max() > 0.1


def test_equal_keys_average_the_visible_values():
    c, n_prefix = 6, 3
    Q = _rand((c, 1, 4), 6)
    K = torch.ones(n_prefix + c, 1, 4).to(torch.bfloat16)
    V = _rand((n_prefix + c, 1, 4), 7)
    out = oracle.chunk_attention(Q, K, V, n_prefix)
    v = V.to(torch.float64).numpy()[:, 0]
    for j in range(c):
        np.testing.assert_allclose(out[j, 0], v[: n_prefix + j + 1].mean(axis=0), rtol=1e-12, atol=1e-14)


def test_first_chunk_without_prefix_is_causal_attention():
    c = 5
    Q, K, V = _rand((c, 2, 8), 8), _rand((c, 2, 8), 9), _rand((c, 2, 8), 10)
    out = oracle.chunk_attention(Q, K, V, 0)
    v = V.to(torch.float64).numpy()
    np.testing.assert_allclose(out[0], v[0], rtol=1e-13, atol=1e-15)    # token 0 sees itself only
