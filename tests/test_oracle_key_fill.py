"""Pins of the oracle's key-cache fill (Eq. 1 with RoPE of Eq. 3 for the retrieval layer's keys)."""
import math

import numpy as np
import torch

import oracle
from workloads.recall_inputs import ROPE_THETA, _rope_inplace


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


def test_position_zero_is_the_plain_projection():
    X, W = _rand((5, 64), 0), _rand((256, 64), 1)
    out = oracle.key_fill(X, W, pos0=0)
    want = (X.to(torch.float64) @ W.to(torch.float64).T).numpy().reshape(5, 2, 128)
    np.testing.assert_allclose(out[0], want[0], rtol=0, atol=1e-12)     # angle 0 at position 0
    assert np.abs(out[1:] - want[1:]).max() > 1e-3                       # later positions turn


def test_one_hot_rows_pick_weight_columns_and_rotate_like_rope():
    # X = rows of the identity: the projection is a column of W^T, i.e. K[t, g, :] is
    # W[g*128:(g+1)*128, t] turned to position pos0 + t; the input generator's RoPE routine is an
    # independent restatement of Eq. 3.
    d_model = 64
    W = _rand((256, d_model), 2)
    X = torch.eye(d_model).to(torch.bfloat16)
    pos0 = 1000
    out = oracle.key_fill(X, W, pos0=pos0)
    base = W.to(torch.float32).T.reshape(d_model, 2, 128).contiguous()  # [t, g, :]
    want = _rope_inplace(base.clone(), pos0).to(torch.float64).numpy()
    np.testing.assert_allclose(out, want, rtol=0, atol=2e-5)            # fp32 tables in the generator


def test_hand_computed_pair():
    # d_model = 1, x = 2, one head whose channel 0 has weight 1.5 and channel 64 weight -0.5;
    # position 3: channel 0 turns by 3 * theta^0 = 3 rad
    W = torch.zeros(128, 1)
    W[0, 0], W[64, 0] = 1.5, -0.5
    X = torch.tensor([[2.0]])
    out = oracle.key_fill(X.to(torch.bfloat16), W.to(torch.bfloat16), pos0=3, theta=10000.0)
    lo, hi = 3.0, -1.0
    assert abs(out[0, 0, 0] - (lo * math.cos(3) - hi * math.sin(3))) < 1e-14
    assert abs(out[0, 0, 64] - (lo * math.sin(3) + hi * math.cos(3))) < 1e-14
    assert np.abs(out[0, 0, 1:64]).max() == 0 and np.abs(out[0, 0, 65:]).max() == 0


def test_bias_linearity_and_pair_norms():
    X, W, b = _rand((7, 128), 3), _rand((128, 128), 4, 0.1), _rand((128,), 5)
    plain = oracle.key_fill(X, W, pos0=11)
    with_b = oracle.key_fill(X, W, pos0=11, bias=b)
    only_b = oracle.key_fill(torch.zeros_like(X), W, pos0=11, bias=b)
    np.testing.assert_allclose(with_b, plain + only_b, rtol=0, atol=1e-11)
    y = (X.to(torch.float64) @ W.to(torch.float64).T).numpy().reshape(7, 1, 128)
    np.testing.assert_allclose(plain[..., :64] ** 2 + plain[..., 64:] ** 2,
                               y[..., :64] ** 2 + y[..., 64:] ** 2, rtol=1e-11, atol=1e-300)


def test_chunked_fill_equals_one_fill_and_feeds_eq7():
    # filling chunk by chunk at the right positions is the same cache as one fill, and Eq. 7 on
    # it moves a key to the position it would have had D positions later
    X, W = _rand((96, 64), 6), _rand((128, 64), 7, 0.2)
    whole = oracle.key_fill(X, W, pos0=0)
    parts = np.concatenate([oracle.key_fill(X[a:a + 32], W, pos0=a) for a in (0, 32, 64)])
    np.testing.assert_allclose(parts, whole, rtol=0, atol=1e-12)
    later = oracle.key_fill(X[:1], W, pos0=64)                          # token 0 placed at position 64
    cache = torch.from_numpy(oracle.round_to_bf16(whole).view(np.int16)).view(torch.bfloat16)
    turned = oracle.dca_rerope(cache.reshape(96, 1, 128), chunk=16, n_sink=0, theta=ROPE_THETA)
    # N_C = 6: chunk 1 (positions 0..15) turns by D = (6 - 1 - 1) * 16 = 64
    np.testing.assert_allclose(turned[0], later[0], rtol=0, atol=0.05)  # bf16 rounding of the cache
