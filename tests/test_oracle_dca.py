"""Pins of the oracle's Eq. 7 (re-rotation of the cached keys under Dual Chunk Attention)."""
import math

import numpy as np
import torch

import oracle
from workloads.recall_inputs import ROPE_THETA, _rope_inplace


def _bf16(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def _chunk_of(t, chunk, n_sink):
    return 1 if t < n_sink else 1 + (t - n_sink) // chunk


def test_hand_computed_pair_rotation():
    # d = 2: one channel pair, theta^0 = 1, so the angle is D itself.  L = 7, chunk = 2, no
    # sink: N_C = 4, chunk 1 (t = 0, 1) turns by D = (4 - 1 - 1) * 2 = 4, chunk 2 by 2, rest 0.
    K = _bf16(np.tile(np.array([[[1.0, 0.0]]]), (7, 1, 1)))
    out = oracle.dca_rerope(K, chunk=2, n_sink=0, theta=10000.0)
    for t, D in enumerate([4, 4, 2, 2, 0, 0, 0]):
        assert abs(out[t, 0, 0] - math.cos(D)) < 1e-15
        assert abs(out[t, 0, 1] - math.sin(D)) < 1e-15


def test_sink_tokens_belong_to_the_first_chunk():
    # L = 11, n_sink = 3, chunk = 2: N_C = 4; positions 0..4 are chunk 1 (D = 4), 5..6 chunk 2
    K = _bf16(np.tile(np.array([[[0.0, 1.0]]]), (11, 1, 1)))
    out = oracle.dca_rerope(K, chunk=2, n_sink=3, theta=7.0)
    Ds = [4] * 5 + [2] * 2 + [0] * 4
    for t, D in enumerate(Ds):
        assert abs(out[t, 0, 0] + math.sin(D)) < 1e-15      # (0,1) -> (-sin, cos)
        assert abs(out[t, 0, 1] - math.cos(D)) < 1e-15


def test_norms_kept_and_last_two_chunks_untouched():
    g = torch.Generator().manual_seed(3)
    K = torch.randn(300, 2, 16, generator=g).to(torch.bfloat16)
    out = oracle.dca_rerope(K, chunk=64, n_sink=4, theta=ROPE_THETA)
    k = K.to(torch.float64).numpy()
    n_in = k[..., :8] ** 2 + k[..., 8:] ** 2
    n_out = out[..., :8] ** 2 + out[..., 8:] ** 2
    np.testing.assert_allclose(n_out, n_in, rtol=1e-12, atol=1e-300)
    # N_C = ceil(296 / 64) = 5: chunks 4 and 5 start at position 4 + 3 * 64
    np.testing.assert_array_equal(out[196:], k[196:])
    assert np.abs(out[:196] - k[:196]).max() > 0.1


def test_rotation_composes_with_rope_positions():
    # A key that carries RoPE at position p, turned by D, is the key with RoPE at p + D.  The
    # input generator's RoPE routine is an independent restatement of Eq. 3.
    g = torch.Generator().manual_seed(5)
    d, chunk, L = 128, 32, 200                     # N_C = 7
    base = torch.randn(1, 3, d, generator=g).to(torch.bfloat16).to(torch.float32)
    pos = torch.arange(L)
    keys = _rope_inplace(base.repeat(L, 1, 1).clone(), 0).to(torch.bfloat16)
    out = oracle.dca_rerope(keys, chunk=chunk, n_sink=0, theta=ROPE_THETA)
    n_chunks = -(-L // chunk)
    half = d // 2
    inv_freq = ROPE_THETA ** (-2.0 * np.arange(half) / d)
    kb = keys.to(torch.float64).numpy()
    for t in (0, 31, 32, 100, 159, 160, 199):
        i = _chunk_of(t, chunk, 0)
        D = (n_chunks - 1 - i) * chunk if i < n_chunks - 1 else 0
        ang = D * inv_freq
        want_lo = kb[t, :, :half] * np.cos(ang) - kb[t, :, half:] * np.sin(ang)
        want_hi = kb[t, :, :half] * np.sin(ang) + kb[t, :, half:] * np.cos(ang)
        np.testing.assert_allclose(out[t, :, :half], want_lo, rtol=0, atol=1e-12)
        np.testing.assert_allclose(out[t, :, half:], want_hi, rtol=0, atol=1e-12)
        # and against RoPE applied at the shifted position to the unrotated base (bf16 rounding
        # of `keys` bounds the agreement)
        shifted = _rope_inplace(base.clone(), t + D).to(torch.float64).numpy()[0]
        np.testing.assert_allclose(out[t], shifted, rtol=0, atol=0.05)
    # keys of different chunks with the same offset inside the chunk coincide after Eq. 7
    np.testing.assert_allclose(out[5], out[32 + 5], rtol=0, atol=0.05)
    np.testing.assert_allclose(out[5], out[4 * 32 + 5], rtol=0, atol=0.05)


def test_logit_identity_with_counter_rotated_query():
    g = torch.Generator().manual_seed(9)
    d, chunk, L = 64, 16, 80                       # N_C = 5
    K = torch.randn(L, 1, d, generator=g).to(torch.bfloat16)
    q = torch.randn(d, generator=g).to(torch.float64).numpy()
    out = oracle.dca_rerope(K, chunk=chunk, n_sink=0, theta=ROPE_THETA)
    half = d // 2
    inv_freq = ROPE_THETA ** (-2.0 * np.arange(half) / d)
    k = K.to(torch.float64).numpy()
    for t in (0, 17, 40, 79):
        i = _chunk_of(t, chunk, 0)
        D = (5 - 1 - i) * chunk if i < 4 else 0
        ang = -D * inv_freq                                            # R(-D) q
        q_lo = q[:half] * np.cos(ang) - q[half:] * np.sin(ang)
        q_hi = q[:half] * np.sin(ang) + q[half:] * np.cos(ang)
        lhs = float(q @ out[t, 0])
        rhs = float(np.concatenate([q_lo, q_hi]) @ k[t, 0])
        assert abs(lhs - rhs) < 1e-10


def test_short_contexts_are_left_alone():
    g = torch.Generator().manual_seed(1)
    K = torch.randn(100, 2, 8, generator=g).to(torch.bfloat16)
    for chunk in (50, 64, 100, 1000):              # N_C <= 2
        out = oracle.dca_rerope(K, chunk=chunk, n_sink=0, theta=ROPE_THETA)
        np.testing.assert_array_equal(out, K.to(torch.float64).numpy())


# ---- Eq. 6: the sink keys of the layers before the retrieval layer ----

def _complex_rotation(x, dist, theta=500000.0):
    """Independent route: the pair (c, c + d/2) as a complex number times e^{i dist w_c}."""
    d = x.shape[-1]
    half = d // 2
    w = theta ** (-2.0 * np.arange(half) / d)
    z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * dist * w)
    return np.concatenate([z.real, z.imag], axis=-1)


def test_sinks_first_two_chunks_see_the_cached_keys():
    g = torch.Generator().manual_seed(3)
    ks = torch.randn(4, 2, 128, generator=g).to(torch.bfloat16)
    for i in (1, 2):
        assert np.array_equal(oracle.dca_rerope_sinks(ks, i, 1024), ks.to(torch.float64).numpy())


def test_sinks_power_of_the_rotation_is_one_rotation_by_the_summed_distance():
    g = torch.Generator().manual_seed(4)
    ks = torch.randn(4, 8, 128, generator=g).to(torch.bfloat16)
    x = ks.to(torch.float64).numpy()
    for i, chunk in ((3, 1024), (4, 1024), (7, 512), (40, 100)):
        got = oracle.dca_rerope_sinks(ks, i, chunk)
        ref = _complex_rotation(x, (i - 2) * chunk)
        assert np.abs(got - ref).max() < 1e-9
        # pair norms are kept
        n0 = x[..., :64] ** 2 + x[..., 64:] ** 2
        n1 = got[..., :64] ** 2 + got[..., 64:] ** 2
        assert np.abs(n0 - n1).max() < 1e-9


def test_sinks_hand_computed_quarter_turn():
    # theta = 1 makes every pair turn by the distance itself; a chunk of pi/2 "positions"
    # cannot be given (integer), so use d = 2, theta = 1, chunk = 1 and check against
    # cos(1), sin(1) applied twice: (1, 0) -> (cos 2, sin 2)
    ks = torch.tensor([[[1.0, 0.0]]]).to(torch.bfloat16)
    got = oracle.dca_rerope_sinks(ks, 4, 1, theta=1.0)
    assert np.allclose(got[0, 0], [np.cos(2.0), np.sin(2.0)], atol=1e-12)


def test_sinks_keep_their_distance_to_the_chunk():
    """What Eq. 6 is for: a sink key cached with RoPE at position s, seen from chunk i, sits
    (i - 2) chunks further along, so its logit against a query at position p of chunk i equals
    the logit of the un-rotated key against a query (i - 2) chunks earlier."""
    g = torch.Generator().manual_seed(5)
    raw_k = torch.randn(1, 1, 128, generator=g, dtype=torch.float64).numpy()
    raw_q = torch.randn(128, generator=g, dtype=torch.float64).numpy()
    s, chunk, i = 2, 256, 6
    k_cached = _complex_rotation(raw_k, s)                       # RoPE at its own position
    kb = torch.from_numpy(k_cached).to(torch.bfloat16)
    k_i = oracle.dca_rerope_sinks(kb, i, chunk)[0, 0]
    p = 4 + (i - 1) * chunk + 17                                  # some position in chunk i
    q_p = _complex_rotation(raw_q[None], p)[0]
    q_back = _complex_rotation(raw_q[None], p - (i - 2) * chunk)[0]
    kb64 = kb.to(torch.float64).numpy()[0, 0]
    assert abs(np.dot(q_p, k_i) - np.dot(q_back, kb64)) < 1e-9
