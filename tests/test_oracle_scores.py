"""Pins for the oracle's Eq. 4 / Eq. 5 part (logits, softmax over keys, max reduction).

Every check compares the C oracle with something fixed by mathematics or by a library
routine, never with the oracle itself.
"""
import numpy as np
import pytest
import torch
from scipy.special import softmax as scipy_softmax

import oracle


def _bf16(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def _f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def _library_scores(K: torch.Tensor, Q: torch.Tensor) -> np.ndarray:
    """Eq. 4 + Eq. 5 through numpy einsum and scipy softmax (fp64)."""
    k, q = _f64(K), _f64(Q)
    L, n_kv, d = k.shape
    q_len, n_q, _ = q.shape
    group = n_q // n_kv
    kv_of_head = np.arange(n_q) // group
    logits = np.einsum("ihc,thc->hit", q, k[:, kv_of_head, :]) / np.sqrt(d)
    probs = scipy_softmax(logits, axis=-1)
    return probs.max(axis=(0, 1))


def test_single_row_is_library_softmax_and_sums_to_one():
    rng = np.random.default_rng(0)
    K = _bf16(rng.standard_normal((257, 1, 16)))
    Q = _bf16(rng.standard_normal((1, 1, 16)))
    a = oracle.scores(K, Q)
    logits = (_f64(K)[:, 0, :] @ _f64(Q)[0, 0, :]) / np.sqrt(16.0)
    np.testing.assert_allclose(a, scipy_softmax(logits), rtol=1e-12, atol=0)
    assert abs(a.sum() - 1.0) < 1e-12


def test_identical_keys_give_one_over_L():
    rng = np.random.default_rng(1)
    key = rng.standard_normal((1, 2, 8))
    K = _bf16(np.repeat(key, 100, axis=0))
    Q = _bf16(rng.standard_normal((3, 4, 8)))
    a = oracle.scores(K, Q)
    np.testing.assert_allclose(a, np.full(100, 0.01), rtol=1e-13)


def test_two_keys_closed_form_pins_the_scale():
    # one head, one query token, d = 4: logits are (q.k)/2, so p0 = 1/(1+exp(-(s0-s1))).
    Q = _bf16([[[1.0, 2.0, 0.0, -1.0]]])
    K = _bf16([[[3.0, 0.5, 7.0, 1.0]], [[-1.0, 1.0, 2.0, 0.0]]])
    s0 = (3.0 + 1.0 + 0.0 - 1.0) / 2.0
    s1 = (-1.0 + 2.0) / 2.0
    p0 = 1.0 / (1.0 + np.exp(-(s0 - s1)))
    a = oracle.scores(K, Q)
    np.testing.assert_allclose(a, [p0, 1.0 - p0], rtol=1e-14)


@pytest.mark.parametrize("n_kv,n_q,q_len,L,d", [(2, 4, 3, 50, 8), (4, 8, 2, 33, 16),
                                                 (1, 3, 5, 20, 4), (8, 32, 2, 64, 128)])
def test_gqa_mapping_and_max_reduction_against_library(n_kv, n_q, q_len, L, d):
    rng = np.random.default_rng(10 + n_q)
    K = _bf16(rng.standard_normal((L, n_kv, d)) * 1.5)
    Q = _bf16(rng.standard_normal((q_len, n_q, d)) * 1.5)
    a, m, z = oracle.scores(K, Q, with_stats=True)
    np.testing.assert_allclose(a, _library_scores(K, Q), rtol=1e-11, atol=0)
    # the row statistics are those of the same logits (row index i * n_q + h)
    k, q = _f64(K), _f64(Q)
    group = n_q // n_kv
    for i in range(q_len):
        for h in range(n_q):
            s = k[:, h // group, :] @ q[i, h, :] / np.sqrt(d)
            assert m[i * n_q + h] == pytest.approx(s.max(), rel=1e-13)
            assert z[i * n_q + h] == pytest.approx(np.exp(s - s.max()).sum(), rel=1e-12)


def test_bounds_and_query_permutation_invariance():
    rng = np.random.default_rng(3)
    K = _bf16(rng.standard_normal((200, 2, 16)))
    Q = _bf16(rng.standard_normal((6, 4, 16)))
    a = oracle.scores(K, Q)
    R = 6 * 4
    assert np.all(a > 0) and np.all(a <= 1)
    assert 1.0 <= a.sum() <= R
    perm = torch.tensor([4, 0, 5, 2, 1, 3])
    a2 = oracle.scores(K, Q[perm])
    np.testing.assert_array_equal(a, a2)
    # duplicating a query token cannot change a max
    a3 = oracle.scores(K, torch.cat([Q, Q[:2]], dim=0))
    np.testing.assert_array_equal(a, a3)
    # swapping two heads of the SAME group leaves A unchanged, swapping across groups does not
    Qs = Q.clone()
    Qs[:, [0, 1]] = Q[:, [1, 0]]
    np.testing.assert_array_equal(a, oracle.scores(K, Qs))
    Qx = Q.clone()
    Qx[:, [0, 2]] = Q[:, [2, 0]]
    assert not np.array_equal(a, oracle.scores(K, Qx))


def test_shift_invariance_with_exact_integers():
    # small integers are exact in bf16: adding one vector to every key shifts each row's
    # logits by a constant, which a softmax ignores.
    rng = np.random.default_rng(4)
    K = rng.integers(-3, 4, size=(64, 2, 8)).astype(np.float32)
    Q = rng.integers(-2, 3, size=(2, 4, 8)).astype(np.float32)
    shift = rng.integers(-2, 3, size=(1, 2, 8)).astype(np.float32)
    a = oracle.scores(_bf16(K), _bf16(Q))
    b = oracle.scores(_bf16(K + shift), _bf16(Q))
    np.testing.assert_allclose(a, b, rtol=1e-12)


def test_scores_at_and_row_stats_subsets_agree_with_full_definition():
    rng = np.random.default_rng(5)
    K = _bf16(rng.standard_normal((300, 2, 32)))
    Q = _bf16(rng.standard_normal((4, 8, 32)))
    lib = _library_scores(K, Q)
    rows = list(range(4 * 8))
    m, z = oracle.row_stats(K, Q, rows)
    pos = [0, 17, 299, 128]
    np.testing.assert_allclose(oracle.scores_at(K, Q, m, z, pos), lib[pos], rtol=1e-11)
    m2, z2 = oracle.row_stats(K, Q, [5, 30])
    assert m2[0] == m[5] and z2[1] == z[30]
