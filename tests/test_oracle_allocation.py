"""Pins for the oracle's Algorithm 1 part (pooling, top-K_m, quota, de-duplication, sort)."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                out[k.strip()] = v.split()
    return out


# ---------------------------------------------------------------- pooling

def _brute_maxpool(a, m):
    return np.array([max(a[c * m:(c + 1) * m]) for c in range((len(a) + m - 1) // m)])


def _brute_window(p, n, op):
    out = []
    for c in range(len(p)):
        lo = c - n // 2
        vals = [p[u] for u in range(lo, lo + n) if 0 <= u < len(p)]
        out.append(sum(vals) / n if op == 0 else max(vals))
    return np.array(out)


@pytest.mark.parametrize("n", [1, 2, 3, 7, 10, 31])
def test_maxpool_brute_force(n):
    rng = np.random.default_rng(n)
    for L in (1, 5, 16, 37):
        a = rng.random(L)
        np.testing.assert_array_equal(oracle.maxpool(a, n), _brute_maxpool(list(a), n))


@pytest.mark.parametrize("op", [0, 1])
@pytest.mark.parametrize("n", [1, 2, 3, 4, 7, 16, 63])
def test_window_pool_brute_force(n, op):
    rng = np.random.default_rng(100 + n)
    for L in (1, 2, 9, 40, 130):
        p = rng.random(L)
        np.testing.assert_allclose(oracle.winpool(p, n, op), _brute_window(list(p), n, op),
                                   rtol=1e-14)


def test_size_one_pooling_is_identity():
    a = np.random.default_rng(0).random(77)
    np.testing.assert_array_equal(oracle.maxpool(a, 1), a)
    np.testing.assert_array_equal(oracle.winpool(a, 1, 0), a)
    np.testing.assert_array_equal(oracle.winpool(a, 1, 1), a)


def test_pooling_known_values():
    # monotone array: strided max pooling picks the last element of every cell
    a = np.arange(10, dtype=np.float64)
    np.testing.assert_array_equal(oracle.maxpool(a, 4), [3, 7, 9])
    # odd window is centred; even window has the extra cell on the left
    p = np.array([1.0, 2.0, 4.0, 8.0, 16.0])
    np.testing.assert_allclose(oracle.winpool(p, 3, 0), np.array([3, 7, 14, 28, 24]) / 3)
    np.testing.assert_allclose(oracle.winpool(p, 2, 0), np.array([1, 3, 6, 12, 24]) / 2)
    np.testing.assert_array_equal(oracle.winpool(p, 4, 1), [2, 4, 8, 16, 16])
    # a constant array stays constant away from the zero-padded edges
    c = oracle.winpool(np.full(20, 0.25), 5, 0)
    np.testing.assert_allclose(c[2:-2], 0.25)
    np.testing.assert_allclose(c[[0, 1, -2, -1]], [0.15, 0.2, 0.2, 0.15])


# ---------------------------------------------------------------- Algorithm 1

def _alg1_with_sets(A, n_sink, B, max_sizes, win_sizes, win_op):
    """Algorithm 1 written with Python sets and full sorts, in the paper's loop order."""
    A = list(A)
    I = set(range(n_sink))
    Ap = A[n_sink:]
    n_comb = len(max_sizes) * len(win_sizes)
    comb = 0
    for m in max_sizes:
        P = [max(Ap[c * m:(c + 1) * m]) for c in range((len(Ap) + m - 1) // m)]
        K_m = B // m + 1 + (1 if len(Ap) % m else 0)
        for n in win_sizes:
            B_c = B // n_comb + (1 if comb < B % n_comb else 0)
            comb += 1
            W = _brute_window(P, n, win_op)
            top = sorted(range(len(P)), key=lambda c: (-W[c], c))[:K_m]
            mapped = [n_sink + t for c in top for t in range(c * m, min(c * m + m, len(Ap)))]
            S_I = 0
            it = iter(mapped)
            while S_I < B_c:
                idx = next(it)
                if idx not in I:
                    I.add(idx)
                    S_I += 1
    return sorted(I)


@pytest.mark.parametrize("seed", range(12))
def test_algorithm1_against_set_transcription(seed):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(20, 90))
    n_sink = int(rng.integers(0, 5))
    B = int(rng.integers(1, (L - n_sink) // 2))
    max_sizes = [[1], [2, 4], [2, 4, 8], [3]][seed % 4]
    win_sizes = [[1, 3], [1, 2, 3, 4], [5], [1, 7, 15]][(seed // 4) % 4 if seed < 8 else seed % 4]
    win_op = seed % 2
    if seed % 3 == 0:       # few distinct values: long runs of exact ties
        A = rng.integers(1, 5, size=L).astype(np.float64) / 8.0
    else:
        A = rng.random(L)
    got = oracle.allocate(A, B, max_sizes, win_sizes, win_op, n_sink)
    assert list(got) == _alg1_with_sets(A, n_sink, B, max_sizes, win_sizes, win_op)


def test_hand_worked_example():
    g = _read_golden("alg1_worked_example.txt")
    A = np.array([float(x) for x in g["A"]])
    got, diag = oracle.allocate(A, int(g["budget"][0]), [int(x) for x in g["max_sizes"]],
                                [int(x) for x in g["win_sizes"]], 0, diagnostics=True)
    assert list(got) == [int(x) for x in g["expected"]]
    assert list(diag["combination_of"]) == [int(x) for x in g["combination_of"]]


def test_hand_worked_tie_rule():
    g = _read_golden("tie_rule_example.txt")
    A = np.array([float(x) for x in g["A"]])
    got = oracle.allocate(A, int(g["budget"][0]), [int(x) for x in g["max_sizes"]],
                          [int(x) for x in g["win_sizes"]], int(g["win_op"][0]))
    assert list(got) == [int(x) for x in g["expected"]]


def test_snapkv_special_case_is_plain_topk_of_average_pool():
    # one max kernel of size 1 + one average kernel == top-B of the average-pooled scores
    rng = np.random.default_rng(42)
    A = rng.random(500)
    n, B = 7, 60
    pooled = np.convolve(A, np.ones(n) / n, mode="same")
    want = np.sort(np.argsort(-pooled, kind="stable")[:B])
    got = oracle.allocate(A, B, [1], [n], 0)
    np.testing.assert_array_equal(got, want)


def test_monotone_scores_give_exact_topk():
    A = np.linspace(0.0, 1.0, 1000) ** 2
    got = oracle.allocate(A, 100, [1], [1], 1)
    np.testing.assert_array_equal(got, np.arange(900, 1000))
    # with max cells of 4 the last 25 cells are taken whole
    got = oracle.allocate(A, 100, [4], [1], 0)
    np.testing.assert_array_equal(got, np.arange(900, 1000))


def test_default_spec_counts_quota_and_invariants():
    rng = np.random.default_rng(7)
    L, B, S = 3000, 500, 4
    A = rng.random(L) ** 4
    max_sizes, win_sizes = [2, 4, 8], list(range(1, 17))
    idx, diag = oracle.allocate(A, B, max_sizes, win_sizes, 0, n_sink=S, diagnostics=True)
    assert len(diag["quota"]) == 48
    assert diag["quota"].sum() == B
    assert set(diag["quota"]) == {B // 48, B // 48 + 1}
    assert list(diag["quota"][: B % 48]) == [B // 48 + 1] * (B % 48)
    np.testing.assert_array_equal(diag["taken"], diag["quota"])
    assert len(idx) == S + B and len(set(idx)) == S + B
    assert np.all(np.diff(idx) > 0)
    assert list(idx[:S]) == list(range(S))
    assert idx.min() >= 0 and idx.max() < L


def test_budget_edges():
    A = np.random.default_rng(1).random(37)
    assert list(oracle.allocate(A, 0, [2], [3], 0, n_sink=3)) == [0, 1, 2]
    # the whole context fits: every position comes back, also with a partial tail cell
    for m in ([1], [2], [4], [8], [5, 3]):
        got = oracle.allocate(A, 37 - 2, m, [1, 4], 0, n_sink=2)
        np.testing.assert_array_equal(got, np.arange(37))
    with pytest.raises(RuntimeError):
        oracle.allocate(A, 36, [1], [1], 0, n_sink=2)


def test_quota_always_reachable_with_partial_tail_cell():
    # termination of the "while S_I < B_c" loop for every (L', m, B) on a small grid
    rng = np.random.default_rng(3)
    for Lp in range(1, 26):
        A = rng.random(Lp)
        for m in (1, 2, 3, 4, 8):
            for B in range(0, Lp + 1):
                idx = oracle.allocate(A, B, [m], [1, 2], 0)
                assert len(set(idx)) == B


def test_multi_kernel_keeps_long_span_whole_single_small_kernel_does_not():
    # A long span in which only a few tokens score high, plus scattered isolated peaks that
    # out-rank the weak span tokens: one size-1 kernel picks the peaks, larger windows pull
    # in the whole span (the lesson of the paper's pooling ablation).
    rng = np.random.default_rng(11)
    L, B = 4000, 128
    A = rng.random(L) * 0.01
    span = np.arange(1000, 1064)
    A[span] = 0.02
    A[span[::8]] = 0.9                                   # 8 strong tokens inside the span
    peaks = rng.choice(np.setdiff1d(np.arange(L), np.arange(900, 1200)), 200, replace=False)
    A[peaks] = 0.5                                       # isolated distractors
    single = set(oracle.allocate(A, B, [1], [1], 0))
    multi = set(oracle.allocate(A, B, [1], [1, 15, 31], 1))
    assert len(single & set(span)) == 8
    assert set(span) <= multi


# ---- the averaging window in single precision (the rounding an fp32 implementation applies) ----

def test_single_precision_average_hand_example():
    # window of 3 around cell 1 covers 1, 2^-24, 2^-24: in float 1 + 2^-24 rounds back to 1
    # (tie to even) twice, so the sum is 1 and the average float(1) / float(3); in double the
    # sum is 1 + 2^-23
    p = np.array([1.0, 2.0 ** -24, 2.0 ** -24, 0.0, 0.0], dtype=np.float64)
    w64 = oracle.winpool(p, 3, 0)
    w32 = oracle.winpool(p, 3, 0, avg_single=True)
    assert w64[1] == (1.0 + 2.0 ** -23) / 3.0
    assert w32[1] == float(np.float32(1.0) / np.float32(3.0))
    # the maximum window is exact either way
    assert np.array_equal(oracle.winpool(p, 3, 1), oracle.winpool(p, 3, 1, avg_single=True))


def test_single_precision_average_is_exact_on_small_integers_and_close_otherwise():
    rng = np.random.default_rng(3)
    ints = rng.integers(0, 64, size=500).astype(np.float64) * 8.0       # sums and /8 exact in float
    assert np.array_equal(oracle.winpool(ints, 8, 0), oracle.winpool(ints, 8, 0, avg_single=True))
    x = np.exp(rng.normal(-10, 3, size=2000)).astype(np.float32).astype(np.float64)
    for n in (2, 7, 31, 200):
        w64, w32 = oracle.winpool(x, n, 0), oracle.winpool(x, n, 0, avg_single=True)
        assert np.all(np.abs(w32 - w64) <= (n + 1) * 2.0 ** -24 * w64)
        assert np.array_equal(w32, w32.astype(np.float32).astype(np.float64))   # results are floats


def test_single_precision_average_can_turn_a_near_tie_into_a_tie():
    # cells 1 and 4 hold 1; cell 3, left neighbour of cell 4, holds 2^-25.  Window 2 covers
    # [c - 1, c]: in double cell 4 averages 0.5 + 2^-26 and ranks first; in float both cells
    # average exactly 0.5 and the lower index ranks first.
    a = np.array([0.0, 1.0, 0.0, 2.0 ** -25, 1.0, 0.0, 0.0, 0.0], dtype=np.float64)
    assert oracle.allocate(a, 1, (1,), (2,), 0).tolist() == [4]
    assert oracle.allocate(a, 1, (1,), (2,), 0, avg_single=True).tolist() == [1]
    # the switch does not leak into later calls
    assert oracle.allocate(a, 1, (1,), (2,), 0).tolist() == [4]
