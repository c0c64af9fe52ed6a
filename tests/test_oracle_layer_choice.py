"""Pins of the oracle's retrieval-layer choice (Section 3.3, first paragraph; Appendix A.1):
worked examples small enough to do by hand, and the invariants of the definition."""
import numpy as np

import oracle


def test_hits_of_a_hand_worked_example():
    # recalled 1 2 3 7 8 12; phrases: [1..3] complete, [7..9] misses 9, [20..21] untouched,
    # [12..12] a one-token phrase that was recalled
    hits = oracle.span_hits([1, 2, 3, 7, 8, 12], [(1, 3), (7, 3), (20, 2), (12, 1)])
    assert hits.tolist() == [3, 2, 0, 1]


def test_exact_match_counts_only_complete_phrases():
    spans = [(10, 4), (100, 2), (200, 3)]
    layers = [
        [10, 11, 12, 100, 101, 200, 201],          # 1 complete (second), first misses 13
        [10, 11, 12, 13, 100, 101, 200, 201, 202],  # all 3
        [10, 11, 12, 13, 100, 101, 200, 201, 202],  # all 3 again: the earlier layer must win
        [5, 6, 7],                                   # none
    ]
    hits, full, l_r = oracle.layer_choice(layers, spans)
    assert hits.tolist() == [[3, 2, 2], [4, 2, 3], [4, 2, 3], [0, 0, 0]]
    assert full.tolist() == [1, 3, 3, 0]
    assert l_r == 1


def test_smallest_index_wins_also_when_nothing_is_retrieved():
    _, full, l_r = oracle.layer_choice([[1], [2], [3]], [(10, 2)])
    assert full.tolist() == [0, 0, 0] and l_r == 0


def test_a_partial_phrase_never_beats_a_complete_one():
    # layer 0 recalls 9 of 10 positions of each phrase (more positions in total), layer 1
    # recalls one phrase completely and nothing of the other
    spans = [(0, 10), (50, 10)]
    l0 = list(range(0, 9)) + list(range(50, 59))
    l1 = list(range(0, 10))
    hits, full, l_r = oracle.layer_choice([l0, l1], spans)
    assert hits.sum(axis=1).tolist() == [18, 10]
    assert full.tolist() == [0, 1] and l_r == 1


def test_invariants_on_random_lists():
    rng = np.random.default_rng(5)
    L = 5000
    begins = np.sort(rng.choice(np.arange(0, L - 64, 64), size=20, replace=False))
    spans = [(int(b), int(rng.integers(1, 40))) for b in begins]          # disjoint
    layers = [np.sort(rng.choice(L, size=n, replace=False)) for n in (0, 100, 2500, L)]
    hits, full, l_r = oracle.layer_choice(layers, spans)
    lens = np.array([n for _, n in spans])
    assert np.all(hits >= 0) and np.all(hits <= lens[None, :])
    assert np.all(hits.sum(axis=1) <= [len(x) for x in layers])            # disjoint phrases
    assert hits[0].sum() == 0 and np.array_equal(hits[3], lens)            # empty / everything
    assert full[3] == len(spans) and l_r == int(np.argmax(full))
    # against numpy's own membership routine
    for l, idx in enumerate(layers):
        ref = [int(np.isin(np.arange(b, b + n), idx).sum()) for b, n in spans]
        assert hits[l].tolist() == ref
