"""The end-to-end index rule of tests/parity.py, checked on the CPU: an allocation produced by
Algorithm 1 on slightly perturbed scores (what a single-precision path does to near-ties),
knock-on effects in later combinations included, must be accepted, and an allocation with a
choice that no near-tie accounts for must be rejected.  The mistakes are planted here, in the
oracle's output."""
import numpy as np
import pytest

import oracle
import parity


def _scores(seed, L):
    rng = np.random.default_rng(seed)
    a = rng.random(L) ** 8                        # heavy head, like attention scores
    a[rng.integers(0, L, L // 20)] = a[rng.integers(0, L, L // 20)]   # exact repeats
    return a / a.sum()


SPECS = [
    (300, (1,), (1, 7, 15), 1, 0),
    (400, (2, 4, 8), (1, 2, 3, 4), 0, 4),
    (257, (3,), (5, 16), 0, 2),
    (96, (1, 2), (1, 5), 0, 1),
    (1000, (2, 4, 8), tuple(range(1, 17)), 0, 4),
]


@pytest.mark.parametrize("seed", range(5))
@pytest.mark.parametrize("spec", SPECS, ids=str)
def test_near_tie_flips_are_accepted_and_planted_errors_rejected(seed, spec):
    budget, max_sizes, win_sizes, win_op, n_sink = spec
    L = 5000
    a = _scores(seed, L)
    ref, diag = oracle.allocate(a, *spec, diagnostics=True)
    assert parity.decisions_within_tolerance(a, diag["combination_of"], *spec, rtol=0.0,
                                             atol=0.0) == []
    # a relative perturbation inside the tolerance, as a single-precision path produces: flips
    # at the cut-offs and their knock-on in later combinations
    rng = np.random.default_rng(100 + seed)
    b = a * (1.0 + 4e-4 * rng.standard_normal(L).clip(-2, 2))
    idx, dg = oracle.allocate(b, *spec, diagnostics=True)
    comb_of = dg["combination_of"]
    assert parity.decisions_within_tolerance(a, comb_of, *spec) == []
    if len(set(idx.tolist()) ^ set(ref.tolist())):
        assert parity.decisions_within_tolerance(a, comb_of, *spec, rtol=0.0, atol=0.0)
    # planted mistake: one recalled position swapped for the lowest-scored free one
    taken = np.flatnonzero(comb_of >= 0)
    victim = taken[np.argmax(a[taken])]
    free = np.flatnonzero(comb_of < 0)
    free = free[free >= n_sink]
    spare = free[np.argmin(a[free])]
    wrong = comb_of.copy()
    wrong[spare], wrong[victim] = wrong[victim], -1
    assert parity.decisions_within_tolerance(a, wrong, *spec)
    # planted mistake: a quota off by one (one position dropped)
    short = comb_of.copy()
    short[victim] = -1
    assert parity.decisions_within_tolerance(a, short, *spec)
    # planted mistake: a position credited to a combination that runs before the one whose
    # turn it was to take it, in exchange for one of that combination's own
    if len(max_sizes) * len(win_sizes) > 1:
        last = comb_of.max()
        a_pos = np.flatnonzero(comb_of == last)
        b_pos = np.flatnonzero(comb_of == 0)
        lo = a_pos[np.argmin(a[a_pos])]
        hi = b_pos[np.argmax(a[b_pos])]
        swapped = comb_of.copy()
        swapped[lo], swapped[hi] = 0, last
        assert parity.decisions_within_tolerance(a, swapped, *spec)
    # planted mistake: a sink position allocated
    if n_sink:
        sunk = comb_of.copy()
        sunk[0] = 0
        assert parity.decisions_within_tolerance(a, sunk, *spec)
