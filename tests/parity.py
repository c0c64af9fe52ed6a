"""Parity rules between the CUDA path and the CPU oracle (helpers for the GPU tests).

scores: |gpu - oracle| <= 2e-3 * |oracle| + 1e-6 per position.
indices: (a) selection logic -- Algorithm 1 run by the oracle on the GPU's own fp32 scores
must give the GPU's index list EXACTLY.  Which cells rank first is an integer decision taken
from the pooled values, so both sides take it in the kernel's precision: the oracle adds the
averaging window left to right and divides in single precision, as the kernel does (the
maximum window is exact in any precision).
(b) end to end against the all-double oracle: with the combination that took every position
known from (a), every combination's choice is judged on the ORACLE's pooled values: no cell
that it left a free token in may rank above the cells it took from by more than the score
tolerance (`decisions_within_tolerance`).  A near-tie at a cut-off may fall either way; what
that changes for the later combinations is judged on what really was free then, not assumed:
one position that no such near-tie accounts for fails.  With `strict=True` (the benchmark
configurations) the index list must also be identical to the all-double oracle's.
"""
from __future__ import annotations

import numpy as np

import oracle

SCORE_RTOL = 2e-3
SCORE_ATOL = 1e-6


def score_errors(gpu: np.ndarray, ref: np.ndarray):
    gpu = np.asarray(gpu, dtype=np.float64)
    err = np.abs(gpu - ref)
    bound = SCORE_RTOL * np.abs(ref) + SCORE_ATOL
    worst = int(np.argmax(err / bound))
    return dict(max_rel=float(np.max(err / np.maximum(np.abs(ref), 1e-300))),
                max_ratio=float(err[worst] / bound[worst]), worst=worst,
                n_bad=int(np.sum(err > bound)))


def decisions_within_tolerance(A: np.ndarray, combination_of: np.ndarray, budget, max_sizes,
                               win_sizes, win_op, n_sink, rtol=SCORE_RTOL, atol=SCORE_ATOL):
    """Checks an allocation, given with the combination that took every position, against
    Algorithm 1 on the scores A (fp64), decision by decision.

    `combination_of[pos]` is the combination that allocated `pos` (-1 = not allocated).  In
    every combination, in loop order, the cells are judged by the pooled values computed from
    A: a cell that still has a free token which the combination did NOT take must not rank
    above the taken cells, i.e. its pooled value may exceed the smallest pooled value among
    the cells the combination took from by at most (rtol, atol).  With a zero tolerance this
    is Algorithm 1's rule itself (up to the order of exactly equal values); with the score
    tolerance it admits precisely the near-ties at each combination's cut-off, and the
    knock-on of a flipped near-tie -- later combinations finding other tokens free -- is
    judged on what really was free at that point instead of being waved through.  Also
    checked: quotas met exactly, nothing allocated twice or inside the sink part.
    Returns a list of violations (empty = consistent)."""
    A = np.asarray(A, dtype=np.float64)
    comb_of = np.asarray(combination_of)
    L = len(A)
    Lp = L - n_sink
    problems = []
    if np.any(comb_of[:n_sink] >= 0):
        problems.append(("sink allocated", -1, 0.0, 0.0))
    free = np.ones(Lp, dtype=bool)
    Ap = A[n_sink:]
    cp = comb_of[n_sink:]
    n_comb = len(max_sizes) * len(win_sizes)
    comb = 0
    for m in max_sizes:
        P = oracle.maxpool(Ap, m)
        n_cells = len(P)
        pad = n_cells * m - Lp
        for n in win_sizes:
            quota = budget // n_comb + (1 if comb < budget % n_comb else 0)
            W = oracle.winpool(P, n, win_op)
            mine = cp == comb
            if int(mine.sum()) != quota:
                problems.append(("quota", comb, float(mine.sum()), float(quota)))
            if np.any(mine & ~free):
                problems.append(("allocated twice", comb, 0.0, 0.0))
            if quota:
                free_cnt = np.pad(free, (0, pad)).reshape(n_cells, m).sum(axis=1)
                mine_cnt = np.pad(mine, (0, pad)).reshape(n_cells, m).sum(axis=1)
                took = mine_cnt > 0
                passed = free_cnt > mine_cnt               # a free token was left behind
                if took.any() and passed.any():
                    cut = W[took].min()
                    over = passed & (W > cut + rtol * abs(cut) + atol)
                    for c in np.flatnonzero(over)[:5]:
                        problems.append((comb, int(n_sink + c * m), float(W[c]), float(cut)))
                # inside a cell tokens go in ascending position: a partly taken cell keeps
                # its first free tokens
                for c in np.flatnonzero(took & passed):
                    lo, hi = c * m, min(c * m + m, Lp)
                    f = np.flatnonzero(free[lo:hi])
                    t = np.flatnonzero(mine[lo:hi])
                    if not np.array_equal(t, f[:len(t)]):
                        problems.append(("order inside cell", comb, float(c), 0.0))
            free &= ~mine
            comb += 1
    return problems


def check_recall(K, Q, w, gpu_idx, gpu_scores, ref_scores=None, ref_idx=None, spec=None,
                 strict=False):
    """Full parity check of one recall; returns a report dict, raises AssertionError on failure.

    `spec` overrides the workload's (budget, max_sizes, win_sizes, win_op, n_sink);
    `strict` demands an index list identical to the all-double oracle's."""
    budget, max_sizes, win_sizes, win_op, n_sink = spec or (
        w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    gpu_idx = np.asarray(gpu_idx)
    gpu_scores = np.asarray(gpu_scores, dtype=np.float64)
    if ref_scores is None:
        ref_scores = oracle.scores(K, Q)
    rep = score_errors(gpu_scores, ref_scores)
    assert rep["n_bad"] == 0, f"scores out of tolerance: {rep}"
    assert len(gpu_idx) == n_sink + budget
    assert np.all(np.diff(gpu_idx) > 0), "indices not strictly ascending"
    # (a) selection logic on the GPU's own scores, decided in the kernel's precision
    own, diag = oracle.allocate(gpu_scores, budget, max_sizes, win_sizes, win_op, n_sink,
                                avg_single=True, diagnostics=True)
    differ = sorted(set(gpu_idx.tolist()) ^ set(own.tolist()))
    rep["logic_diff"] = len(differ)
    assert not differ, f"selection logic differs from Algorithm 1 at {differ[:10]}"
    # (b) end to end against the oracle's own selection
    if ref_idx is None:
        ref_idx = oracle.allocate(ref_scores, budget, max_sizes, win_sizes, win_op, n_sink)
    rep["e2e_diff"] = len(set(gpu_idx.tolist()) ^ set(ref_idx.tolist()))
    if strict:
        assert rep["e2e_diff"] == 0, f"index list differs from the oracle's: {rep['e2e_diff']}"
    bad = decisions_within_tolerance(ref_scores, diag["combination_of"], budget, max_sizes,
                                     win_sizes, win_op, n_sink)
    rep["e2e_unexplained"] = len(bad)
    assert not bad, f"choices that no near-tie at a cut-off accounts for: {bad[:10]}"
    return rep
