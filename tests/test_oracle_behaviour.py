"""The oracle on the smallest benchmark configuration: planted needle spans come back."""
import numpy as np

import oracle
from workloads import CONFIGS, make_inputs


def test_config1_planted_spans_are_recovered():
    x = make_inputs(CONFIGS["cfg1_L4k"])
    w = x.workload
    idx, a = oracle.recall(x.K, x.Q, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    planted = set(x.planted_positions().tolist())
    assert len(planted) == 4 * 32
    assert planted <= set(idx.tolist())
    assert len(idx) == w.budget and np.all(np.diff(idx) > 0)
    # every needle outscores 99% of the background keys
    mask = np.zeros(w.L, dtype=bool)
    mask[list(planted)] = True
    assert a[mask].min() > np.quantile(a[~mask], 0.99)


def test_generator_is_deterministic_and_seeded():
    a = make_inputs(CONFIGS["cfg1_L4k"])
    b = make_inputs(CONFIGS["cfg1_L4k"])
    assert (a.K.view(dtype=a.K.dtype) == b.K).all() and (a.Q == b.Q).all() and a.spans == b.spans
