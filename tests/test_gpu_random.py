"""Seeded random configurations of the recall through the C ABI against the oracle: odd head
layouts, lengths, budgets, pooling specs and sinks drawn together, each checked three ways (one
call, key shards at random cuts, the host entry point)."""
import random

import numpy as np
import pytest
import torch

import oracle
import parity
from workloads import make_inputs, small_workload

pytestmark = pytest.mark.gpu


def _draw(seed):
    rng = random.Random(seed)
    n_kv = rng.choice([1, 2, 4, 8])
    n_q = n_kv * rng.choice([1, 2, 4, 7])
    L = rng.choice([rng.randint(1, 300), rng.randint(300, 6000), rng.randint(6000, 40000)])
    q_len = rng.choice([1, 2, 5, 16, 33, 64]) if L < 6000 else rng.choice([1, 4, 16])
    n_sink = min(rng.choice([0, 0, 1, 4]), L)
    budget = rng.randint(0, min(L - n_sink, 500))
    max_sizes = tuple(sorted(rng.sample([1, 2, 3, 4, 8, 16, 64], rng.randint(1, 3))))
    win_sizes = tuple(sorted(rng.sample([1, 2, 3, 4, 5, 7, 8, 15, 16, 31, 63, 200], rng.randint(1, 4))))
    w = small_workload(L, q_len, seed=1000 + seed, n_kv_heads=n_kv, n_q_heads=n_q,
                       n_spans=2 if L >= 256 else 0, budget=budget, max_sizes=max_sizes,
                       win_sizes=win_sizes, win_op=rng.randint(0, 1), n_sink=n_sink,
                       key_kind=rng.choice(["gauss", "lowrank", "outlier"]))
    n_cut = rng.randint(0, 3)
    cuts = sorted(set([0, L] + [rng.randint(1, L) for _ in range(n_cut)]))
    return w, cuts


@pytest.mark.parametrize("seed", range(32))
def test_random_configuration(seed):
    from paper_2508_17892_b200 import IlreRecall
    w, cuts = _draw(seed)
    x = make_inputs(w)
    spec = (w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    eng = IlreRecall(max_L=w.L, max_q_len=w.q_len, max_budget=max(w.budget, 1), max_combinations=48,
                     n_kv_heads=w.n_kv_heads, n_q_heads=w.n_q_heads, host_staging=True)
    K, Q = x.K.cuda(), x.Q.cuda()
    a = oracle.scores(x.K, x.Q)
    idx, sc = eng.run(K, Q, *spec, want_scores=True)
    torch.cuda.synchronize()
    eng.check_status()
    parity.check_recall(x.K, x.Q, w, idx.cpu().numpy(), sc.cpu().numpy(), ref_scores=a)
    shards = [K[p:q] for p, q in zip(cuts[:-1], cuts[1:])]
    stats = torch.stack([eng.shard_stats(k, Q) for k in shards])
    sc2 = torch.cat([eng.shard_scores(k, Q, stats) for k in shards])
    idx2 = eng.allocate(sc2, *spec)
    torch.cuda.synchronize()
    eng.check_status()
    parity.check_recall(x.K, x.Q, w, idx2.cpu().numpy(), sc2.cpu().numpy(), ref_scores=a)
    idx3, _ = eng.run_host(x.K, x.Q, *spec)
    eng.check_status()
    assert np.array_equal(idx3.numpy(), idx.cpu().numpy())
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def _draw_many(seed):
    rng = random.Random(900 + seed)
    L = rng.choice([rng.randint(200, 3000), rng.randint(3000, 40000), rng.randint(40000, 150000)])
    n_sink = rng.choice([0, 4, 37])
    budget = min(rng.choice([rng.randint(48, 600), rng.randint(600, 5000), 4096]), L - n_sink - 1)
    max_sizes = tuple(sorted(rng.sample([1, 2, 3, 4, 8, 16, 32, 64], rng.randint(2, 6))))
    win_sizes = tuple(sorted(rng.sample([1, 2, 3, 5, 7, 9, 11, 13, 15, 31, 63], rng.randint(4, 8))))
    return small_workload(L, rng.choice([1, 2, 4]), seed=5000 + seed, n_spans=3 if L >= 256 else 0,
                          budget=budget, max_sizes=max_sizes, win_sizes=win_sizes,
                          win_op=rng.randint(0, 1), n_sink=n_sink,
                          key_kind=rng.choice(["gauss", "lowrank", "outlier"]))


@pytest.mark.parametrize("seed", range(12))
def test_random_configuration_with_many_combinations(seed):
    """8 to 48 (max size, window size) combinations at once, as in Algorithm 1's default pooling:
    many candidate lists of very different lengths share the grid."""
    from paper_2508_17892_b200 import IlreRecall
    w = _draw_many(seed)
    x = make_inputs(w)
    eng = IlreRecall(max_L=w.L, max_q_len=w.q_len, max_budget=max(w.budget, 1), max_combinations=48,
                     n_kv_heads=w.n_kv_heads, n_q_heads=w.n_q_heads)
    idx, sc = eng.run(x.K.cuda(), x.Q.cuda(), w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                      want_scores=True)
    torch.cuda.synchronize()
    eng.check_status()
    parity.check_recall(x.K, x.Q, w, idx.cpu().numpy(), sc.cpu().numpy())
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()
