"""GPU parity of the key-range sharded recall's per-rank steps, called through the C ABI.
The shards are processed one after another on one GPU (no kernel waits on another), which
computes exactly what P ranks compute between their two all-gathers."""
import numpy as np
import pytest
import torch

import oracle
import parity
from workloads import CONFIGS, make_inputs, small_workload

pytestmark = pytest.mark.gpu

LOG2E = 1.4426950408889634


def _engine(w, **kw):
    from paper_2508_17892_b200 import IlreRecall
    args = dict(max_L=w.L, max_q_len=w.q_len, max_budget=max(w.budget, 1), max_combinations=48,
                n_kv_heads=w.n_kv_heads, n_q_heads=w.n_q_heads)
    args.update(kw)
    return IlreRecall(**args)


def _sharded(eng, K, Q, cuts, w):
    """cuts: shard boundaries [0, ..., L].  Returns (idx, scores, per-shard statistics)."""
    shards = [K[a:b] for a, b in zip(cuts[:-1], cuts[1:])]
    stats = torch.stack([eng.shard_stats(k, Q) for k in shards])
    scores = torch.cat([eng.shard_scores(k, Q, stats) for k in shards])
    idx = eng.allocate(scores, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    torch.cuda.synchronize()
    eng.check_status()
    return idx.cpu().numpy(), scores.cpu().numpy(), stats.cpu().numpy()


@pytest.mark.parametrize("name,cuts", [
    ("cfg1_L4k", [0, 4096]),
    ("cfg1_L4k", [0, 1408, 4096]),
    ("cfg2_L32k", [0, 10880, 21888, 32768]),
    ("cfg3_L128k", [0, 16384, 32768, 49152, 65536, 81920, 98304, 114688, 131072]),
])
def test_sharded_steps_match_oracle(name, cuts):
    x = make_inputs(CONFIGS[name])
    w = x.workload
    eng = _engine(w)
    K, Q = x.K.cuda(), x.Q.cuda()
    idx, sc, stats = _sharded(eng, K, Q, cuts, w)
    a, m, z = oracle.scores(x.K, x.Q, with_stats=True)
    # every shard's statistics against the oracle's over the same key range (sampled rows)
    rows = np.unique(np.linspace(0, w.q_len * w.n_q_heads - 1, 24).astype(int))
    for s, (lo, hi) in enumerate(zip(cuts[:-1], cuts[1:])):
        ms, zs = oracle.row_stats(x.K[lo:hi].contiguous(), x.Q, rows)
        lse_ref = ms + np.log(zs)
        lse_gpu = stats[s, rows, 0] / LOG2E + np.log(stats[s, rows, 1].astype(np.float64))
        assert np.abs(lse_gpu - lse_ref).max() < 5e-4
        # the reported maximum is the row's true maximum (the sum is relative to it)
        assert np.abs(stats[s, rows, 0] / LOG2E - ms).max() < 1e-4 * np.maximum(1, np.abs(ms)).max()
    rep = parity.check_recall(x.K, x.Q, w, idx, sc, ref_scores=a)
    gpu_lse = eng.row_lse(w.q_len).cpu().numpy().reshape(-1)
    assert np.abs(gpu_lse - (m + np.log(z))).max() < 5e-4
    print(name, len(cuts) - 1, rep)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"


def test_one_shard_is_the_unsharded_run_bit_for_bit():
    x = make_inputs(CONFIGS["cfg2_L32k"])
    w = x.workload
    eng = _engine(w)
    K, Q = x.K.cuda(), x.Q.cuda()
    idx0, sc0 = eng.run(K, Q, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                        want_scores=True)
    idx0, sc0 = idx0.cpu().numpy(), sc0.cpu().numpy()
    idx, sc, _ = _sharded(eng, K, Q, [0, w.L], w)
    assert np.array_equal(sc, sc0)
    assert np.array_equal(idx, idx0)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"


def test_ragged_shards_sinks_and_strided_pooling():
    """Shard lengths that are not multiples of the key tile, a shard shorter than one tile,
    sink tokens, strided max-pooling and the averaging window."""
    w = small_workload(5000 + 77, 5, seed=23, budget=200, max_sizes=(1, 2, 4), win_sizes=(1, 7, 15),
                       win_op=0, n_sink=4)
    x = make_inputs(w)
    eng = _engine(w)
    idx, sc, _ = _sharded(eng, x.K.cuda(), x.Q.cuda(), [0, 100, 1900, 1901, 4000, w.L], w)
    rep = parity.check_recall(x.K, x.Q, w, idx, sc)
    print(rep)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"


@pytest.mark.parametrize("win_op", [0, 1])
@pytest.mark.parametrize("L", [1, 333, 70001])
def test_allocate_on_given_scores_is_algorithm_1(L, win_op):
    """Algorithm 1 from caller-supplied scores (no attention involved): heavy-tailed random
    scores with exact repeats, against the oracle's allocation on the same fp32 values."""
    rng = np.random.default_rng(L + win_op)
    a = np.exp(rng.normal(-12.0, 3.0, size=L)).astype(np.float32)
    if L > 10:
        a[rng.integers(0, L, size=L // 5)] = a[rng.integers(0, L, size=L // 5)]   # ties
    n_sink = 2 if L > 4 else 0
    budget = min(L - n_sink, 300)
    max_sizes, win_sizes = (1, 2, 8), (1, 3, 9)
    w = small_workload(L, 1, budget=budget)
    eng = _engine(w)
    idx = eng.allocate(torch.from_numpy(a).cuda(), budget, max_sizes, win_sizes, win_op, n_sink)
    torch.cuda.synchronize()
    eng.check_status()
    idx = idx.cpu().numpy()
    # the decision is taken in the kernel's precision on both sides: single-precision averages
    ref = oracle.allocate(a.astype(np.float64), budget, max_sizes, win_sizes, win_op, n_sink,
                          avg_single=True)
    assert len(idx) == n_sink + budget and np.all(np.diff(idx) > 0)
    assert np.array_equal(idx, ref)


def test_argument_errors():
    from paper_2508_17892_b200 import IlreError
    w = small_workload(1024, 2)
    x = make_inputs(w)
    eng = _engine(w)
    K, Q = x.K.cuda(), x.Q.cuda()
    big = torch.zeros(w.L + 1, dtype=torch.float32, device="cuda")
    with pytest.raises(IlreError):            # beyond the handle's max_L
        eng.allocate(big, 8, (1,), (1,))
    with pytest.raises(IlreError):            # budget beyond the context
        eng.allocate(big[:16], 17, (1,), (1,))
    stats = eng.shard_stats(K, Q)
    with pytest.raises(IlreError):            # zero shards
        eng.shard_scores(K, Q, stats.new_empty(0, w.q_len * w.n_q_heads, 2))
    torch.cuda.synchronize()
    eng.check_status()


def test_helper_with_a_single_rank_group():
    """sharded_recall (the exchange code) on a 1-rank NCCL group gives the unsharded result."""
    import torch.distributed as dist
    from paper_2508_17892_b200.sharded import sharded_recall
    x = make_inputs(CONFIGS["cfg1_L4k"])
    w = x.workload
    eng = _engine(w)
    K, Q = x.K.cuda(), x.Q.cuda()
    own = not dist.is_initialized()
    if own:
        dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29747", rank=0, world_size=1)
    try:
        idx, sc = sharded_recall(eng, K, Q, w.L, w.budget, w.max_sizes, w.win_sizes, w.win_op,
                                 w.n_sink, want_scores=True)
        torch.cuda.synchronize()
    finally:
        if own:
            dist.destroy_process_group()
    idx0, sc0 = eng.run(K, Q, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                        want_scores=True)
    assert torch.equal(idx, idx0) and torch.equal(sc, sc0)
