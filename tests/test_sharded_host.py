"""Host side of the key-range sharded recall: the shard boundaries, and the two exchanges on
gloo ranks with an engine whose three steps are the CPU oracle's (the exchange code is the
same one the GPU ranks run over NCCL; only the engine differs)."""
import math
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
LOG2E = 1.4426950408889634


def test_shard_bounds_cover_the_context_in_order():
    from paper_2508_17892_b200.sharded import shard_bounds
    for L in (1, 127, 128, 129, 1000, 4096, 131072, 1048576 + 77):
        for world in (1, 2, 3, 8):
            prev = 0
            sizes = []
            for r in range(world):
                lo, hi = shard_bounds(L, world, r)
                assert lo == prev and hi >= lo
                assert lo % 128 == 0 or lo == L
                prev = hi
                sizes.append(hi - lo)
            assert prev == L
            # balanced to within one tile (the last shard also absorbs the ragged tail)
            assert max(sizes) - min(sizes) <= 128 + 127


class OracleEngine:
    """shard_stats / shard_scores / allocate computed by the oracle on CPU tensors."""

    def shard_stats(self, K_shard, Q):
        import oracle
        rows = np.arange(Q.shape[0] * Q.shape[1])
        m, z = oracle.row_stats(K_shard, Q, rows)
        return torch.from_numpy(np.stack([m * LOG2E, z], axis=1).astype(np.float32))

    def shard_scores(self, K_shard, Q, stats_all, out):
        import oracle
        st = stats_all.numpy().astype(np.float64)
        M = st[:, :, 0].max(axis=0)
        Z = (st[:, :, 1] * np.exp2(st[:, :, 0] - M)).sum(axis=0)
        a = oracle.scores_at(K_shard, Q, M / LOG2E, Z, np.arange(K_shard.shape[0]))
        out.copy_(torch.from_numpy(a.astype(np.float32)))
        return out

    def allocate(self, scores, budget, max_sizes, win_sizes, win_op, n_sink):
        import oracle
        return torch.from_numpy(oracle.allocate(scores.numpy().astype(np.float64), budget,
                                                max_sizes, win_sizes, win_op, n_sink))


def _worker(rank, world, port, L, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2508_17892_b200.sharded import shard_bounds, sharded_recall
    from workloads import make_inputs, small_workload
    w = small_workload(L, 3, seed=11, n_kv_heads=2, n_q_heads=4, budget=48, max_sizes=(1, 2),
                       win_sizes=(1, 5), win_op=0, n_sink=2)
    x = make_inputs(w)
    lo, hi = shard_bounds(L, world, rank)
    idx, sc = sharded_recall(OracleEngine(), x.K[lo:hi].contiguous(), x.Q, L, w.budget,
                             w.max_sizes, w.win_sizes, w.win_op, w.n_sink, want_scores=True)
    q.put((rank, idx.numpy().tolist(), sc.numpy().tolist()))
    dist.destroy_process_group()


@pytest.mark.parametrize("world,L,port", [(2, 1000, 29741), (3, 300, 29743)])
def test_sharded_recall_on_gloo_ranks_matches_the_unsharded_oracle(world, L, port):
    """L = 300 on three ranks leaves the last rank with 44 keys; L = 1000 on two gives
    512 + 488."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, L, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=240) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sys.path.insert(0, ROOT)
    import oracle
    import parity
    from workloads import make_inputs, small_workload
    w = small_workload(L, 3, seed=11, n_kv_heads=2, n_q_heads=4, budget=48, max_sizes=(1, 2),
                       win_sizes=(1, 5), win_op=0, n_sink=2)
    x = make_inputs(w)
    a = oracle.scores(x.K, x.Q)
    ref = oracle.allocate(a, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    for rank, idx, sc in got:
        assert idx == got[0][1], "ranks disagree on the recalled indices"
        sc = np.asarray(sc)
        assert sc.shape == (L,)
        # statistics and scores crossed the wire as fp32
        assert np.all(np.abs(sc - a) <= 2e-5 * a + 1e-12)
        assert len(idx) == w.n_sink + w.budget and idx == sorted(set(idx))
        own, diag = oracle.allocate(sc, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                                    diagnostics=True)
        assert own.tolist() == idx
        assert not parity.decisions_within_tolerance(a, diag["combination_of"], w.budget,
                                                     w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                                                     1e-4, 1e-12)
