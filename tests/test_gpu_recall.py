"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import parity
from workloads import (CONFIGS, PAPER_DEFAULT_MAX_SIZES, PAPER_DEFAULT_WIN_SIZES, make_inputs,
                       small_workload)

pytestmark = pytest.mark.gpu


def _engine(w, **kw):
    from paper_2508_17892_b200 import IlreRecall
    args = dict(max_L=w.L, max_q_len=w.q_len, max_budget=max(w.budget, 1), max_combinations=48,
                n_kv_heads=w.n_kv_heads, n_q_heads=w.n_q_heads)
    args.update(kw)
    return IlreRecall(**args)


def _run(eng, x, spec=None):
    w = x.workload
    budget, max_sizes, win_sizes, win_op, n_sink = spec or (
        w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    idx, sc = eng.run(x.K.cuda(), x.Q.cuda(), budget, max_sizes, win_sizes, win_op, n_sink,
                      want_scores=True)
    torch.cuda.synchronize()
    eng.check_status()
    return idx.cpu().numpy(), sc.cpu().numpy()


@pytest.fixture(scope="module")
def cases():
    cache = {}

    def get(name):
        if name not in cache:
            x = make_inputs(CONFIGS[name])
            a, m, z = oracle.scores(x.K, x.Q, with_stats=True)
            cache[name] = (x, a, m + np.log(z))
        return cache[name]
    return get


@pytest.mark.parametrize("name", ["cfg1_L4k", "cfg2_L32k", "cfg3_L128k", "cfg4_L512k"])
def test_benchmark_configs_match_oracle(cases, name):
    x, a, lse = cases(name)
    w = x.workload
    eng = _engine(w)
    idx, sc = _run(eng, x)
    rep = parity.check_recall(x.K, x.Q, w, idx, sc, ref_scores=a, strict=True)
    gpu_lse = eng.row_lse(w.q_len).cpu().numpy().reshape(-1)
    assert np.abs(gpu_lse - lse).max() < 5e-4
    assert eng.last_launch_count() > 0
    print(name, rep)
    # the planted spans are what the oracle recovers too
    planted = set(x.planted_positions().tolist())
    ref_idx = oracle.allocate(a, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    assert len(planted & set(idx.tolist())) == len(planted & set(ref_idx.tolist()))
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


@pytest.mark.parametrize("name", ["cfg1_L4k", "cfg2_L32k"])
@pytest.mark.parametrize("variant", ["avg", "paper_default", "paper_default_sink4"])
def test_other_pooling_specs(cases, name, variant):
    x, a, _ = cases(name)
    w = x.workload
    if variant == "avg":
        spec = (w.budget, w.max_sizes, w.win_sizes, 0, 0)
    elif variant == "paper_default":
        spec = (w.budget, PAPER_DEFAULT_MAX_SIZES, PAPER_DEFAULT_WIN_SIZES, 0, 0)
    else:
        spec = (w.budget, PAPER_DEFAULT_MAX_SIZES, PAPER_DEFAULT_WIN_SIZES, 0, 4)
    eng = _engine(w)
    idx, sc = _run(eng, x, spec)
    rep = parity.check_recall(x.K, x.Q, w, idx, sc, ref_scores=a, spec=spec)
    print(name, variant, rep)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


RAGGED = [
    # L, q_len, n_kv, n_q, budget, max_sizes, win_sizes, win_op, n_sink
    (1, 1, 8, 32, 1, (1,), (1,), 0, 0),
    (127, 1, 8, 32, 16, (1,), (1, 3), 1, 0),
    (129, 17, 8, 32, 40, (2,), (1, 2, 4), 0, 4),
    (1000, 16, 8, 32, 100, (2, 4, 8), (1, 2, 3, 4), 0, 4),
    (4097, 64, 8, 32, 512, (1,), (1, 7, 15), 1, 0),
    (5000, 130, 8, 32, 256, (3,), (5, 16), 0, 2),        # 520 rows per kv head: two row blocks
    (3001, 256, 8, 32, 300, (1,), (1, 63), 1, 0),
    (2049, 33, 4, 28, 128, (2, 8), (1, 6), 0, 1),        # 7 query heads per kv head
    (777, 9, 2, 2, 64, (1,), (1, 7), 1, 0),              # no grouping
    (20000, 40, 1, 8, 999, (4,), (1, 2), 0, 3),
    (300, 5, 8, 32, 296, (8,), (1, 4), 0, 4),            # budget = L - n_sink with a partial cell
    (300, 5, 8, 32, 0, (2,), (3,), 0, 4),                # empty budget: sinks only
    (50, 3, 8, 32, 0, (2,), (3,), 0, 0),                 # empty budget, no sinks: an empty list
]


@pytest.mark.parametrize("case", RAGGED, ids=lambda c: f"L{c[0]}_q{c[1]}_kv{c[2]}_h{c[3]}_B{c[4]}")
def test_ragged_shapes_match_oracle(case):
    L, q_len, n_kv, n_q, budget, max_sizes, win_sizes, win_op, n_sink = case
    w = small_workload(L, q_len, seed=L + q_len, n_kv_heads=n_kv, n_q_heads=n_q,
                       n_spans=2 if L >= 256 else 0, budget=budget, max_sizes=max_sizes,
                       win_sizes=win_sizes, win_op=win_op, n_sink=n_sink)
    x = make_inputs(w)
    eng = _engine(w)
    idx, sc = _run(eng, x)
    rep = parity.check_recall(x.K, x.Q, w, idx, sc)
    print(case, rep)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


BIG = [
    # L, q_len, budget, max_sizes, win_sizes, win_op, n_sink -- paths of the selection kernel
    # that the benchmark shapes do not reach
    (40000, 4, 9000, (1,), (1, 5), 1, 0),          # K_m > 8192: ranking staged in two chunks
    (60000, 2, 16382, (1,), (1,), 0, 0),           # largest budget: one staging buffer only
    (1200000, 1, 4096, (1,), (1, 15), 1, 4),       # bitmap too large for shared memory
    (1100000, 1, 2000, (2, 64), (1, 3), 0, 3),     # strided max-pool sources at 1M, m = 64
    # ascending output pass: word list with a long sink part that ends inside a bitmap word,
    # a word count that is no multiple of four, a context just past one word per thread
    (70001, 1, 3000, (1, 4), (1, 7), 1, 5003),
    (32801, 2, 1500, (1,), (3,), 0, 33),
    (1200070, 1, 1000, (1,), (1,), 1, 40000),      # the same with the bitmap in global memory
]


@pytest.mark.parametrize("case", BIG, ids=lambda c: f"L{c[0]}_q{c[1]}_B{c[2]}_m{len(c[3])}")
def test_selection_kernel_edge_paths(case):
    L, q_len, budget, max_sizes, win_sizes, win_op, n_sink = case
    w = small_workload(L, q_len, seed=L % 1000 + budget, n_spans=4, span_len=(16, 64),
                       budget=budget, max_sizes=max_sizes, win_sizes=win_sizes, win_op=win_op,
                       n_sink=n_sink)
    x = make_inputs(w)
    eng = _engine(w)
    idx, sc = _run(eng, x)
    rep = parity.check_recall(x.K, x.Q, w, idx, sc)
    print(case, rep)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


@pytest.mark.parametrize("pattern", ["all_equal", "two_levels", "blocks_of_equal", "all_equal_40k",
                                     "blocks_of_equal_40k", "all_equal_40k_B6000",
                                     "blocks_of_equal_40k_B6000"])
@pytest.mark.parametrize("win_op", [0, 1])
def test_massive_ties_follow_the_cell_order(pattern, win_op):
    """Keys that repeat make whole stretches of the scores bit-identical, so the K_m-th value
    is held by thousands of cells and the lower cell index has to decide (reading 11).  The
    plateaus are shorter (one CTA sorts the tied cells out) or longer (further passes over the
    whole array) than what the selection sets aside for one CTA, sometimes both in one call."""
    import dataclasses
    # the larger budget makes lists of 1024 to 8192 candidates: ranked inside value buckets
    # whose sampled splitters then differ in the cell index only
    budget = 6000 if pattern.endswith("_B6000") else 700
    pattern = pattern.replace("_B6000", "")
    L, q_len = (40000, 2) if pattern.endswith("_40k") else (9000, 3)
    pattern = pattern.replace("_40k", "")
    w = small_workload(L, q_len, seed=3, n_spans=0, budget=budget, max_sizes=(1, 2), win_sizes=(1, 3),
                       win_op=win_op, n_sink=2)
    x = make_inputs(w)
    g = torch.Generator().manual_seed(17)
    K = x.K.clone()
    if pattern == "all_equal":
        K[:] = K[0]
    elif pattern == "two_levels":
        K[: L // 2] = K[0]
        K[L // 2:] = K[1]
    else:
        protos = torch.randn(9, 8, 128, generator=g).to(torch.bfloat16)
        for b in range(9):
            K[b * (L // 9):(b + 1) * (L // 9)] = protos[b]
    x = dataclasses.replace(x, K=K.contiguous())
    eng = _engine(w)
    idx, sc = _run(eng, x)
    rep = parity.check_recall(x.K, x.Q, w, idx, sc)
    # the device scores really are bit-identical inside a stretch
    if pattern == "all_equal":
        assert np.unique(sc).size == 1
    print(pattern, win_op, rep)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_handle_reuse_and_determinism(cases):
    # one handle, different shapes back to back, and bit-identical repeats
    big = make_inputs(CONFIGS["cfg2_L32k"])
    eng = _engine(big.workload)
    first = _run(eng, big)
    x1, a1, _ = cases("cfg1_L4k")
    small = _run(eng, x1)
    parity.check_recall(x1.K, x1.Q, x1.workload, small[0], small[1], ref_scores=a1)
    again = _run(eng, big)
    np.testing.assert_array_equal(first[0], again[0])
    np.testing.assert_array_equal(first[1], again[1])
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_run_host_matches_run(cases):
    x, a, _ = cases("cfg1_L4k")
    w = x.workload
    eng = _engine(w, host_staging=True)
    idx_dev, _ = _run(eng, x)
    sc_host = torch.empty(w.L, dtype=torch.float32).pin_memory()
    idx_host, _ = eng.run_host(x.K.pin_memory(), x.Q.pin_memory(), w.budget, w.max_sizes,
                               w.win_sizes, w.win_op, w.n_sink, out_scores=sc_host)
    eng.check_status()
    np.testing.assert_array_equal(idx_host.numpy(), idx_dev)
    parity.check_recall(x.K, x.Q, w, idx_host.numpy(), sc_host.numpy(), ref_scores=a)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


@pytest.mark.parametrize("name", ["cfg3_L128k", "cfg4_L512k"])
def test_run_host_pipelined_upload_matches_oracle(cases, name):
    """Long contexts go up in pieces (2 at 128K, 8 at 512K) whose row statistics are merged
    like those of key shards: checked against the oracle, pageable and pinned host memory."""
    x, a, lse = cases(name)
    w = x.workload
    eng = _engine(w, host_staging=True)
    sc_host = torch.empty(w.L, dtype=torch.float32).pin_memory()
    for K_host in (x.K.pin_memory(), x.K):
        idx_host, _ = eng.run_host(K_host, x.Q, w.budget, w.max_sizes, w.win_sizes, w.win_op,
                                   w.n_sink, out_scores=sc_host)
        eng.check_status()
        parity.check_recall(x.K, x.Q, w, idx_host.numpy(), sc_host.numpy(), ref_scores=a)
        gpu_lse = eng.row_lse(w.q_len).cpu().numpy().reshape(-1)
        assert np.abs(gpu_lse - lse).max() < 5e-4
    # twice in a row on one handle: same result (the staging buffer is reused)
    idx2, _ = eng.run_host(x.K, x.Q, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    np.testing.assert_array_equal(idx2.numpy(), idx_host.numpy())
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_recall_can_be_captured_in_a_cuda_graph(cases):
    """run() allocates nothing, never synchronises and only launches kernels (one of them
    cooperative): it can be captured once and replayed, e.g. to shave launch overhead off short
    contexts.  The replay must give what the direct call gives."""
    x, _, _ = cases("cfg2_L32k")
    w = x.workload
    eng = _engine(w)
    K, Q = x.K.cuda(), x.Q.cuda()
    out = torch.empty(w.n_sink + w.budget, dtype=torch.int32, device="cuda")
    spec = (w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    eng.run(K, Q, *spec, out_idx=out)
    torch.cuda.synchronize()
    direct = out.clone()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            eng.run(K, Q, *spec, out_idx=out, stream=side)
    for _ in range(3):
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, direct)
    eng.check_status()
    del graph
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_in_kernel_sm_clock_is_plausible(cases):
    x, _, _ = cases("cfg2_L32k")
    eng = _engine(x.workload)
    assert eng.sm_clock_mhz() == 0.0                      # nothing profiled yet
    eng.set_profiling(True)
    _run(eng, x)
    mhz = eng.sm_clock_mhz()
    eng.set_profiling(False)
    assert 300.0 < mhz < 2500.0, mhz
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_error_codes_on_device(cases):
    from paper_2508_17892_b200 import IlreError
    x, _, _ = cases("cfg1_L4k")
    w = x.workload
    eng = _engine(w)
    K, Q = x.K.cuda(), x.Q.cuda()

    def code(**kw):
        args = dict(K=K, Q=Q, budget=w.budget, max_sizes=(1,), win_sizes=(1,), win_op=0, n_sink=0)
        args.update(kw)
        with pytest.raises(IlreError) as e:
            eng.run(**args)
        return e.value.code

    assert code(budget=w.budget + 1) == -3                     # above max_budget
    assert code(n_sink=w.L, budget=1) == -4                    # budget > L - n_sink
    assert code(win_sizes=(0,)) == -1
    assert code(max_sizes=(65,)) == -2
    assert code(win_sizes=tuple(range(1, 50))) == -3           # 49 combinations > 48
    assert code(win_op=2) == -1
    Kmis = torch.empty(w.L * 8 * 128 + 1, dtype=torch.bfloat16, device="cuda")[1:].view(w.L, 8, 128)
    assert code(K=Kmis) == -5
    big = torch.zeros(w.L + 1, 8, 128, dtype=torch.bfloat16, device="cuda")
    assert code(K=big) == -3
    assert eng.status() == 0
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_full_size_1m_config_against_the_full_oracle():
    """L = 1M, q_len = 256 (the benchmark configuration, same launch geometry as bench.py),
    against the oracle run in full: the statistics of all 8192 rows over all 1M keys, all 1M
    scores from the oracle's own statistics, and the index list, which must be identical.
    The oracle needs about two minutes of the host's cores for its 4.4e12 flops."""
    w = CONFIGS["cfg5_L1m"]
    x = make_inputs(w)
    eng = _engine(w)
    idx, sc = _run(eng, x)
    gpu_lse = eng.row_lse(w.q_len).cpu().numpy().reshape(-1).astype(np.float64)
    a, m, z = oracle.scores(x.K, x.Q, with_stats=True)
    lse = m + np.log(z)
    assert np.abs(gpu_lse - lse).max() < 5e-4
    rep = parity.check_recall(x.K, x.Q, w, idx, sc, ref_scores=a, strict=True)
    print("cfg5_L1m", rep, "max lse error", np.abs(gpu_lse - lse).max())
    assert np.all(np.isfinite(sc)) and sc.min() > 0 and sc.max() <= 1
    rng = np.random.default_rng(0)
    rows = np.unique(np.concatenate([rng.integers(0, w.q_len * w.n_q_heads, 40),
                                     [0, w.q_len * w.n_q_heads - 1]]))
    # The same context as eight key shards of 131072 positions (the per-rank steps bench.py
    # times with --shards 8): merged statistics, all scores and the index list
    # against the oracle, and the scores against the unsharded run's.
    from paper_2508_17892_b200.sharded import shard_bounds
    K, Q = x.K.cuda(), x.Q.cuda()
    bounds = [shard_bounds(w.L, 8, r) for r in range(8)]
    stats = torch.stack([eng.shard_stats(K[lo:hi], Q) for lo, hi in bounds])
    sc8 = torch.cat([eng.shard_scores(K[lo:hi], Q, stats) for lo, hi in bounds])
    idx8 = eng.allocate(sc8, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    torch.cuda.synchronize()
    eng.check_status()
    sc8, idx8 = sc8.cpu().numpy(), idx8.cpu().numpy()
    lse8 = eng.row_lse(w.q_len).cpu().numpy().reshape(-1).astype(np.float64)
    assert np.abs(lse8 - lse).max() < 5e-4
    assert np.abs(lse8 - gpu_lse).max() < 1e-5
    # per-shard statistics of sampled rows against the oracle on the same key range
    a0, b0 = bounds[3]
    m3, z3 = oracle.row_stats(x.K[a0:b0].contiguous(), x.Q, rows.tolist())
    st3 = stats[3].cpu().numpy().astype(np.float64)[rows]
    assert np.abs(st3[:, 0] * np.log(2.0) + np.log(st3[:, 1]) - (m3 + np.log(z3))).max() < 5e-4
    rep8 = parity.check_recall(x.K, x.Q, w, idx8, sc8, ref_scores=a)
    print("cfg5_L1m in 8 shards", rep8)
    assert np.abs(sc8 - sc).max() <= 2e-5 * sc.max() and np.all(np.abs(sc8 - sc) <= 1e-4 * sc)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_recalls_in_a_row_on_a_side_stream_keep_their_own_results():
    """The kernels of a recall start while the one before them still runs and wait before they
    read its output.  Recalls queued back to back on one stream without a synchronisation in
    between -- different keys, queries and lengths each time, work of another library before
    and between them on the same stream -- must each give the list and the scores that the
    same recall gives alone."""
    ws = [small_workload(L, q_len, seed=70 + i, n_spans=3, budget=b, max_sizes=(1, 2), win_sizes=(1, 5),
                         win_op=i % 2, n_sink=2)
          for i, (L, q_len, b) in enumerate([(9000, 16, 300), (30000, 4, 700), (5000, 33, 128),
                                             (30000, 4, 700), (12000, 64, 512)])]
    xs = [make_inputs(w) for w in ws]
    w0 = max(ws, key=lambda w: w.L)
    eng = _engine(w0, max_q_len=max(w.q_len for w in ws), max_budget=max(w.budget for w in ws))
    alone = []
    for w, x in zip(ws, xs):
        idx, sc = _run(eng, x)
        alone.append((idx, sc))
    side = torch.cuda.Stream()
    Ks = [x.K.cuda() for x in xs]
    Qs = [x.Q.cuda() for x in xs]
    scratch = torch.zeros(1 << 22, device="cuda")
    torch.cuda.synchronize()
    outs = []
    with torch.cuda.stream(side):
        for rep in range(3):
            for w, K, Q in zip(ws, Ks, Qs):
                scratch.add_(1.0)                              # a foreign kernel before the recall
                idx, sc = eng.run(K, Q, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                                  want_scores=True, stream=side)
                outs.append((idx, sc))
    side.synchronize()
    eng.check_status()
    for n, (idx, sc) in enumerate(outs):
        ref_idx, ref_sc = alone[n % len(ws)]
        assert np.array_equal(idx.cpu().numpy(), ref_idx), f"recall {n}"
        assert np.array_equal(sc.cpu().numpy(), ref_sc), f"scores of recall {n}"
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()
