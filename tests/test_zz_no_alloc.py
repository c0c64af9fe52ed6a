"""The allocation-free top-k entry point against the regular recall entry point.

Some callers of the library cannot allocate device memory (a framework-owned memory pool, a
thread that must never hit cudaMalloc's implicit synchronisation).  For them the library has
one call that needs no handle and keeps its scratch in a fixed array inside the library.  Here
its result is compared, through the C ABI, with what ``ilre_recall_run`` returns for the
equivalent pooling spec (one max kernel of size 1, one window of size 1, no sink), on two
calls in a row -- the second call reuses the scratch the first one left behind -- and with
the CPU oracle's Algorithm 1 for that spec.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from workloads import CONFIGS, make_inputs, small_workload

pytestmark = pytest.mark.gpu


def _reference_topk(eng, K, Q, budget):
    idx, scores = eng.run(K, Q, budget, (1,), (1,), 0, 0, want_scores=True)
    torch.cuda.synchronize()
    eng.check_status()
    return idx, scores


def test_noalloc_topk_matches_recall_run_twice_in_a_row():
    from paper_2508_17892_b200 import IlreRecall, load_library, topk_positions_noalloc
    x = make_inputs(CONFIGS["cfg1_L4k"])
    w = x.workload
    eng = IlreRecall(max_L=w.L, max_q_len=w.q_len, max_budget=w.budget)
    K, Q = x.K.cuda(), x.Q.cuda()
    ref_a, scores = _reference_topk(eng, K, Q, 512)
    ref_b, _ = _reference_topk(eng, K, Q, 100)
    out_a = torch.empty(512, dtype=torch.int32, device="cuda")
    out_b = torch.empty(100, dtype=torch.int32, device="cuda")
    topk_positions_noalloc(scores, 512, out_idx=out_a)      # first call: sets the scratch up
    topk_positions_noalloc(scores, 100, out_idx=out_b)      # second call: scratch holds old bits
    torch.cuda.synchronize()
    assert torch.equal(out_a, ref_a)                        # integer positions: bit-exact
    assert torch.equal(out_b, ref_b)
    # and against the oracle: Algorithm 1 with one size-1 max kernel and one size-1 window
    sc64 = scores.cpu().numpy().astype(np.float64)
    assert np.array_equal(out_a.cpu().numpy(), oracle.allocate(sc64, 512, [1], [1], 1))
    assert np.array_equal(out_b.cpu().numpy(), oracle.allocate(sc64, 100, [1], [1], 1))
    eng.close()

    # a ragged length with exact ties (scores quantised to few levels), k = 0 and k = L
    w2 = small_workload(5003, 8, seed=3, budget=700)
    x2 = make_inputs(w2)
    eng2 = IlreRecall(max_L=w2.L, max_q_len=w2.q_len, max_budget=5003)
    _, s2 = _reference_topk(eng2, x2.K.cuda(), x2.Q.cuda(), 700)
    coarse = (s2 * 4096).round() / 4096                     # many equal values
    want = torch.sort(torch.sort(coarse, descending=True, stable=True).indices[:700]).values
    got = topk_positions_noalloc(coarse, 700)
    torch.cuda.synchronize()
    assert torch.equal(got.long(), want)
    assert np.array_equal(got.cpu().numpy(),
                          oracle.allocate(coarse.cpu().numpy().astype(np.float64), 700, [1], [1], 1))
    # zeros of either sign are one value: ties among them go to the lower position
    zeros = coarse.clone()
    zeros[::3] = 0.0
    zeros[1::3] = -0.0
    zeros[2::3] = torch.where(zeros[2::3] > 0.01, zeros[2::3], torch.zeros_like(zeros[2::3]))
    n_pos = int((zeros > 0).sum())
    got0 = topk_positions_noalloc(zeros, n_pos + 40)
    torch.cuda.synchronize()
    assert np.array_equal(got0.cpu().numpy(),
                          oracle.allocate(zeros.cpu().numpy().astype(np.float64), n_pos + 40,
                                          [1], [1], 1))
    assert topk_positions_noalloc(coarse, 0).numel() == 0
    assert torch.equal(topk_positions_noalloc(coarse, 5003).long().cpu(), torch.arange(5003))
    eng2.close()

    # sizes beyond the fixed scratch are refused before anything is launched
    lib = load_library()
    from paper_2508_17892_b200 import NOALLOC_MAX_L
    st = torch.cuda.current_stream().cuda_stream
    assert lib.ilre_topk_positions_noalloc(scores.data_ptr(), NOALLOC_MAX_L + 1, 1,
                                           out_a.data_ptr(), st) == -3
    assert lib.ilre_topk_positions_noalloc(scores.data_ptr(), 10, 11, out_a.data_ptr(), st) == -4
    assert lib.ilre_topk_positions_noalloc(None, 10, 1, out_a.data_ptr(), st) == -1
