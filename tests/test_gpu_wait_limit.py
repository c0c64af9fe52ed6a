"""The give-up path of the kernels' bounded waits, reached without faulting anything: one wait
is made impossible to complete and given a short spin budget; the kernel must return by
itself, the handle must report ILRE_ERR_DEVICE_WAIT, and the next ordinary run on the same
handle must be correct again."""
import numpy as np
import pytest
import torch

import parity
from workloads import make_inputs, small_workload

pytestmark = pytest.mark.gpu

ILRE_ERR_DEVICE_WAIT = -7
GRID_BARRIER, MISSING_KEY_TILE = 1, 2


def _setup():
    from paper_2508_17892_b200 import IlreRecall
    w = small_workload(9000, 8, seed=21, budget=200, win_sizes=(1, 7), win_op=1)
    x = make_inputs(w)
    eng = IlreRecall(max_L=w.L, max_q_len=w.q_len, max_budget=w.budget)
    spec = (w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink)
    return w, x, eng, spec, x.K.cuda(), x.Q.cuda()


def _good_run(eng, x, w, spec, K, Q):
    idx, sc = eng.run(K, Q, *spec, want_scores=True)
    torch.cuda.synchronize()
    assert eng.status() == 0
    parity.check_recall(x.K, x.Q, w, idx.cpu().numpy(), sc.cpu().numpy())
    return idx.clone()


@pytest.mark.parametrize("what", [GRID_BARRIER, MISSING_KEY_TILE])
def test_a_wait_that_cannot_complete_gives_up_and_the_handle_recovers(what):
    w, x, eng, spec, K, Q = _setup()
    want = _good_run(eng, x, w, spec, K, Q)
    eng.selftest_wait(200_000, what)                    # about 0.1 ms of spinning, then give up
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    eng.run(K, Q, *spec)
    t1.record()
    torch.cuda.synchronize()                             # the kernels returned by themselves
    assert t0.elapsed_time(t1) < 200.0                   # ms: nowhere near the default budget
    assert eng.status() == ILRE_ERR_DEVICE_WAIT
    assert eng.status() == 0                             # reading the status clears it
    # injection off, default budget: the same handle computes the right answer again
    eng.selftest_wait(0, 0)
    got = _good_run(eng, x, w, spec, K, Q)
    assert torch.equal(got, want)
    # a short budget alone (nothing injected) does not disturb a run of this size
    eng.selftest_wait(50_000_000, 0)
    assert torch.equal(_good_run(eng, x, w, spec, K, Q), want)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_selftest_arguments_are_checked():
    from paper_2508_17892_b200 import IlreError
    _, _, eng, _, _, _ = _setup()
    for bad in [(-1, 0), (0, 3), (0, -1)]:
        with pytest.raises(IlreError) as e:
            eng.selftest_wait(*bad)
        assert e.value.code == -1
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()
