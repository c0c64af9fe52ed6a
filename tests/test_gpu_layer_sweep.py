"""GPU parity of the offline retrieval-layer choice (Section 3.3; Appendix A.1), through the
C ABI: the hit counting / layer choice on given lists, and the whole sweep (one recall per
candidate layer, then the choice) against the oracle's."""
import numpy as np
import pytest
import torch

import oracle
from workloads import layer_sweep_workloads, make_inputs, small_workload

pytestmark = pytest.mark.gpu


def _gpu_choice(lists, spans):
    from paper_2508_17892_b200 import layer_recall
    idx = torch.tensor(np.asarray(lists, dtype=np.int32).reshape(len(lists), -1), device="cuda")
    sb = torch.tensor([b for b, _ in spans], dtype=torch.int32, device="cuda")
    sl = torch.tensor([n for _, n in spans], dtype=torch.int32, device="cuda")
    hits, full, layer = layer_recall(idx, sb, sl)
    torch.cuda.synchronize()
    return hits.cpu().numpy(), full.cpu().numpy(), int(layer.item())


@pytest.mark.parametrize("n_layers,n_idx,n_spans,L", [(1, 1, 1, 8), (4, 64, 5, 1000),
                                                      (32, 1024, 20, 131072), (3, 0, 4, 100),
                                                      (5, 300, 0, 5000), (1024, 16, 3, 400)])
def test_choice_on_random_lists_is_bit_exact(n_layers, n_idx, n_spans, L):
    rng = np.random.default_rng(n_layers * 7 + n_idx)
    seg = L // max(n_spans, 1)
    spans = [(s * seg + int(rng.integers(0, max(seg // 2, 1))), int(rng.integers(1, max(seg // 2, 2))))
             for s in range(n_spans)]
    lists = []
    for l in range(n_layers):
        if l % 3 == 2 and lists:
            lists.append(lists[-1].copy())                      # equal layers: lowest index wins
            continue
        base = rng.choice(L, size=n_idx, replace=False) if n_idx else np.empty(0, dtype=np.int64)
        if n_spans and n_idx:                                     # bias some lists into the phrases
            want = np.concatenate([np.arange(b, b + n) for b, n in spans[: 1 + l % n_spans]])[:n_idx]
            base = np.unique(np.concatenate([want, base]))[:n_idx]
            while len(base) < n_idx:
                base = np.unique(np.concatenate([base, rng.choice(L, size=n_idx)]))[:n_idx]
        lists.append(np.sort(base))
    hits, full, layer = _gpu_choice(lists, spans)
    r_hits, r_full, r_layer = oracle.layer_choice(lists, spans)
    assert np.array_equal(hits, r_hits.reshape(hits.shape))
    assert np.array_equal(full, r_full)
    assert layer == r_layer


def test_capacity_and_argument_errors():
    from paper_2508_17892_b200 import IlreError, layer_recall
    z = torch.zeros(1025, 4, dtype=torch.int32, device="cuda")
    s = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(IlreError):
        layer_recall(z, s, s + 1)


def test_sweep_over_candidate_layers_matches_the_oracle():
    """Six candidate layers of one context (same planted phrases, per-layer query, keys and
    needle strength): the recall of each layer on the GPU, then the layer choice, against the
    oracle doing both."""
    from paper_2508_17892_b200 import IlreRecall
    base = small_workload(16384, 8, seed=31, n_spans=8, span_len=(8, 24), budget=256,
                          max_sizes=(1, 2), win_sizes=(1, 7, 15), win_op=0, n_sink=4)
    ws = layer_sweep_workloads(base, [0.2, 0.65, 0.8, 3.0, 3.0, 0.9])
    eng = IlreRecall(max_L=base.L, max_q_len=base.q_len, max_budget=base.budget)
    idx = torch.empty(len(ws), base.n_sink + base.budget, dtype=torch.int32, device="cuda")
    ref_lists, spans = [], None
    for l, w in enumerate(ws):
        x = make_inputs(w)
        spans = spans or x.spans
        assert x.spans == spans
        eng.run(x.K.cuda(), x.Q.cuda(), w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                out_idx=idx[l])
        a = oracle.scores(x.K, x.Q)
        ref_lists.append(oracle.allocate(a, w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink))
    torch.cuda.synchronize()
    eng.check_status()
    gpu_lists = idx.cpu().numpy()
    hits, full, layer = _gpu_choice(gpu_lists, spans)
    # the counting kernel on the GPU's own lists: bit-exact
    o_hits, o_full, o_layer = oracle.layer_choice(gpu_lists, spans)
    assert np.array_equal(hits, o_hits) and np.array_equal(full, o_full) and layer == o_layer
    # the whole sweep against the oracle's: same retrieved-phrase counts and the same layer
    r_hits, r_full, r_layer = oracle.layer_choice(ref_lists, spans)
    assert np.array_equal(full, r_full), (full, r_full)
    assert layer == r_layer
    assert full[layer] == full.max() and np.all(full[:layer] < full.max())
    assert len(set(full.tolist())) >= 3          # the layers do differ
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
