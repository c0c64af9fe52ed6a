"""GPU parity of the Dual Chunk Attention key re-rotation (Eq. 7) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import parity
from workloads import make_inputs, small_workload

pytestmark = pytest.mark.gpu

# One bf16 rounding of an fp32 result: half a unit in the last place is at most 2^-8 of the
# value (8 significant bits).  Before it, the fp32 rotation carries an absolute error of a few
# 2^-24 of the INPUT magnitudes (two products, one sum, an fp32 table entry), which matters
# where the two products cancel: inputs here stay below 16, hence 16 * 4 * 2^-24 ~ 4e-6.
REL_TOL = 2.0 ** -8 * (1 + 1e-3)
ABS_TOL = 4e-6


def _engine(n_kv=8, n_q=32, max_L=70000):
    from paper_2508_17892_b200 import IlreRecall
    return IlreRecall(max_L=max_L, max_q_len=64, max_budget=512, n_kv_heads=n_kv, n_q_heads=n_q)


def _as_f64(t: torch.Tensor) -> np.ndarray:
    return t.cpu().to(torch.float64).numpy()


CASES = [
    # L, n_kv, chunk, n_sink
    (4096, 8, 1024, 0),
    (5000, 8, 1024, 4),          # ragged last chunk, sink in the first chunk
    (777, 2, 64, 4),
    (300, 8, 100, 0),            # N_C = 3: only the first chunk turns
    (200, 8, 100, 0),            # N_C = 2: nothing turns
    (65, 1, 1, 3),               # chunk of one position
    (65552, 8, 8, 0),            # 8194 chunks: exactly the capacity of the angle table
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"L{c[0]}_kv{c[1]}_c{c[2]}_s{c[3]}")
def test_rerope_matches_oracle(case):
    L, n_kv, chunk, n_sink = case
    g = torch.Generator().manual_seed(L + chunk)
    K = (torch.randn(L, n_kv, 128, generator=g) * 2.0).to(torch.bfloat16)
    want = oracle.dca_rerope(K, chunk, n_sink)
    eng = _engine(n_kv=n_kv, n_q=n_kv * 4, max_L=max(L, 4096))
    Kd = K.cuda()
    out = torch.empty_like(Kd)
    eng.rerope_keys(Kd, chunk, n_sink, out=out)            # separate output
    inplace = Kd.clone()
    eng.rerope_keys(inplace, chunk, n_sink)                # in place
    torch.cuda.synchronize()
    eng.check_status()
    assert torch.equal(out, inplace)
    assert torch.equal(Kd.cpu(), K)                        # the input of the first call is intact
    got = _as_f64(out)
    err = np.abs(got - want)
    assert np.all(err <= REL_TOL * np.abs(want) + ABS_TOL), float((err / (np.abs(want) + 1e-30)).max())
    # almost every element is the correctly rounded value of the exact rotation
    exact = oracle.round_to_bf16(want)
    same = out.cpu().view(torch.int16).numpy().view(np.uint16) == exact
    assert same.mean() > 0.999, same.mean()
    # the last two chunks are bit-identical to the input
    n_chunks = -(-(L - n_sink) // chunk)
    keep_from = n_sink + max(n_chunks - 2, 0) * chunk
    assert torch.equal(out[keep_from:].cpu(), K[keep_from:])
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_too_many_chunks_is_refused():
    from paper_2508_17892_b200 import IlreError
    eng = _engine(max_L=70000)
    K = torch.zeros(66000, 8, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(IlreError) as e:
        eng.rerope_keys(K, 4)                              # 16500 chunks > 8192 + 2
    assert e.value.code == -3
    with pytest.raises(IlreError) as e:
        eng.rerope_keys(K, 0)
    assert e.value.code == -1
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_recall_on_rerotated_keys_matches_oracle():
    # Eq. 7 followed by the recall: the oracle runs on the oracle's own re-rotated keys (rounded
    # to bf16, as a cache holds them); the device output may differ from that rounding in rare
    # elements by one unit in the last place, so its scores are checked at the score tolerance.
    w = small_workload(6000, 16, seed=11, n_spans=3, span_len=(16, 32), budget=256,
                       win_sizes=(1, 7, 15), win_op=1)
    x = make_inputs(w)
    chunk, n_sink = 1024, 0
    ref_keys = torch.from_numpy(oracle.round_to_bf16(oracle.dca_rerope(x.K, chunk, n_sink))
                                .view(np.int16)).view(torch.bfloat16).reshape(x.K.shape)
    from paper_2508_17892_b200 import IlreRecall
    eng = IlreRecall(max_L=w.L, max_q_len=w.q_len, max_budget=w.budget)
    Kd = x.K.cuda()
    eng.rerope_keys(Kd, chunk, n_sink)
    idx, sc = eng.run(Kd, x.Q.cuda(), w.budget, w.max_sizes, w.win_sizes, w.win_op, w.n_sink,
                      want_scores=True)
    torch.cuda.synchronize()
    eng.check_status()
    # exact parity of the recall itself on the device's own re-rotated keys
    parity.check_recall(Kd.cpu(), x.Q, w, idx.cpu().numpy(), sc.cpu().numpy())
    # and against the all-oracle pipeline: a key that differs by one bf16 unit moves a logit by
    # at most |q_c| * 2^-8 |k_c| / sqrt(d), far below what separates planted spans from the rest
    ref_idx, ref_scores = oracle.recall(ref_keys, x.Q, w.budget, w.max_sizes, w.win_sizes, w.win_op,
                                        w.n_sink)
    rel = np.abs(sc.cpu().numpy() - ref_scores) / ref_scores
    assert np.quantile(rel, 0.999) < 2e-3 and rel.max() < 0.05
    planted = set(x.planted_positions().tolist())
    assert len(planted & set(idx.cpu().tolist())) == len(planted & set(ref_idx.tolist()))
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


@pytest.mark.parametrize("name,chunk,n_sink", [("cfg2_L32k", 1024, 0), ("cfg3_L128k", 4096, 4)])
def test_recall_with_dca_against_the_oracle_pipeline(name, chunk, n_sink):
    """DCA on (Eq. 7 -> Eq. 4, Eq. 5, Algorithm 1) as one path against the oracle's pipeline
    `dca_rerope -> round to bf16 -> scores -> allocate`, position by position.

    The device's re-rotated cache differs from the oracle's correctly rounded one in rare
    elements by one bf16 unit.  What such a difference can do to a score is bounded from the
    inputs alone: a logit of position t moves by at most
    delta_t = max_r |q_r . (K_dev[t] - K_ref[t])| / sqrt(d), every row's lse by at most
    delta_lse (taken from the oracle's statistics on the two caches), so a score moves by at
    most the factor exp(delta_t + delta_lse).  Where the two caches agree (delta_t = 0) the
    plain score tolerance (plus delta_lse) applies."""
    from workloads import CONFIGS
    from paper_2508_17892_b200 import IlreRecall
    w = CONFIGS[name]
    x = make_inputs(w)
    ref_keys = torch.from_numpy(oracle.round_to_bf16(oracle.dca_rerope(x.K, chunk, n_sink))
                                .view(np.int16)).view(torch.bfloat16).reshape(x.K.shape)
    eng = IlreRecall(max_L=w.L, max_q_len=w.q_len, max_budget=w.budget)
    Kd = torch.empty_like(x.K, device="cuda")
    eng.rerope_keys(x.K.cuda(), chunk, n_sink, out=Kd)
    spec = (w.budget, w.max_sizes, w.win_sizes, w.win_op, n_sink)
    idx, sc = eng.run(Kd, x.Q.cuda(), *spec, want_scores=True)
    torch.cuda.synchronize()
    eng.check_status()
    idx, sc, Kd = idx.cpu().numpy(), sc.cpu().numpy().astype(np.float64), Kd.cpu()
    same_rows = (Kd.view(torch.int16) == ref_keys.view(torch.int16)).all(dim=2).all(dim=1).numpy()
    assert same_rows.mean() > 0.1                     # plenty of positions with identical keys
    # the recall itself, exactly, on the device's own cache
    a_dev, m_d, z_d = oracle.scores(Kd, x.Q, with_stats=True)
    parity.check_recall(Kd, x.Q, w, idx, sc, ref_scores=a_dev, spec=spec)
    # the whole path against the oracle's pipeline
    a_ref, m_r, z_r = oracle.scores(ref_keys, x.Q, with_stats=True)
    delta_lse = np.abs((m_d + np.log(z_d)) - (m_r + np.log(z_r))).max()
    diff = Kd.to(torch.float64) - ref_keys.to(torch.float64)             # [L, n_kv, d], sparse
    q = x.Q.to(torch.float64)
    group = w.n_q_heads // w.n_kv_heads
    delta = np.zeros(w.L)
    touched = np.flatnonzero(~same_rows)
    for g in range(w.n_kv_heads):
        qg = q[:, g * group:(g + 1) * group, :].reshape(-1, w.d)        # rows of this kv head
        dl = (diff[touched, g, :] @ qg.T).abs().max(dim=1).values.numpy() / np.sqrt(w.d)
        delta[touched] = np.maximum(delta[touched], dl)
    assert delta.max() < 0.05
    bound = parity.SCORE_RTOL * a_ref + parity.SCORE_ATOL + a_ref * np.expm1(delta + delta_lse)
    err = np.abs(sc - a_ref)
    assert np.all(err <= bound), (int(np.argmax(err / bound)), float((err / bound).max()))
    assert np.all(err[same_rows] <= (parity.SCORE_RTOL + 2 * delta_lse) * a_ref[same_rows]
                  + parity.SCORE_ATOL)
    # the index list: every combination's choice judged on the oracle pipeline's pooled
    # values, near-ties widened by what the differing cache elements can move a score
    own, diag = oracle.allocate(sc, *spec, avg_single=True, diagnostics=True)
    assert np.array_equal(own, idx)
    bad = parity.decisions_within_tolerance(
        a_ref, diag["combination_of"], *spec,
        rtol=parity.SCORE_RTOL + float(np.expm1(delta.max() + delta_lse)))
    assert not bad, bad[:10]
    ref_idx = oracle.allocate(a_ref, *spec)
    print(name, "positions with identical keys", same_rows.mean(), "max delta", delta.max(),
          "delta_lse", delta_lse, "index differences", len(set(idx.tolist()) ^ set(ref_idx.tolist())))
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


# ---- Eq. 6: sink keys of the layers before the retrieval layer ----

SINK_CASES = [
    # n_sink, n_kv, chunk, chunk_index
    (4, 8, 1024, 1), (4, 8, 1024, 2), (4, 8, 1024, 3), (4, 8, 1024, 4), (4, 8, 1024, 1024),
    (1, 2, 64, 7), (64, 4, 512, 100), (4, 8, 8, 8194),
]


@pytest.mark.parametrize("case", SINK_CASES, ids=lambda c: f"S{c[0]}_kv{c[1]}_c{c[2]}_i{c[3]}")
def test_sink_rerope_matches_oracle(case):
    n_sink, n_kv, chunk, i = case
    g = torch.Generator().manual_seed(100 + i)
    ks = (4.0 * torch.randn(n_sink, n_kv, 128, generator=g)).to(torch.bfloat16)
    eng = _engine(n_kv=n_kv, n_q=n_kv)
    ref = oracle.dca_rerope_sinks(ks, i, chunk)
    src = ks.cuda()
    out = eng.rerope_sinks(src, chunk, i)
    torch.cuda.synchronize()
    eng.check_status()
    assert torch.equal(src.cpu(), ks)                       # the cached keys are left alone
    got = _as_f64(out)
    if i <= 2:
        assert np.array_equal(got, ref)
    else:
        assert np.all(np.abs(got - ref) <= REL_TOL * np.abs(ref) + ABS_TOL)
        assert not np.array_equal(got, _as_f64(ks))
    # in place gives the same bytes
    inplace = ks.cuda()
    eng.rerope_sinks(inplace, chunk, i, out=inplace)
    torch.cuda.synchronize()
    assert torch.equal(inplace, out)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_sink_rerope_chunk_by_chunk_and_with_eq7_on_one_handle():
    """Chunks arrive in order (the angle table grows ahead of them); Eq. 7 on the same handle
    in between, with another chunk size, must not disturb later calls."""
    from paper_2508_17892_b200 import IlreError
    g = torch.Generator().manual_seed(9)
    ks = torch.randn(4, 8, 128, generator=g).to(torch.bfloat16)
    eng = _engine()
    src = ks.cuda()
    for i in list(range(1, 140)) + [70, 3]:
        got = _as_f64(eng.rerope_sinks(src, 256, i))
        ref = oracle.dca_rerope_sinks(ks, i, 256)
        assert np.all(np.abs(got - ref) <= REL_TOL * np.abs(ref) + ABS_TOL), i
        if i == 100:
            x = make_inputs(small_workload(3000, 1, seed=5))
            eng.rerope_keys(x.K.cuda(), 500, 0)
    with pytest.raises(IlreError):
        eng.rerope_sinks(src, 256, 8195)                     # beyond the angle table
    with pytest.raises(IlreError):
        eng.rerope_sinks(src, 256, 0)
    torch.cuda.synchronize()
    eng.check_status()
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()
