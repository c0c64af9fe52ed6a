"""GPU parity of the key-cache fill (key projection + RoPE, Eq. 1 / Eq. 3) against the oracle."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _rand(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


def _engine(n_kv, max_L):
    from paper_2508_17892_b200 import IlreRecall
    return IlreRecall(max_L=max_L, max_q_len=16, max_budget=64, n_kv_heads=n_kv, n_q_heads=n_kv)


def _check(got: torch.Tensor, want: np.ndarray, X, W, bias):
    """One bf16 rounding (at most 2^-8 of the value) on top of an fp32 accumulation whose
    absolute error is bounded by a few 2^-24 per term of sum |x_k w_k| (+ |b|)."""
    g = got.cpu().to(torch.float64).numpy()
    mag = (X.to(torch.float64).abs() @ W.to(torch.float64).abs().T).numpy()
    if bias is not None:
        mag = mag + bias.to(torch.float64).abs().numpy()[None, :]
    mag = mag.reshape(want.shape)
    half = want.shape[-1] // 2
    pair = mag[..., :half] + mag[..., half:]                # both channels of a pair feed a result
    bound = 2.0 ** -8 * (1 + 1e-3) * np.abs(want) + 1e-6 * np.concatenate([pair, pair], axis=-1)
    err = np.abs(g - want)
    assert np.all(err <= bound), float((err / bound).max())
    exact = oracle.round_to_bf16(want)
    same = got.cpu().view(torch.int16).numpy().view(np.uint16) == exact
    assert same.mean() > 0.99, same.mean()


CASES = [
    # n_tok, d_model, n_kv, pos0, bias
    (128, 64, 8, 0, False),
    (1024, 4096, 8, 0, False),        # one prefill chunk of the Llama-3.1-8B shape
    (1000, 512, 8, 5000, True),       # ragged token tile, offset positions, bias
    (300, 256, 2, 123456, True),
    (129, 64, 1, 1023, False),        # one head; positions cross a table-row boundary
    (20000, 128, 8, 0, False),        # two heads per tile, several tiles per CTA
    (1, 64, 8, 7, True),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"n{c[0]}_d{c[1]}_kv{c[2]}_p{c[3]}_b{int(c[4])}")
def test_fill_matches_oracle(case):
    n_tok, d_model, n_kv, pos0, with_bias = case
    X = _rand((n_tok, d_model), n_tok + 1)
    W = _rand((n_kv * 128, d_model), d_model + 2, 1.0 / np.sqrt(d_model))
    bias = _rand((n_kv * 128,), 3) if with_bias else None
    want = oracle.key_fill(X, W, pos0, bias=bias)
    L = pos0 + n_tok + 5
    eng = _engine(n_kv, max(L, 1024))
    cache = torch.full((L, n_kv, 128), 7.0, dtype=torch.bfloat16, device="cuda")
    eng.fill_keys(X.cuda(), W.cuda(), cache, pos0, bias=bias.cuda() if with_bias else None)
    torch.cuda.synchronize()
    eng.check_status()
    _check(cache[pos0:pos0 + n_tok], want, X, W, bias)
    # rows outside the filled range keep their contents
    assert torch.all(cache[:pos0] == 7.0) and torch.all(cache[pos0 + n_tok:] == 7.0)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_chunked_fill_equals_one_call_and_feeds_the_recall():
    from paper_2508_17892_b200 import IlreRecall
    n_kv, d_model, L, chunk = 8, 256, 3000, 1024
    X = _rand((L, d_model), 21)
    W = _rand((n_kv * 128, d_model), 22, 1.0 / 16)
    Q = _rand((8, 32, 128), 23)
    eng = IlreRecall(max_L=L, max_q_len=8, max_budget=128)
    Xd, Wd = X.cuda(), W.cuda()
    whole = torch.zeros(L, n_kv, 128, dtype=torch.bfloat16, device="cuda")
    parts = torch.zeros_like(whole)
    eng.fill_keys(Xd, Wd, whole, 0)
    for a in range(0, L, chunk):
        eng.fill_keys(Xd[a:a + chunk].contiguous(), Wd, parts, a)
    torch.cuda.synchronize()
    eng.check_status()
    assert torch.equal(whole, parts)
    # the filled cache goes straight into Eq. 7 and the recall
    import parity
    from workloads import small_workload
    w = small_workload(L, 8, budget=128, win_sizes=(1, 7), win_op=1)
    eng.rerope_keys(whole, chunk)
    idx, sc = eng.run(whole, Q.cuda(), w.budget, w.max_sizes, w.win_sizes, w.win_op, 0,
                      want_scores=True)
    torch.cuda.synchronize()
    eng.check_status()
    parity.check_recall(whole.cpu(), Q, w, idx.cpu().numpy(), sc.cpu().numpy())
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_fill_argument_errors():
    from paper_2508_17892_b200 import IlreError
    eng = _engine(8, 2048)
    X = torch.zeros(64, 96, dtype=torch.bfloat16, device="cuda")          # 96 % 64 != 0
    W = torch.zeros(1024, 96, dtype=torch.bfloat16, device="cuda")
    cache = torch.zeros(2048, 8, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(IlreError) as e:
        eng.fill_keys(X, W, cache, 0)
    assert e.value.code == -2
    X = torch.zeros(64, 128, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(1024, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(IlreError) as e:
        eng.fill_keys(X, W, cache, 2000)                                   # runs past the cache
    assert e.value.code == -3
    assert eng.status() == 0
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()


def test_gather_input_ids_is_plain_indexing():
    from paper_2508_17892_b200 import gather_input_ids
    g = torch.Generator().manual_seed(0)
    ids = torch.randint(0, 128000, (5000,), generator=g, dtype=torch.int32)
    idx = torch.sort(torch.randperm(5000, generator=g)[:700]).values.to(torch.int32)
    query = torch.randint(0, 128000, (37,), generator=g, dtype=torch.int32)
    out = gather_input_ids(ids.cuda(), idx.cuda(), query.cuda())
    want = np.concatenate([ids.numpy()[idx.numpy()], query.numpy()])     # C~ = C[I], then the query
    np.testing.assert_array_equal(out.cpu().numpy(), want)
    bad = torch.tensor([0, 4999, 5000, -1], dtype=torch.int32)
    out = gather_input_ids(ids.cuda(), bad.cuda(), query[:0].cuda())
    np.testing.assert_array_equal(out.cpu().numpy(), [ids[0].item(), ids[4999].item(), -1, -1])


def test_fill_and_re_rotation_replay_from_a_graph_on_another_stream():
    """Once the handle holds the angle tables (built by a first call, here on the default
    stream), the fill and the Eq. 7 re-rotation can be captured on another stream and replayed:
    the replay writes what the direct calls write."""
    from paper_2508_17892_b200 import IlreRecall
    n_kv, d_model, L, chunk = 8, 256, 2500, 512
    X = _rand((L, d_model), 31).cuda()
    W = _rand((n_kv * 128, d_model), 32, 1.0 / 16).cuda()
    eng = IlreRecall(max_L=L, max_q_len=8, max_budget=128)
    direct = torch.zeros(L, n_kv, 128, dtype=torch.bfloat16, device="cuda")
    eng.fill_keys(X, W, direct, 0)
    eng.rerope_keys(direct, chunk)
    torch.cuda.synchronize()
    replayed = torch.zeros_like(direct)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    views = [X[a:a + chunk] for a in range(0, L, chunk)]
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i, v in enumerate(views):
                eng.fill_keys(v, W, replayed, i * chunk, stream=side)
            eng.rerope_keys(replayed, chunk, stream=side)
    assert not replayed.any()                              # nothing ran during the capture
    graph.replay()
    torch.cuda.synchronize()
    eng.check_status()
    assert torch.equal(replayed, direct)
    assert eng.check_guards() == 0, "a kernel wrote past the end of a workspace buffer"
    eng.close()
    # a handle without the tables refuses to build them inside a capture (a replay could not
    # tell that they are stale); the capture itself stays valid
    from paper_2508_17892_b200.recall import IlreError
    fresh = IlreRecall(max_L=L, max_q_len=8, max_budget=128)
    import warnings
    graph2 = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side), warnings.catch_warnings():
        warnings.simplefilter("ignore")                    # the captured graph stays empty
        with torch.cuda.graph(graph2, stream=side):
            with pytest.raises(IlreError) as e1:
                fresh.fill_keys(views[0], W, replayed, 0, stream=side)
            with pytest.raises(IlreError) as e2:
                fresh.rerope_keys(replayed, chunk, stream=side)
    assert e1.value.code == -2 and e2.value.code == -2
    torch.cuda.synchronize()
    fresh.fill_keys(views[0], W, replayed, 0)              # the handle works as before
    torch.cuda.synchronize()
    fresh.check_status()
    fresh.close()
