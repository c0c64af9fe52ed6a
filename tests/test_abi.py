"""The C-ABI library: loads without a GPU, exports what the header declares, and rejects bad
arguments before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2508_17892_b200 import build, recall
    build.build()
    return recall.load_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "ilre_recall.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ilre_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2508_17892_b200 import EXPORTED_SYMBOLS
    declared = _declared_symbols()
    assert declared == sorted(EXPORTED_SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_strerror_covers_all_codes(lib):
    from paper_2508_17892_b200 import strerror
    seen = {strerror(c) for c in range(0, -10, -1)}
    assert len(seen) == 10 and "unknown status" not in seen
    assert strerror(-99) == "unknown status"


def test_create_rejects_bad_configs_without_a_device(lib):
    from paper_2508_17892_b200 import IlreConfig
    out = ctypes.c_void_p()
    good = dict(n_kv_heads=8, n_q_heads=32, head_dim=128, max_L=4096, max_q_len=16,
                max_budget=512, max_combinations=48, device=0, host_staging=0)

    def create(**kw):
        cfg = IlreConfig(**{**good, **kw})
        return lib.ilre_recall_create(ctypes.byref(cfg), ctypes.byref(out))

    assert lib.ilre_recall_create(None, ctypes.byref(out)) == -1
    assert create(head_dim=64) == -2
    assert create(n_q_heads=30) == -2
    assert create(max_L=0) == -1
    assert create(max_budget=20000) == -3
    assert create(max_combinations=65) == -3
    assert create(max_L=2 ** 31) == -3
    assert out.value is None


def test_null_handle_calls_return_invalid_arg(lib):
    assert lib.ilre_recall_status(None) == -1
    assert lib.ilre_recall_destroy(None) == -1
    assert lib.ilre_recall_set_profiling(None, 1) == -1
    assert lib.ilre_recall_selftest_wait(None, 0, 0) == -1
    assert lib.ilre_recall_last_launch_count(None) == -1
    assert lib.ilre_recall_check_guards(None) == -1
    assert lib.ilre_recall_run(None, None, 1, None, 1, 0, None, None, None, None) == -1
    assert lib.ilre_recall_run_host(None, None, 1, None, 1, 0, None, None, None, None) == -1
    assert lib.ilre_recall_shard_stats(None, None, 1, None, 1, None, None) == -1
    assert lib.ilre_recall_shard_scores(None, None, 1, None, 1, None, 1, None, None) == -1
    assert lib.ilre_recall_allocate(None, None, 1, 0, None, None, None) == -1
    assert lib.ilre_recall_fill_keys(None, None, 1, 64, None, None, 0, 500000.0, None, 1, None) == -1
    assert lib.ilre_recall_rerope_keys(None, None, None, 1, 1, 0, 500000.0, None) == -1
    assert lib.ilre_recall_rerope_sinks(None, None, None, 1, 1, 1, 500000.0, None) == -1
    assert lib.ilre_recall_chunk_attention(None, None, None, None, 1, 0, None, None) == -1
    assert lib.ilre_recall_copy_row_lse(None, None, 1, None) == -1
    assert lib.ilre_recall_sm_clock(None, None) == -1
    assert lib.ilre_recall_stage_times(None, None, 0) == -1


def test_handle_free_calls_validate_their_arguments(lib):
    # no device is touched before validation
    assert lib.ilre_layer_recall(None, 0, 0, None, None, 0, None, None, None, None) == -1   # no layers
    assert lib.ilre_layer_recall(None, 1, 4, None, None, 0, None, None, None, None) == -1   # no outputs
    assert lib.ilre_gather_input_ids(None, 0, None, 0, None, 0, None, None) == -1
    assert lib.ilre_topk_positions_noalloc(None, 16, 4, None, None) != 0


def test_create_without_gpu_reports_cuda_error(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2508_17892_b200 import IlreError, IlreRecall
    with pytest.raises(IlreError) as e:
        IlreRecall(max_L=4096, max_q_len=16)
    assert e.value.code == -6
