"""B200 (sm_100a) implementation of ILRe's token-recall path behind a C ABI.

``IlreRecall`` wraps ``libilre_recall.so`` (built in-tree by ``paper_2508_17892_b200.build``).
"""
from .recall import (EXPORTED_SYMBOLS, LIB_PATH, NOALLOC_MAX_L, STAGE_NAMES, IlreConfig, IlreError,
                     IlrePoolSpec, IlreRecall, gather_input_ids, layer_recall, load_library,
                     strerror,
                     topk_positions_noalloc)

__all__ = ["EXPORTED_SYMBOLS", "LIB_PATH", "STAGE_NAMES", "IlreConfig", "IlreError",
           "IlrePoolSpec", "IlreRecall", "NOALLOC_MAX_L", "gather_input_ids", "layer_recall", "load_library", "strerror",
           "topk_positions_noalloc"]
