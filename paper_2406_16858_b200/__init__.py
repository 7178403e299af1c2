"""B200 (sm_100a) library for the data-parallel hot path of EAGLE-2's draft-and-verify cycle.

The product is ``libeagle2.so`` (hand-written CUDA kernels behind the C ABI of ``include/eagle2.h``);
this package is its thin Python binding.  PyTorch is used for device memory and streams only.
Build the library first: ``python -m paper_2406_16858_b200.build``.
"""
from .binding import (  # noqa: F401
    Eagle2Error, OP_ACCEPT, OP_EXPAND, OP_KV_COMPACT, OP_RERANK, OP_TREE_ATTENTION, OP_TREE_MASK,
    STATUS_BAD_TREE, STATUS_KV_OVERFLOW, STATUS_NONFINITE_LOGIT, STATUS_NOT_CLOSED,
    EXPAND_BY_CONFIDENCE, STATUS_TIMEOUT, accept, expand, expand_static, expand_variant, kv_compact, lib, lib_path, lm_head, lm_head_expand, OP_LM_HEAD_EXPAND,
    rerank, rerank_mask, rerank_skipped, set_wait_limit, strerror, tree_attention, tree_attention_launches, tree_mask, version, workspace_bytes, workspace_init)
