"""Sparse verification attention for speculative decoding on B200 (sm_100a).

CUDA library (csrc/, built into libsv.so) + a ctypes binding with the names of include/sv.h +
``SparseVerifier``, a small driver that runs the per-layer select -> attention sequence for a stack of
layers.  Importing the package loads the compiled library and fails if it is missing.
"""
from .binding import (EXPORTS, LIB_PATH, SV_NOALLOC_SCRATCH_BYTES, SV_OK, SV_STATUS_INDEX, SV_STATUS_NO_LIST,  # noqa: F401
                      SV_STATUS_WAIT_MASK, SV_TAIL_BLOCK, SvError, make_geom, make_kv, sv_accept, sv_anchor_jaccard,
                      sv_block_reps, sv_block_reps_bf16, sv_budget_blocks, sv_geom, sv_kv, sv_kv_append,
                      sv_pick_anchors, sv_select_blocks, sv_select_blocks_bf16reps, sv_select_blocks_global,
                      sv_select_blocks_tokens, sv_status_word_check, sv_token_overlap, sv_verify_attn,
                      sv_verify_attn_noalloc, sv_verify_attn_reused, sv_verify_attn_splits, sv_workspace_bytes)
from .engine import SparseVerifier  # noqa: F401
