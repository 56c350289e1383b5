"""ctypes binding of libsv.so: the same entry points as include/sv.h, taking torch CUDA tensors.

Argument marshalling only -- every step of the path runs in the library's CUDA kernels.  torch is
used for device memory and streams.  There is no CPU fallback: importing this module fails if the
compiled library is missing.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsv.so")

SV_OK = 0
SV_TAIL_BLOCK = -1   # sv_block_reps(block_begin=SV_TAIL_BLOCK): refresh only each sequence's last block
STATUS_NAMES = {0: "SV_OK", 1: "SV_ERR_NULL", 2: "SV_ERR_SHAPE", 3: "SV_ERR_ALIGN", 4: "SV_ERR_BUDGET",
                5: "SV_ERR_WORKSPACE", 6: "SV_ERR_UNSUPPORTED", 7: "SV_ERR_CUDA", 8: "SV_ERR_SCRATCH_LIMIT",
                9: "SV_ERR_INDEX"}
# bits of the device status word (see sv.h)
SV_STATUS_WAIT_MASK, SV_STATUS_INDEX, SV_STATUS_NO_LIST = 0x0FF, 0x100, 0x200
SV_NOALLOC_SCRATCH_BYTES = 4 * 1024 * 1024   # size of the library's built-in scratch (sv_verify_attn_noalloc)

EXPORTS = ("sv_strerror", "sv_status_word_check", "sv_budget_blocks", "sv_workspace_bytes", "sv_block_reps", "sv_select_blocks",
           "sv_verify_attn", "sv_verify_attn_reused", "sv_verify_attn_splits", "sv_verify_attn_noalloc", "sv_kv_append", "sv_anchor_jaccard", "sv_pick_anchors",
           "sv_select_blocks_tokens", "sv_token_overlap", "sv_select_blocks_global", "sv_accept",
           "sv_block_reps_bf16", "sv_select_blocks_bf16reps")


class SvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} ({_strerror(status)})")


class sv_geom(ctypes.Structure):
    _fields_ = [("n_seq", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block_size", ctypes.c_int32), ("max_blocks", ctypes.c_int32),
                ("n_draft", ctypes.c_int32)]


class sv_kv(ctypes.Structure):
    _fields_ = [("k_pool", ctypes.c_void_p), ("v_pool", ctypes.c_void_p), ("block_table", ctypes.c_void_p),
                ("seq_lens", ctypes.c_void_p), ("n_pages", ctypes.c_int32)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_21911_b200.build` "
                          "(there is no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, f64, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_double,
                                  ctypes.c_size_t)
    gp, kp = ctypes.POINTER(sv_geom), ctypes.POINTER(sv_kv)
    lib.sv_strerror.restype = ctypes.c_char_p
    lib.sv_strerror.argtypes = [ctypes.c_int]
    lib.sv_status_word_check.restype = ctypes.c_int
    lib.sv_status_word_check.argtypes = [i32]
    lib.sv_budget_blocks.restype = i32
    lib.sv_budget_blocks.argtypes = [i64, i64, f64, i32, i32, i32]
    lib.sv_workspace_bytes.restype = sz
    lib.sv_workspace_bytes.argtypes = [gp, i32]
    lib.sv_verify_attn_splits.restype = i32
    lib.sv_verify_attn_splits.argtypes = [gp, i32]
    lib.sv_block_reps.restype = ctypes.c_int
    lib.sv_block_reps.argtypes = [gp, kp, i32, i32, vp, vp]
    lib.sv_select_blocks.restype = ctypes.c_int
    lib.sv_select_blocks.argtypes = [gp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, i32, vp, vp]
    lib.sv_verify_attn.restype = ctypes.c_int
    lib.sv_verify_attn.argtypes = [gp, vp, kp, vp, vp, vp, vp, vp, i32, f32, vp, vp, vp, sz, vp, vp]
    lib.sv_verify_attn_reused.restype = ctypes.c_int
    lib.sv_verify_attn_reused.argtypes = lib.sv_verify_attn.argtypes
    lib.sv_anchor_jaccard.restype = ctypes.c_int
    lib.sv_anchor_jaccard.argtypes = [gp, i32, vp, vp, i32, vp, vp, vp]
    lib.sv_pick_anchors.restype = ctypes.c_int
    lib.sv_pick_anchors.argtypes = [vp, vp, i32, i32, i32, vp, vp]
    lib.sv_kv_append.restype = ctypes.c_int
    lib.sv_kv_append.argtypes = [gp, vp, vp, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
    lib.sv_select_blocks_tokens.restype = ctypes.c_int
    lib.sv_select_blocks_tokens.argtypes = [gp, vp, vp, vp, vp, i32, i32, vp, vp, i32, vp]
    lib.sv_token_overlap.restype = ctypes.c_int
    lib.sv_token_overlap.argtypes = [gp, vp, vp, i32, vp, vp]
    lib.sv_select_blocks_global.restype = ctypes.c_int
    lib.sv_select_blocks_global.argtypes = [gp, vp, vp, vp, vp, i32, i32, vp, vp, i32, vp, vp]
    lib.sv_block_reps_bf16.restype = ctypes.c_int
    lib.sv_block_reps_bf16.argtypes = [gp, kp, i32, i32, vp, vp]
    lib.sv_select_blocks_bf16reps.restype = ctypes.c_int
    lib.sv_select_blocks_bf16reps.argtypes = [gp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, i32, vp, vp]
    lib.sv_accept.restype = ctypes.c_int
    lib.sv_accept.argtypes = [i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sv_verify_attn_noalloc.restype = ctypes.c_int
    lib.sv_verify_attn_noalloc.argtypes = [gp, vp, kp, vp, vp, vp, vp, vp, i32, f32, vp, vp, vp, vp]
    return lib


_lib = _load()


def _strerror(status: int) -> str:
    return _lib.sv_strerror(int(status)).decode()


def _ptr(t: Optional[torch.Tensor], dtype: torch.dtype, name: str) -> Optional[int]:
    """Device pointer of a contiguous CUDA tensor of the given dtype (None -> NULL)."""
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def _check(status: int, where: str) -> None:
    if status != SV_OK:
        raise SvError(status, where)


def make_geom(n_seq, n_q_heads, n_kv_heads, head_dim, block_size, max_blocks, n_draft) -> sv_geom:
    return sv_geom(n_seq, n_q_heads, n_kv_heads, head_dim, block_size, max_blocks, n_draft)


def make_kv(k_pool: torch.Tensor, v_pool: Optional[torch.Tensor], block_table: torch.Tensor,
            seq_lens: torch.Tensor) -> sv_kv:
    """Paged KV descriptor.  Pools are bf16 [n_pages][Hkv][B][D]; the tensors must outlive the calls."""
    return sv_kv(_ptr(k_pool, torch.bfloat16, "k_pool"), _ptr(v_pool, torch.bfloat16, "v_pool"),
                 _ptr(block_table, torch.int32, "block_table"), _ptr(seq_lens, torch.int32, "seq_lens"),
                 int(k_pool.shape[0]))


def sv_status_word_check(value: int) -> int:
    """Status code for a device status word the caller has read back (0 = SV_OK)."""
    return int(_lib.sv_status_word_check(int(value)))


def sv_budget_blocks(L_seq: int, L0: int, rho: float, block_size: int, n_sink: int = 0, n_local: int = 0) -> int:
    return int(_lib.sv_budget_blocks(L_seq, L0, rho, block_size, n_sink, n_local))


def sv_workspace_bytes(geom: sv_geom, max_sel: int) -> int:
    return int(_lib.sv_workspace_bytes(ctypes.byref(geom), max_sel))


def sv_verify_attn_splits(geom: sv_geom, max_sel: int) -> int:
    return int(_lib.sv_verify_attn_splits(ctypes.byref(geom), max_sel))


def sv_block_reps(geom: sv_geom, kv: sv_kv, reps: torch.Tensor, block_begin: int = 0, block_end: int = -1,
                  stream=None) -> None:
    _check(_lib.sv_block_reps(ctypes.byref(geom), ctypes.byref(kv), block_begin, block_end,
                              _ptr(reps, torch.float32, "reps"), _stream(stream)), "sv_block_reps")


def sv_block_reps_bf16(geom: sv_geom, kv: sv_kv, reps_bf16: torch.Tensor, block_begin: int = 0, block_end: int = -1,
                       stream=None) -> None:
    """sv_block_reps with the representatives stored in bfloat16."""
    _check(_lib.sv_block_reps_bf16(ctypes.byref(geom), ctypes.byref(kv), block_begin, block_end,
                                   _ptr(reps_bf16, torch.bfloat16, "reps_bf16"), _stream(stream)), "sv_block_reps_bf16")


def sv_select_blocks_bf16reps(geom: sv_geom, q, reps_bf16, seq_lens, budget_blocks, n_sink: int, n_local: int, out_idx,
                              out_cnt, reuse_prev: bool = False, prev_idx=None, prev_cnt=None, out_scores=None,
                              stream=None) -> None:
    """sv_select_blocks reading bfloat16 representatives."""
    _check(_lib.sv_select_blocks_bf16reps(ctypes.byref(geom), _ptr(q, torch.bfloat16, "q"),
                                          _ptr(reps_bf16, torch.bfloat16, "reps_bf16"),
                                          _ptr(seq_lens, torch.int32, "seq_lens"),
                                          _ptr(budget_blocks, torch.int32, "budget_blocks"), n_sink, n_local,
                                          1 if reuse_prev else 0, _ptr(prev_idx, torch.int32, "prev_idx"),
                                          _ptr(prev_cnt, torch.int32, "prev_cnt"), _ptr(out_idx, torch.int32, "out_idx"),
                                          _ptr(out_cnt, torch.int32, "out_cnt"), int(out_idx.shape[-1]),
                                          _ptr(out_scores, torch.float32, "out_scores"), _stream(stream)),
           "sv_select_blocks_bf16reps")


def sv_select_blocks(geom: sv_geom, q, reps, seq_lens, budget_blocks, n_sink: int, n_local: int, out_idx, out_cnt,
                     reuse_prev: bool = False, prev_idx=None, prev_cnt=None, out_scores=None, stream=None) -> None:
    max_sel = int(out_idx.shape[-1])
    _check(_lib.sv_select_blocks(ctypes.byref(geom), _ptr(q, torch.bfloat16, "q"), _ptr(reps, torch.float32, "reps"),
                                 _ptr(seq_lens, torch.int32, "seq_lens"),
                                 _ptr(budget_blocks, torch.int32, "budget_blocks"), n_sink, n_local,
                                 1 if reuse_prev else 0, _ptr(prev_idx, torch.int32, "prev_idx"),
                                 _ptr(prev_cnt, torch.int32, "prev_cnt"), _ptr(out_idx, torch.int32, "out_idx"),
                                 _ptr(out_cnt, torch.int32, "out_cnt"), max_sel,
                                 _ptr(out_scores, torch.float32, "out_scores"), _stream(stream)), "sv_select_blocks")


def sv_verify_attn(geom: sv_geom, q, kv: sv_kv, draft_k, draft_v, parent, sel_idx, sel_cnt, out, lse=None,
                   workspace=None, softmax_scale: float = 0.0, status_word=None, stream=None, _fn=None, _name="sv_verify_attn") -> None:
    max_sel = int(sel_idx.shape[-1]) if sel_idx is not None else int(geom.max_blocks)
    ws_ptr = workspace.data_ptr() if workspace is not None else None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    if workspace is not None and not workspace.is_cuda:
        raise TypeError("workspace must be a CUDA tensor")
    _check((_fn or _lib.sv_verify_attn)(ctypes.byref(geom), _ptr(q, torch.bfloat16, "q"), ctypes.byref(kv),
                               _ptr(draft_k, torch.bfloat16, "draft_k"), _ptr(draft_v, torch.bfloat16, "draft_v"),
                               _ptr(parent, torch.int32, "parent"), _ptr(sel_idx, torch.int32, "sel_idx"),
                               _ptr(sel_cnt, torch.int32, "sel_cnt"), max_sel, float(softmax_scale),
                               _ptr(out, torch.bfloat16, "out"), _ptr(lse, torch.float32, "lse"), ws_ptr, ws_bytes,
                               _ptr(status_word, torch.int32, "status_word"), _stream(stream)), _name)


def sv_verify_attn_reused(geom: sv_geom, q, kv: sv_kv, draft_k, draft_v, parent, sel_idx, sel_cnt, out, lse=None,
                          workspace=None, softmax_scale: float = 0.0, status_word=None, stream=None) -> None:
    """sv_verify_attn for a layer that reuses an earlier layer's block list: the caller vouches that the list, the tables,
    the lengths and the K/V pools are not written by the kernel just before, and the gather starts ahead of it."""
    sv_verify_attn(geom, q, kv, draft_k, draft_v, parent, sel_idx, sel_cnt, out, lse=lse, workspace=workspace,
                   softmax_scale=softmax_scale, status_word=status_word, stream=stream, _fn=_lib.sv_verify_attn_reused,
                   _name="sv_verify_attn_reused")


def sv_verify_attn_noalloc(geom: sv_geom, q, kv: sv_kv, draft_k, draft_v, parent, sel_idx, sel_cnt, out, lse=None,
                           softmax_scale: float = 0.0, status_word=None, stream=None) -> None:
    """sv_verify_attn without a caller workspace: the split-KV partials go to the scratch array built into
    the library (SV_NOALLOC_SCRATCH_BYTES).  For callers that cannot allocate device memory where they
    need the attention -- a server whose HBM is fully reserved by its KV-cache pool, code that runs under
    another component's allocator.  Nothing is allocated here, by torch or otherwise: only the caller's
    input and output tensors are passed through.  Problems whose partials do not fit raise
    SvError(SV_ERR_SCRATCH_LIMIT).  All calls on a device share that array, so calls that may overlap on
    the GPU must be serialised by the caller; make the first call on a device outside any stream capture."""
    max_sel = int(sel_idx.shape[-1]) if sel_idx is not None else int(geom.max_blocks)
    _check(_lib.sv_verify_attn_noalloc(ctypes.byref(geom), _ptr(q, torch.bfloat16, "q"), ctypes.byref(kv),
                                       _ptr(draft_k, torch.bfloat16, "draft_k"),
                                       _ptr(draft_v, torch.bfloat16, "draft_v"), _ptr(parent, torch.int32, "parent"),
                                       _ptr(sel_idx, torch.int32, "sel_idx"), _ptr(sel_cnt, torch.int32, "sel_cnt"),
                                       max_sel, float(softmax_scale), _ptr(out, torch.bfloat16, "out"),
                                       _ptr(lse, torch.float32, "lse"), _ptr(status_word, torch.int32, "status_word"),
                                       _stream(stream)), "sv_verify_attn_noalloc")


def sv_kv_append(geom: sv_geom, k_pool, v_pool, block_table, seq_lens, draft_k, draft_v, accept_idx, n_accept,
                 seq_lens_out, reps=None, stream=None) -> None:
    """Commit accepted draft tokens to the paged cache (pools modified in place), write the new lengths to
    seq_lens_out (a different tensor than seq_lens) and refresh the representatives of the grown blocks."""
    _check(_lib.sv_kv_append(ctypes.byref(geom), _ptr(k_pool, torch.bfloat16, "k_pool"), _ptr(v_pool, torch.bfloat16, "v_pool"),
                             int(k_pool.shape[0]), _ptr(block_table, torch.int32, "block_table"),
                             _ptr(seq_lens, torch.int32, "seq_lens"), _ptr(draft_k, torch.bfloat16, "draft_k"),
                             _ptr(draft_v, torch.bfloat16, "draft_v"), _ptr(accept_idx, torch.int32, "accept_idx"),
                             _ptr(n_accept, torch.int32, "n_accept"), int(accept_idx.shape[-1]),
                             _ptr(seq_lens_out, torch.int32, "seq_lens_out"), _ptr(reps, torch.float32, "reps"),
                             _stream(stream)), "sv_kv_append")


def sv_anchor_jaccard(geom: sv_geom, sel_idx_all, sel_cnt_all, inter, uni, stream=None) -> None:
    """Eq. 7 set sizes between adjacent layers.  sel_idx_all int32 [layers][S][Hkv][max_sel], sel_cnt_all int32
    [layers][S][Hkv]; inter / uni int32 [layers][S] (outputs)."""
    _check(_lib.sv_anchor_jaccard(ctypes.byref(geom), int(sel_idx_all.shape[0]), _ptr(sel_idx_all, torch.int32, "sel_idx_all"),
                                  _ptr(sel_cnt_all, torch.int32, "sel_cnt_all"), int(sel_idx_all.shape[-1]),
                                  _ptr(inter, torch.int32, "inter"), _ptr(uni, torch.int32, "uni"), _stream(stream)),
           "sv_anchor_jaccard")


def sv_select_blocks_tokens(geom: sv_geom, q, reps, seq_lens, budget_blocks, n_sink: int, n_local: int, out_idx,
                            out_cnt, stream=None) -> None:
    """Every draft token retrieves with its own query.  out_idx int32 [T][S][Hkv][max_sel], out_cnt int32 [T][S][Hkv]."""
    _check(_lib.sv_select_blocks_tokens(ctypes.byref(geom), _ptr(q, torch.bfloat16, "q"), _ptr(reps, torch.float32, "reps"),
                                        _ptr(seq_lens, torch.int32, "seq_lens"),
                                        _ptr(budget_blocks, torch.int32, "budget_blocks"), n_sink, n_local,
                                        _ptr(out_idx, torch.int32, "out_idx"), _ptr(out_cnt, torch.int32, "out_cnt"),
                                        int(out_idx.shape[-1]), _stream(stream)), "sv_select_blocks_tokens")


def sv_token_overlap(geom: sv_geom, sel_idx_all, sel_cnt_all, inter, stream=None) -> None:
    """|Sel_i n Sel_j| for every pair of draft tokens: inter int32 [S][Hkv][T][T] (output)."""
    _check(_lib.sv_token_overlap(ctypes.byref(geom), _ptr(sel_idx_all, torch.int32, "sel_idx_all"),
                                 _ptr(sel_cnt_all, torch.int32, "sel_cnt_all"), int(sel_idx_all.shape[-1]),
                                 _ptr(inter, torch.int32, "inter"), _stream(stream)), "sv_token_overlap")


def sv_select_blocks_global(geom: sv_geom, q, reps, seq_lens, budget_blocks, n_sink: int, n_local: int, out_idx,
                            out_cnt, scores, stream=None) -> None:
    """Budget shared by the KV heads: the budget * Hkv best (head, block) pairs of every sequence.
    out_idx int32 [S][Hkv][max_sel >= max_blocks], out_cnt int32 [S][Hkv], scores float32 [S][Hkv][max_blocks]."""
    _check(_lib.sv_select_blocks_global(ctypes.byref(geom), _ptr(q, torch.bfloat16, "q"), _ptr(reps, torch.float32, "reps"),
                                        _ptr(seq_lens, torch.int32, "seq_lens"),
                                        _ptr(budget_blocks, torch.int32, "budget_blocks"), n_sink, n_local,
                                        _ptr(out_idx, torch.int32, "out_idx"), _ptr(out_cnt, torch.int32, "out_cnt"),
                                        int(out_idx.shape[-1]), _ptr(scores, torch.float32, "scores"), _stream(stream)),
           "sv_select_blocks_global")


def sv_accept(p_target, p_draft, tokens, parent, u_accept, u_next, path, n_path, next_token, alpha=None, stream=None) -> None:
    """Acceptance walk (Eq. 2-3).  p_target, p_draft float32 [S][T][V]; tokens int32 [S][T]; parent int32 [S][T] or
    None (chain); u_accept float32 [S][T]; u_next float32 [S]; outputs path int32 [S][T], n_path int32 [S],
    next_token int32 [S], optional alpha float32 [S][T]."""
    S, T, V = (int(x) for x in p_target.shape)
    if tuple(p_draft.shape) != (S, T, V) or tuple(tokens.shape) != (S, T) or tuple(path.shape) != (S, T):
        raise ValueError("sv_accept: shapes disagree")
    _check(_lib.sv_accept(S, T, V, _ptr(p_target, torch.float32, "p_target"), _ptr(p_draft, torch.float32, "p_draft"),
                          _ptr(tokens, torch.int32, "tokens"), _ptr(parent, torch.int32, "parent"),
                          _ptr(u_accept, torch.float32, "u_accept"), _ptr(u_next, torch.float32, "u_next"),
                          _ptr(path, torch.int32, "path"), _ptr(n_path, torch.int32, "n_path"),
                          _ptr(next_token, torch.int32, "next_token"), _ptr(alpha, torch.float32, "alpha"),
                          _stream(stream)), "sv_accept")


def sv_pick_anchors(inter, uni, n_anchors: int):
    """Eq. 8 on host arrays (numpy int32 [layers][samples]).  Returns (anchors bool [layers], J float64 [layers])."""
    import numpy as np
    inter = np.ascontiguousarray(inter, dtype=np.int32)
    uni = np.ascontiguousarray(uni, dtype=np.int32)
    n_layers, n_samples = inter.shape
    anchors = np.zeros(n_layers, dtype=np.uint8)
    J = np.zeros(n_layers, dtype=np.float64)
    _check(_lib.sv_pick_anchors(inter.ctypes.data, uni.ctypes.data, n_layers, n_samples, int(n_anchors), anchors.ctypes.data,
                                J.ctypes.data), "sv_pick_anchors")
    return anchors.astype(bool), J
