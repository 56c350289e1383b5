"""fp64 CPU oracle of the sparse verification attention path -- TEST INFRASTRUCTURE.

Only ``tests/``, ``__graft_entry__.smoke()`` and the CPU-baseline / reference
leg of ``bench.py`` may import this package.  It is a thin ctypes wrapper over
``sv_oracle.c`` (compiled with gcc on first use) and shares no code with the
CUDA library.  Tensors are numpy arrays; bfloat16 tensors are passed as their
uint16 bit patterns.

Paper passages: Section 3.1 (Eq. 4, Eq. 5, top-N with sink/local blocks),
Section 3.2 (Eq. 6), Section 3.3 (Eq. 9), Section 2.2 (one block set shared by
all draft tokens).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sv_oracle.c")
_LIB = os.path.join(_HERE, "libsv_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile sv_oracle.c into libsv_oracle.so next to it (gcc, -O2, OpenMP)."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".{os.getpid()}.tmp"
            cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(a, dtype):
    """Pointer to a C-contiguous numpy array of the given dtype (None -> NULL)."""
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (a.dtype, dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(_load().svo_num_threads())


def _nbmax(block_table):
    return int(block_table.shape[1])


def block_reps(k_pool, block_table, seq_lens):
    """Mean key of every block (Eq. 5).  k_pool uint16 [pages][Hkv][B][D] -> fp64 [S][Hkv][NBmax][D]."""
    _, Hkv, B, D = k_pool.shape
    S, NBmax = block_table.shape
    reps = np.zeros((S, Hkv, NBmax, D), dtype=np.float64)
    rc = _load().svo_block_reps(S, Hkv, D, B, NBmax, _p(k_pool, np.uint16), _p(block_table, np.int32),
                                _p(seq_lens, np.int32), _p(reps, np.float64))
    assert rc == 0, rc
    return reps


def group_query(q, Hkv):
    """Retrieval query: mean of the first draft token's query over the GQA group.  q uint16 [S][T][Hq][D]."""
    S, T, Hq, D = q.shape
    qbar = np.zeros((S, Hkv, D), dtype=np.float64)
    rc = _load().svo_group_query(S, T, Hq, Hkv, D, _p(q, np.uint16), _p(qbar, np.float64))
    assert rc == 0, rc
    return qbar


def scores(qbar, reps, seq_lens, B):
    """Importance scores (Eq. 5): fp64 [S][Hkv][NBmax]; entries past the last block are -inf."""
    S, Hkv, NBmax, D = reps.shape
    sc = np.full((S, Hkv, NBmax), -np.inf, dtype=np.float64)
    rc = _load().svo_scores(S, Hkv, D, B, NBmax, _p(qbar, np.float64), _p(reps, np.float64),
                            _p(seq_lens, np.int32), _p(sc, np.float64))
    assert rc == 0, rc
    return sc


def select(sc, seq_lens, budget, B, n_sink, n_local, max_sel):
    """Top-N blocks with sink/local blocks kept (Section 3.1).  Returns (idx [S][Hkv][max_sel], cnt [S][Hkv])."""
    S, Hkv, NBmax = sc.shape
    idx = np.full((S, Hkv, max_sel), -1, dtype=np.int32)
    cnt = np.zeros((S, Hkv), dtype=np.int32)
    rc = _load().svo_select(S, Hkv, B, NBmax, _p(np.ascontiguousarray(sc), np.float64), _p(seq_lens, np.int32),
                            _p(budget, np.int32), n_sink, n_local, max_sel, _p(idx, np.int32), _p(cnt, np.int32))
    if rc == 2:
        raise ValueError("forced sink/local blocks exceed the budget")
    if rc == 3:
        raise ValueError("selected set does not fit max_sel")
    assert rc == 0, rc
    return idx, cnt


def select_blocks(q, k_pool, block_table, seq_lens, budget, n_sink, n_local, max_sel):
    """Representatives -> retrieval query -> scores -> selection, the order of Section 3.1."""
    _, Hkv, B, _ = k_pool.shape
    reps = block_reps(k_pool, block_table, seq_lens)
    qbar = group_query(q, Hkv)
    sc = scores(qbar, reps, seq_lens, B)
    idx, cnt = select(sc, seq_lens, budget, B, n_sink, n_local, max_sel)
    return idx, cnt, sc


def select_layers(layers, anchors, budget, n_sink, n_local, max_sel):
    """Inter-layer retrieval reuse (Eq. 9): anchor layers retrieve, the others take the set of the
    nearest preceding anchor.  ``layers`` is a list of dicts with q, k_pool, block_table, seq_lens;
    ``anchors`` a list of bools (layer 0 must be an anchor).  Returns a list of (idx, cnt)."""
    assert anchors[0], "the first layer has no preceding anchor (J(M_1, M_0) = 0 makes it one)"
    out = []
    for l, lay in enumerate(layers):
        if anchors[l]:
            idx, cnt, _ = select_blocks(lay["q"], lay["k_pool"], lay["block_table"], lay["seq_lens"], budget,
                                        n_sink, n_local, max_sel)
        else:
            a = max(i for i in range(l) if anchors[i])
            idx, cnt = out[a][0].copy(), out[a][1].copy()
        out.append((idx, cnt))
    return out


def _samples_arg(samples):
    if samples is None:
        return 0, None
    samples = np.ascontiguousarray(np.asarray(samples, dtype=np.int32).reshape(-1, 3))
    return samples.shape[0], samples


def verify_attn(q, k_pool, v_pool, block_table, seq_lens, draft_k, draft_v, parent, sel_idx, sel_cnt,
                scale=None, samples=None):
    """Sparse verification attention.  Returns (out fp64 [S][T][Hq][D], lse fp64 [S][T][Hq]) or, with
    ``samples`` (rows of (s, i, hq)), ([n][D], [n])."""
    S, T, Hq, D = q.shape
    _, Hkv, B, _ = k_pool.shape
    NBmax = _nbmax(block_table)
    max_sel = sel_idx.shape[2]
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    n, smp = _samples_arg(samples)
    if smp is None:
        out = np.zeros((S, T, Hq, D), dtype=np.float64)
        lse = np.zeros((S, T, Hq), dtype=np.float64)
    else:
        out = np.zeros((n, D), dtype=np.float64)
        lse = np.zeros((n,), dtype=np.float64)
    lib = _load()
    rc = lib.svo_verify_attn(S, T, Hq, Hkv, D, B, NBmax, _p(q, np.uint16), _p(k_pool, np.uint16),
                             _p(v_pool, np.uint16), _p(block_table, np.int32), _p(seq_lens, np.int32),
                             _p(draft_k, np.uint16), _p(draft_v, np.uint16), _p(parent, np.int32),
                             _p(np.ascontiguousarray(sel_idx), np.int32), _p(np.ascontiguousarray(sel_cnt), np.int32),
                             max_sel, ctypes.c_double(scale), n, _p(smp, np.int32), _p(out, np.float64),
                             _p(lse, np.float64))
    assert rc == 0, rc
    return out, lse


def dense_verify_attn(q, k_pool, v_pool, block_table, seq_lens, draft_k, draft_v, parent, scale=None,
                      samples=None):
    """Dense ("strict") verification attention over the whole prefix; same return convention."""
    S, T, Hq, D = q.shape
    _, Hkv, B, _ = k_pool.shape
    NBmax = _nbmax(block_table)
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    n, smp = _samples_arg(samples)
    if smp is None:
        out = np.zeros((S, T, Hq, D), dtype=np.float64)
        lse = np.zeros((S, T, Hq), dtype=np.float64)
    else:
        out = np.zeros((n, D), dtype=np.float64)
        lse = np.zeros((n,), dtype=np.float64)
    rc = _load().svo_dense_verify_attn(S, T, Hq, Hkv, D, B, NBmax, _p(q, np.uint16), _p(k_pool, np.uint16),
                                       _p(v_pool, np.uint16), _p(block_table, np.int32), _p(seq_lens, np.int32),
                                       _p(draft_k, np.uint16), _p(draft_v, np.uint16), _p(parent, np.int32),
                                       ctypes.c_double(scale), n, _p(smp, np.int32), _p(out, np.float64),
                                       _p(lse, np.float64))
    assert rc == 0, rc
    return out, lse


def budget_blocks(L, L0, rho, B, n_sink=0, n_local=0) -> int:
    """Piecewise budget (Eq. 6) in blocks per KV head."""
    lib = _load()
    lib.svo_budget_blocks.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_double, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_int]
    return int(lib.svo_budget_blocks(int(L), int(L0), float(rho), int(B), int(n_sink), int(n_local)))


def kv_append(k_pool, v_pool, block_table, seq_lens, draft_k, draft_v, accept_idx, n_accept, reps=None):
    """Commit accepted draft tokens to the paged cache (in place) and refresh the representatives of the
    blocks that grew.  accept_idx int32 [S][A], n_accept int32 [S].  Returns the new lengths (int32 [S])."""
    _, Hkv, B, D = k_pool.shape
    S, NBmax = block_table.shape
    T = draft_k.shape[1]
    A = accept_idx.shape[1]
    out = np.zeros(S, dtype=np.int32)
    rc = _load().svo_kv_append(S, T, Hkv, D, B, NBmax, _p(k_pool, np.uint16), _p(v_pool, np.uint16),
                               _p(block_table, np.int32), _p(seq_lens, np.int32), _p(draft_k, np.uint16),
                               _p(draft_v, np.uint16), _p(np.ascontiguousarray(accept_idx), np.int32),
                               _p(np.ascontiguousarray(n_accept), np.int32), A, _p(out, np.int32), _p(reps, np.float64))
    if rc:
        raise ValueError(f"kv_append: bad argument ({rc})")
    return out


def jaccard_adjacent(idx_all, cnt_all):
    """Eq. 7 between adjacent layers.  idx_all int32 [layers][S][Hkv][max_sel], cnt_all int32 [layers][S][Hkv].
    Returns (inter int32 [layers][S], union int32 [layers][S], J fp64 [layers]); J[0] = 0 by definition."""
    n_layers, S, Hkv, max_sel = idx_all.shape
    inter = np.zeros((n_layers, S), np.int32)
    uni = np.zeros((n_layers, S), np.int32)
    J = np.zeros(n_layers, np.float64)
    rc = _load().svo_jaccard_adjacent(n_layers, S, Hkv, max_sel, _p(np.ascontiguousarray(idx_all), np.int32),
                                      _p(np.ascontiguousarray(cnt_all), np.int32), _p(inter, np.int32), _p(uni, np.int32),
                                      _p(J, np.float64))
    assert rc == 0, rc
    return inter, uni, J


def pick_anchors(J, K):
    """Eq. 8: the K layers least similar to their predecessor.  Returns a bool array [layers]."""
    J = np.ascontiguousarray(J, dtype=np.float64)
    anchors = np.zeros(J.shape[0], np.uint8)
    rc = _load().svo_pick_anchors(J.shape[0], _p(J, np.float64), int(K), _p(anchors, np.uint8))
    if rc:
        raise ValueError("K must be between 1 and the number of layers")
    return anchors.astype(bool)


# ------------------------------------------------------------------ retrieval variants the paper discusses


def group_query_row(q, Hkv, row):
    """Retrieval query of draft token ``row`` (Section 2.2): group mean of that token's query heads."""
    S, T, Hq, D = q.shape
    qbar = np.zeros((S, Hkv, D), dtype=np.float64)
    rc = _load().svo_group_query_row(S, T, Hq, Hkv, D, _p(q, np.uint16), int(row), _p(qbar, np.float64))
    if rc:
        raise ValueError("row outside the draft tokens")
    return qbar


def select_global(sc, seq_lens, budget, B, n_sink, n_local, max_sel):
    """Budget shared by the KV heads (Eq. 6 read over all heads): the budget*Hkv best (head, block) pairs.
    Returns (idx [S][Hkv][max_sel], cnt [S][Hkv])."""
    S, Hkv, NBmax = sc.shape
    idx = np.full((S, Hkv, max_sel), -1, dtype=np.int32)
    cnt = np.zeros((S, Hkv), dtype=np.int32)
    rc = _load().svo_select_global(S, Hkv, B, NBmax, _p(np.ascontiguousarray(sc), np.float64),
                                   _p(seq_lens, np.int32), _p(budget, np.int32), n_sink, n_local, max_sel,
                                   _p(idx, np.int32), _p(cnt, np.int32))
    if rc == 2:
        raise ValueError("forced sink/local blocks exceed the budget")
    if rc == 3:
        raise ValueError("a head's set does not fit max_sel")
    assert rc == 0, rc
    return idx, cnt


def select_tokens(q, k_pool, block_table, seq_lens, budget, n_sink, n_local, max_sel):
    """Every draft token retrieves with its own query.  Returns (idx [T][S][Hkv][max_sel], cnt [T][S][Hkv])."""
    S, T, _, _ = q.shape
    _, Hkv, B, _ = k_pool.shape
    reps = block_reps(k_pool, block_table, seq_lens)
    idx_all = np.full((T, S, Hkv, max_sel), -1, dtype=np.int32)
    cnt_all = np.zeros((T, S, Hkv), dtype=np.int32)
    for i in range(T):
        sc = scores(group_query_row(q, Hkv, i), reps, seq_lens, B)
        idx_all[i], cnt_all[i] = select(sc, seq_lens, budget, B, n_sink, n_local, max_sel)
    return idx_all, cnt_all


def pair_overlap(idx_all, cnt_all):
    """|Sel_i n Sel_j| for every pair of draft tokens: int32 [S][Hkv][T][T]."""
    T, S, Hkv, max_sel = idx_all.shape
    inter = np.zeros((S, Hkv, T, T), np.int32)
    rc = _load().svo_pair_overlap(T, S, Hkv, max_sel, _p(np.ascontiguousarray(idx_all), np.int32),
                                  _p(np.ascontiguousarray(cnt_all), np.int32), _p(inter, np.int32))
    assert rc == 0, rc
    return inter


def overlap_by_distance(inter, cnt_all, position):
    """The statistic of the block-overlap figure (Section 2.2): for token pairs i != j at positional distance
    |position[i] - position[j]|, the intersection of their retrieved blocks divided by the number of blocks a
    token retrieves, averaged over pairs, heads and sequences.  Returns {distance: mean ratio}."""
    S, Hkv, T, _ = inter.shape
    acc = {}
    for i in range(T):
        for j in range(T):
            if i == j:
                continue
            d = abs(int(position[i]) - int(position[j]))
            for s in range(S):
                for h in range(Hkv):
                    n = max(int(cnt_all[i, s, h]), int(cnt_all[j, s, h]))
                    r = float(inter[s, h, i, j]) / n if n else 1.0
                    acc.setdefault(d, []).append(r)
    return {d: float(np.mean(v)) for d, v in sorted(acc.items())}


# ------------------------------------------------------------------ acceptance (Eq. 2-3)


def accept(p_target, p_draft, tokens, parent, u_accept, u_next, want_dist=False):
    """Acceptance walk of Section 2.1.  p_target, p_draft float32 [S][T][V]; tokens int32 [S][T]; parent int32
    [S][T] or None (chain); u_accept float32 [S][T], u_next float32 [S] uniform numbers in [0, 1).
    Returns dict(path int32 [S][T] (-1 padded), n_path int32 [S], next_token int32 [S], alpha float64 [S][T],
    final_dist float64 [S][V] or None)."""
    S, T, V = p_target.shape
    path = np.full((S, T), -1, np.int32)
    n_path = np.zeros(S, np.int32)
    nxt = np.zeros(S, np.int32)
    alpha = np.zeros((S, T), np.float64)
    dist = np.zeros((S, V), np.float64) if want_dist else None
    rc = _load().svo_accept(S, T, V, _p(np.ascontiguousarray(p_target), np.float32),
                            _p(np.ascontiguousarray(p_draft), np.float32), _p(np.ascontiguousarray(tokens), np.int32),
                            _p(None if parent is None else np.ascontiguousarray(parent), np.int32),
                            _p(np.ascontiguousarray(u_accept), np.float32), _p(np.ascontiguousarray(u_next), np.float32),
                            _p(path, np.int32), _p(n_path, np.int32), _p(nxt, np.int32), _p(alpha, np.float64),
                            _p(dist, np.float64))
    if rc == 2:
        raise ValueError("token id outside the vocabulary")
    assert rc == 0, rc
    return dict(path=path, n_path=n_path, next_token=nxt, alpha=alpha, final_dist=dist)


def round_bf16(x):
    """Nearest bfloat16 (ties to even) of fp64 values, returned as fp64."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty_like(x)
    rc = _load().svo_round_bf16(ctypes.c_int64(x.size), _p(x, np.float64), _p(y, np.float64))
    assert rc == 0, rc
    return y


def block_reps_bf16(k_pool, block_table, seq_lens):
    """Block representatives kept in bfloat16: the fp64 means of Eq. 5 rounded once."""
    return round_bf16(block_reps(k_pool, block_table, seq_lens))
