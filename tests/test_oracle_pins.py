"""Pins of the fp64 CPU oracle to what the paper and the mathematics fix (no GPU needed).

Each test ties one oracle function to something other than itself: a hand-worked fixture under
tests/golden/, a closed form, brute force on tiny inputs, a library routine, or an invariant of
the definition.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
import sv_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_fixture(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


def _bits(x):
    return si.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _tiny_case(S=2, Hq=4, Hkv=2, D=8, B=4, T=3, lens=(13, 6), seed=0, tree=False, scale=1.0):
    """Small random case with an out-of-order page table (values rounded to bf16)."""
    g = np.random.default_rng(seed)
    lens = np.array(lens, dtype=np.int32)
    nb = (lens + B - 1) // B
    n_pages = int(nb.sum()) + 2
    perm = g.permutation(n_pages)
    bt = np.zeros((S, int(nb.max())), dtype=np.int32)
    o = 0
    for s in range(S):
        bt[s, :nb[s]] = perm[o:o + nb[s]]
        o += nb[s]
    c = dict(
        q=_bits(g.standard_normal((S, T, Hq, D)) * scale),
        k_pool=_bits(g.standard_normal((n_pages, Hkv, B, D)) * scale),
        v_pool=_bits(g.standard_normal((n_pages, Hkv, B, D))),
        draft_k=_bits(g.standard_normal((S, T, Hkv, D)) * scale),
        draft_v=_bits(g.standard_normal((S, T, Hkv, D))),
        block_table=bt, seq_lens=lens, n_blocks=nb, B=B, Hkv=Hkv, parent=None)
    if tree:
        par = np.full((S, T), -1, dtype=np.int32)
        for s in range(S):
            for i in range(1, T):
                par[s, i] = g.integers(0, i)
        c["parent"] = par
    return c


def _gather_tokens(pool, bt, s, h, L, B):
    """[L][D] fp64 rows of one (sequence, KV head), gathered with numpy indexing (independent of the C code)."""
    t = np.arange(L)
    return si.bf16_bits_to_f64(pool[bt[s, t // B], h, t % B, :])


# --------------------------------------------------------------------------- O1-O3: Eq. 5

def test_eq5_hand_worked_fixture():
    fx = _read_fixture("eq5_block_scores.txt")
    q = _bits(fx["q_heads"].reshape(1, 1, 2, 2))
    k_pool = np.zeros((3, 1, 2, 2), dtype=np.uint16)
    keys = fx["keys"].reshape(5, 2)
    bt = np.array([[2, 0, 1]], dtype=np.int32)          # pages out of order on purpose
    for t in range(5):
        k_pool[bt[0, t // 2], 0, t % 2] = _bits(keys[t])
    k_pool[bt[0, 2], 0, 1] = _bits([99.0, 99.0])        # slot past the end of the sequence: must be ignored
    lens = np.array([5], dtype=np.int32)
    reps = oracle.block_reps(k_pool, bt, lens)
    np.testing.assert_array_equal(reps[0, 0], fx["reps"].reshape(3, 2))
    qbar = oracle.group_query(q, 1)
    np.testing.assert_array_equal(qbar[0, 0], [2.0, 0.0])
    sc = oracle.scores(qbar, reps, lens, 2)
    np.testing.assert_array_equal(sc[0, 0], fx["scores"])


def test_eq5_literal_sum_matches_representative_form():
    """Eq. 5 as printed (mean over the block of q0.k) against the oracle's q0 . mean(k)."""
    c = _tiny_case(seed=3)
    B, Hkv = c["B"], c["Hkv"]
    reps = oracle.block_reps(c["k_pool"], c["block_table"], c["seq_lens"])
    qbar = oracle.group_query(c["q"], Hkv)
    sc = oracle.scores(qbar, reps, c["seq_lens"], B)
    G = c["q"].shape[2] // Hkv
    for s in range(2):
        L = int(c["seq_lens"][s])
        for h in range(Hkv):
            keys = _gather_tokens(c["k_pool"], c["block_table"], s, h, L, B)
            q0 = si.bf16_bits_to_f64(c["q"][s, 0, h * G:(h + 1) * G]).sum(axis=0) / G
            dots = keys @ q0
            for b in range(int(c["n_blocks"][s])):
                lit = dots[b * B:min((b + 1) * B, L)].mean()
                assert abs(sc[s, h, b] - lit) < 1e-12
            assert np.all(np.isneginf(sc[s, h, int(c["n_blocks"][s]):]))


def test_planted_shift_closed_form():
    """A block whose keys are all c*u (u = q0/|q0|), others zero: score is exactly c*|q0|, others 0."""
    D, B = 4, 4
    q = _bits(np.array([3.0, 0.0, 4.0, 0.0]).reshape(1, 1, 1, D))     # |q0| = 5, u = (0.6, 0, 0.8, 0)
    k_pool = np.zeros((4, 1, B, D), dtype=np.uint16)
    u = np.array([0.75, 0.0, 1.0, 0.0])                                # 1.25*u, exactly representable
    k_pool[2, 0] = _bits(np.tile(u, (B, 1)))
    bt = np.array([[0, 1, 2, 3]], dtype=np.int32)
    lens = np.array([16], dtype=np.int32)
    idx, cnt, sc = oracle.select_blocks(q, k_pool, bt, lens, np.array([1], np.int32), 0, 0, 4)
    np.testing.assert_array_equal(sc[0, 0], [0.0, 0.0, 1.25 * 5.0, 0.0])
    assert cnt[0, 0] == 1 and idx[0, 0, 0] == 2


# --------------------------------------------------------------------------- O4: selection

def _brute_force_select(sc, nb, N, n_sink, n_local):
    if N >= nb:
        return list(range(nb))
    forced = [b for b in range(nb) if b < n_sink or b >= nb - n_local]
    rest = [b for b in range(nb) if b not in forced]
    best, best_sum = None, -math.inf
    for comb in itertools.combinations(rest, N - len(forced)):     # lexicographic: smaller indices first
        tot = sum(sc[b] for b in comb)
        if tot > best_sum:
            best, best_sum = comb, tot
    return sorted(forced + list(best))


@pytest.mark.parametrize("n_sink,n_local", [(0, 0), (1, 1), (2, 3)])
def test_select_equals_brute_force(n_sink, n_local):
    g = np.random.default_rng(11)
    B = 4
    for trial in range(12):
        nb = int(g.integers(n_sink + n_local + 1, 13))
        N = int(g.integers(n_sink + n_local, nb + 2))
        L = nb * B - int(g.integers(0, B))
        sc = np.full((1, 1, 12), -np.inf)
        sc[0, 0, :nb] = g.standard_normal(nb)
        idx, cnt = oracle.select(sc, np.array([L], np.int32), np.array([N], np.int32), B, n_sink, n_local, 12)
        want = _brute_force_select(sc[0, 0], nb, N, n_sink, n_local)
        assert cnt[0, 0] == len(want) == min(N, nb)
        assert idx[0, 0, :cnt[0, 0]].tolist() == want


def test_select_ties_prefer_smaller_index_and_errors():
    sc = np.zeros((1, 1, 8))
    idx, cnt = oracle.select(sc, np.array([32], np.int32), np.array([4], np.int32), 4, 1, 1, 8)
    assert idx[0, 0, :4].tolist() == [0, 1, 2, 7]
    with pytest.raises(ValueError):
        oracle.select(sc, np.array([32], np.int32), np.array([1], np.int32), 4, 1, 1, 8)
    with pytest.raises(ValueError):
        oracle.select(sc, np.array([32], np.int32), np.array([5], np.int32), 4, 1, 1, 4)


def test_selection_ignores_later_draft_tokens_and_is_shared():
    """Only the first draft token retrieves (Section 2.2): other query rows cannot change the set."""
    geom = si.make_geometry(si.WORKLOADS["cfg0"])
    c = si.make_layer(geom)
    a = oracle.select_blocks(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, 16)
    q2 = c["q"].copy()
    q2[:, 1:] = _bits(np.random.default_rng(5).standard_normal(q2[:, 1:].shape))
    b = oracle.select_blocks(q2, c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, 16)
    np.testing.assert_array_equal(a[0], b[0])
    assert a[0].shape == (1, 2, 16)        # one list per (sequence, KV head), none per draft token


def test_generator_plants_and_repairs_gap():
    geom = si.make_geometry(si.WORKLOADS["cfg0"])
    c = si.make_layer(geom)
    idx, cnt, sc = oracle.select_blocks(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, 16)
    assert c["min_gap_ratio"] >= 1.0 and c["delta"] > 0
    for (s, h), planted in c["planted"].items():
        sel = set(idx[s, h, :cnt[s, h]].tolist())
        assert set(planted.tolist()) <= sel and {0, 63} <= sel
        rest = np.setdiff1d(np.arange(64), list(sel))
        assert sc[s, h, list(sel - {0, 63})].min() - sc[s, h, rest].max() >= c["delta"] * 0.999


@pytest.mark.parametrize("forced", [(1, 1), (0, 0), (2, 3)])
def test_generator_repairs_gap_on_ragged_lengths_with_partly_filled_last_blocks(forced):
    """The generator scores blocks with its own copy of Eq. 5 to plant and repair the gap.  Where the last block
    of a sequence is only partly filled, that copy has to divide by the tokens the block holds, as the oracle does
    (with n_local = 0 the last block competes on its score): the oracle's own scores must show the promised gap
    between kept and evicted blocks for every sequence of a ragged batch."""
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=5, seq_len=(700, 3000), budget_blocks=9, n_sink=forced[0], n_local=forced[1])
    geom = si.make_geometry(w)
    assert any(int(L) % w.block_size for L in geom["seq_lens"])          # ragged: partly filled last blocks exist
    c = si.make_layer(geom, sharp=True)
    idx, cnt, sc = oracle.select_blocks(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], forced[0],
                                        forced[1], c["max_sel"])
    assert c["min_gap_ratio"] >= 1.0 and c["delta"] > 0
    gaps = []
    for s in range(w.n_seq):
        nb = int(c["n_blocks"][s])
        forced_set = set(range(min(forced[0], nb))) | set(range(max(0, nb - forced[1]), nb))
        for h in range(w.n_kv_heads):
            sel = set(idx[s, h, :cnt[s, h]].tolist())
            assert forced_set <= sel and set(c["planted"][(s, h)].tolist()) <= sel
            rest = np.setdiff1d(np.arange(nb), list(sel))
            chosen = list(sel - forced_set)
            if len(rest) and len(chosen):     # the generator's own smallest gap must be the oracle's too
                gap = sc[s, h, chosen].min() - sc[s, h, rest].max()
                assert gap >= c["min_gap"] * (1 - 1e-9) - 1e-15 and gap > 0
                gaps.append(gap)
    assert abs(min(gaps) - c["min_gap"]) <= 1e-12 * max(1.0, abs(c["min_gap"]))


# --------------------------------------------------------------------------- O5: inter-layer reuse (Eq. 9)

def test_reuse_copies_nearest_preceding_anchor():
    w = si.shrink(si.WORKLOADS["cfg0"], seq_len=(1024, 1024), budget_blocks=6, planted=3)
    geom = si.make_geometry(w)
    layers = [si.make_layer(geom, layer=l) for l in range(5)]
    anchors = [True, False, True, False, False]
    res = oracle.select_layers(layers, anchors, geom["budget"], 1, 1, geom["max_sel"])
    ind = oracle.select_layers(layers, [True] * 5, geom["budget"], 1, 1, geom["max_sel"])
    for l, a in enumerate([0, 0, 2, 2, 2]):
        np.testing.assert_array_equal(res[l][0], ind[a][0])
        np.testing.assert_array_equal(res[l][1], ind[a][1])
    for l in range(5):      # all anchors == independent per-layer retrieval
        one = oracle.select_blocks(layers[l]["q"], layers[l]["k_pool"], geom["block_table"], geom["seq_lens"],
                                   geom["budget"], 1, 1, geom["max_sel"])
        np.testing.assert_array_equal(ind[l][0], one[0])
    assert any(not np.array_equal(ind[0][0], ind[l][0]) for l in range(1, 5))


# --------------------------------------------------------------------------- O6: attention

def _all_blocks(c, max_sel=None):
    S, Hkv = c["block_table"].shape[0], c["Hkv"]
    nbmax = int(c["n_blocks"].max())
    max_sel = max_sel or nbmax
    idx = np.full((S, Hkv, max_sel), -1, dtype=np.int32)
    cnt = np.zeros((S, Hkv), dtype=np.int32)
    for s in range(S):
        idx[s, :, :c["n_blocks"][s]] = np.arange(c["n_blocks"][s])
        cnt[s] = c["n_blocks"][s]
    return idx, cnt


def _attn(c, idx, cnt, **kw):
    return oracle.verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"],
                              c["draft_v"], c["parent"], idx, cnt, **kw)


def _dense(c, **kw):
    return oracle.dense_verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"],
                                    c["draft_k"], c["draft_v"], c["parent"], **kw)


def test_attention_hand_worked_fixture():
    fx = _read_fixture("softmax_attention.txt")
    k_pool = np.zeros((2, 1, 2, 2), np.uint16)
    v_pool = np.zeros((2, 1, 2, 2), np.uint16)
    bt = np.array([[1, 0]], np.int32)
    for t in range(3):
        k_pool[bt[0, t // 2], 0, t % 2] = _bits(fx["keys"].reshape(3, 2)[t])
        v_pool[bt[0, t // 2], 0, t % 2] = _bits(fx["values"].reshape(3, 2)[t])
    k_pool[bt[0, 1], 0, 1] = _bits([40.0, 40.0])      # past the end: must not contribute
    v_pool[bt[0, 1], 0, 1] = _bits([1e4, 1e4])
    args = (_bits(fx["q"].reshape(1, 1, 1, 2)), k_pool, v_pool, bt, np.array([3], np.int32),
            _bits(fx["draft_k"].reshape(1, 1, 1, 2)), _bits(fx["draft_v"].reshape(1, 1, 1, 2)), None)
    ln2 = math.log(2.0)
    cases = [([0, 1], [1.0, 14.0], math.log(15.0)), ([0], [-105.0 / 11, 270.0 / 11], math.log(11.0)),
             ([1], [0.0, 15.0], math.log(12.0))]
    for sel, o_want, lse_want in cases:
        idx = np.array([[sel + [-1] * (2 - len(sel))]], np.int32)
        cnt = np.array([[len(sel)]], np.int32)
        o, lse = oracle.verify_attn(*args, idx, cnt, scale=ln2)
        np.testing.assert_allclose(o[0, 0, 0], o_want, rtol=0, atol=1e-13)
        assert abs(lse[0, 0, 0] - lse_want) < 1e-13
    o, lse = oracle.dense_verify_attn(*args, scale=ln2)
    np.testing.assert_allclose(o[0, 0, 0], [1.0, 14.0], rtol=0, atol=1e-13)
    assert abs(lse[0, 0, 0] - math.log(15.0)) < 1e-13


@pytest.mark.parametrize("tree", [False, True])
def test_all_blocks_equals_dense_and_library_sdpa(tree):
    c = _tiny_case(S=2, Hq=4, Hkv=2, D=8, B=4, T=5, lens=(13, 8), seed=7, tree=tree)
    idx, cnt = _all_blocks(c)
    o, lse = _attn(c, idx, cnt)
    od, lsed = _dense(c)
    np.testing.assert_allclose(o, od, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lsed, rtol=0, atol=1e-12)
    # library routine: torch scaled_dot_product_attention in fp64 with an explicit boolean mask
    S, T, Hq, D = c["q"].shape
    G = Hq // c["Hkv"]
    for s in range(S):
        L = int(c["seq_lens"][s])
        for hq in range(Hq):
            h = hq // G
            K = np.concatenate([_gather_tokens(c["k_pool"], c["block_table"], s, h, L, 4),
                                si.bf16_bits_to_f64(c["draft_k"][s, :, h])])
            V = np.concatenate([_gather_tokens(c["v_pool"], c["block_table"], s, h, L, 4),
                                si.bf16_bits_to_f64(c["draft_v"][s, :, h])])
            Q = si.bf16_bits_to_f64(c["q"][s, :, hq])
            mask = np.ones((T, L + T), dtype=bool)
            for i in range(T):
                vis = set()
                a = i
                while a >= 0:
                    vis.add(a)
                    a = (a - 1) if c["parent"] is None else int(c["parent"][s, a])
                for j in range(T):
                    mask[i, L + j] = j in vis
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
                attn_mask=torch.from_numpy(mask)[None]).numpy()[0]
            np.testing.assert_allclose(o[s, :, hq], ref, rtol=0, atol=1e-12)


def test_prefix_blocks_equal_dense_on_truncated_prefix():
    c = _tiny_case(S=1, Hq=2, Hkv=1, D=8, B=4, T=2, lens=(19,), seed=9)
    idx = np.array([[[0, 1, 2, -1, -1]]], np.int32)
    cnt = np.array([[3]], np.int32)
    o, lse = _attn(c, idx, cnt)
    c2 = dict(c)
    c2["seq_lens"] = np.array([12], np.int32)
    od, lsed = _dense(c2)
    np.testing.assert_allclose(o, od, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lsed, rtol=0, atol=1e-12)


def test_softmax_weights_sum_to_one():
    """With every value vector equal to ones the output is the sum of the softmax weights."""
    c = _tiny_case(seed=13, tree=True, scale=3.0)
    c["v_pool"][...] = _bits(1.0)
    c["draft_v"][...] = _bits(1.0)
    idx = np.array([[[0, 2, -1, -1]] * 2, [[1, -1, -1, -1]] * 2], np.int32)
    cnt = np.array([[2, 2], [1, 1]], np.int32)
    o, _ = _attn(c, idx, cnt)
    np.testing.assert_allclose(o, 1.0, rtol=0, atol=1e-12)


def test_single_draft_token_is_plain_decode_attention():
    c = _tiny_case(S=1, Hq=2, Hkv=1, D=8, B=4, T=1, lens=(10,), seed=17)
    idx, cnt = _all_blocks(c)
    o, lse = _attn(c, idx, cnt)
    K = np.concatenate([_gather_tokens(c["k_pool"], c["block_table"], 0, 0, 10, 4), si.bf16_bits_to_f64(c["draft_k"][0, :, 0])])
    V = np.concatenate([_gather_tokens(c["v_pool"], c["block_table"], 0, 0, 10, 4), si.bf16_bits_to_f64(c["draft_v"][0, :, 0])])
    for hq in range(2):
        z = K @ si.bf16_bits_to_f64(c["q"][0, 0, hq]) / math.sqrt(8)
        p = np.exp(z - z.max())
        np.testing.assert_allclose(o[0, 0, hq], (p / p.sum()) @ V, rtol=0, atol=1e-12)
        assert abs(lse[0, 0, hq] - (z.max() + math.log(p.sum()))) < 1e-12


def test_tree_with_linear_parents_is_chain():
    c = _tiny_case(seed=19, T=4)
    idx, cnt = _all_blocks(c)
    o_chain, _ = _attn(c, idx, cnt)
    c["parent"] = np.tile(np.arange(-1, 3, dtype=np.int32), (2, 1))
    o_tree, _ = _attn(c, idx, cnt)
    np.testing.assert_array_equal(o_chain, o_tree)


def test_tree_siblings_do_not_see_each_other():
    """Two children of the root: each equals a 2-token chain made of the root and itself."""
    c = _tiny_case(S=1, Hq=2, Hkv=1, D=8, B=4, T=3, lens=(8,), seed=23)
    idx, cnt = _all_blocks(c)
    c["parent"] = np.array([[-1, 0, 0]], np.int32)
    o, _ = _attn(c, idx, cnt)
    c2 = dict(c)
    keep = [0, 2]
    c2.update(q=c["q"][:, keep].copy(), draft_k=c["draft_k"][:, keep].copy(), draft_v=c["draft_v"][:, keep].copy(),
              parent=None)
    o2, _ = _attn(c2, idx, cnt)
    np.testing.assert_allclose(o[:, 2], o2[:, 1], rtol=0, atol=1e-13)


def test_split_merge_by_log_sum_exp():
    """Attention over Sel1 u Sel2 equals the log-sum-exp merge of attention over each half
    (the draft tokens go with one half only; the other half is computed with T-less inputs via lse)."""
    c = _tiny_case(S=1, Hq=2, Hkv=1, D=8, B=4, T=1, lens=(16,), seed=29, scale=2.0)
    full_idx, full_cnt = _all_blocks(c)
    o, lse = _attn(c, full_idx, full_cnt)
    # half A: blocks {0,1} + draft token; half B: blocks {2,3} + draft token.  The draft token is in both,
    # so remove its contribution once: w_draft = exp(z_draft - lse_X).
    oa, la = _attn(c, np.array([[[0, 1, -1, -1]]], np.int32), np.array([[2]], np.int32))
    ob, lb = _attn(c, np.array([[[2, 3, -1, -1]]], np.int32), np.array([[2]], np.int32))
    on, ln_ = _attn(c, np.array([[[-1, -1, -1, -1]]], np.int32), np.array([[0]], np.int32))   # draft token only
    for hq in range(2):
        # sums of exponentials: E_A = e^{la}, E_B = e^{lb}, E_draft = e^{ln}; union = E_A + E_B - E_draft
        m = max(la[0, 0, hq], lb[0, 0, hq])
        ea, eb, en = (math.exp(x - m) for x in (la[0, 0, hq], lb[0, 0, hq], ln_[0, 0, hq]))
        tot = ea + eb - en
        merged = (ea * oa[0, 0, hq] + eb * ob[0, 0, hq] - en * on[0, 0, hq]) / tot
        np.testing.assert_allclose(o[0, 0, hq], merged, rtol=0, atol=1e-11)
        assert abs(lse[0, 0, hq] - (m + math.log(tot))) < 1e-11


def test_sampled_rows_match_full_output():
    c = _tiny_case(seed=31, tree=True)
    idx = np.array([[[0, 3, -1, -1]] * 2, [[0, 1, -1, -1]] * 2], np.int32)
    cnt = np.array([[2, 2], [2, 2]], np.int32)
    o, lse = _attn(c, idx, cnt)
    smp = [(1, 2, 3), (0, 0, 0), (0, 1, 2)]
    os_, ls = _attn(c, idx, cnt, samples=smp)
    od, ld = _dense(c)
    ods, lds = _dense(c, samples=smp)
    for r, (s, i, hq) in enumerate(smp):
        np.testing.assert_array_equal(os_[r], o[s, i, hq])
        assert ls[r] == lse[s, i, hq]
        np.testing.assert_array_equal(ods[r], od[s, i, hq])
        assert lds[r] == ld[s, i, hq]


def test_full_budget_selection_gives_dense_attention_on_workload_shape():
    """The paper's fixed point on a generator-made case: budget = all blocks => dense verification."""
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=2, seq_len=(300, 700), n_q_heads=8, n_kv_heads=2, budget_blocks=10**6)
    geom = si.make_geometry(w)
    c = si.make_layer(geom, sharp=True)
    idx, cnt, _ = oracle.select_blocks(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1,
                                       geom["max_blocks"])
    np.testing.assert_array_equal(cnt, np.repeat(geom["n_blocks"][:, None], 2, axis=1))
    o, lse = oracle.verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"],
                                c["draft_v"], None, idx, cnt)
    od, lsed = oracle.dense_verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"],
                                        c["draft_k"], c["draft_v"], None)
    np.testing.assert_allclose(o, od, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lsed, rtol=0, atol=1e-12)


# --------------------------------------------------------------------------- O7: budget (Eq. 6)

def test_budget_closed_form():
    assert oracle.budget_blocks(4096, 4096, 0.1, 64) == 64           # L <= L0: nothing evicted
    assert oracle.budget_blocks(1000, 4096, 0.1, 64) == 16
    assert oracle.budget_blocks(32768, 4096, 0.1, 64) == 109         # (28672*0.1 + 4096)/64 = 108.8
    assert oracle.budget_blocks(131072, 4096, 0.5, 128) == 528       # (126976*0.5 + 4096)/128 = 528
    assert oracle.budget_blocks(5000, 64, 0.001, 64, 2, 4) == 6      # never fewer than the forced blocks
    assert oracle.budget_blocks(4097, 4096, 0.999, 64) == 65         # never more than the blocks that exist
    for L in (5000, 20000, 77777):
        for rho in (0.05, 0.1, 0.3):
            n = oracle.budget_blocks(L, 2048, rho, 1)
            assert n == math.ceil((L - 2048) * rho + 2048)


def test_budget_reproduces_table2_sparsity_column():
    """Weak cross-check: one effective length per dataset reproduces the printed s_a at all three L0."""
    rows = []
    with open(os.path.join(GOLDEN, "table2_sparsity.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, L0, sa = line.split()
                rows.append((name, int(L0), float(sa)))
    for name, L in (("GovReport", 6300), ("2WikiMQA", 6900)):
        for n, L0, sa in rows:
            if n == name:
                kept = oracle.budget_blocks(L, L0, 0.1, 1)
                assert abs((1 - kept / L) - sa) < 0.035, (name, L0, 1 - kept / L, sa)


# --------------------------------------------------------------------------- commit of accepted tokens

def _append_case(seed=41):
    c = _tiny_case(S=2, Hq=4, Hkv=2, D=8, B=4, T=5, lens=(9, 6), seed=seed)
    # room for growth: table of 5 blocks per sequence, fresh pages for the blocks that will be entered
    S, NB = 2, 5
    n_pages = S * NB + 1
    g = np.random.default_rng(seed)
    perm = g.permutation(n_pages)
    bt = perm[:S * NB].reshape(S, NB).astype(np.int32)
    k_pool = _bits(g.standard_normal((n_pages, 2, 4, 8)))
    v_pool = _bits(g.standard_normal((n_pages, 2, 4, 8)))
    c.update(block_table=bt, k_pool=k_pool, v_pool=v_pool, n_blocks=(c["seq_lens"] + 3) // 4)
    return c


def test_kv_append_places_rows_and_updates_lengths_and_reps():
    c = _append_case()
    accept = np.array([[0, 2, 3, 0, 0], [0, 1, 0, 0, 0]], np.int32)     # sequence 0 keeps drafts 0,2,3; sequence 1 keeps 0,1
    n_acc = np.array([3, 2], np.int32)
    old_k = [_gather_tokens(c["k_pool"], c["block_table"], s, h, int(c["seq_lens"][s]), 4) for s in range(2) for h in range(2)]
    old_v = [_gather_tokens(c["v_pool"], c["block_table"], s, h, int(c["seq_lens"][s]), 4) for s in range(2) for h in range(2)]
    reps = oracle.block_reps(c["k_pool"], c["block_table"], c["seq_lens"])
    untouched = reps.copy()
    new_len = oracle.kv_append(c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"], c["draft_v"],
                               accept, n_acc, reps)
    assert new_len.tolist() == [12, 8]
    i = 0
    for s in range(2):
        for h in range(2):
            want_k = np.concatenate([old_k[i], si.bf16_bits_to_f64(c["draft_k"][s, accept[s, :n_acc[s]], h])])
            want_v = np.concatenate([old_v[i], si.bf16_bits_to_f64(c["draft_v"][s, accept[s, :n_acc[s]], h])])
            np.testing.assert_array_equal(_gather_tokens(c["k_pool"], c["block_table"], s, h, int(new_len[s]), 4), want_k)
            np.testing.assert_array_equal(_gather_tokens(c["v_pool"], c["block_table"], s, h, int(new_len[s]), 4), want_v)
            for b in range((int(new_len[s]) + 3) // 4):        # every block's representative is the mean of its tokens
                np.testing.assert_allclose(reps[s, h, b], want_k[4 * b:4 * b + 4].mean(axis=0), rtol=0, atol=1e-14)
            i += 1
    # blocks that received nothing keep their representative bit for bit
    np.testing.assert_array_equal(reps[0, :, :2], untouched[0, :, :2])
    np.testing.assert_array_equal(reps[1, :, :1], untouched[1, :, :1])


def test_kv_append_at_once_equals_token_by_token_and_zero_accept_is_a_no_op():
    a = _append_case(43)
    b = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in a.items()}
    accept = np.array([[1, 4, 2, 0, 0], [3, 0, 0, 0, 0]], np.int32)
    n_acc = np.array([3, 0], np.int32)
    ra = oracle.block_reps(a["k_pool"], a["block_table"], a["seq_lens"])
    rb = ra.copy()
    la = oracle.kv_append(a["k_pool"], a["v_pool"], a["block_table"], a["seq_lens"], a["draft_k"], a["draft_v"], accept, n_acc, ra)
    lens = b["seq_lens"].copy()
    for step in range(3):
        lens = oracle.kv_append(b["k_pool"], b["v_pool"], b["block_table"], lens, b["draft_k"], b["draft_v"],
                                accept[:, step:step + 1].copy(), np.array([1, 0], np.int32), rb)
    assert la.tolist() == lens.tolist() == [12, 6]
    np.testing.assert_array_equal(a["k_pool"], b["k_pool"])
    np.testing.assert_array_equal(a["v_pool"], b["v_pool"])
    np.testing.assert_allclose(ra, rb, rtol=0, atol=1e-14)
    with pytest.raises(ValueError):
        oracle.kv_append(a["k_pool"], a["v_pool"], a["block_table"], la, a["draft_k"], a["draft_v"],
                         np.array([[7], [0]], np.int32), np.array([1, 0], np.int32), ra)     # draft index out of range


def test_attention_after_append_sees_the_committed_tokens():
    """After committing draft tokens 0..2 of a chain, the next step's dense attention over the cache equals
    attention over a prefix that already contained them."""
    c = _append_case(47)
    accept = np.tile(np.arange(5, dtype=np.int32), (2, 1))
    n_acc = np.array([3, 3], np.int32)
    new_len = oracle.kv_append(c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"], c["draft_v"],
                               accept, n_acc, None)
    # verification of draft token 3 before the commit: it saw the old prefix and drafts 0..3 (chain);
    # after the commit the same query with a single draft token (the old draft 3) sees prefix' + itself
    q1 = c["q"][:, 3:4].copy()
    dk1, dv1 = c["draft_k"][:, 3:4].copy(), c["draft_v"][:, 3:4].copy()
    after, _ = oracle.dense_verify_attn(q1, c["k_pool"], c["v_pool"], c["block_table"], new_len, dk1, dv1, None)
    c0 = _append_case(47)
    before, _ = oracle.dense_verify_attn(c0["q"], c0["k_pool"], c0["v_pool"], c0["block_table"], c0["seq_lens"],
                                         c0["draft_k"], c0["draft_v"], None)
    np.testing.assert_allclose(after[:, 0], before[:, 3], rtol=0, atol=1e-12)


# --------------------------------------------------------------------------- anchor calibration (Eq. 7-8)

def _random_selection_stack(n_layers=6, S=3, Hkv=2, nb=40, n_keep=9, seed=3, p_keep=0.7):
    """Selection lists with inter-layer correlation: a layer keeps each block of the previous layer with
    probability p_keep (layer 3 is redrawn from scratch)."""
    g = np.random.default_rng(seed)
    idx = np.full((n_layers, S, Hkv, n_keep + 3), -1, np.int32)
    cnt = np.zeros((n_layers, S, Hkv), np.int32)
    for s in range(S):
        for h in range(Hkv):
            cur = set(g.choice(nb, n_keep, replace=False).tolist())
            for l in range(n_layers):
                if l == 3:
                    cur = set(g.choice(nb, n_keep, replace=False).tolist())
                elif l > 0:
                    keep = {b for b in cur if g.random() < p_keep}
                    rest = [b for b in range(nb) if b not in cur]
                    cur = keep | set(g.choice(rest, max(0, n_keep + int(g.integers(0, 3)) - len(keep)), replace=False).tolist())
                lst = sorted(cur)
                idx[l, s, h, :len(lst)] = lst
                cnt[l, s, h] = len(lst)
    return idx, cnt


def test_jaccard_matches_python_sets_and_first_layer_is_zero():
    idx, cnt = _random_selection_stack()
    inter, uni, J = oracle.jaccard_adjacent(idx, cnt)
    L, S, H, _ = idx.shape
    assert J[0] == 0.0 and (inter[0] == 0).all() and (uni[0] == 0).all()
    for l in range(1, L):
        js = []
        for s in range(S):
            a = {(h, b) for h in range(H) for b in idx[l, s, h, :cnt[l, s, h]].tolist()}
            b_ = {(h, b) for h in range(H) for b in idx[l - 1, s, h, :cnt[l - 1, s, h]].tolist()}
            assert inter[l, s] == len(a & b_) and uni[l, s] == len(a | b_)
            js.append(len(a & b_) / len(a | b_))
        assert abs(J[l] - np.mean(js)) < 1e-15
    assert J[3] == J[1:].min()                    # the redrawn layer is the least similar to its predecessor
    same = np.stack([idx[0]] * 3), np.stack([cnt[0]] * 3)
    assert oracle.jaccard_adjacent(*same)[2].tolist() == [0.0, 1.0, 1.0]


def test_pick_anchors_is_topk_of_dissimilarity():
    idx, cnt = _random_selection_stack(n_layers=9, seed=8)
    J = oracle.jaccard_adjacent(idx, cnt)[2]
    for K in (1, 3, 9):
        a = oracle.pick_anchors(J, K)
        want = np.argsort(-(1.0 - J), kind="stable")[:K]
        assert sorted(np.flatnonzero(a).tolist()) == sorted(want.tolist())
        assert a[0]                                # J = 0 makes the first layer the most dissimilar one
    assert oracle.pick_anchors(np.array([0.0, 0.5, 0.5, 0.5]), 2).tolist() == [True, True, False, False]
    with pytest.raises(ValueError):
        oracle.pick_anchors(J, 0)


# ---------------------------------------------------------------------------- retrieval variants (Sections 2.2, 3.2)


def test_group_query_row_zero_is_the_first_token_and_rows_follow_a_roll():
    c = _tiny_case(T=4)
    np.testing.assert_array_equal(oracle.group_query_row(c["q"], 2, 0), oracle.group_query(c["q"], 2))
    for i in range(1, 4):
        rolled = np.ascontiguousarray(np.roll(c["q"], -i, axis=1))
        np.testing.assert_array_equal(oracle.group_query_row(c["q"], 2, i), oracle.group_query(rolled, 2))
    # literal group mean of the widened values
    want = si.bf16_bits_to_f64(c["q"])[:, 2].reshape(2, 2, 2, 8).mean(axis=2)
    np.testing.assert_allclose(oracle.group_query_row(c["q"], 2, 2), want, rtol=0, atol=1e-15)
    with pytest.raises(ValueError):
        oracle.group_query_row(c["q"], 2, 4)


def _brute_force_select_global(sc, nb, total, n_sink, n_local):
    """Best-sum subset of (head, block) pairs of size `total` that contains the forced pairs."""
    Hkv = sc.shape[0]
    pairs = [(h, b) for h in range(Hkv) for b in range(nb)]
    if total >= len(pairs):
        return set(pairs)
    forced = [(h, b) for (h, b) in pairs if b < n_sink or b >= nb - n_local]
    rest = [x for x in pairs if x not in forced]
    best, best_sum = None, -math.inf
    for comb in itertools.combinations(rest, total - len(forced)):
        tot = sum(sc[h, b] for (h, b) in comb)
        if tot > best_sum:
            best, best_sum = comb, tot
    return set(forced) | set(best)


@pytest.mark.parametrize("n_sink,n_local", [(0, 0), (1, 1)])
def test_select_global_equals_brute_force_over_head_block_pairs(n_sink, n_local):
    g = np.random.default_rng(23)
    B, Hkv = 4, 2
    for trial in range(10):
        nb = int(g.integers(n_sink + n_local + 2, 8))
        N = int(g.integers(n_sink + n_local, nb))          # per-head average; total = N * Hkv
        L = nb * B - int(g.integers(0, B))
        sc = np.full((1, Hkv, 8), -np.inf)
        sc[0, :, :nb] = g.standard_normal((Hkv, nb))
        idx, cnt = oracle.select_global(sc, np.array([L], np.int32), np.array([N], np.int32), B, n_sink, n_local, 8)
        got = {(h, int(b)) for h in range(Hkv) for b in idx[0, h, :cnt[0, h]]}
        assert got == _brute_force_select_global(sc[0], nb, N * Hkv, n_sink, n_local)
        assert int(cnt.sum()) == N * Hkv
        for h in range(Hkv):
            assert np.all(np.diff(idx[0, h, :cnt[0, h]]) > 0)


def test_select_global_special_cases():
    g = np.random.default_rng(29)
    B, nb = 4, 10
    L = np.array([nb * B - 1], np.int32)
    # one KV head: the shared budget is the per-head budget
    sc1 = g.standard_normal((1, 1, nb))
    for N in (3, 6, 10, 12):
        a = oracle.select_global(sc1, L, np.array([N], np.int32), B, 1, 1, nb)
        b = oracle.select(sc1, L, np.array([N], np.int32), B, 1, 1, nb)
        np.testing.assert_array_equal(a[0], b[0])
        np.testing.assert_array_equal(a[1], b[1])
    # numpy statement: forced pairs, then the best of the rest by (score desc, head asc, block asc)
    Hkv, N = 3, 4
    sc = g.standard_normal((1, Hkv, nb))
    sc[0, 1, 4] = sc[0, 0, 7]                                  # a tie across heads: the smaller head wins
    idx, cnt = oracle.select_global(sc, L, np.array([N], np.int32), B, 1, 1, nb)
    forced = {(h, b) for h in range(Hkv) for b in (0, nb - 1)}
    rest = [(h, b) for h in range(Hkv) for b in range(1, nb - 1)]
    order = np.lexsort(([b for _, b in rest], [h for h, _ in rest], [-sc[0, h, b] for h, b in rest]))
    want = forced | {rest[i] for i in order[:N * Hkv - len(forced)]}
    got = {(h, int(b)) for h in range(Hkv) for b in idx[0, h, :cnt[0, h]]}
    assert got == want
    # a head with uniformly higher scores takes the whole free budget
    sc2 = g.standard_normal((1, 2, nb))
    sc2[0, 1] += 100.0
    idx, cnt = oracle.select_global(sc2, L, np.array([5], np.int32), B, 1, 1, nb)
    assert cnt[0].tolist() == [2, 8]
    with pytest.raises(ValueError):
        oracle.select_global(sc2, L, np.array([1], np.int32), B, 1, 1, nb)       # forced pairs exceed the total
    with pytest.raises(ValueError):
        oracle.select_global(sc2, L, np.array([5], np.int32), B, 1, 1, 5)        # head 1 needs 8 slots


def test_per_token_retrieval_and_pair_overlap_match_python_sets():
    geom = si.make_geometry(si.WORKLOADS["cfg0"])
    c = si.make_layer(geom)
    T = c["q"].shape[1]
    idx_all, cnt_all = oracle.select_tokens(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, 16)
    first = oracle.select_blocks(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, 16)
    np.testing.assert_array_equal(idx_all[0], first[0])        # token 0 is the adopted strategy
    np.testing.assert_array_equal(cnt_all[0], first[1])
    inter = oracle.pair_overlap(idx_all, cnt_all)
    S, Hkv = cnt_all.shape[1:]
    for s in range(S):
        for h in range(Hkv):
            sets = [set(idx_all[i, s, h, :cnt_all[i, s, h]].tolist()) for i in range(T)]
            for i in range(T):
                for j in range(T):
                    assert inter[s, h, i, j] == len(sets[i] & sets[j])
    np.testing.assert_array_equal(inter, inter.transpose(0, 1, 3, 2))
    # identical queries retrieve identical blocks: overlap ratio 1 at every distance
    c2 = dict(c)
    q_same = c["q"].copy()
    q_same[:, 1:] = q_same[:, :1]
    ia, ca = oracle.select_tokens(q_same, c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, 16)
    ratios = oracle.overlap_by_distance(oracle.pair_overlap(ia, ca), ca, np.arange(T))
    assert set(ratios) == set(range(1, T)) and all(abs(v - 1.0) < 1e-15 for v in ratios.values())
    # hand-made sets: {0,1,2,3} vs {2,3,4,5} share half of their blocks
    idx2 = np.array([[[[0, 1, 2, 3]]], [[[2, 3, 4, 5]]]], np.int32)
    cnt2 = np.full((2, 1, 1), 4, np.int32)
    r = oracle.overlap_by_distance(oracle.pair_overlap(idx2, cnt2), cnt2, [0, 1])
    assert r == {1: 0.5}


# ---------------------------------------------------------------------------- acceptance (Eq. 2-3)


def _dists(g, *shape):
    p = g.random(shape).astype(np.float64) ** 3 + 1e-3            # a few dominant tokens, none with zero mass
    p = (p / p.sum(-1, keepdims=True)).astype(np.float32)
    return p


def test_accept_identical_models_accept_every_draft_and_sample_from_the_target():
    g = np.random.default_rng(51)
    S, T, V = 6, 5, 37
    p = _dists(g, S, T, V)
    tok = g.integers(0, V, (S, T)).astype(np.int32)
    u, un = g.random((S, T)).astype(np.float32), g.random(S).astype(np.float32)
    r = oracle.accept(p, p.copy(), tok, None, u, un, want_dist=True)
    assert r["n_path"].tolist() == [T] * S
    assert r["path"].tolist() == [list(range(T))] * S
    assert np.all(r["alpha"][:, 1:] == 1.0) and np.all(np.isnan(r["alpha"][:, 0]))
    for s in range(S):
        last = p[s, T - 1].astype(np.float64)
        np.testing.assert_allclose(r["final_dist"][s], last / last.sum(), rtol=0, atol=1e-15)
        cdf = np.cumsum(last)
        assert r["next_token"][s] == int(np.searchsorted(cdf, np.float64(un[s]) * cdf[-1], side="left"))


def test_accept_with_a_deterministic_target_is_greedy_prefix_matching():
    """One-hot target rows: a draft token is kept exactly when it is the target's token, the first mismatch cuts
    the rest and is replaced by the target's token (norm(max(0, p - q)) is the one-hot itself)."""
    g = np.random.default_rng(52)
    S, T, V = 8, 6, 11
    want = g.integers(0, V, (S, T)).astype(np.int32)               # the target's token after each row
    p = np.zeros((S, T, V), np.float32)
    for s in range(S):
        p[s, np.arange(T), want[s]] = 1.0
    q = _dists(g, S, T, V)
    tok = np.zeros((S, T), np.int32)
    n_match = g.integers(0, T, S)
    for s in range(S):
        for i in range(1, T):
            tok[s, i] = want[s, i - 1] if i <= n_match[s] else (want[s, i - 1] + 1 + g.integers(0, V - 1)) % V
    r = oracle.accept(p, q, tok, None, g.random((S, T)).astype(np.float32), g.random(S).astype(np.float32))
    for s in range(S):
        assert r["n_path"][s] == 1 + n_match[s]
        assert r["path"][s, :r["n_path"][s]].tolist() == list(range(1 + n_match[s]))
        assert r["next_token"][s] == want[s, n_match[s]]


def test_accept_one_draft_token_keeps_the_target_distribution():
    """The purpose of Eq. 2-3: the first new token is distributed as the target, whatever the draft model is.
    Exact check: sum over the draft token d ~ q of  alpha_d [x = d] + (1 - alpha_d) residual_d(x)  equals p(x)."""
    g = np.random.default_rng(53)
    V = 9
    p, q = _dists(g, 1, 2, V), _dists(g, 1, 2, V)
    out = np.zeros(V)
    for d in range(V):
        tok = np.array([[0, d]], np.int32)
        acc = oracle.accept(p, q, tok, None, np.zeros((1, 2), np.float32), np.zeros(1, np.float32))
        a = acc["alpha"][0, 1]
        assert a == min(1.0, float(p[0, 0, d]) / float(q[0, 0, d]))
        out[d] += float(q[0, 0, d]) * a
        if a < 1.0:
            rej = oracle.accept(p, q, tok, None, np.full((1, 2), 0.9999999, np.float32), np.zeros(1, np.float32), want_dist=True)
            assert rej["n_path"][0] == 1
            out += float(q[0, 0, d]) * (1.0 - a) * rej["final_dist"][0]
    np.testing.assert_allclose(out, p[0, 0].astype(np.float64) / p[0, 0].astype(np.float64).sum(), rtol=0, atol=1e-7)


def test_accept_two_siblings_keep_the_target_distribution():
    """Tree step with two children drawn independently from q: try the first, on rejection adjust p and try the
    second, on rejection adjust again and resample.  The emitted token is again distributed as the target."""
    g = np.random.default_rng(54)
    V = 6
    p, q = _dists(g, 1, 3, V), _dists(g, 1, 3, V)
    par = np.array([[-1, 0, 0]], np.int32)
    q0 = q[0, 0].astype(np.float64)
    out = np.zeros(V)
    hi = np.float32(0.9999999)
    for d1 in range(V):
        for d2 in range(V):
            w = q0[d1] * q0[d2]
            tok = np.array([[0, d1, d2]], np.int32)
            a1 = oracle.accept(p, q, tok, par, np.zeros((1, 3), np.float32), np.zeros(1, np.float32))["alpha"][0, 1]
            out[d1] += w * a1
            if a1 == 1.0:
                continue
            r2 = oracle.accept(p, q, tok, par, np.array([[0, hi, 0]], np.float32), np.zeros(1, np.float32))
            a2 = r2["alpha"][0, 2]
            assert a2 == 0.0 or r2["path"][0, :2].tolist() == [0, 2]      # a repeated rejected token has no mass left
            out[d2] += w * (1 - a1) * a2
            if a2 == 1.0:
                continue
            r3 = oracle.accept(p, q, tok, par, np.array([[0, hi, hi]], np.float32), np.zeros(1, np.float32), want_dist=True)
            assert r3["n_path"][0] == 1
            out += w * (1 - a1) * (1 - a2) * r3["final_dist"][0]
    want = p[0, 0].astype(np.float64)
    np.testing.assert_allclose(out, want / want.sum(), rtol=0, atol=1e-7)


def test_accept_inverts_the_cumulative_sum_and_walks_a_tree():
    g = np.random.default_rng(55)
    S, T, V = 5, 7, 23
    p, q = _dists(g, S, T, V), _dists(g, S, T, V)
    par = np.full((S, T), -1, np.int32)
    for s in range(S):
        for i in range(1, T):
            par[s, i] = g.integers(0, i)
    tok = g.integers(0, V, (S, T)).astype(np.int32)
    u, un = g.random((S, T)).astype(np.float32), g.random(S).astype(np.float32)
    r = oracle.accept(p, q, tok, par, u, un, want_dist=True)
    for s in range(S):
        n = r["n_path"][s]
        path = r["path"][s, :n]
        assert path[0] == 0 and all(par[s, path[k]] == path[k - 1] for k in range(1, n))     # a root-to-node path
        assert all(u[s, c] < r["alpha"][s, c] for c in path[1:])
        tried = ~np.isnan(r["alpha"][s])
        assert all(par[s, c] in path for c in np.nonzero(tried)[0])                          # only children of kept rows
        assert all(u[s, c] >= r["alpha"][s, c] for c in np.nonzero(tried)[0] if c not in path)
        cdf = np.cumsum(r["final_dist"][s])
        x = r["next_token"][s]
        lo = cdf[x - 1] if x > 0 else 0.0
        assert lo - 1e-12 <= np.float64(un[s]) <= cdf[x] + 1e-12
    with pytest.raises(ValueError):
        oracle.accept(p, q, np.full((S, T), V, np.int32), par, u, un)


def test_round_bf16_is_nearest_representable_with_ties_to_even():
    g = np.random.default_rng(61)
    x = np.concatenate([g.standard_normal(4000) * 10.0 ** g.integers(-6, 6, 4000), [0.0, 1.0, -1.0, 255.0, 256.5]])
    y = oracle.round_bf16(x)
    # representable: a float32 whose low 16 bits are zero
    bits = y.astype(np.float32).view(np.uint32)
    assert np.all(y.astype(np.float32).astype(np.float64) == y) and np.all(bits & 0xFFFF == 0)
    # nearest: no bfloat16 neighbour is closer
    up = (bits + 0x10000).view(np.float32).astype(np.float64)
    dn = (bits - 0x10000).view(np.float32).astype(np.float64)
    nz = x != 0
    assert np.all(np.abs(y - x)[nz] <= np.abs(up - x)[nz]) and np.all(np.abs(y - x)[nz] <= np.abs(dn - x)[nz])
    # ties go to the even significand: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert oracle.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert oracle.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    assert oracle.round_bf16(np.array([-(1.0 + 2.0 ** -8)]))[0] == -1.0
    # agrees with the float32 -> bfloat16 conversion of the input generator wherever float32 holds x exactly
    x32 = x.astype(np.float32)
    np.testing.assert_array_equal(oracle.round_bf16(x32.astype(np.float64)), si.bf16_bits_to_f64(si.f32_to_bf16_bits(x32)))
