"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU oracle, element by element,
on the same seeded bf16 inputs.

Bars: kept block indices and counts bit-exact; attention outputs within max-abs 1e-2 and mean-abs 1e-3
(the stated tolerance) and, because those are loose for the N(0,1)/sqrt(128) generator, also a
per-row relative L2 error <= 1e-2 and |lse - lse*| <= 1e-3; every case also runs with the
"sharp" generator (logit std ~3), where a wrong mask, a dropped block or a wrong tail bound
fails by orders of magnitude.
"""
import numpy as np
import pytest
import torch

import oracle
import sv_inputs as si

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sv():
    import paper_2512_21911_b200 as pkg
    return pkg


def bf16_dev(a):
    return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()


def bf16_host(t):
    return si.bf16_bits_to_f64(t.cpu().view(torch.int16).numpy().view(np.uint16))


class Dev:
    """Device copies of a generated case + the geometry descriptors."""

    def __init__(self, sv, c):
        w = c["workload"]
        self.c, self.w = c, w
        self.geom = sv.make_geom(w.n_seq, w.n_q_heads, w.n_kv_heads, w.head_dim, w.block_size, c["max_blocks"], w.n_draft)
        self.q, self.k_pool, self.v_pool = bf16_dev(c["q"]), bf16_dev(c["k_pool"]), bf16_dev(c["v_pool"])
        self.draft_k, self.draft_v = bf16_dev(c["draft_k"]), bf16_dev(c["draft_v"])
        self.block_table = torch.from_numpy(c["block_table"]).cuda()
        self.seq_lens = torch.from_numpy(c["seq_lens"]).cuda()
        self.budget = torch.from_numpy(c["budget"]).cuda()
        self.parent = torch.from_numpy(c["parent"]).cuda() if c["parent"] is not None else None
        self.kv = sv.make_kv(self.k_pool, self.v_pool, self.block_table, self.seq_lens)
        self.reps = torch.full((w.n_seq, w.n_kv_heads, c["max_blocks"], w.head_dim), float("nan"), device="cuda")


def gpu_select(sv, d, n_sink, n_local, max_sel, scores=False):
    sv.sv_block_reps(d.geom, d.kv, d.reps)
    idx = torch.full((d.w.n_seq, d.w.n_kv_heads, max_sel), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((d.w.n_seq, d.w.n_kv_heads), -7, dtype=torch.int32, device="cuda")
    sc = torch.full((d.w.n_seq, d.w.n_kv_heads, d.c["max_blocks"]), float("nan"), device="cuda") if scores else None
    sv.sv_select_blocks(d.geom, d.q, d.reps, d.seq_lens, d.budget, n_sink, n_local, idx, cnt, out_scores=sc)
    return idx, cnt, sc


def gpu_attn(sv, d, idx, cnt):
    w = d.w
    out = torch.full((w.n_seq, w.n_draft, w.n_q_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((w.n_seq, w.n_draft, w.n_q_heads), float("nan"), device="cuda")
    max_sel = idx.shape[-1] if idx is not None else d.c["max_blocks"]
    ws = torch.empty(max(16, sv.sv_workspace_bytes(d.geom, max_sel)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.sv_verify_attn(d.geom, d.q, d.kv, d.draft_k, d.draft_v, d.parent, idx, cnt, out, lse=lse, workspace=ws,
                      status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return bf16_host(out), lse.cpu().numpy().astype(np.float64)


def check_attn(o, lse, o_ref, lse_ref, what=""):
    assert np.isfinite(o).all() and np.isfinite(lse).all(), what
    err = np.abs(o - o_ref)
    scale = max(1.0, float(np.abs(o_ref).max()))
    assert err.max() <= 1e-2 * scale, (what, err.max())
    assert err.mean() <= 1e-3 * scale, (what, err.mean())
    rel = np.linalg.norm(o - o_ref, axis=-1) / np.linalg.norm(o_ref, axis=-1)
    assert rel.max() <= 1e-2, (what, rel.max())
    assert np.abs(lse - lse_ref).max() <= 1e-3, (what, np.abs(lse - lse_ref).max())


def oracle_select(c, n_sink, n_local, max_sel):
    return oracle.select_blocks(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], n_sink, n_local, max_sel)


def oracle_attn(c, idx, cnt, samples=None):
    return oracle.verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"],
                              c["draft_v"], c["parent"], idx, cnt, samples=samples)


def run_pipeline(sv, c, n_sink=None, n_local=None, what=""):
    """reps -> select -> attention on the GPU, compared stage by stage with the oracle."""
    n_sink = c["n_sink"] if n_sink is None else n_sink
    n_local = c["n_local"] if n_local is None else n_local
    d = Dev(sv, c)
    idx, cnt, sc = gpu_select(sv, d, n_sink, n_local, c["max_sel"], scores=True)
    torch.cuda.synchronize()
    idx_ref, cnt_ref, sc_ref = oracle_select(c, n_sink, n_local, c["max_sel"])
    reps_ref = oracle.block_reps(c["k_pool"], c["block_table"], c["seq_lens"])
    reps = d.reps.cpu().numpy().astype(np.float64)
    for s in range(d.w.n_seq):
        nb = int(c["n_blocks"][s])
        np.testing.assert_allclose(reps[s, :, :nb], reps_ref[s, :, :nb], rtol=1e-5, atol=1e-6 * max(1.0, np.abs(reps_ref).max()))
        assert np.isnan(reps[s, :, nb:]).all()                       # blocks past the end are not written
        tol = 1e-5 * max(1.0, float(np.abs(sc_ref[s, :, :nb]).max()))
        np.testing.assert_allclose(sc.cpu().numpy()[s, :, :nb], sc_ref[s, :, :nb], rtol=0, atol=tol)
    cnt_h, idx_h = cnt.cpu().numpy(), idx.cpu().numpy()
    np.testing.assert_array_equal(cnt_h, cnt_ref)
    for s in range(d.w.n_seq):
        for h in range(d.w.n_kv_heads):
            n = cnt_ref[s, h]
            np.testing.assert_array_equal(idx_h[s, h, :n], idx_ref[s, h, :n], err_msg=f"{what} s={s} h={h}")
            assert (idx_h[s, h, n:] == -7).all()
    o, lse = gpu_attn(sv, d, idx, cnt)
    o_ref, lse_ref = oracle_attn(c, idx_ref, cnt_ref)
    check_attn(o, lse, o_ref, lse_ref, what)
    return d, idx, cnt, o, lse


def check_lists(idx_h, cnt_h, idx_ref, cnt_ref, what=""):
    np.testing.assert_array_equal(cnt_h, cnt_ref, err_msg=what)
    for s in range(cnt_ref.shape[0]):
        for h in range(cnt_ref.shape[1]):
            n = cnt_ref[s, h]
            np.testing.assert_array_equal(idx_h[s, h, :n], idx_ref[s, h, :n], err_msg=f"{what} s={s} h={h}")
            assert (idx_h[s, h, n:] == -7).all()


def run_sampled(sv, c, samples, what=""):
    """select + attention on a full-size case: lists bit-exact, attention checked on the sampled (s, i, hq) rows."""
    d = Dev(sv, c)
    idx, cnt, _ = gpu_select(sv, d, c["n_sink"], c["n_local"], c["max_sel"])
    torch.cuda.synchronize()
    idx_ref, cnt_ref, _ = oracle_select(c, c["n_sink"], c["n_local"], c["max_sel"])
    check_lists(idx.cpu().numpy(), cnt.cpu().numpy(), idx_ref, cnt_ref, what)
    o, lse = gpu_attn(sv, d, idx, cnt)
    o_ref, lse_ref = oracle_attn(c, idx_ref, cnt_ref, samples=samples)
    check_attn(np.stack([o[s, i, hq] for s, i, hq in samples]), np.array([lse[s, i, hq] for s, i, hq in samples]),
               o_ref, lse_ref, what)
    assert np.isfinite(o).all()
    return d


SMALL = {
    # rows = G*T: 16 (1 warp row), 32, 20 (ragged batch), 64, 128 (block 128, tree)
    "cfg0": si.WORKLOADS["cfg0"],
    "cfg1_full": si.shrink(si.WORKLOADS["cfg1"], n_layers=1),      # the benchmark's layer shape, for the variant tests
    "cfg1_small": si.shrink(si.WORKLOADS["cfg1"], seq_len=(4096, 4096), budget_blocks=20, n_layers=1),
    "cfg2_small": si.shrink(si.WORKLOADS["cfg2"], n_seq=5, seq_len=(700, 3000), budget_blocks=9),
    "rows64": si.shrink(si.WORKLOADS["cfg1"], seq_len=(2500, 2500), budget_blocks=12, n_draft=16, n_layers=1, tree=True),
    "cfg3_small": si.shrink(si.WORKLOADS["cfg3"], n_seq=2, seq_len=(5000, 9000), budget_blocks=11, planted=3),
    "rows4": si.shrink(si.WORKLOADS["cfg1"], seq_len=(2048, 2048), budget_blocks=8, n_draft=1, n_layers=1),
    "t32": si.shrink(si.WORKLOADS["cfg0"], seq_len=(1000, 1000), budget_blocks=5, n_draft=32, tree=True, planted=2),
    # multi-head attention (G = 1), a wide GQA group (G = 16, 128 rows), block 128 whose tail holds <= 64 tokens
    "mha": si.shrink(si.WORKLOADS["cfg0"], n_q_heads=4, n_kv_heads=4, seq_len=(1200, 1200), budget_blocks=6, planted=2),
    "g16": si.shrink(si.WORKLOADS["cfg0"], n_q_heads=32, n_kv_heads=2, seq_len=(1500, 1500), budget_blocks=6, n_draft=8, planted=2),
    # 65-128 rows (one softmax thread per row) with idle warps and padding rows: 80 rows (3 of 4 warps), 104 rows
    "rows80_tree": si.shrink(si.WORKLOADS["cfg1"], seq_len=(2100, 2100), budget_blocks=9, n_draft=20, n_layers=1, tree=True, planted=2),
    "rows104": si.shrink(si.WORKLOADS["cfg3"], n_seq=2, seq_len=(1500, 2600), budget_blocks=5, n_draft=13, planted=2),
    # more than 128 query rows per KV head (several row tiles) and more than 32 draft tokens (64-bit ancestor masks)
    "t60_tree": si.shrink(si.WORKLOADS["cfg1"], seq_len=(3000, 3000), budget_blocks=10, n_draft=60, n_layers=1, tree=True, planted=3),
    "t40_chain_2seq": si.shrink(si.WORKLOADS["cfg2"], n_seq=2, seq_len=(900, 2100), budget_blocks=7, n_draft=40, planted=2),
    "g8_t24_b128": si.shrink(si.WORKLOADS["cfg3"], n_seq=2, seq_len=(2000, 4000), budget_blocks=6, n_draft=24, planted=2),
    "g16_t64": si.shrink(si.WORKLOADS["cfg0"], n_q_heads=32, n_kv_heads=2, seq_len=(1100, 1100), budget_blocks=5, n_draft=64, tree=True, planted=2),
    # an odd number of row tiles (3 x 128 rows: 16 + 16 + 8 draft tokens), one CTA per row tile
    "g8_t40_tree_3tiles": si.shrink(si.WORKLOADS["cfg3"], n_seq=2, seq_len=(1800, 3100), budget_blocks=6, n_draft=40, planted=2),
    # more row-tile CTAs than SMs: one CTA serves a pair of row tiles from one gather (2 tiles: 10 x 8 x 2 = 160 CTAs
    # otherwise; 3 tiles, the last pair holding one: 7 x 8 x 3 = 168)
    "t24_tile_pairs": si.shrink(si.WORKLOADS["cfg3"], n_seq=10, seq_len=(700, 1900), budget_blocks=5, n_draft=24, planted=2),
    "t40_tree_tile_pairs_odd": si.shrink(si.WORKLOADS["cfg3"], n_seq=7, seq_len=(600, 1500), budget_blocks=4, n_draft=40, tree=True, planted=1),
    # more (sequence, KV head) pairs than SMs: several waves of CTAs, one split each
    "many_seqs": si.shrink(si.WORKLOADS["cfg2"], n_seq=40, seq_len=(300, 1100), budget_blocks=6, planted=1),
    "b128_short_tail": si.shrink(si.WORKLOADS["cfg3"], n_seq=2, seq_len=(128 * 9 + 30, 128 * 9 + 30), n_q_heads=16, n_kv_heads=4,
                                 budget_blocks=5, n_draft=6, planted=2),
}


@pytest.mark.parametrize("name", list(SMALL))
@pytest.mark.parametrize("sharp", [False, True])
def test_pipeline_parity_small(sv, name, sharp):
    c = si.make_layer(si.make_geometry(SMALL[name]), sharp=sharp)
    assert c["min_gap_ratio"] >= 1.0
    run_pipeline(sv, c, what=f"{name} sharp={sharp}")


def test_full_size_cfg3_one_pair_in_full(sv):
    """The long-context tree configuration: besides random samples, every draft row and query head of one
    (sequence, KV head) pair -- all 128 query rows of one CTA group."""
    c = si.make_layer(si.make_geometry(si.WORKLOADS["cfg3"]), sharp=True)
    w = c["workload"]
    G = w.n_q_heads // w.n_kv_heads
    smp = [(2, i, 5 * G + g) for i in range(w.n_draft) for g in range(G)]
    run_sampled(sv, c, smp, what="cfg3, sequence 2, KV head 5")


def test_full_size_cfg3_dense_sampled(sv):
    """Dense verification of the 4 x 131072-token tree configuration (2 GiB of K/V per call) on sampled rows."""
    c = si.make_layer(si.make_geometry(si.WORKLOADS["cfg3"]), sharp=True)
    d = Dev(sv, c)
    o, lse = gpu_attn(sv, d, None, None)
    g = np.random.default_rng(23)
    w = c["workload"]
    smp = [(int(g.integers(0, w.n_seq)), int(g.integers(0, w.n_draft)), int(g.integers(0, w.n_q_heads))) for _ in range(32)]
    o_ref, lse_ref = oracle.dense_verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"],
                                              c["draft_k"], c["draft_v"], c["parent"], samples=smp)
    check_attn(np.stack([o[s, i, h] for s, i, h in smp]), np.array([lse[s, i, h] for s, i, h in smp]), o_ref, lse_ref,
               "cfg3 dense")


@pytest.mark.parametrize("point", [(8192, 1 / 16, 8), (8192, 1 / 4, 16), (32768, 1 / 16, 4), (32768, 1 / 4, 8),
                                   (131072, 1 / 16, 16), (131072, 1 / 32, 8), (131072, 1 / 4, 1)])
def test_more_sweep_points(sv, point):
    """Further points of the context x budget x draft-length sweep: every context, the 1/16 budget, 8 draft tokens."""
    c = si.make_layer(si.make_geometry(si.sweep_workload(*point)), sharp=True)
    g = np.random.default_rng(19)
    w = c["workload"]
    smp = [(0, int(g.integers(0, w.n_draft)), int(g.integers(0, w.n_q_heads))) for _ in range(32)]
    run_sampled(sv, c, smp, what=f"sweep {point}")


@pytest.mark.parametrize("forced", [(0, 0), (2, 4)])
def test_sink_local_variants(sv, forced):
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=3, seq_len=(900, 2000), budget_blocks=10, n_sink=forced[0], n_local=forced[1])
    c = si.make_layer(si.make_geometry(w), sharp=True)
    run_pipeline(sv, c, what=f"forced={forced}")


def test_nan_in_unused_tail_slots_is_harmless(sv):
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=3, seq_len=(900, 2000), budget_blocks=10)
    c = si.make_layer(si.make_geometry(w), sharp=True, tail_fill=None)
    run_pipeline(sv, c, what="nan tail")


def test_budget_covering_all_blocks_is_dense(sv):
    """Fixed point: nothing evicted -> the sparse path equals dense verification; sel_idx=NULL is the same."""
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=3, seq_len=(500, 1500), budget_blocks=10**6)
    geom = si.make_geometry(w)
    geom["max_sel"] = geom["max_blocks"]
    c = si.make_layer(geom, sharp=True)
    d, idx, cnt, o, lse = run_pipeline(sv, c, what="full budget")
    np.testing.assert_array_equal(cnt.cpu().numpy(), np.repeat(c["n_blocks"][:, None], w.n_kv_heads, axis=1))
    od_ref, lsed_ref = oracle.dense_verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"],
                                                c["draft_k"], c["draft_v"], c["parent"])
    check_attn(o, lse, od_ref, lsed_ref, "sparse(all) vs dense oracle")
    o2, lse2 = gpu_attn(sv, d, None, None)
    check_attn(o2, lse2, od_ref, lsed_ref, "dense entry")


def test_selection_ties_and_first_token_only(sv):
    """All-zero keys: every score ties, smaller indices win.  Other draft rows never change the set."""
    w = si.shrink(si.WORKLOADS["cfg0"], seq_len=(1500, 1500), budget_blocks=7)
    c = si.make_layer(si.make_geometry(w))
    z = dict(c)
    z["k_pool"] = np.zeros_like(c["k_pool"])
    d = Dev(sv, z)
    idx, cnt, _ = gpu_select(sv, d, 1, 1, 7)
    torch.cuda.synchronize()
    assert (cnt.cpu().numpy() == 7).all()
    assert (idx.cpu().numpy() == np.array([0, 1, 2, 3, 4, 5, 23])).all()
    idx_ref, _, _ = oracle_select(z, 1, 1, 7)
    np.testing.assert_array_equal(idx.cpu().numpy(), idx_ref)
    d1 = Dev(sv, c)
    a, _, _ = gpu_select(sv, d1, 1, 1, 7)
    c2 = dict(c)
    c2["q"] = c["q"].copy()
    c2["q"][:, 1:] = si.f32_to_bf16_bits(np.random.default_rng(1).standard_normal(c["q"][:, 1:].shape).astype(np.float32))
    b, _, _ = gpu_select(sv, Dev(sv, c2), 1, 1, 7)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_reuse_prev_copies_previous_layer(sv):
    w = si.shrink(si.WORKLOADS["cfg0"], seq_len=(1500, 1500), budget_blocks=7)
    c = si.make_layer(si.make_geometry(w))
    d = Dev(sv, c)
    idx, cnt, _ = gpu_select(sv, d, 1, 1, 7)
    idx2, cnt2 = torch.zeros_like(idx), torch.zeros_like(cnt)
    sv.sv_select_blocks(d.geom, None, None, None, None, 1, 1, idx2, cnt2, reuse_prev=True, prev_idx=idx, prev_cnt=cnt)
    torch.cuda.synchronize()
    assert torch.equal(idx, idx2) and torch.equal(cnt, cnt2)
    with pytest.raises(sv.SvError):
        sv.sv_select_blocks(d.geom, None, None, None, None, 1, 1, idx2, cnt2, reuse_prev=True)


@pytest.mark.parametrize("name", ["cfg1_small", "cfg3_small", "t60_tree", "rows4"])
def test_reused_list_variant_matches_oracle(sv, name):
    """sv_verify_attn_reused (the gather starts ahead of the dependency wait; for layers that reuse a list, Eq. 9):
    same results as the oracle on a list written well before the call, sparse and dense, called back to back so that
    each call's gather overlaps the previous call's tail."""
    c = si.make_layer(si.make_geometry(SMALL[name]), sharp=True)
    d = Dev(sv, c)
    idx, cnt, _ = gpu_select(sv, d, c["n_sink"], c["n_local"], c["max_sel"])
    torch.cuda.synchronize()
    idx_ref, cnt_ref, _ = oracle_select(c, c["n_sink"], c["n_local"], c["max_sel"])
    w = d.w
    ws = torch.empty(max(16, sv.sv_workspace_bytes(d.geom, c["max_blocks"])), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs = [torch.full((w.n_seq, w.n_draft, w.n_q_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
            for _ in range(4)]
    lses = [torch.full((w.n_seq, w.n_draft, w.n_q_heads), float("nan"), device="cuda") for _ in range(4)]
    for k in range(4):      # sparse, dense, sparse, dense
        sparse = k % 2 == 0
        sv.sv_verify_attn_reused(d.geom, d.q, d.kv, d.draft_k, d.draft_v, d.parent, idx if sparse else None,
                                 cnt if sparse else None, outs[k], lse=lses[k], workspace=ws, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o_ref, lse_ref = oracle_attn(c, idx_ref, cnt_ref)
    o_dense, lse_dense = oracle.dense_verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"],
                                                  c["draft_k"], c["draft_v"], c["parent"])
    for k in range(4):
        ref = (o_ref, lse_ref) if k % 2 == 0 else (o_dense, lse_dense)
        check_attn(bf16_host(outs[k]), lses[k].cpu().numpy().astype(np.float64), ref[0], ref[1], f"reused {name} call {k}")


def test_block_reps_range_update(sv):
    """Only the requested block range is rewritten (a decoding loop refreshes the tail block only)."""
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=3, seq_len=(900, 2000), budget_blocks=10)
    c = si.make_layer(si.make_geometry(w))
    d = Dev(sv, c)
    sv.sv_block_reps(d.geom, d.kv, d.reps)
    full = d.reps.clone()
    d.reps.fill_(123.0)
    sv.sv_block_reps(d.geom, d.kv, d.reps, 3, 6)
    torch.cuda.synchronize()
    assert torch.equal(d.reps[:, :, 3:6], full[:, :, 3:6])
    assert (d.reps[:, :, :3] == 123.0).all() and (d.reps[:, :, 6:] == 123.0).all()
    # tail-only refresh: exactly the last block of every (ragged) sequence
    d.reps.fill_(123.0)
    sv.sv_block_reps(d.geom, d.kv, d.reps, sv.SV_TAIL_BLOCK)
    torch.cuda.synchronize()
    for s in range(3):
        t = int(c["n_blocks"][s]) - 1
        assert torch.equal(d.reps[s, :, t], full[s, :, t])
        assert (d.reps[s, :, :t] == 123.0).all() and (d.reps[s, :, t + 1:] == 123.0).all()


def test_empty_prefix_and_empty_selection(sv):
    """A sequence with no cached tokens attends to its draft tokens only; so does an empty block list."""
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=3, seq_len=(300, 900), budget_blocks=4, tree=True)
    geom = si.make_geometry(w)
    c = si.make_layer(geom, sharp=True)
    c["seq_lens"] = c["seq_lens"].copy()
    c["seq_lens"][1] = 0
    c["n_blocks"] = ((c["seq_lens"] + 63) // 64).astype(np.int32)
    d = Dev(sv, c)
    idx, cnt, _ = gpu_select(sv, d, 1, 1, c["max_sel"])
    torch.cuda.synchronize()
    idx_ref, cnt_ref, _ = oracle_select(c, 1, 1, c["max_sel"])
    np.testing.assert_array_equal(cnt.cpu().numpy(), cnt_ref)
    assert (cnt_ref[1] == 0).all()
    o, lse = gpu_attn(sv, d, idx, cnt)
    o_ref, lse_ref = oracle_attn(c, idx_ref, cnt_ref)
    check_attn(o, lse, o_ref, lse_ref, "empty prefix")
    cnt0 = torch.zeros_like(cnt)
    o, lse = gpu_attn(sv, d, idx, cnt0)
    o_ref, lse_ref = oracle_attn(c, idx_ref, np.zeros_like(cnt_ref))
    check_attn(o, lse, o_ref, lse_ref, "empty selection")


def test_more_splits_than_blocks(sv):
    """One (sequence, KV head) pair: the split count is capped by the block count, some CTAs get one block."""
    w = si.shrink(si.WORKLOADS["cfg0"], n_q_heads=4, n_kv_heads=1, seq_len=(2000, 2000), budget_blocks=10, planted=1)
    c = si.make_layer(si.make_geometry(w), sharp=True)
    d = run_pipeline(sv, c, what="10 blocks")[0]
    assert sv.sv_verify_attn_splits(d.geom, 10) == 10
    # a list of a few units is not split at all (the merge would cost more than the gather)
    w = si.shrink(si.WORKLOADS["cfg0"], n_q_heads=4, n_kv_heads=1, seq_len=(2000, 2000), budget_blocks=3, planted=1)
    c = si.make_layer(si.make_geometry(w), sharp=True)
    d = run_pipeline(sv, c, what="3 blocks")[0]
    assert sv.sv_verify_attn_splits(d.geom, 3) == 1 and sv.sv_workspace_bytes(d.geom, 3) == 0


def test_workspace_too_small_is_rejected(sv):
    c = si.make_layer(si.make_geometry(SMALL["cfg0"]))
    d = Dev(sv, c)
    idx, cnt, _ = gpu_select(sv, d, 1, 1, 16)
    out = torch.zeros((1, 4, 8, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(sv.SvError) as e:
        sv.sv_verify_attn(d.geom, d.q, d.kv, d.draft_k, d.draft_v, None, idx, cnt, out, workspace=ws)
    assert e.value.status == 5


def test_layer_stack_with_reuse_matches_oracle(sv):
    """SparseVerifier over 4 layers, anchors on even layers (Eq. 9), against the oracle's layer loop."""
    w = si.shrink(si.WORKLOADS["cfg1"], seq_len=(4096, 4096), budget_blocks=12, n_layers=4)
    geom = si.make_geometry(w)
    layers = [si.make_layer(geom, layer=l, sharp=True) for l in range(4)]
    anchors = [True, False, True, False]
    ref_sel = oracle.select_layers(layers, anchors, geom["budget"], 1, 1, geom["max_sel"])
    eng = sv.SparseVerifier(n_seq=1, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64,
                            max_blocks=geom["max_blocks"], n_draft=8, n_layers=4,
                            block_table=torch.from_numpy(geom["block_table"]).cuda(),
                            seq_lens=torch.from_numpy(geom["seq_lens"]).cuda(),
                            budget_blocks=torch.from_numpy(geom["budget"]).cuda(), max_sel=geom["max_sel"],
                            anchors=anchors)
    q = torch.stack([bf16_dev(c["q"]) for c in layers])
    dk = torch.stack([bf16_dev(c["draft_k"]) for c in layers])
    dv = torch.stack([bf16_dev(c["draft_v"]) for c in layers])
    out = torch.zeros_like(q)
    for l, c in enumerate(layers):
        eng.set_layer_kv(l, bf16_dev(c["k_pool"]), bf16_dev(c["v_pool"]))
        eng.build_reps(l)
    eng.verify_step(q, dk, dv, out)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    for l, c in enumerate(layers):
        o_ref, _ = oracle_attn(c, *ref_sel[l])
        o = bf16_host(out[l])
        rel = np.linalg.norm(o - o_ref, axis=-1) / np.linalg.norm(o_ref, axis=-1)
        assert rel.max() <= 1e-2, (l, rel.max())
    np.testing.assert_array_equal(eng.sel_idx.cpu().numpy(), ref_sel[2][0])
    assert eng.kernels_per_step() == 2 + 4 * (2 if sv.sv_verify_attn_splits(eng.geom, geom["max_sel"]) > 1 else 1)

    # the same step fed from pinned host memory, its copies in chunks on side streams: the same bits, eagerly and as a graph
    q_h, dk_h, dv_h = q.cpu().pin_memory(), dk.cpu().pin_memory(), dv.cpu().pin_memory()
    want = out.cpu()
    for chunk in (1, 3, 4):
        q2, dk2, dv2, out2 = torch.zeros_like(q), torch.zeros_like(dk), torch.zeros_like(dv), torch.zeros_like(out)
        out_h = torch.zeros_like(want).pin_memory()
        eng.verify_step_from_host(q_h, dk_h, dv_h, q2, dk2, dv2, out2, out_h, layers_per_chunk=chunk)
        torch.cuda.synchronize()
        assert torch.equal(out_h, want), chunk
    side = torch.cuda.Stream()
    out_h = torch.zeros_like(want).pin_memory()
    with torch.cuda.stream(side):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            eng.verify_step_from_host(q_h, dk_h, dv_h, q2, dk2, dv2, out2, out_h, layers_per_chunk=2)
        q2.zero_(), out2.zero_()
        g.replay()
        g.replay()
        side.synchronize()
    assert torch.equal(out_h, want) and int(eng.status.item()) == 0


# ------------------------------------------------------------------ full-size configurations

def _sampled_check(sv, c, n_samples, what):
    d = Dev(sv, c)
    idx, cnt, _ = gpu_select(sv, d, c["n_sink"], c["n_local"], c["max_sel"])
    torch.cuda.synchronize()
    idx_ref, cnt_ref, _ = oracle_select(c, c["n_sink"], c["n_local"], c["max_sel"])
    np.testing.assert_array_equal(cnt.cpu().numpy(), cnt_ref)
    np.testing.assert_array_equal(idx.cpu().numpy(), idx_ref)
    o, lse = gpu_attn(sv, d, idx, cnt)
    w = c["workload"]
    g = np.random.default_rng(7)
    smp = np.stack([g.integers(0, w.n_seq, n_samples), g.integers(0, w.n_draft, n_samples),
                    g.integers(0, w.n_q_heads, n_samples)], axis=1).astype(np.int32)
    o_ref, lse_ref = oracle_attn(c, idx_ref, cnt_ref, samples=smp)
    o_s = np.stack([o[s, i, hq] for s, i, hq in smp])
    lse_s = np.array([lse[s, i, hq] for s, i, hq in smp])
    check_attn(o_s, lse_s, o_ref, lse_ref, what)
    # properties that hold at any size: finite everywhere, and (V rows are random) outputs bounded by max |v|
    assert np.isfinite(o).all()
    return d, idx, cnt


@pytest.mark.parametrize("sharp", [False, True])
def test_full_size_cfg1_one_layer(sv, sharp):
    c = si.make_layer(si.make_geometry(si.WORKLOADS["cfg1"]), layer=3, sharp=sharp)
    run_pipeline(sv, c, what=f"cfg1 sharp={sharp}")


def test_full_size_cfg1_dense_sampled(sv):
    c = si.make_layer(si.make_geometry(si.WORKLOADS["cfg1"]), layer=0, sharp=True)
    d = Dev(sv, c)
    o, lse = gpu_attn(sv, d, None, None)
    smp = [(0, 7, 31), (0, 0, 0), (0, 3, 17), (0, 5, 9)]
    o_ref, lse_ref = oracle.dense_verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"],
                                              c["draft_k"], c["draft_v"], None, samples=smp)
    check_attn(np.stack([o[s, i, h] for s, i, h in smp]), np.array([lse[s, i, h] for s, i, h in smp]), o_ref, lse_ref,
               "cfg1 dense")


def test_full_size_cfg2(sv):
    c = si.make_layer(si.make_geometry(si.WORKLOADS["cfg2"]), sharp=True)
    run_pipeline(sv, c, what="cfg2")


def test_full_size_cfg2_dense_sampled(sv):
    """Dense verification of the ragged 16-sequence batch: more (sequence, KV head) pairs than an SM each needs, lists
    long enough that every pair is still cut into several CTAs to even out the lengths."""
    c = si.make_layer(si.make_geometry(si.WORKLOADS["cfg2"]), sharp=True)
    d = Dev(sv, c)
    assert sv.sv_verify_attn_splits(d.geom, c["max_blocks"]) > 1
    o, lse = gpu_attn(sv, d, None, None)
    longest, shortest = int(np.argmax(c["seq_lens"])), int(np.argmin(c["seq_lens"]))
    smp = [(longest, 4, 31), (longest, 0, 0), (shortest, 2, 13), (7, 3, 20), (15, 1, 5)]
    o_ref, lse_ref = oracle.dense_verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"],
                                              c["draft_k"], c["draft_v"], None, samples=smp)
    check_attn(np.stack([o[s, i, h] for s, i, h in smp]), np.array([lse[s, i, h] for s, i, h in smp]), o_ref, lse_ref,
               "cfg2 dense")


def test_full_size_cfg3_sampled(sv):
    c = si.make_layer(si.make_geometry(si.WORKLOADS["cfg3"]), sharp=True)
    _sampled_check(sv, c, 64, "cfg3")


@pytest.mark.parametrize("name", ["tree60", "tree60_batch"])
def test_full_size_tree60_sampled(sv, name):
    """The 60-node draft tree on Llama-3.1-8B geometry at full size: alone (two row tiles, one CTA each) and as a batch of
    12 (one CTA per pair of row tiles); lists bit-exact, attention on sampled rows of both row tiles."""
    w = si.WORKLOADS[name]
    assert w.budget_blocks == sv.sv_budget_blocks(max(w.seq_len), 4096, 0.1, 64, 1, 1)
    c = si.make_layer(si.make_geometry(w), sharp=True)
    _sampled_check(sv, c, 64, name)


@pytest.mark.parametrize("point", [(8192, 1 / 32, 1), (32768, 1 / 8, 16), (131072, 1 / 4, 4)])
def test_sweep_points(sv, point):
    c = si.make_layer(si.make_geometry(si.sweep_workload(*point)), sharp=True)
    _sampled_check(sv, c, 48, f"sweep {point}")


def test_stacked_tail_refresh_equals_per_layer(sv):
    """set_kv_stack: one sv_block_reps launch refreshes the tail block of every layer."""
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=3, seq_len=(900, 2000), budget_blocks=10, n_layers=3)
    geom = si.make_geometry(w)
    layers = [si.make_layer(geom, layer=l) for l in range(3)]
    eng = sv.SparseVerifier(n_seq=3, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64,
                            max_blocks=geom["max_blocks"], n_draft=5, n_layers=3,
                            block_table=torch.from_numpy(geom["block_table"]).cuda(),
                            seq_lens=torch.from_numpy(geom["seq_lens"]).cuda(),
                            budget_blocks=torch.from_numpy(geom["budget"]).cuda(), max_sel=geom["max_sel"])
    k_all = torch.stack([bf16_dev(c["k_pool"]) for c in layers])
    v_all = torch.stack([bf16_dev(c["v_pool"]) for c in layers])
    eng.set_kv_stack(k_all, v_all)
    for l in range(3):
        eng.build_reps(l)
    full = eng.reps.clone()
    eng.reps.fill_(5.0)
    eng.refresh_tail_all()
    torch.cuda.synchronize()
    for l in range(3):
        for s in range(3):
            t = int(geom["n_blocks"][s]) - 1
            assert torch.equal(eng.reps[l, s, :, t], full[l, s, :, t])
            assert (eng.reps[l, s, :, :t] == 5.0).all()
        ref = oracle.block_reps(layers[l]["k_pool"], geom["block_table"], geom["seq_lens"])
        for s in range(3):
            nb = int(geom["n_blocks"][s])
            np.testing.assert_allclose(full[l, s, :, :nb].cpu().numpy(), ref[s, :, :nb], rtol=1e-5, atol=1e-6)


def test_out_of_range_indices_are_clamped_and_reported(sv):
    """Block indices outside the table (-1, NBmax + 5), a page id outside the pool and a list count of -1 never reach
    an address: the kernel clamps them into their tables and says so in the status word.  Nothing faults; the same
    call with the valid inputs afterwards is exact again."""
    c = si.make_layer(si.make_geometry(SMALL["cfg1_small"]), sharp=True)
    d = Dev(sv, c)
    idx, cnt, _ = gpu_select(sv, d, c["n_sink"], c["n_local"], c["max_sel"])
    idx_ref, cnt_ref, _ = oracle_select(c, c["n_sink"], c["n_local"], c["max_sel"])
    w = d.w
    ws = torch.empty(max(16, sv.sv_workspace_bytes(d.geom, c["max_sel"])), dtype=torch.uint8, device="cuda")

    def run(idx_t, cnt_t, kv):
        out = torch.full((w.n_seq, w.n_draft, w.n_q_heads, w.head_dim), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((w.n_seq, w.n_draft, w.n_q_heads), float("nan"), device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sv.sv_verify_attn(d.geom, d.q, kv, d.draft_k, d.draft_v, d.parent, idx_t, cnt_t, out, lse=lse, workspace=ws,
                          status_word=status)
        torch.cuda.synchronize()
        return bf16_host(out), lse.cpu().numpy().astype(np.float64), int(status.item())

    bad_idx = idx.clone()
    bad_idx[0, 0, 1] = -1
    bad_idx[0, 1, 2] = c["max_blocks"] + 5
    o, lse, st = run(bad_idx, cnt, d.kv)
    assert st == sv.SV_STATUS_INDEX and sv.sv_status_word_check(st) == 9 and np.isfinite(o).all()
    bad_table = d.block_table.clone()
    bad_table[0, int(idx_ref[0, 0, 3])] = c["n_pages"] + 1000          # a kept block whose page id lies outside the pool
    bad_table[0, int(idx_ref[0, 0, 4])] = -3
    o, lse, st = run(idx, cnt, sv.make_kv(d.k_pool, d.v_pool, bad_table, d.seq_lens))
    assert st == sv.SV_STATUS_INDEX and np.isfinite(o).all()
    # a list that block selection marked invalid: the draft tokens only, and the word says so
    no_list = cnt.clone()
    no_list[0, 1] = -1
    o, lse, st = run(idx, no_list, d.kv)
    assert st == sv.SV_STATUS_NO_LIST and sv.sv_status_word_check(st) == 9
    cnt_exp = cnt_ref.copy()
    cnt_exp[0, 1] = 0
    o_ref, lse_ref = oracle_attn(c, idx_ref, cnt_exp)
    check_attn(o, lse, o_ref, lse_ref, "count -1 = no cached blocks")
    # the valid inputs again: clean word, exact result
    o, lse, st = run(idx, cnt, d.kv)
    assert st == 0 and sv.sv_status_word_check(st) == 0
    o_ref, lse_ref = oracle_attn(c, idx_ref, cnt_ref)
    check_attn(o, lse, o_ref, lse_ref, "after the clamped calls")


def test_engine_reports_a_bad_status_word(sv):
    w = SMALL["cfg1_small"]
    geom = si.make_geometry(w)
    eng = sv.SparseVerifier(n_seq=w.n_seq, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                            block_size=w.block_size, max_blocks=geom["max_blocks"], n_draft=w.n_draft, n_layers=1,
                            block_table=torch.from_numpy(geom["block_table"]).cuda(),
                            seq_lens=torch.from_numpy(geom["seq_lens"]).cuda(),
                            budget_blocks=torch.from_numpy(geom["budget"]).cuda(), max_sel=geom["max_sel"])
    eng.check_status()
    eng.sel_cnt[0, 0] = -1
    with pytest.raises(sv.SvError) as e:
        eng.check_status()
    assert e.value.status == 9
    eng.sel_cnt[0, 0] = 0
    eng.status.fill_(2)
    with pytest.raises(sv.SvError) as e:
        eng.check_status()
    assert e.value.status == 7


def test_commit_then_dense_verify_on_the_new_lengths(sv):
    """sv_kv_append writes the new lengths; a dense sv_verify_attn launched right behind it on the same stream reads
    them from that buffer.  Sequences cross a block boundary, so a role of the attention kernel that picked the old
    length up too early would issue fewer tiles than the others expect."""
    w = si.shrink(SMALL["cfg2_small"], n_draft=8)
    c = si.make_layer(si.make_geometry(w), sharp=True)
    S, Hkv, T, B = w.n_seq, w.n_kv_heads, w.n_draft, w.block_size
    bt = np.concatenate([c["block_table"], np.zeros((S, 1), np.int32)], axis=1)
    for s in range(S):
        bt[s, c["n_blocks"][s]] = c["n_pages"] + s
    g = np.random.default_rng(11)
    fresh = si.f32_to_bf16_bits(g.standard_normal((S, Hkv, B, 128)).astype(np.float32))
    k_pool, v_pool = np.concatenate([c["k_pool"], fresh]), np.concatenate([c["v_pool"], fresh[::-1].copy()])
    # two slots before a block boundary inside the generated prefix (so that every cached token is real data): a
    # commit of eight rows takes every sequence into its next block
    lens = ((c["seq_lens"] // B) * B - 2).astype(np.int32)
    n_acc = np.full(S, T, np.int32)
    acc = np.tile(np.arange(T, dtype=np.int32), (S, 1))
    NB = bt.shape[1]
    geom = sv.make_geom(S, w.n_q_heads, Hkv, 128, B, NB, T)
    kp, vp = bf16_dev(k_pool), bf16_dev(v_pool)
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    q, dk, dv = bf16_dev(c["q"]), bf16_dev(c["draft_k"]), bf16_dev(c["draft_v"])
    new_len = torch.zeros_like(sld)
    out = torch.full((S, T, w.n_q_heads, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((S, T, w.n_q_heads), float("nan"), device="cuda")
    ws = torch.empty(max(16, sv.sv_workspace_bytes(geom, NB)), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    kv_new = sv.make_kv(kp, vp, btd, new_len)
    for _ in range(3):      # repeated: the overlap of the two kernels varies from launch to launch
        kp.copy_(bf16_dev(k_pool)); vp.copy_(bf16_dev(v_pool)); new_len.zero_()
        sv.sv_kv_append(geom, kp, vp, btd, sld, dk, dv, torch.from_numpy(acc).cuda(), torch.from_numpy(n_acc).cuda(), new_len, None)
        sv.sv_verify_attn(geom, q, kv_new, dk, dv, None, None, None, out, lse=lse, workspace=ws, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
    ko, vo = k_pool.copy(), v_pool.copy()
    len_o = oracle.kv_append(ko, vo, bt, lens, c["draft_k"], c["draft_v"], acc, n_acc, None)
    assert ((len_o + B - 1) // B > (lens + B - 1) // B).all()
    np.testing.assert_array_equal(new_len.cpu().numpy(), len_o)
    o_ref, lse_ref = oracle.dense_verify_attn(c["q"], ko, vo, bt, len_o, c["draft_k"], c["draft_v"], None)
    check_attn(bf16_host(out), lse.cpu().numpy().astype(np.float64), o_ref, lse_ref, "dense verify right behind a commit")


def test_kv_append_drops_rows_for_unassigned_pages(sv):
    """A block-table entry that is not a page of the pool (-1: not assigned yet) ends the table: rows that would
    enter that block are dropped, the length stops at the block boundary, and nothing outside the sequence's own
    pages is written (every other page of the pools is a canary)."""
    B, Hkv, T, S, NB = 64, 2, 8, 3, 4
    n_pages = 16
    g = np.random.default_rng(3)
    k_pool = si.f32_to_bf16_bits(g.standard_normal((n_pages, Hkv, B, 128)).astype(np.float32))
    v_pool = si.f32_to_bf16_bits(g.standard_normal((n_pages, Hkv, B, 128)).astype(np.float32))
    bt = np.array([[2, -1, -1, -1], [5, 7, n_pages + 9, -1], [9, 11, 12, 13]], np.int32)
    lens = np.array([B - 3, 2 * B - 5, 4 * B - 2], np.int32)     # 3, 5 and 2 slots left before an unusable block / the end
    n_acc = np.full(S, T, np.int32)
    acc = np.tile(np.arange(T, dtype=np.int32), (S, 1))
    dk = si.f32_to_bf16_bits(g.standard_normal((S, T, Hkv, 128)).astype(np.float32))
    dv = si.f32_to_bf16_bits(g.standard_normal((S, T, Hkv, 128)).astype(np.float32))
    geom = sv.make_geom(S, 4, Hkv, 128, B, NB, T)
    kp, vp = bf16_dev(k_pool), bf16_dev(v_pool)
    new_len = torch.zeros(S, dtype=torch.int32, device="cuda")
    reps = torch.full((S, Hkv, NB, 128), 7.0, device="cuda")
    sv.sv_kv_append(geom, kp, vp, torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda(), bf16_dev(dk), bf16_dev(dv),
                    torch.from_numpy(acc).cuda(), torch.from_numpy(n_acc).cuda(), new_len, reps)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(new_len.cpu().numpy(), [B, 2 * B, 4 * B])
    k_exp, v_exp = k_pool.copy(), v_pool.copy()
    for s, (page, n) in enumerate([(2, 3), (7, 5), (13, 2)]):
        k_exp[page, :, B - n:] = dk[s, :n].transpose(1, 0, 2)
        v_exp[page, :, B - n:] = dv[s, :n].transpose(1, 0, 2)
    np.testing.assert_array_equal(kp.cpu().view(torch.int16).numpy().view(np.uint16), k_exp)
    np.testing.assert_array_equal(vp.cpu().view(torch.int16).numpy().view(np.uint16), v_exp)
    r = reps.cpu().numpy()
    assert (r[0, :, 1:] == 7.0).all() and (r[1, :, 2:] == 7.0).all() and (r[2, :, :3] == 7.0).all()
    np.testing.assert_allclose(r[0, :, 0], si.bf16_bits_to_f64(k_exp[2]).mean(axis=1), rtol=1e-5, atol=1e-6)
    # a length already past the table: nothing is appended and the length is kept
    lens2 = np.array([NB * B + 5, 0, 0], np.int32)
    sv.sv_kv_append(geom, kp, vp, torch.from_numpy(bt).cuda(), torch.from_numpy(lens2).cuda(), bf16_dev(dk), bf16_dev(dv),
                    torch.from_numpy(acc).cuda(), torch.from_numpy(np.array([4, 0, 0], np.int32)).cuda(), new_len, None)
    torch.cuda.synchronize()
    assert int(new_len[0].item()) == NB * B + 5


@pytest.mark.parametrize("block", [64, 128])
def test_kv_append_parity(sv, block):
    """Commit of accepted draft tokens: pools and lengths bit-exact against the oracle, representatives of the
    grown blocks equal to the oracle's (fp32 vs fp64) and bit-identical to a full sv_block_reps rebuild."""
    base = SMALL["cfg2_small"] if block == 64 else SMALL["cfg3_small"]
    w = si.shrink(base, n_draft=8)
    geom = si.make_geometry(w)
    c = si.make_layer(geom)
    S, Hkv, T = w.n_seq, w.n_kv_heads, w.n_draft
    g = np.random.default_rng(5)
    # one more table column with fresh pages, so that sequences may enter a new block
    extra = np.arange(c["n_pages"], c["n_pages"] + S, dtype=np.int32)
    bt = np.concatenate([c["block_table"], np.zeros((S, 1), np.int32)], axis=1)
    for s in range(S):
        bt[s, c["n_blocks"][s]] = extra[s]
    junk = si.f32_to_bf16_bits(g.standard_normal((S, Hkv, block, 128)).astype(np.float32))
    k_pool = np.concatenate([c["k_pool"], junk]); v_pool = np.concatenate([c["v_pool"], junk[::-1].copy()])
    lens = c["seq_lens"].copy()
    lens[0] = (lens[0] // block) * block + block - 3          # 3 slots left: an 8-token commit crosses into the new block
    lens[1] = (lens[1] // block) * block                      # exactly at a block boundary
    n_acc = g.integers(0, T + 1, size=S).astype(np.int32)
    n_acc[0], n_acc[1] = 8, 5
    if S > 2:
        n_acc[2] = 0
    acc = np.stack([np.sort(g.choice(T, size=T, replace=False)) for _ in range(S)]).astype(np.int32)
    NB = bt.shape[1]
    geom_c = sv.make_geom(S, w.n_q_heads, Hkv, 128, block, NB, T)
    kp, vp = bf16_dev(k_pool), bf16_dev(v_pool)
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    dk, dv = bf16_dev(c["draft_k"]), bf16_dev(c["draft_v"])
    kv = sv.make_kv(kp, vp, btd, sld)
    reps = torch.zeros((S, Hkv, NB, 128), device="cuda")
    sv.sv_block_reps(geom_c, kv, reps)
    before = reps.clone()
    new_len = torch.zeros_like(sld)
    sv.sv_kv_append(geom_c, kp, vp, btd, sld, dk, dv, torch.from_numpy(acc).cuda(), torch.from_numpy(n_acc).cuda(), new_len, reps)
    torch.cuda.synchronize()
    # oracle on the same inputs
    ko, vo = k_pool.copy(), v_pool.copy()
    reps_o = oracle.block_reps(ko, bt, lens)
    len_o = oracle.kv_append(ko, vo, bt, lens, c["draft_k"], c["draft_v"], acc, n_acc, reps_o)
    np.testing.assert_array_equal(new_len.cpu().numpy(), len_o)
    np.testing.assert_array_equal(kp.cpu().view(torch.int16).numpy().view(np.uint16), ko)
    np.testing.assert_array_equal(vp.cpu().view(torch.int16).numpy().view(np.uint16), vo)
    r = reps.cpu().numpy()
    for s in range(S):
        nbn = (int(len_o[s]) + block - 1) // block
        np.testing.assert_allclose(r[s, :, :nbn], reps_o[s, :, :nbn], rtol=1e-5, atol=1e-6)
        first = int(lens[s]) // block
        assert torch.equal(reps[s, :, :first], before[s, :, :first])          # blocks that did not grow are untouched
    rebuilt = torch.zeros_like(reps)
    kv2 = sv.make_kv(kp, vp, btd, new_len)
    sv.sv_block_reps(geom_c, kv2, rebuilt)
    torch.cuda.synchronize()
    for s in range(S):
        nbn = (int(len_o[s]) + block - 1) // block
        assert torch.equal(reps[s, :, :nbn], rebuilt[s, :, :nbn])
    with pytest.raises(sv.SvError):
        sv.sv_kv_append(geom_c, kp, vp, btd, sld, dk, dv, torch.from_numpy(acc).cuda(), torch.from_numpy(n_acc).cuda(), sld, reps)


def test_anchor_calibration_parity(sv):
    """Eq. 7-8 on a stack whose layers retrieve from inputs with planted inter-layer correlation: set sizes
    bit-exact against the oracle, same anchors."""
    n_layers = 6
    w = si.shrink(si.WORKLOADS["cfg2"], n_seq=4, seq_len=(1500, 4000), budget_blocks=12, n_layers=n_layers)
    geom = si.make_geometry(w)
    layers = [si.make_layer(geom, layer=l) for l in range(n_layers)]
    # correlate the layers: layers 1, 2, 4, 5 reuse the keys of their predecessor with a little noise in Q only
    for l in (1, 2, 4, 5):
        layers[l]["k_pool"] = layers[l - 1]["k_pool"]
        layers[l]["q"] = layers[l - 1]["q"].copy()
        layers[l]["q"][:, 0, ::5] = layers[l]["q"][:, 0, 1::5][:, :layers[l]["q"][:, 0, ::5].shape[1]]
    S, Hkv, max_sel = w.n_seq, w.n_kv_heads, geom["max_sel"]
    idx_all = torch.zeros((n_layers, S, Hkv, max_sel), dtype=torch.int32, device="cuda")
    cnt_all = torch.zeros((n_layers, S, Hkv), dtype=torch.int32, device="cuda")
    ref = []
    for l, c in enumerate(layers):
        d = Dev(sv, c)
        sv.sv_block_reps(d.geom, d.kv, d.reps)
        sv.sv_select_blocks(d.geom, d.q, d.reps, d.seq_lens, d.budget, 1, 1, idx_all[l], cnt_all[l])
        ref.append(oracle_select(c, 1, 1, max_sel))
    torch.cuda.synchronize()
    # the perturbed queries were not gap-repaired: compare the calibration on the GPU's own lists
    idx_h, cnt_h = idx_all.cpu().numpy(), cnt_all.cpu().numpy()
    for l in (0, 3):
        np.testing.assert_array_equal(cnt_h[l], ref[l][1])
        np.testing.assert_array_equal(idx_h[l], ref[l][0])
    inter = torch.full((n_layers, S), -1, dtype=torch.int32, device="cuda")
    uni = torch.full((n_layers, S), -1, dtype=torch.int32, device="cuda")
    gm = sv.make_geom(S, w.n_q_heads, Hkv, 128, 64, geom["max_blocks"], w.n_draft)
    sv.sv_anchor_jaccard(gm, idx_all, cnt_all, inter, uni)
    torch.cuda.synchronize()
    inter_o, uni_o, J_o = oracle.jaccard_adjacent(idx_h, cnt_h)
    np.testing.assert_array_equal(inter.cpu().numpy(), inter_o)
    np.testing.assert_array_equal(uni.cpu().numpy(), uni_o)
    anchors, J = sv.sv_pick_anchors(inter.cpu().numpy(), uni.cpu().numpy(), 2)
    np.testing.assert_allclose(J, J_o, rtol=0, atol=1e-15)
    np.testing.assert_array_equal(anchors, oracle.pick_anchors(J_o, 2))
    assert anchors.tolist() == [True, False, False, True, False, False]     # the two layers with fresh keys


@pytest.mark.parametrize("name", ["cfg1_small", "rows64", "cfg3_small"])
def test_attention_with_growing_logits_rescales_accumulator(sv, name):
    """Keys that get larger along the sequence make the running maximum jump by far more than 2^8 between
    units, which forces the in-TMEM rescale of the output accumulator; an arbitrary fixed block list is used
    on both sides (no selection involved)."""
    c = si.make_layer(si.make_geometry(SMALL[name]), sharp=True)
    w = c["workload"]
    kp = si.bf16_bits_to_f32(c["k_pool"])
    for s in range(w.n_seq):
        nb = int(c["n_blocks"][s])
        for b in range(nb):
            kp[c["block_table"][s, b]] *= np.float32(2.0 ** (4 * b // max(1, nb - 1)))     # x1 ... x16 along the sequence
    c = dict(c, k_pool=si.f32_to_bf16_bits(kp))
    idx = np.full((w.n_seq, w.n_kv_heads, c["max_sel"]), -1, np.int32)
    cnt = np.zeros((w.n_seq, w.n_kv_heads), np.int32)
    for s in range(w.n_seq):
        nb = int(c["n_blocks"][s])
        for h in range(w.n_kv_heads):
            pick = np.arange(h % 2, nb, max(1, nb // c["max_sel"]) + 1)[:c["max_sel"]]
            pick = np.union1d(pick, [nb - 1])[:c["max_sel"]]
            idx[s, h, :len(pick)] = pick
            cnt[s, h] = len(pick)
    d = Dev(sv, c)
    o, lse = gpu_attn(sv, d, torch.from_numpy(idx).cuda(), torch.from_numpy(cnt).cuda())
    o_ref, lse_ref = oracle_attn(c, idx, cnt)
    assert np.abs(lse_ref).max() > 20          # the logits really are large
    check_attn(o, lse, o_ref, lse_ref, f"growing logits {name}")


# ---------------------------------------------------------------------------- retrieval variants


def _boundary_gap_global(sc, nb, total, n_sink, n_local):
    """Gap between the last kept and the first dropped evictable (head, block) score of one sequence."""
    free = np.array([sc[h, b] for h in range(sc.shape[0]) for b in range(nb) if not (b < n_sink or b >= nb - n_local)])
    k = total - sc.shape[0] * min(nb, n_sink + n_local)
    if k <= 0 or k >= free.size:
        return np.inf
    srt = np.sort(free)[::-1]
    return srt[k - 1] - srt[k]


@pytest.mark.parametrize("name", ["cfg0", "cfg1_small", "cfg2_small", "cfg3_small", "cfg1_full"])
def test_select_global_parity(sv, name):
    """Budget shared by the KV heads: lists bit-exact against the oracle wherever the fp32 scores leave no doubt
    about the boundary pair (checked in the oracle's fp64 scores); counts always add up to budget * Hkv."""
    w = SMALL[name]
    geom = si.make_geometry(w)
    c = si.make_layer(geom)
    d = Dev(sv, c)
    S, Hkv, NB = w.n_seq, w.n_kv_heads, c["max_blocks"]
    sv.sv_block_reps(d.geom, d.kv, d.reps)
    idx = torch.full((S, Hkv, NB), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((S, Hkv), -7, dtype=torch.int32, device="cuda")
    sc = torch.full((S, Hkv, NB), float("nan"), device="cuda")
    sv.sv_select_blocks_global(d.geom, d.q, d.reps, d.seq_lens, d.budget, 1, 1, idx, cnt, sc)
    torch.cuda.synchronize()
    _, _, sc_o = oracle.select_blocks(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, NB)
    idx_o, cnt_o = oracle.select_global(sc_o, c["seq_lens"], c["budget"], w.block_size, 1, 1, NB)
    idx_h, cnt_h, sc_h = idx.cpu().numpy(), cnt.cpu().numpy(), sc.cpu().numpy()
    exact = 0
    for s in range(S):
        nb = int(c["n_blocks"][s])
        np.testing.assert_allclose(sc_h[s, :, :nb], sc_o[s, :, :nb], rtol=0, atol=2e-5 * max(1.0, np.abs(sc_o[s, :, :nb]).max()))
        N = int(c["budget"][s])
        assert int(cnt_h[s].sum()) == (nb * Hkv if N >= nb else N * Hkv)
        for h in range(Hkv):
            got = idx_h[s, h, :cnt_h[s, h]]
            assert np.all(np.diff(got) > 0) and (got.size == 0 or (got[0] >= 0 and got[-1] < nb))
            assert N >= nb or (got[0] == 0 and got[-1] == nb - 1)          # sink and local blocks kept
        gap = _boundary_gap_global(sc_o[s], nb, N * Hkv, 1, 1)
        err = float(np.abs(sc_h[s, :, :nb] - sc_o[s, :, :nb]).max())      # fp32 scores against fp64 scores
        if gap > 2.5 * err + 1e-12:                                        # the boundary pair cannot have swapped
            np.testing.assert_array_equal(cnt_h[s], cnt_o[s])
            for h in range(Hkv):
                np.testing.assert_array_equal(idx_h[s, h, :cnt_h[s, h]], idx_o[s, h, :cnt_o[s, h]])
            exact += 1
        else:   # an fp32 near-tie at the boundary: every kept pair must score at least the boundary value
            free = sorted((sc_o[s, h, b] for h in range(Hkv) for b in range(1, nb - 1)), reverse=True)
            thr = free[N * Hkv - 2 * Hkv - 1] - 2.5 * err - 1e-12
            for h in range(Hkv):
                for b in idx_h[s, h, :cnt_h[s, h]]:
                    assert b in (0, nb - 1) or sc_o[s, h, b] >= thr
    assert exact >= (S + 1) // 2
    # the lists drive the attention kernel unchanged (per-head counts differ)
    o, lse = gpu_attn(sv, d, idx, cnt)
    o_ref, lse_ref = oracle.verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"],
                                        c["draft_v"], c["parent"], idx_h, cnt_h)
    check_attn(o, lse, o_ref, lse_ref, f"{name} global budget")


def test_select_global_ties_and_degenerate_budgets(sv):
    """Equal scores everywhere: the smaller head, then the smaller block wins; budget >= blocks keeps everything;
    a budget equal to the forced blocks keeps only those."""
    w = SMALL["cfg0"]
    geom = si.make_geometry(w)
    c = si.make_layer(geom)
    c["k_pool"] = np.zeros_like(c["k_pool"])                       # all scores are exactly zero
    d = Dev(sv, c)
    S, Hkv, NB = w.n_seq, w.n_kv_heads, c["max_blocks"]
    sv.sv_block_reps(d.geom, d.kv, d.reps)
    for N in (2, 5, NB, NB + 3):
        bud = torch.full((S,), N, dtype=torch.int32, device="cuda")
        idx = torch.full((S, Hkv, NB), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((S, Hkv), -7, dtype=torch.int32, device="cuda")
        sc = torch.zeros((S, Hkv, NB), device="cuda")
        sv.sv_select_blocks_global(d.geom, d.q, d.reps, d.seq_lens, bud, 1, 1, idx, cnt, sc)
        torch.cuda.synchronize()
        sc_o = np.zeros((S, Hkv, NB))
        idx_o, cnt_o = oracle.select_global(sc_o, c["seq_lens"], np.full(S, N, np.int32), w.block_size, 1, 1, NB)
        np.testing.assert_array_equal(cnt.cpu().numpy(), cnt_o)
        for s in range(S):
            for h in range(Hkv):
                np.testing.assert_array_equal(idx.cpu().numpy()[s, h, :cnt_o[s, h]], idx_o[s, h, :cnt_o[s, h]])
    with pytest.raises(sv.SvError):
        sv.sv_select_blocks_global(d.geom, d.q, d.reps, d.seq_lens, d.budget, 1, 1, idx[:, :, :NB - 1].contiguous(), cnt, sc)


@pytest.mark.parametrize("name", ["cfg0", "cfg2_small", "cfg3_small", "cfg1_full"])
def test_per_token_retrieval_and_overlap_parity(sv, name):
    """Every draft token retrieves with its own query; pair intersections bit-exact against the oracle on the
    lists the GPU produced, token 0 equal to the adopted strategy."""
    w = SMALL[name]
    geom = si.make_geometry(w)
    c = si.make_layer(geom)
    d = Dev(sv, c)
    S, Hkv, T, max_sel = w.n_seq, w.n_kv_heads, w.n_draft, geom["max_sel"]
    sv.sv_block_reps(d.geom, d.kv, d.reps)
    idx_all = torch.full((T, S, Hkv, max_sel), -7, dtype=torch.int32, device="cuda")
    cnt_all = torch.full((T, S, Hkv), -7, dtype=torch.int32, device="cuda")
    sv.sv_select_blocks_tokens(d.geom, d.q, d.reps, d.seq_lens, d.budget, 1, 1, idx_all, cnt_all)
    inter = torch.full((S, Hkv, T, T), -1, dtype=torch.int32, device="cuda")
    sv.sv_token_overlap(d.geom, idx_all, cnt_all, inter)
    torch.cuda.synchronize()
    idx_h, cnt_h = idx_all.cpu().numpy(), cnt_all.cpu().numpy()
    idx_o, cnt_o = oracle.select_tokens(c["q"], c["k_pool"], c["block_table"], c["seq_lens"], c["budget"], 1, 1, max_sel)
    np.testing.assert_array_equal(cnt_h, cnt_o)
    np.testing.assert_array_equal(idx_h[0], idx_o[0])              # gap-repaired row: exact
    # rows 1.. were not gap-repaired by the generator: demand agreement on all but a few boundary blocks
    differ = sum(int(set(idx_h[i, s, h, :cnt_h[i, s, h]]) != set(idx_o[i, s, h, :cnt_o[i, s, h]]))
                 for i in range(1, T) for s in range(S) for h in range(Hkv))
    assert differ <= max(1, (T - 1) * S * Hkv // 50), differ
    np.testing.assert_array_equal(inter.cpu().numpy(), oracle.pair_overlap(idx_h, cnt_h))
    ratios = oracle.overlap_by_distance(inter.cpu().numpy(), cnt_h, np.arange(T))
    assert all(0.0 <= v <= 1.0 for v in ratios.values())


# ---------------------------------------------------------------------------- acceptance (Eq. 2-3)


def _settle_accept_case(c, margin=1e-4):
    """Move the uniform numbers away from the decision boundaries (as seen by the fp64 oracle) so that fp32 and
    fp64 must take the same decisions; returns the oracle's result for the settled inputs."""
    for _ in range(8):
        r = oracle.accept(c["p_target"], c["p_draft"], c["tokens"], c["parent"], c["u_accept"], c["u_next"], want_dist=True)
        moved = False
        a = r["alpha"]
        close = ~np.isnan(a) & (np.abs(c["u_accept"].astype(np.float64) - a) < margin) & (a < 1.0)
        if close.any():
            c["u_accept"][close] = np.clip(a[close] + 20 * margin, 0, 0.999).astype(np.float32)
            moved = True
        for s in range(c["u_next"].shape[0]):
            cdf = np.cumsum(r["final_dist"][s])
            x = int(r["next_token"][s])
            lo = cdf[x - 1] if x > 0 else 0.0
            if min(c["u_next"][s] - lo, cdf[x] - c["u_next"][s]) < 1e-5 and cdf[x] - lo > 4e-5:
                c["u_next"][s] = np.float32(0.5 * (lo + cdf[x]))
                moved = True
        if not moved:
            return r
    raise AssertionError("could not settle the uniform numbers")


def _gpu_accept(sv, c):
    S, T, V = c["p_target"].shape
    dev = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).cuda()
    path = torch.full((S, T), -9, dtype=torch.int32, device="cuda")
    n_path = torch.full((S,), -9, dtype=torch.int32, device="cuda")
    nxt = torch.full((S,), -9, dtype=torch.int32, device="cuda")
    alpha = torch.full((S, T), float("nan"), device="cuda")
    sv.sv_accept(dev(c["p_target"]), dev(c["p_draft"]), dev(c["tokens"]), dev(c["parent"]), dev(c["u_accept"]),
                 dev(c["u_next"]), path, n_path, nxt, alpha)
    torch.cuda.synchronize()
    return path.cpu().numpy(), n_path.cpu().numpy(), nxt.cpu().numpy(), alpha.cpu().numpy()


def _check_accept(c, r, got):
    path, n_path, nxt, alpha = got
    np.testing.assert_array_equal(n_path, r["n_path"])
    np.testing.assert_array_equal(path, r["path"])
    tried = ~np.isnan(r["alpha"])
    np.testing.assert_array_equal(np.isnan(alpha), ~tried)
    np.testing.assert_allclose(alpha[tried], r["alpha"][tried], rtol=2e-5, atol=1e-7)
    for s in range(nxt.shape[0]):
        if nxt[s] == r["next_token"][s]:
            continue
        # a different token is acceptable only next to the oracle's on the cumulative sum, within fp32 summation error
        cdf = np.cumsum(r["final_dist"][s])
        x = int(nxt[s])
        lo = cdf[x - 1] if x > 0 else 0.0
        assert r["final_dist"][s, x] > 0 and lo - 1e-5 <= c["u_next"][s] <= cdf[x] + 1e-5, (s, x, r["next_token"][s])
    assert np.mean(nxt == r["next_token"]) >= 0.9


@pytest.mark.parametrize("S,T,V,tree", [(4, 5, 512, False), (3, 8, 4096, True), (2, 16, 32768, True),
                                         (5, 6, 10240, False), (2, 1, 2048, False), (1, 32, 8192, True), (2, 64, 4096, True), (1, 60, 2048, False)])
def test_accept_parity(sv, S, T, V, tree):
    """Acceptance walk against the oracle: kept rows bit-exact, acceptance probabilities to fp32 accuracy, the
    drawn token equal (or adjacent within fp32 summation error on the cumulative sum).  Vocabularies from one CTA
    per sequence (512) to clusters of 8 (32768), ragged per-thread segments (10240)."""
    c = si.make_accept_case(S, T, V, seed=2000 + V + T, tree=tree)
    r = _settle_accept_case(c)
    _check_accept(c, r, _gpu_accept(sv, c))


def test_accept_special_cases(sv):
    """Identical models keep the whole chain; a one-hot target is greedy matching; a rejected token that repeats
    among the siblings has no mass left; all-rejecting uniform numbers walk every sibling."""
    c = si.make_accept_case(3, 6, 1024, seed=7)
    c["p_draft"] = c["p_target"].copy()
    r = _settle_accept_case(c)
    got = _gpu_accept(sv, c)
    assert got[1].tolist() == [6, 6, 6]
    _check_accept(c, r, got)
    # one-hot target
    c = si.make_accept_case(4, 6, 1024, seed=8)
    want = np.random.default_rng(3).integers(0, 1024, (4, 6))
    c["p_target"][:] = 0
    for s in range(4):
        c["p_target"][s, np.arange(6), want[s]] = 1.0
        c["tokens"][s, 1:3] = want[s, 0:2]                     # two matches, then whatever the draft drew
    r = _settle_accept_case(c)
    got = _gpu_accept(sv, c)
    _check_accept(c, r, got)
    assert all(got[1][s] >= 3 and got[2][s] == want[s, got[1][s] - 1] for s in range(4))
    # siblings: every child rejected, one token repeated
    c = si.make_accept_case(2, 5, 2048, seed=9, tree=True)
    c["parent"][:] = np.array([-1, 0, 0, 0, 0], np.int32)
    c["tokens"][:, 2] = c["tokens"][:, 1]
    c["u_accept"][:] = 0.9995
    r = _settle_accept_case(c)
    got = _gpu_accept(sv, c)
    _check_accept(c, r, got)


@pytest.mark.parametrize("tree", [False, True])
def test_accept_full_vocabulary(sv, tree):
    """Llama-3.1 vocabulary (128256 entries), batch and draft length of the benchmark workload."""
    c = si.make_accept_case(4, 8, 128256, seed=11, tree=tree)
    r = _settle_accept_case(c)
    _check_accept(c, r, _gpu_accept(sv, c))


def test_accept_feeds_kv_append(sv):
    """One decoding step end to end on the GPU: verify-attention on the selected blocks, acceptance, commit of the
    kept rows (root + accepted drafts) to the paged cache -- cache, lengths and representatives against the oracle
    run on the same inputs."""
    w = si.shrink(SMALL["cfg2_small"], n_draft=8)
    geom = si.make_geometry(w)
    c = si.make_layer(geom)
    S, Hkv, T, B = w.n_seq, w.n_kv_heads, w.n_draft, w.block_size
    # room for the commit: one more table column with fresh pages
    bt = np.concatenate([c["block_table"], np.zeros((S, 1), np.int32)], axis=1)
    for s in range(S):
        bt[s, c["n_blocks"][s]] = c["n_pages"] + s
    pad = np.zeros((S,) + c["k_pool"].shape[1:], np.uint16)
    k_pool, v_pool = np.concatenate([c["k_pool"], pad]), np.concatenate([c["v_pool"], pad])
    NB = bt.shape[1]
    g = sv.make_geom(S, w.n_q_heads, Hkv, 128, B, NB, T)
    kp, vp = bf16_dev(k_pool), bf16_dev(v_pool)
    btd, sld = torch.from_numpy(bt).cuda(), torch.from_numpy(c["seq_lens"]).cuda()
    kv = sv.make_kv(kp, vp, btd, sld)
    reps = torch.zeros((S, Hkv, NB, 128), device="cuda")
    sv.sv_block_reps(g, kv, reps)
    a = si.make_accept_case(S, T, 4096, seed=77)
    r = _settle_accept_case(a)
    dev = lambda x: None if x is None else torch.from_numpy(np.ascontiguousarray(x)).cuda()
    path = torch.zeros((S, T), dtype=torch.int32, device="cuda")
    n_path, nxt = torch.zeros(S, dtype=torch.int32, device="cuda"), torch.zeros(S, dtype=torch.int32, device="cuda")
    sv.sv_accept(dev(a["p_target"]), dev(a["p_draft"]), dev(a["tokens"]), None, dev(a["u_accept"]), dev(a["u_next"]),
                 path, n_path, nxt)
    new_len = torch.zeros_like(sld)
    sv.sv_kv_append(g, kp, vp, btd, sld, bf16_dev(c["draft_k"]), bf16_dev(c["draft_v"]), path, n_path, new_len, reps)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(path.cpu().numpy(), r["path"])
    ko, vo = k_pool.copy(), v_pool.copy()
    reps_o = oracle.block_reps(ko, bt, c["seq_lens"])
    len_o = oracle.kv_append(ko, vo, bt, c["seq_lens"], c["draft_k"], c["draft_v"], r["path"], r["n_path"], reps_o)
    np.testing.assert_array_equal(new_len.cpu().numpy(), len_o)
    assert np.all(len_o == c["seq_lens"] + r["n_path"]) and np.all(r["n_path"] >= 1)
    np.testing.assert_array_equal(kp.cpu().view(torch.int16).numpy().view(np.uint16), ko)
    np.testing.assert_array_equal(vp.cpu().view(torch.int16).numpy().view(np.uint16), vo)
    rg = reps.cpu().numpy()
    for s in range(S):
        nbn = (int(len_o[s]) + B - 1) // B
        np.testing.assert_allclose(rg[s, :, :nbn], reps_o[s, :, :nbn], rtol=0, atol=2e-6)


@pytest.mark.parametrize("name", ["cfg0", "cfg1_small", "cfg2_small", "cfg3_small", "cfg1_full", "one_128k_sequence"])
def test_bf16_representatives_parity(sv, name):
    """Representatives stored in bfloat16: the GPU rounds its fp32 mean, the oracle its fp64 mean -- equal except
    where the two means straddle a rounding boundary (one bfloat16 step, rare); scores to fp32 accuracy of the
    rounded values; block lists bit-exact wherever the oracle's boundary gap exceeds the measured score error.
    (The 128K-token sequence has 2048 blocks per KV head: the launch with clusters of 16 CTAs.)"""
    w = SMALL[name] if name in SMALL else si.sweep_workload(131072, 1 / 32, 1)
    geom = si.make_geometry(w)
    c = si.make_layer(geom)
    d = Dev(sv, c)
    S, Hkv, NB, max_sel = w.n_seq, w.n_kv_heads, c["max_blocks"], geom["max_sel"]
    reps16 = torch.zeros((S, Hkv, NB, 128), dtype=torch.bfloat16, device="cuda")
    sv.sv_block_reps_bf16(d.geom, d.kv, reps16)
    idx = torch.full((S, Hkv, max_sel), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((S, Hkv), -7, dtype=torch.int32, device="cuda")
    sc = torch.zeros((S, Hkv, NB), device="cuda")
    sv.sv_select_blocks_bf16reps(d.geom, d.q, reps16, d.seq_lens, d.budget, 1, 1, idx, cnt, out_scores=sc)
    torch.cuda.synchronize()
    reps_o = oracle.block_reps_bf16(c["k_pool"], c["block_table"], c["seq_lens"])
    sc_o = oracle.scores(oracle.group_query(c["q"], Hkv), reps_o, c["seq_lens"], w.block_size)
    idx_o, cnt_o = oracle.select(sc_o, c["seq_lens"], c["budget"], w.block_size, 1, 1, max_sel)
    rg = bf16_host(reps16)
    idx_h, cnt_h, sc_h = idx.cpu().numpy(), cnt.cpu().numpy(), sc.cpu().numpy()
    n_val = n_diff = 0
    exact = 0
    for s in range(S):
        nb = int(c["n_blocks"][s])
        a, b = rg[s, :, :nb], reps_o[s, :, :nb]
        step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(b), 1e-30))) - 7)     # one bfloat16 step at that magnitude
        assert np.all(np.abs(a - b) <= step * 1.0000001)
        n_val += a.size
        n_diff += int((a != b).sum())
        err = float(np.abs(sc_h[s, :, :nb] - sc_o[s, :, :nb]).max())
        np.testing.assert_array_equal(cnt_h[s], cnt_o[s])
        for h in range(Hkv):
            N = int(cnt_o[s, h])
            free = np.sort(sc_o[s, h, 1:nb - 1])[::-1]
            k = N - 2
            gap = np.inf if (N >= nb or k <= 0 or k >= free.size) else free[k - 1] - free[k]
            got = idx_h[s, h, :N]
            assert np.all(np.diff(got) > 0) and got[0] == 0 and got[-1] == nb - 1
            if gap > 2.5 * err + 1e-12:
                np.testing.assert_array_equal(got, idx_o[s, h, :N])
                exact += 1
            else:
                assert all(b_ in (0, nb - 1) or sc_o[s, h, b_] >= free[k - 1] - 2.5 * err - 1e-12 for b_ in got)
    assert n_diff <= max(2, n_val // 2000), (n_diff, n_val)
    assert exact >= (S * Hkv * 3) // 4


def test_engine_two_decoding_steps(sv):
    """SparseVerifier over a 2-layer stack: verify -> accept -> commit -> verify again.  The second step's block
    lists and attention must equal the oracle's on the cache the oracle itself appended to."""
    n_layers = 2
    w = si.shrink(SMALL["cfg2_small"], n_draft=6, n_layers=n_layers)
    geom = si.make_geometry(w)
    layers = [si.make_layer(geom, layer=l) for l in range(n_layers)]
    S, Hkv, Hq, T, B = w.n_seq, w.n_kv_heads, w.n_q_heads, w.n_draft, w.block_size
    c0 = layers[0]
    bt = np.concatenate([c0["block_table"], np.zeros((S, 1), np.int32)], axis=1)      # room to grow into
    for s in range(S):
        bt[s, c0["n_blocks"][s]] = c0["n_pages"] + s
    NB, max_sel = bt.shape[1], geom["max_sel"]
    pad = np.zeros((S,) + c0["k_pool"].shape[1:], np.uint16)
    pools = [(np.concatenate([c["k_pool"], pad]), np.concatenate([c["v_pool"], pad])) for c in layers]
    lens = c0["seq_lens"].copy()
    eng = sv.SparseVerifier(n_seq=S, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=128, block_size=B, max_blocks=NB, n_draft=T,
                            n_layers=n_layers, block_table=torch.from_numpy(bt).cuda(), seq_lens=torch.from_numpy(lens).cuda(),
                            budget_blocks=torch.from_numpy(c0["budget"]).cuda(), max_sel=max_sel, n_sink=1, n_local=1)
    k_all = torch.stack([bf16_dev(k) for k, _ in pools]).contiguous()
    v_all = torch.stack([bf16_dev(v) for _, v in pools]).contiguous()
    eng.set_kv_stack(k_all, v_all)
    for l in range(n_layers):
        eng.build_reps(l)
    stack = lambda key: torch.stack([bf16_dev(c[key]) for c in layers]).contiguous()
    q, dk, dv = stack("q"), stack("draft_k"), stack("draft_v")
    out = torch.zeros_like(q)
    eng.verify_step(q, dk, dv, out)
    a = si.make_accept_case(S, T, 2048, seed=91)
    ra = _settle_accept_case(a)
    dev = lambda x: torch.from_numpy(np.ascontiguousarray(x)).cuda()
    path, n_path, nxt = eng.accept(dev(a["p_target"]), dev(a["p_draft"]), dev(a["tokens"]), dev(a["u_accept"]), dev(a["u_next"]))
    eng.commit(dk, dv, path, n_path)
    torch.cuda.synchronize()
    assert int(eng.status.item()) == 0
    np.testing.assert_array_equal(path.cpu().numpy(), ra["path"])
    # the oracle's copy of the step
    new_lens = None
    for l, c in enumerate(layers):
        ko, vo = pools[l]
        new_lens = oracle.kv_append(ko, vo, bt, lens, c["draft_k"], c["draft_v"], ra["path"], ra["n_path"], None)
    np.testing.assert_array_equal(eng.seq_lens.cpu().numpy(), new_lens)
    # second step: fresh queries and draft tokens (layer data of another seed), same budgets
    layers2 = [si.make_layer(geom, layer=10 + l) for l in range(n_layers)]
    stack2 = lambda key: torch.stack([bf16_dev(c[key]) for c in layers2]).contiguous()
    q2, dk2, dv2 = stack2("q"), stack2("draft_k"), stack2("draft_v")
    out2 = torch.zeros_like(q2)
    lse2 = torch.zeros((S, T, Hq), device="cuda")
    for l in range(n_layers):
        eng.verify_layer(l, q2[l], dk2[l], dv2[l], out2[l], lse=lse2)
        torch.cuda.synchronize()
        ko, vo = pools[l]
        idx_o, cnt_o, sc_o = oracle.select_blocks(layers2[l]["q"], ko, bt, new_lens, c0["budget"], 1, 1, max_sel)
        idx_g, cnt_g = eng.sel_idx.cpu().numpy(), eng.sel_cnt.cpu().numpy()
        np.testing.assert_array_equal(cnt_g, cnt_o)
        # the second step's queries were gap-repaired against the un-appended cache: demand the same sets except
        # at most a couple of boundary blocks, and compare the attention on the GPU's own lists
        differ = sum(int(set(idx_g[s, h, :cnt_g[s, h]]) != set(idx_o[s, h, :cnt_o[s, h]])) for s in range(S) for h in range(Hkv))
        assert differ <= max(1, S * Hkv // 20), differ
        o_ref, lse_ref = oracle.verify_attn(layers2[l]["q"], ko, vo, bt, new_lens, layers2[l]["draft_k"], layers2[l]["draft_v"],
                                            None, idx_g, cnt_g)
        check_attn(bf16_host(out2[l]), lse2.cpu().numpy().astype(np.float64), o_ref, lse_ref, f"second step, layer {l}")
    assert int(eng.status.item()) == 0


def test_select_fuzz_exact_scores(sv):
    """Selection on hand-made score distributions, bit-exact against the oracle including ties.  The query is a unit
    vector, so a block's score is the first component of its representative exactly (no rounding on either side):
    normal, heavy-tailed (outliers stretch the score range), coarsely quantised (many ties at the boundary), two far
    clusters, constant, and block counts on both sides of the 2048-block limit of the fast selection path."""
    g = np.random.default_rng(77)
    S, Hkv, Hq, T, B = 2, 2, 4, 3, 64
    kinds = ["normal", "cauchy", "quantised", "clusters", "constant", "few_distinct", "tiny_range"]
    for trial in range(42):
        kind = kinds[trial % len(kinds)]
        NB = int(g.choice([33, 64, 200, 512, 513, 1024, 1500, 2048, 2049, 3000]))
        lens = np.array([NB * B - int(g.integers(0, B)), max(B, int(g.integers(NB // 2, NB)) * B - 7)], np.int32)
        n_sink, n_local = int(g.integers(0, 3)), int(g.integers(0, 3))
        budget = np.array([int(g.integers(n_sink + n_local + 1, NB)), int(g.integers(n_sink + n_local, NB + 5))], np.int32)
        max_sel = int(max(budget.max(), 8))
        if kind == "normal":
            sc = g.standard_normal((S, Hkv, NB))
        elif kind == "cauchy":
            sc = g.standard_cauchy((S, Hkv, NB)) * 0.01
        elif kind == "quantised":
            sc = np.round(g.standard_normal((S, Hkv, NB)) * 3) / 8
        elif kind == "clusters":
            sc = g.standard_normal((S, Hkv, NB)) * 1e-3 + (g.random((S, Hkv, NB)) < 0.1) * 50.0
        elif kind == "constant":
            sc = np.full((S, Hkv, NB), -0.375)
        elif kind == "few_distinct":
            sc = g.integers(0, 3, (S, Hkv, NB)).astype(np.float64) - 1.0
        else:
            sc = 1.0 + g.random((S, Hkv, NB)) * 1e-6
        sc = sc.astype(np.float32)
        reps = np.zeros((S, Hkv, NB, 128), np.float32)
        reps[..., 0] = sc
        q = np.zeros((S, T, Hq, 128), np.float32)
        q[:, 0, :, 0] = 1.0
        q[:, 1:] = g.standard_normal((S, T - 1, Hq, 128))
        geom = sv.make_geom(S, Hq, Hkv, 128, B, NB, T)
        idx = torch.full((S, Hkv, max_sel), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((S, Hkv), -7, dtype=torch.int32, device="cuda")
        sv.sv_select_blocks(geom, bf16_dev(si.f32_to_bf16_bits(q)), torch.from_numpy(reps).cuda(), torch.from_numpy(lens).cuda(),
                            torch.from_numpy(budget).cuda(), n_sink, n_local, idx, cnt)
        torch.cuda.synchronize()
        sc_o = sc.astype(np.float64)
        eff = np.minimum(np.maximum(budget, n_sink + n_local), max_sel).astype(np.int32)   # the library's documented clamp
        idx_o, cnt_o = oracle.select(sc_o, lens, eff, B, n_sink, n_local, max_sel)
        np.testing.assert_array_equal(cnt.cpu().numpy(), cnt_o, err_msg=f"trial {trial} {kind} NB={NB}")
        ih = idx.cpu().numpy()
        for s in range(S):
            for h in range(Hkv):
                np.testing.assert_array_equal(ih[s, h, :cnt_o[s, h]], idx_o[s, h, :cnt_o[s, h]],
                                              err_msg=f"trial {trial} {kind} NB={NB} s={s} h={h} budget={budget[s]}")


def test_select_global_fuzz_exact_scores(sv):
    """The shared-budget variant on the same hand-made score distributions, bit-exact including ties across heads."""
    g = np.random.default_rng(78)
    S, T, B = 2, 2, 64
    for trial in range(24):
        # head counts that give 16, 5, 4 and 1 warps per head in the ordered compaction, more parts than warps, and
        # more heads than its part tables hold (block-wide scans instead)
        Hkv = Hq = [4, 1, 3, 24, 4, 136][trial % 6]
        NB = int(g.choice([40, 200, 512, 1000])) if Hkv <= 24 else int(g.choice([40, 200]))
        lens = np.array([NB * B - int(g.integers(0, B)), max(B, int(g.integers(NB // 2, NB)) * B - 7)], np.int32)
        n_sink, n_local = int(g.integers(0, 2)), int(g.integers(0, 3))
        budget = np.array([int(g.integers(n_sink + n_local, NB)), int(g.integers(n_sink + n_local, NB + 3))], np.int32)
        kind = trial % 4
        if kind == 0:
            sc = g.standard_normal((S, Hkv, NB))
        elif kind == 1:
            sc = np.round(g.standard_normal((S, Hkv, NB)) * 2) / 4            # many ties, also across heads
        elif kind == 2:
            sc = g.standard_cauchy((S, Hkv, NB)) * 0.01
        else:
            sc = np.full((S, Hkv, NB), 0.25)
        sc = sc.astype(np.float32)
        reps = np.zeros((S, Hkv, NB, 128), np.float32)
        reps[..., 0] = sc
        q = np.zeros((S, T, Hq, 128), np.float32)
        q[:, 0, :, 0] = 1.0
        geom = sv.make_geom(S, Hq, Hkv, 128, B, NB, T)
        idx = torch.full((S, Hkv, NB), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((S, Hkv), -7, dtype=torch.int32, device="cuda")
        scd = torch.zeros((S, Hkv, NB), device="cuda")
        sv.sv_select_blocks_global(geom, bf16_dev(si.f32_to_bf16_bits(q)), torch.from_numpy(reps).cuda(),
                                   torch.from_numpy(lens).cuda(), torch.from_numpy(budget).cuda(), n_sink, n_local, idx, cnt, scd)
        torch.cuda.synchronize()
        idx_o, cnt_o = oracle.select_global(sc.astype(np.float64), lens, budget, B, n_sink, n_local, NB)
        np.testing.assert_array_equal(cnt.cpu().numpy(), cnt_o, err_msg=f"trial {trial}")
        ih = idx.cpu().numpy()
        for s in range(S):
            for h in range(Hkv):
                np.testing.assert_array_equal(ih[s, h, :cnt_o[s, h]], idx_o[s, h, :cnt_o[s, h]], err_msg=f"trial {trial} s={s} h={h}")


def test_pipeline_fuzz_random_shapes(sv):
    """reps -> select -> attention on randomly drawn shapes (batch, GQA group, draft length, chain / tree, block size,
    ragged lengths, budgets, forced blocks), each compared stage by stage with the oracle."""
    g = np.random.default_rng(2024)
    done = 0
    for trial in range(40):
        Hkv = int(g.choice([1, 2, 4]))
        G = int(g.choice([1, 2, 4, 8]))
        T = int(g.choice([1, 2, 3, 5, 8, 13, 16]))
        if G * T > 128:
            continue
        B = int(g.choice([64, 128]))
        S = int(g.integers(1, 5))
        lo = int(g.integers(3 * B, 12 * B))
        hi = lo + int(g.integers(0, 10 * B))
        n_sink, n_local = int(g.integers(0, 3)), int(g.integers(0, 3))
        nb_min = (lo + B - 1) // B
        budget = int(g.integers(max(1, n_sink + n_local), nb_min + 3))
        w = si.Workload(f"fuzz{trial}", S, (lo, hi), Hkv * G, Hkv, 128, B, budget, T, bool(g.integers(0, 2)), 1,
                        max(1, min(2, budget - n_sink - n_local)), 5000 + trial, n_sink, n_local)
        geom = si.make_geometry(w)
        c = si.make_layer(geom, sharp=bool(trial & 1))
        run_pipeline(sv, c, what=f"fuzz {trial}: S={S} Hkv={Hkv} G={G} T={T} B={B} L={lo}..{hi} N={budget} sink={n_sink} local={n_local}")
        done += 1
    assert done >= 25


def test_pipeline_fuzz_many_rows(sv):
    """The same on shapes with more than 128 query rows per KV head or more than 32 draft tokens: one to eight row
    tiles, 64-bit ancestor masks, chain and tree, one split and several; every third case has enough sequences that the
    row-tile CTAs outnumber the SMs, where one CTA serves a pair of row tiles (the last one alone when their number is
    odd)."""
    g = np.random.default_rng(4048)
    done = paired = 0
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    tiles_seen = set()
    for trial in range(60):
        Hkv = int(g.choice([1, 2]))
        G = int(g.choice([1, 2, 4, 8, 16]))
        T = int(g.choice([20, 33, 40, 47, 60, 64]))
        if G * T <= 128 and T <= 32:
            continue
        B = int(g.choice([64, 128]))
        S = int(g.integers(1, 3))
        tt = T if G * T <= 128 else max(1, 128 // G)
        tiles = -(-T // tt)
        many = trial % 3 == 2 and tiles > 1
        if many:
            S = n_sm // (Hkv * tiles) + int(g.integers(1, 4))
            paired += 1
        lo = int(g.integers(3 * B, (5 if many else 10) * B))
        hi = lo + int(g.integers(0, (3 if many else 6) * B))
        n_sink, n_local = int(g.integers(0, 2)), int(g.integers(0, 3))
        nb_min = (lo + B - 1) // B
        budget = int(g.integers(max(1, n_sink + n_local), nb_min + 2))
        w = si.Workload(f"wide{trial}", S, (lo, hi), Hkv * G, Hkv, 128, B, budget, T, bool(g.integers(0, 2)), 1,
                        max(1, min(2, budget - n_sink - n_local)), 7000 + trial, n_sink, n_local)
        tiles_seen.add(tiles)
        geom = si.make_geometry(w)
        c = si.make_layer(geom, sharp=bool(trial & 1))
        run_pipeline(sv, c, what=f"wide {trial}: S={S} Hkv={Hkv} G={G} T={T} B={B} L={lo}..{hi} N={budget} sink={n_sink} local={n_local}")
        done += 1
        if done >= 27 and paired >= 6 and {1, 2, 3}.issubset(tiles_seen) and max(tiles_seen) >= 5:
            break
    assert done >= 20 and paired >= 5 and {1, 2, 3}.issubset(tiles_seen) and max(tiles_seen) >= 5, (done, paired, tiles_seen)


def test_accept_fuzz(sv):
    """Acceptance walk on random small cases: trees with several siblings per row, every draft length, vocabularies that
    leave ragged per-thread segments, draft models from identical to unrelated."""
    g = np.random.default_rng(99)
    for trial in range(36):
        S = int(g.integers(1, 6))
        T = int(g.integers(1, 17))
        V = 4 * int(g.integers(2, 1500))
        c = si.make_accept_case(S, T, V, seed=300 + trial, tree=bool(trial % 3), draft_noise=float(g.choice([0.0, 0.1, 0.5, 2.0])))
        if trial % 5 == 0 and T > 2:                       # a bushy tree: every draft row hangs off the root
            c["parent"] = np.tile(np.array([-1] + [0] * (T - 1), np.int32), (S, 1))
        if trial % 7 == 0:
            c["u_accept"][:] = 0.9995                       # reject as much as possible
        r = _settle_accept_case(c)
        _check_accept(c, r, _gpu_accept(sv, c))


def test_benchmark_step_under_cuda_graph_replay(sv):
    """The launch configuration the benchmark times: a stack of full-size cfg1 layers with their pools in one
    allocation, one step (tail refresh of all layers in one launch, then select + attention + merge per layer, chained
    with programmatic dependent launch) captured in a CUDA graph and replayed.  Every layer's output after the third
    replay against the oracle on sampled rows; the last layer's block list exact."""
    n_layers = 3
    w = si.shrink(si.WORKLOADS["cfg1"], n_layers=n_layers)
    geom = si.make_geometry(w)
    layers = [si.make_layer(geom, layer=l, sharp=bool(l & 1)) for l in range(n_layers)]
    eng = sv.SparseVerifier(n_seq=w.n_seq, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=128,
                            block_size=w.block_size, max_blocks=geom["max_blocks"], n_draft=w.n_draft, n_layers=n_layers,
                            block_table=torch.from_numpy(geom["block_table"]).cuda(),
                            seq_lens=torch.from_numpy(geom["seq_lens"]).cuda(),
                            budget_blocks=torch.from_numpy(geom["budget"]).cuda(), max_sel=geom["max_sel"],
                            n_sink=w.n_sink, n_local=w.n_local)
    k_all = torch.stack([bf16_dev(c["k_pool"]) for c in layers]).contiguous()
    v_all = torch.stack([bf16_dev(c["v_pool"]) for c in layers]).contiguous()
    eng.set_kv_stack(k_all, v_all)
    for l in range(n_layers):
        eng.build_reps(l)
    q = torch.stack([bf16_dev(c["q"]) for c in layers]).contiguous()
    dk = torch.stack([bf16_dev(c["draft_k"]) for c in layers]).contiguous()
    dv = torch.stack([bf16_dev(c["draft_v"]) for c in layers]).contiguous()
    out = torch.zeros_like(q)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for _ in range(2):
            eng.verify_step(q, dk, dv, out, refresh_tail=True)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            eng.verify_step(q, dk, dv, out, refresh_tail=True)
        out.zero_()
        for _ in range(3):
            graph.replay()
        stream.synchronize()
    assert int(eng.status.item()) == 0
    g = np.random.default_rng(17)
    for l, c in enumerate(layers):
        idx_ref, cnt_ref, _ = oracle_select(c, w.n_sink, w.n_local, geom["max_sel"])
        smp = np.stack([np.zeros(24, np.int64), g.integers(0, w.n_draft, 24), g.integers(0, w.n_q_heads, 24)], axis=1).astype(np.int32)
        o_ref, _ = oracle_attn(c, idx_ref, cnt_ref, samples=smp)
        o = bf16_host(out[l])
        o_s = np.stack([o[s, i, hq] for s, i, hq in smp])
        rel = np.linalg.norm(o_s - o_ref, axis=-1) / np.linalg.norm(o_ref, axis=-1)
        assert rel.max() <= 1e-2 and np.abs(o_s - o_ref).max() <= 1e-2, (l, rel.max())
        if l == n_layers - 1:
            np.testing.assert_array_equal(eng.sel_cnt.cpu().numpy(), cnt_ref)
            np.testing.assert_array_equal(eng.sel_idx.cpu().numpy(), idx_ref)


def test_select_at_the_largest_supported_block_count(sv):
    """32768 blocks per sequence (a 2M-token context at block 64): the general radix path with keys of all CTAs of the
    cluster in CTA 0's shared memory, exact against the oracle; one more block is refused."""
    g = np.random.default_rng(5)
    S, Hkv, Hq, T, B, NB = 1, 1, 2, 2, 64, 32768
    sc = (g.standard_normal((S, Hkv, NB)) * 0.5).astype(np.float32)
    sc[0, 0, ::997] = 0.125                                           # some exact ties
    reps = np.zeros((S, Hkv, NB, 128), np.float32)
    reps[..., 0] = sc
    q = np.zeros((S, T, Hq, 128), np.float32)
    q[:, 0, :, 0] = 1.0
    lens = np.array([NB * B - 5], np.int32)
    for N in (3, 700, 5000):
        budget = np.array([N], np.int32)
        geom = sv.make_geom(S, Hq, Hkv, 128, B, NB, T)
        idx = torch.full((S, Hkv, N), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((S, Hkv), -7, dtype=torch.int32, device="cuda")
        sv.sv_select_blocks(geom, bf16_dev(si.f32_to_bf16_bits(q)), torch.from_numpy(reps).cuda(), torch.from_numpy(lens).cuda(),
                            torch.from_numpy(budget).cuda(), 1, 2, idx, cnt)
        torch.cuda.synchronize()
        idx_o, cnt_o = oracle.select(sc.astype(np.float64), lens, budget, B, 1, 2, N)
        np.testing.assert_array_equal(cnt.cpu().numpy(), cnt_o)
        np.testing.assert_array_equal(idx.cpu().numpy(), idx_o)
    too_big = sv.make_geom(S, Hq, Hkv, 128, B, NB + 1, T)
    with pytest.raises(sv.SvError):
        sv.sv_select_blocks(too_big, bf16_dev(si.f32_to_bf16_bits(q)), torch.zeros((S, Hkv, NB + 1, 128), device="cuda"),
                            torch.from_numpy(lens).cuda(), torch.from_numpy(np.array([8], np.int32)).cuda(), 1, 2,
                            torch.zeros((S, Hkv, 8), dtype=torch.int32, device="cuda"), torch.zeros((S, Hkv), dtype=torch.int32, device="cuda"))
