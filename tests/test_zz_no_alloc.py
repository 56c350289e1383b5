"""sv_verify_attn_noalloc: the variant of the attention call for callers that cannot allocate device
memory (a server whose HBM is fully reserved by its KV-cache pool, code running under another
component's allocator).  It keeps the split-KV partials in a scratch array built into the library
instead of a caller workspace.  Checked here, through the C ABI, against the ordinary entry point on
the same inputs (and against the CPU oracle), twice in a row (the array is shared by all calls and keeps the previous call's
contents, which must not matter).  This file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import sv_inputs as si

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()


def _host(t):
    return si.bf16_bits_to_f64(t.cpu().view(torch.int16).numpy().view(np.uint16))


def _case(sv, w, sharp, layer):
    c = si.make_layer(si.make_geometry(w), layer=layer, sharp=sharp)
    geom = sv.make_geom(w.n_seq, w.n_q_heads, w.n_kv_heads, w.head_dim, w.block_size, c["max_blocks"], w.n_draft)
    t = dict(q=_dev(c["q"]), k=_dev(c["k_pool"]), v=_dev(c["v_pool"]), dk=_dev(c["draft_k"]), dv=_dev(c["draft_v"]),
             bt=torch.from_numpy(c["block_table"]).cuda(), sl=torch.from_numpy(c["seq_lens"]).cuda(),
             bud=torch.from_numpy(c["budget"]).cuda(),
             parent=torch.from_numpy(c["parent"]).cuda() if c["parent"] is not None else None)
    kv = sv.make_kv(t["k"], t["v"], t["bt"], t["sl"])
    reps = torch.zeros((w.n_seq, w.n_kv_heads, c["max_blocks"], w.head_dim), device="cuda")
    idx = torch.zeros((w.n_seq, w.n_kv_heads, c["max_sel"]), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((w.n_seq, w.n_kv_heads), dtype=torch.int32, device="cuda")
    sv.sv_block_reps(geom, kv, reps)
    sv.sv_select_blocks(geom, t["q"], reps, t["sl"], t["bud"], w.n_sink, w.n_local, idx, cnt)
    return c, geom, t, kv, idx, cnt


def test_noalloc_matches_workspace_entry_point_twice():
    import paper_2512_21911_b200 as sv
    shapes = [si.shrink(si.WORKLOADS["cfg1"], seq_len=(8192, 8192), budget_blocks=24, n_layers=1),   # 24 splits' worth
              si.shrink(si.WORKLOADS["cfg1"], seq_len=(2500, 2500), budget_blocks=12, n_draft=16, n_layers=1, tree=True)]
    for call, (w, sharp) in enumerate(zip(shapes, (True, False))):
        c, geom, t, kv, idx, cnt = _case(sv, w, sharp, layer=call)
        assert sv.sv_verify_attn_splits(geom, c["max_sel"]) > 1          # the scratch is really used
        assert sv.sv_workspace_bytes(geom, c["max_sel"]) <= sv.SV_NOALLOC_SCRATCH_BYTES
        shape = (w.n_seq, w.n_draft, w.n_q_heads)
        out_ref = torch.zeros(shape + (w.head_dim,), dtype=torch.bfloat16, device="cuda")
        lse_ref = torch.zeros(shape, device="cuda")
        ws = torch.empty(sv.sv_workspace_bytes(geom, c["max_sel"]), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        sv.sv_verify_attn(geom, t["q"], kv, t["dk"], t["dv"], t["parent"], idx, cnt, out_ref, lse=lse_ref, workspace=ws,
                          status_word=status)
        out = torch.full_like(out_ref, float("nan"))
        lse = torch.full_like(lse_ref, float("nan"))
        sv.sv_verify_attn_noalloc(geom, t["q"], kv, t["dk"], t["dv"], t["parent"], idx, cnt, out, lse=lse,
                                  status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        o, o_ref = _host(out), _host(out_ref)
        assert np.isfinite(o).all()
        # the bar of the other attention tests: max-abs 1e-2, mean-abs 1e-3 (scaled for O(1) outputs), rel-L2 1e-2
        scale = max(1.0, float(np.abs(o_ref).max()))
        assert np.abs(o - o_ref).max() <= 1e-2 * scale and np.abs(o - o_ref).mean() <= 1e-3 * scale
        rel = np.linalg.norm(o - o_ref, axis=-1) / np.linalg.norm(o_ref, axis=-1)
        assert rel.max() <= 1e-2
        assert np.abs(lse.cpu().numpy() - lse_ref.cpu().numpy()).max() <= 1e-3
        # and against the oracle directly, on the lists the library selected
        o_cpu, lse_cpu = oracle.verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"],
                                            c["draft_v"], c["parent"], idx.cpu().numpy(), cnt.cpu().numpy())
        scale = max(1.0, float(np.abs(o_cpu).max()))
        assert np.abs(o - o_cpu).max() <= 1e-2 * scale and np.abs(o - o_cpu).mean() <= 1e-3 * scale
        assert (np.linalg.norm(o - o_cpu, axis=-1) / np.linalg.norm(o_cpu, axis=-1)).max() <= 1e-2
        assert np.abs(lse.cpu().numpy() - lse_cpu).max() <= 1e-3


def test_noalloc_runs_a_large_batch_that_needs_no_partials():
    """256 (sequence, KV head) pairs of 128 query rows: every SM has a pair and the lists are short, so one CTA per
    pair writes the output itself.  No partials exist, so the size of the built-in scratch does not matter and the
    call must run (counted as if it were split, the partials would be four times the scratch)."""
    import paper_2512_21911_b200 as sv
    w = si.shrink(si.WORKLOADS["cfg3"], n_seq=32, seq_len=(600, 1024), budget_blocks=5, planted=1)
    c, geom, t, kv, idx, cnt = _case(sv, w, True, layer=0)
    assert sv.sv_verify_attn_splits(geom, c["max_sel"]) == 1 and sv.sv_workspace_bytes(geom, c["max_sel"]) == 0
    rows = (w.n_q_heads // w.n_kv_heads) * w.n_draft
    assert w.n_seq * w.n_kv_heads * rows * 520 > sv.SV_NOALLOC_SCRATCH_BYTES
    shape = (w.n_seq, w.n_draft, w.n_q_heads)
    out = torch.full(shape + (w.head_dim,), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full(shape, float("nan"), device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.sv_verify_attn_noalloc(geom, t["q"], kv, t["dk"], t["dv"], t["parent"], idx, cnt, out, lse=lse, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    smp = [(s, i, hq) for s in (0, 17, 31) for i in (0, 7, 15) for hq in (0, 9, 63)]
    o_cpu, lse_cpu = oracle.verify_attn(c["q"], c["k_pool"], c["v_pool"], c["block_table"], c["seq_lens"], c["draft_k"],
                                        c["draft_v"], c["parent"], idx.cpu().numpy(), cnt.cpu().numpy(), samples=smp)
    o = _host(out)
    for n, (s_, i, hq) in enumerate(smp):
        assert np.linalg.norm(o[s_, i, hq] - o_cpu[n]) <= 1e-2 * np.linalg.norm(o_cpu[n])
        assert abs(float(lse[s_, i, hq]) - lse_cpu[n]) <= 1e-3


def test_noalloc_rejects_problems_beyond_the_built_in_scratch():
    import paper_2512_21911_b200 as sv
    # the long-context configuration (4 sequences x 8 KV heads x 4 splits x 128 query rows) needs ~8.5 MB of
    # partials: more than the 4 MiB built into the library, so the call must refuse and launch nothing
    geom = sv.make_geom(4, 64, 8, 128, 128, 1024, 16)
    assert sv.sv_workspace_bytes(geom, 32) > sv.SV_NOALLOC_SCRATCH_BYTES
    q = torch.zeros((4, 16, 64, 128), dtype=torch.bfloat16, device="cuda")
    kp = torch.zeros((8, 8, 128, 128), dtype=torch.bfloat16, device="cuda")
    bt = torch.zeros((4, 1024), dtype=torch.int32, device="cuda")
    sl = torch.zeros(4, dtype=torch.int32, device="cuda")
    dk = torch.zeros((4, 16, 8, 128), dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros((4, 8, 32), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    kv = sv.make_kv(kp, kp, bt, sl)
    out = torch.full_like(q, 3.0)
    with pytest.raises(sv.SvError) as e:
        sv.sv_verify_attn_noalloc(geom, q, kv, dk, dk, None, idx, cnt, out)
    assert e.value.status == 8 and "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert (out == 3.0).all()


def test_noalloc_runs_unsplit_where_only_the_balancing_split_would_not_fit():
    """Dense verification of the ragged 16-sequence batch: the ordinary entry point cuts every (sequence, KV head) list
    into several CTAs to even out the lengths, which needs more partials than the built-in scratch holds; every SM has
    a pair anyway, so the no-alloc call runs the same problem without that split instead of refusing it."""
    import paper_2512_21911_b200 as sv
    w = si.WORKLOADS["cfg2"]
    c, geom, t, kv, _, _ = _case(sv, w, True, layer=0)
    nb = c["max_blocks"]
    assert sv.sv_verify_attn_splits(geom, nb) > 1 and sv.sv_workspace_bytes(geom, nb) > sv.SV_NOALLOC_SCRATCH_BYTES
    shape = (w.n_seq, w.n_draft, w.n_q_heads)
    out_ref = torch.zeros(shape + (w.head_dim,), dtype=torch.bfloat16, device="cuda")
    lse_ref = torch.zeros(shape, device="cuda")
    ws = torch.empty(sv.sv_workspace_bytes(geom, nb), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sv.sv_verify_attn(geom, t["q"], kv, t["dk"], t["dv"], t["parent"], None, None, out_ref, lse=lse_ref, workspace=ws,
                      status_word=status)
    out = torch.full_like(out_ref, float("nan"))
    lse = torch.full_like(lse_ref, float("nan"))
    sv.sv_verify_attn_noalloc(geom, t["q"], kv, t["dk"], t["dv"], t["parent"], None, None, out, lse=lse, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o, o_ref = _host(out), _host(out_ref)
    assert np.isfinite(o).all()
    scale = max(1.0, float(np.abs(o_ref).max()))
    assert np.abs(o - o_ref).max() <= 1e-2 * scale and np.abs(o - o_ref).mean() <= 1e-3 * scale
    assert np.abs(lse.cpu().numpy() - lse_ref.cpu().numpy()).max() <= 1e-3
