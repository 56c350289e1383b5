"""Host-side checks that need no GPU: the library loads, exports every declared symbol, validates
arguments before touching the device, and its budget helper follows Eq. 6."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def svb():
    # build through the file path: importing the package would already load a stale library
    subprocess.run([sys.executable, os.path.join(ROOT, "paper_2512_21911_b200", "build.py")], check=True,
                   capture_output=True)
    import paper_2512_21911_b200.binding as b
    return b


def test_exports_every_declared_symbol(svb):
    header = open(os.path.join(ROOT, "include", "sv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(sv_[a-z0-9_]+)\s*\(", header))
    assert declared == set(svb.EXPORTS)
    lib = ctypes.CDLL(svb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_exports_nothing_else(svb):
    """The library's dynamic symbol table holds the entry points of sv.h and nothing more (no development hooks)."""
    import shutil
    import subprocess
    nm = shutil.which("nm")
    if nm is None:
        pytest.skip("binutils nm not available")
    out = subprocess.run([nm, "-D", "--defined-only", svb.LIB_PATH], capture_output=True, text=True, check=True).stdout
    names = {line.split()[-1] for line in out.splitlines() if line.strip()}
    assert names == set(svb.EXPORTS), names ^ set(svb.EXPORTS)


def test_strerror_texts(svb):
    texts = {svb._strerror(i) for i in range(10)}
    assert len(texts) == 10 and "ok" in texts and "unknown status" not in texts
    assert "scratch" in svb._strerror(8) and "index" in svb._strerror(9)
    assert set(svb.STATUS_NAMES) == set(range(10))
    assert svb._strerror(10) == svb._strerror(99) == "unknown status"


def test_status_word_check(svb):
    assert svb.sv_status_word_check(0) == 0
    for wait_bit in (1, 2, 4, 8, 16, 32):
        assert svb.sv_status_word_check(wait_bit) == 7
        assert svb.sv_status_word_check(wait_bit | svb.SV_STATUS_INDEX) == 7     # a give-up outranks a clamp
    assert svb.sv_status_word_check(svb.SV_STATUS_INDEX) == 9
    assert svb.sv_status_word_check(svb.SV_STATUS_NO_LIST) == 9
    assert svb.sv_status_word_check(1 << 20) == 7                                # unknown bits are not "ok"


def test_budget_matches_eq6_and_oracle(svb):
    for L in (100, 4096, 4097, 6300, 32768, 131072, 1000003):
        for L0 in (1024, 4096):
            for rho in (0.05, 0.1, 0.5):
                for B in (64, 128):
                    for forced in ((0, 0), (1, 1), (2, 4)):
                        assert svb.sv_budget_blocks(L, L0, rho, B, *forced) == oracle.budget_blocks(L, L0, rho, B, *forced)
    assert svb.sv_budget_blocks(32768, 4096, 0.1, 64) == 109


def test_argument_validation_without_device(svb):
    g = svb.make_geom(1, 8, 2, 128, 64, 64, 4)
    lib = svb._lib
    null_kv = svb.sv_kv(None, None, None, None, 1)
    assert lib.sv_block_reps(ctypes.byref(g), ctypes.byref(null_kv), 0, -1, None, None) == 1      # SV_ERR_NULL
    bad = svb.make_geom(1, 8, 3, 128, 64, 64, 4)
    assert lib.sv_block_reps(ctypes.byref(bad), ctypes.byref(null_kv), 0, -1, None, None) == 2    # SV_ERR_SHAPE
    for kw, code in ((dict(head_dim=64), 6), (dict(block_size=32), 6), (dict(n_draft=65), 6), (dict(n_draft=0), 2)):
        args = dict(n_seq=1, n_q_heads=8, n_kv_heads=2, head_dim=128, block_size=64, max_blocks=64, n_draft=4)
        args.update(kw)
        gg = svb.make_geom(**args)
        assert lib.sv_block_reps(ctypes.byref(gg), ctypes.byref(null_kv), 0, -1, None, None) == code
    big = svb.make_geom(1, 64, 2, 128, 64, 64, 64)       # G = 32: 4 draft tokens per row tile, 16 tiles
    assert lib.sv_block_reps(ctypes.byref(big), ctypes.byref(null_kv), 0, -1, None, None) == 6
    ok = svb.make_geom(1, 64, 2, 128, 64, 64, 8)         # 32 * 8 = 256 query rows per KV head: two row tiles
    assert lib.sv_block_reps(ctypes.byref(ok), ctypes.byref(null_kv), 0, -1, None, None) == 1      # only the pointers are missing
    # misaligned pool pointer
    kv = svb.sv_kv(0x1008, 0x2000, 0x3000, 0x4000, 4)
    assert lib.sv_block_reps(ctypes.byref(g), ctypes.byref(kv), 0, -1, 0x5000, None) == 3        # SV_ERR_ALIGN
    # select: outputs missing, forced blocks above max_sel, reuse without a previous list
    assert lib.sv_select_blocks(ctypes.byref(g), 0x1000, 0x2000, 0x3000, 0x4000, 1, 1, 0, None, None, None, None,
                                16, None, None) == 1
    assert lib.sv_select_blocks(ctypes.byref(g), 0x1000, 0x2000, 0x3000, 0x4000, 9, 9, 0, None, None, 0x5000,
                                0x6000, 16, None, None) == 4
    assert lib.sv_select_blocks(ctypes.byref(g), None, None, None, None, 1, 1, 1, None, None, 0x5000, 0x6000, 16,
                                None, None) == 1
    # retrieval variants: missing outputs, a list too narrow for one head to hold every block, too many pairs
    assert lib.sv_select_blocks_tokens(ctypes.byref(g), 0x1000, 0x2000, 0x3000, 0x4000, 1, 1, None, None, 16, None) == 1
    assert lib.sv_token_overlap(ctypes.byref(g), 0x1000, 0x2000, 16, None, None) == 1
    assert lib.sv_select_blocks_global(ctypes.byref(g), 0x1000, 0x2000, 0x3000, 0x4000, 1, 1, 0x5000, 0x6000, 64,
                                       None, None) == 1
    assert lib.sv_select_blocks_global(ctypes.byref(g), 0x1000, 0x2000, 0x3000, 0x4000, 1, 1, 0x5000, 0x6000, 63,
                                       0x7000, None) == 2
    wide = svb.make_geom(1, 32, 8, 128, 64, 8192, 4)
    assert lib.sv_select_blocks_global(ctypes.byref(wide), 0x1000, 0x2000, 0x3000, 0x4000, 1, 1, 0x5000, 0x6000, 8192,
                                       0x7000, None) == 6
    assert lib.sv_token_overlap(ctypes.byref(svb.make_geom(1, 32, 8, 128, 64, 32768, 32)), 0x1000, 0x2000, 16, 0x3000,
                                None) == 6
    # acceptance: missing outputs, too many rows, vocabulary not a multiple of 4, misaligned distributions
    acc = lambda S, T, V, pt=0x1000, out=0x7000: lib.sv_accept(S, T, V, pt, 0x2000, 0x3000, None, 0x4000, 0x5000, out,
                                                               0x8000, 0x9000, None, None)
    assert acc(1, 8, 1024, out=None) == 1
    assert acc(0, 8, 1024) == 2 and acc(1, 0, 1024) == 2 and acc(1, 8, 0) == 2
    assert acc(1, 65, 1024) == 6
    assert acc(1, 8, 1022) == 3 and acc(1, 8, 1024, pt=0x1004) == 3
    # attention: missing output
    kv = svb.sv_kv(0x1000, 0x2000, 0x3000, 0x4000, 4)
    assert lib.sv_verify_attn(ctypes.byref(g), 0x1000, ctypes.byref(kv), 0x1000, 0x1000, None, None, None, 0, 0.0,
                              None, None, None, 0, None, None) == 1


def test_workspace_size_formula(svb):
    g = svb.make_geom(1, 32, 8, 128, 64, 512, 8)
    splits = svb.sv_verify_attn_splits(g, 64)
    assert 1 <= splits <= 64
    assert svb.sv_workspace_bytes(g, 64) == 1 * 8 * splits * 32 * 130 * 4 + 256
    assert svb.sv_workspace_bytes(svb.make_geom(1, 8, 3, 128, 64, 64, 4), 16) == 0


def test_split_rule_on_a_148_sm_device(svb):
    """The split counts of the shapes the profiles quote (the library assumes 148 SMs when it has no device to ask, and a
    B200 has 148): few units unsplit; the benchmark layer 16 splits; 240-row trees one CTA per row tile while those fit
    the SMs (1 / 2 / 4 / 8 sequences: 9 / 4 / 2 / 1 splits -- with a pair of row tiles per CTA it would be 18 / 9 / 4 / 2),
    and no split once there are more row-tile CTAs than SMs; the workspace follows the split count."""
    assert svb.sv_verify_attn_splits(svb.make_geom(1, 32, 8, 128, 64, 128, 8), 4) == 1
    assert svb.sv_verify_attn_splits(svb.make_geom(1, 32, 8, 128, 64, 512, 8), 64) == 16
    for n_seq, want in ((1, 9), (2, 4), (4, 2), (8, 1), (12, 1), (24, 1)):
        g = svb.make_geom(n_seq, 32, 8, 128, 64, 512, 60)
        assert svb.sv_verify_attn_splits(g, 70) == want, n_seq
        assert svb.sv_workspace_bytes(g, 70) == (0 if want == 1 else n_seq * 8 * want * 240 * 130 * 4 + 256)


def test_pick_anchors_matches_oracle_on_host(svb):
    import numpy as np
    g = np.random.default_rng(2)
    uni = g.integers(5, 40, size=(12, 7)).astype(np.int32)
    inter = (uni * g.random((12, 7))).astype(np.int32)
    inter[0] = 0
    uni[0] = 0
    for K in (1, 5, 12):
        a, J = svb.sv_pick_anchors(inter, uni, K)
        Jo = np.concatenate([[0.0], (inter[1:] / uni[1:]).mean(axis=1)])
        np.testing.assert_allclose(J, Jo, rtol=0, atol=1e-15)
        np.testing.assert_array_equal(a, oracle.pick_anchors(Jo, K))
    with pytest.raises(svb.SvError):
        svb.sv_pick_anchors(inter, uni, 13)
