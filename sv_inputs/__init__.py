"""Seeded synthetic inputs for the sparse verification attention path.

This module only *constructs inputs* (and names the workload shapes); it holds
no part of the method that is under test.  Both the CUDA library's tests and
the CPU oracle's tests are fed from here, so that the two sides see the same
bfloat16 bits.

Recipe (stand-in for the paper's long-context workloads: Llama-3.1-8B head
geometry, 4K-128K token prefixes, chain or tree drafts; the paper's datasets
and weights are not used):

* Q, K, V and the draft tokens' K/V are i.i.d. N(0, sigma^2) with
  sigma = 1/sqrt(128) (``sharp`` variant: sigma_q = sigma_k = sqrt(3), sigma_v = 1,
  which gives attention logits with a standard deviation of about 3).
* Per (sequence, KV head) a seeded set of "planted" blocks has every key
  shifted by ``1.5 * u``, ``u`` the unit vector along the mean of the first
  draft token's query over the GQA group, so that these blocks score far above
  the rest.
* Gap repair: block selection is an integer result decided by floating-point
  compares, so the inputs are built with a margin.  After bfloat16 rounding the
  block scores are evaluated in fp64; any block that is not among the kept ones
  but scores within ``delta`` of the last kept one has its keys nudged along
  ``-u`` until the gap between the last kept and the first evicted block is at
  least ``delta`` (= 2 % of the standard deviation of the unplanted blocks' scores).  The minimum gap is reported.
* Tensors are rounded to bfloat16 (round-to-nearest-even) and returned as
  uint16 bit patterns in the paged layout the library uses:
  ``pool[page][kv_head][token_in_block][dim]`` with a seeded page permutation.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Tuple

import numpy as np

__all__ = ["Workload", "WORKLOADS", "sweep_workload", "make_geometry", "make_layer", "f32_to_bf16_bits",
           "bf16_bits_to_f32", "bf16_bits_to_f64"]


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even.  Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


@dataclass(frozen=True)
class Workload:
    name: str
    n_seq: int                      # S
    seq_len: Tuple[int, int]        # prefix length L_s: (lo, hi) inclusive, lo == hi -> fixed
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block_size: int                 # B
    budget_blocks: int              # N kept blocks per (sequence, KV head)
    n_draft: int                    # T
    tree: bool                      # draft tree given as a parent array (else causal chain)
    n_layers: int
    planted: float                  # >= 1: count per (s, h); < 1: fraction of the blocks
    seed: int
    n_sink: int = 1
    n_local: int = 1

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


# The named configurations (shapes of the benchmark and parity cases).
WORKLOADS = {
    # tiny single-layer case
    "cfg0": Workload("cfg0", 1, (4096, 4096), 8, 2, 128, 64, 16, 4, False, 1, 6, 1000),
    # Llama-3.1-8B-shaped attention stack, 32K context, 4096-token budget
    "cfg1": Workload("cfg1", 1, (32768, 32768), 32, 8, 128, 64, 64, 8, False, 32, 0.05, 1001),
    # batched verification with ragged prefixes, 2048-token budget
    "cfg2": Workload("cfg2", 16, (4096, 16384), 32, 8, 128, 64, 32, 5, False, 1, 0.05, 1002),
    # long context, GQA 8, 16-node draft tree, 4096-token budget
    "cfg3": Workload("cfg3", 4, (131072, 131072), 64, 8, 128, 128, 32, 16, True, 1, 0.02, 1003),
    # the paper's verification shape (Section 2.2, Section 4.1): a 60-node draft tree on Llama-3.1-8B geometry, 240 query
    # rows per KV head; the budgets are Eq. 6 with rho = 0.1, L0 = 4K at 32768 and at 10000 cached tokens.  Alone, and
    # as a batch of 12 on ragged prefixes.
    "tree60": Workload("tree60", 1, (32768, 32768), 32, 8, 128, 64, 109, 60, True, 1, 0.05, 1060),
    "tree60_batch": Workload("tree60_batch", 12, (6000, 10000), 32, 8, 128, 64, 74, 60, True, 1, 0.05, 1061),
}


def sweep_workload(context: int, budget_frac: float, n_draft: int) -> Workload:
    """One point of the single-layer sweep: 32 query / 8 KV heads, block 64, batch 1."""
    nb = context // 64
    return Workload(f"sweep_L{context}_f{budget_frac:g}_T{n_draft}", 1, (context, context), 32, 8, 128, 64,
                    max(2, int(round(nb * budget_frac))), n_draft, False, 1, 0.05, 1004)


def _rng(seed: int, *key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, *key])))


def make_geometry(w: Workload, permute_pages: bool = True, spare_pages: int = 3) -> dict:
    """Layer-independent part of a case: lengths, page table, draft structure, budgets."""
    g = _rng(w.seed, 0xA11)
    lo, hi = w.seq_len
    seq_lens = (np.full(w.n_seq, lo) if lo == hi else g.integers(lo, hi + 1, size=w.n_seq)).astype(np.int32)
    B = w.block_size
    nb = (seq_lens.astype(np.int64) + B - 1) // B
    max_blocks = int(max(1, nb.max()))
    n_pages = int(nb.sum()) + spare_pages
    pages = g.permutation(n_pages) if permute_pages else np.arange(n_pages)
    block_table = np.zeros((w.n_seq, max_blocks), dtype=np.int32)
    o = 0
    for s in range(w.n_seq):
        block_table[s, : nb[s]] = pages[o : o + nb[s]]
        o += int(nb[s])
    parent = None
    if w.tree:
        parent = np.full((w.n_seq, w.n_draft), -1, dtype=np.int32)
        for s in range(w.n_seq):
            for i in range(1, w.n_draft):
                parent[s, i] = g.integers(0, i)
    budget = np.full(w.n_seq, w.budget_blocks, dtype=np.int32)
    return dict(workload=w, seq_lens=seq_lens, n_blocks=nb.astype(np.int32), max_blocks=max_blocks,
                n_pages=n_pages, block_table=block_table, parent=parent, budget=budget,
                n_sink=w.n_sink, n_local=w.n_local, max_sel=int(max(1, min(w.budget_blocks, max_blocks))))


def _forced_mask(nb: int, n_sink: int, n_local: int) -> np.ndarray:
    b = np.arange(nb)
    return (b < n_sink) | (b >= nb - n_local)


def _block_scores(kbits: np.ndarray, qbar: np.ndarray, L: int, B: int) -> np.ndarray:
    """fp64 scores of the blocks in ``kbits`` ([nb][B][D] bf16 bits, block 0 first) -- generator-side
    margin bookkeeping only."""
    nb = kbits.shape[0]
    k = bf16_bits_to_f32(kbits)
    cnt = np.minimum(B, L - np.arange(nb) * B).astype(np.float64)
    valid = (np.arange(B)[None, :] < cnt[:, None])
    sums = np.add.reduce(np.where(valid[:, :, None], k, np.float32(0)), axis=1, dtype=np.float64)
    return (sums / cnt[:, None]) @ qbar


def make_layer(geom: dict, layer: int = 0, sharp: bool = False, tail_fill: Optional[float] = 50.0,
               delta_rel: float = 0.02) -> dict:
    """Tensors of one layer of a case (see the module docstring for the recipe).

    Returns q, k_pool, v_pool, draft_k, draft_v as uint16 bf16 bits plus the geometry entries,
    ``min_gap`` (smallest kept-vs-evicted score gap over all (s, h)), ``delta`` (largest per-(s, h) margin
    asked for), ``min_gap_ratio`` (smallest gap / delta of any (s, h); >= 1 after repair) and ``planted``.
    ``tail_fill``: value written to K and V slots past the end of a sequence inside its last page
    (a correct kernel never lets them contribute); ``None`` writes NaN bit patterns.
    """
    w: Workload = geom["workload"]
    S, T, Hq, Hkv, D, B = w.n_seq, w.n_draft, w.n_q_heads, w.n_kv_heads, w.head_dim, w.block_size
    G = w.group
    sig_q = sig_k = np.sqrt(3.0) if sharp else 1.0 / np.sqrt(128.0)
    sig_v = 1.0 if sharp else 1.0 / np.sqrt(128.0)
    fill_bits = np.uint16(0x7FC0) if tail_fill is None else f32_to_bf16_bits(np.float32(tail_fill))[()]

    gq = _rng(w.seed, 1, layer)
    q = f32_to_bf16_bits((gq.standard_normal((S, T, Hq, D), dtype=np.float32) * np.float32(sig_q)))
    draft_k = f32_to_bf16_bits(gq.standard_normal((S, T, Hkv, D), dtype=np.float32) * np.float32(sig_k))
    draft_v = f32_to_bf16_bits(gq.standard_normal((S, T, Hkv, D), dtype=np.float32) * np.float32(sig_v))

    n_pages = geom["n_pages"]
    k_pool = np.empty((n_pages, Hkv, B, D), dtype=np.uint16)
    v_pool = np.empty((n_pages, Hkv, B, D), dtype=np.uint16)
    # spare pages hold junk that nothing may read
    k_pool[...] = fill_bits
    v_pool[...] = fill_bits

    min_gap = np.inf
    min_ratio = np.inf
    delta_used = 0.0
    planted_sets = {}
    for s in range(S):
        L = int(geom["seq_lens"][s])
        nb = int(geom["n_blocks"][s])
        if nb == 0:
            continue
        pages = geom["block_table"][s, :nb]
        N = int(min(geom["budget"][s], nb))
        forced = _forced_mask(nb, w.n_sink, w.n_local)
        cand = np.flatnonzero(~forced)
        need = N - int(forced.sum())
        n_plant = int(w.planted) if w.planted >= 1 else int(round(w.planted * nb))
        n_plant = min(n_plant, cand.size)
        tok_valid = (np.arange(nb * B) < L).reshape(nb, B)
        for h in range(Hkv):
            g = _rng(w.seed, 2, layer, s, h)
            k = g.standard_normal((nb, B, D), dtype=np.float32) * np.float32(sig_k)
            v = g.standard_normal((nb, B, D), dtype=np.float32) * np.float32(sig_v)
            qbar = bf16_bits_to_f64(q[s, 0, h * G:(h + 1) * G, :]).mean(axis=0)
            qn = float(np.linalg.norm(qbar))
            u = (qbar / qn).astype(np.float32)
            planted = np.sort(g.choice(cand, size=n_plant, replace=False)) if n_plant else np.zeros(0, np.int64)
            planted_sets[(s, h)] = planted
            # 1.5 (sharp: 2.0) lifts a planted block's score by shift * |qbar|: > 100 (sharp: ~9) score sigmas
            shift = np.float32(2.0 if sharp else 1.5)
            k[planted] += shift * u
            kb = f32_to_bf16_bits(k)
            if 0 < need < cand.size:
                sc = _block_scores(kb, qbar, L, B)
                plain = np.setdiff1d(cand, planted)
                delta = delta_rel * float(np.std(sc[plain if plain.size > 1 else cand]))
                delta_used = max(delta_used, delta)
                for _ in range(200):
                    order = cand[np.argsort(-sc[cand], kind="stable")]
                    s_last = sc[order[need - 1]]
                    rest = order[need:]
                    close = rest[sc[rest] > s_last - delta]
                    if close.size == 0:
                        break
                    k[close] -= np.float32(2.0 * delta / qn) * u
                    kb[close] = f32_to_bf16_bits(k[close])
                    cl_sorted = np.sort(close)
                    # recompute the nudged blocks only
                    for b in cl_sorted:
                        c = min(B, L - b * B)
                        sc[b] = (np.add.reduce(bf16_bits_to_f32(kb[b, :c]), axis=0, dtype=np.float64) / c) @ qbar
                else:
                    raise RuntimeError("gap repair did not converge")
                order = cand[np.argsort(-sc[cand], kind="stable")]
                gap = float(sc[order[need - 1]] - sc[order[need]])
                min_gap = min(min_gap, gap)
                min_ratio = min(min_ratio, gap / delta)
            vb = f32_to_bf16_bits(v)
            kb[~tok_valid] = fill_bits
            vb[~tok_valid] = fill_bits
            k_pool[pages, h] = kb
            v_pool[pages, h] = vb

    out = dict(geom)
    out.update(q=q, k_pool=k_pool, v_pool=v_pool, draft_k=draft_k, draft_v=draft_v, layer=layer,
               min_gap=min_gap, delta=delta_used, min_gap_ratio=min_ratio, planted=planted_sets, sharp=sharp)
    return out


def shrink(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (tests use smaller contexts of the same shape)."""
    return replace(w, **kw)


def make_accept_case(n_seq, n_draft, vocab, seed=2000, tree=False, temperature=0.35, draft_noise=0.2):
    """Seeded inputs for the acceptance step: target and draft distributions per row (softmax of correlated
    Gaussian logits, peaked like language-model outputs: `temperature` sharpens, `draft_noise` is how far the
    draft model's logits stray from the target's), draft tokens drawn from the draft distribution of their
    parent row, and the uniform numbers the step consumes.  Row 0 is the root.  float32 / int32 arrays."""
    g = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, n_seq, n_draft, vocab])))
    lt = g.standard_normal((n_seq, n_draft, vocab)) / temperature
    ld = lt + draft_noise * g.standard_normal((n_seq, n_draft, vocab)) / temperature

    def softmax(z):
        z = z - z.max(-1, keepdims=True)
        e = np.exp(z)
        return (e / e.sum(-1, keepdims=True)).astype(np.float32)

    p_target, p_draft = softmax(lt), softmax(ld)
    parent = np.full((n_seq, n_draft), -1, np.int32)
    for s in range(n_seq):
        for i in range(1, n_draft):
            parent[s, i] = g.integers(0, i) if tree else i - 1
    tokens = np.zeros((n_seq, n_draft), np.int32)
    for s in range(n_seq):
        tokens[s, 0] = g.integers(0, vocab)
        for i in range(1, n_draft):
            q = p_draft[s, parent[s, i]].astype(np.float64)
            tokens[s, i] = g.choice(vocab, p=q / q.sum())
    return dict(p_target=p_target, p_draft=p_draft, tokens=tokens, parent=parent if tree else None,
                u_accept=g.random((n_seq, n_draft), dtype=np.float32), u_next=g.random(n_seq, dtype=np.float32))
