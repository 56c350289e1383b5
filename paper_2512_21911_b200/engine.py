"""SparseVerifier: runs block selection and sparse verification attention for a stack of layers.

A thin driver over the C-ABI calls: it owns the per-layer representatives, the shared block list,
the split-KV workspace and the outputs, and enqueues, per layer, ``sv_select_blocks`` (anchor
layers) or the reuse of the previous layer's list (Eq. 9), then ``sv_verify_attn``; after verification,
``accept`` (Eq. 2-3) and ``commit`` (append the kept rows to the cache) close the decoding step.  All compute
is in the library's kernels; this class only holds buffers and calls them in order.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as sv


class SparseVerifier:
    def __init__(self, *, n_seq: int, n_q_heads: int, n_kv_heads: int, head_dim: int, block_size: int,
                 max_blocks: int, n_draft: int, n_layers: int, block_table: torch.Tensor, seq_lens: torch.Tensor,
                 budget_blocks: torch.Tensor, max_sel: int, n_sink: int = 1, n_local: int = 1,
                 anchors: Optional[Sequence[bool]] = None, parent: Optional[torch.Tensor] = None,
                 device: str = "cuda"):
        self.geom = sv.make_geom(n_seq, n_q_heads, n_kv_heads, head_dim, block_size, max_blocks, n_draft)
        self.n_layers = n_layers
        self.block_table, self.seq_lens, self.budget, self.parent = block_table, seq_lens, budget_blocks, parent
        self.n_sink, self.n_local, self.max_sel = n_sink, n_local, max_sel
        self.anchors = list(anchors) if anchors is not None else [True] * n_layers
        assert self.anchors[0], "layer 0 has no preceding layer to reuse"
        dev = torch.device(device)
        self.reps = torch.zeros((n_layers, n_seq, n_kv_heads, max_blocks, head_dim), dtype=torch.float32, device=dev)
        self.sel_idx = torch.zeros((n_seq, n_kv_heads, max_sel), dtype=torch.int32, device=dev)
        self.sel_cnt = torch.zeros((n_seq, n_kv_heads), dtype=torch.int32, device=dev)
        self.workspace = torch.empty(max(16, sv.sv_workspace_bytes(self.geom, max_sel)), dtype=torch.uint8, device=dev)
        self.dense_workspace = None
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.kv: List[Optional[sv.sv_kv]] = [None] * n_layers
        self._pools = [None] * n_layers   # keep the tensors alive
        self._stack_kv = None
        self._copy_streams = None

    def set_layer_kv(self, layer: int, k_pool: torch.Tensor, v_pool: torch.Tensor) -> None:
        self._pools[layer] = (k_pool, v_pool)
        self.kv[layer] = sv.make_kv(k_pool, v_pool, self.block_table, self.seq_lens)

    def set_kv_stack(self, k_all: torch.Tensor, v_all: torch.Tensor) -> None:
        """All layers' pools in one allocation, bf16 [layers][n_pages][Hkv][B][D].  Besides the per-layer
        descriptors this builds a stacked view in which (layer, sequence) is the batch dimension, so that
        the tail-block refresh of every layer is a single sv_block_reps launch."""
        n_layers, n_pages = int(k_all.shape[0]), int(k_all.shape[1])
        assert n_layers == self.n_layers and k_all.is_contiguous() and v_all.is_contiguous()
        for l in range(n_layers):
            self.set_layer_kv(l, k_all[l], v_all[l])
        g = self.geom
        self._stack_offs = (torch.arange(n_layers, device=k_all.device, dtype=torch.int32) * n_pages).view(n_layers, 1, 1)
        self._stack_table = torch.empty((n_layers * g.n_seq, g.max_blocks), dtype=torch.int32, device=k_all.device)
        self._stack_pages = n_pages
        self.sync_block_table()
        self._stack_lens = self.seq_lens.repeat(n_layers).contiguous()
        self._stack_geom = sv.make_geom(g.n_seq * n_layers, g.n_q_heads, g.n_kv_heads, g.head_dim, g.block_size,
                                        g.max_blocks, g.n_draft)
        self._stack_pools = (k_all, v_all)
        self._stack_kv = sv.make_kv(k_all.view(n_layers * n_pages, *k_all.shape[2:]),
                                    v_all.view(n_layers * n_pages, *v_all.shape[2:]), self._stack_table,
                                    self._stack_lens)

    def sync_block_table(self) -> None:
        """Rebuild the stacked page table from block_table (call after assigning pages to a sequence; commit does it
        itself).  Entries that are not pages of a layer's pool stay invalid in every layer."""
        bt = self.block_table.unsqueeze(0)
        ok = (bt >= 0) & (bt < self._stack_pages)
        self._stack_table.copy_(torch.where(ok, bt + self._stack_offs, -1).reshape(self._stack_table.shape))

    def refresh_tail_all(self) -> None:
        """Recompute the representative of every sequence's last block in all layers (one launch)."""
        sv.sv_block_reps(self._stack_geom, self._stack_kv, self.reps.view(-1, *self.reps.shape[2:]), sv.SV_TAIL_BLOCK)

    def build_reps(self, layer: int, block_begin: int = 0, block_end: int = -1) -> None:
        """(Re)compute block representatives of a layer; a decoding loop only refreshes the tail block."""
        sv.sv_block_reps(self.geom, self.kv[layer], self.reps[layer], block_begin, block_end)

    def verify_layer(self, layer: int, q, draft_k, draft_v, out, lse=None, behind_own_layer: bool = False) -> None:
        """select (anchor) or reuse (non-anchor), then sparse verification attention, on the current stream.

        behind_own_layer: the kernel just before this call in the stream is the preceding layer's attention / merge
        (as inside verify_step), which writes neither the block list nor the cache: a layer that reuses the list
        then starts its gather while that kernel drains (sv_verify_attn_reused)."""
        if self.anchors[layer]:
            sv.sv_select_blocks(self.geom, q, self.reps[layer], self.seq_lens, self.budget, self.n_sink,
                                self.n_local, self.sel_idx, self.sel_cnt)
        else:   # Eq. 9: same list as the preceding layer; in place, so nothing is launched
            sv.sv_select_blocks(self.geom, None, None, None, None, self.n_sink, self.n_local, self.sel_idx,
                                self.sel_cnt, reuse_prev=True, prev_idx=self.sel_idx, prev_cnt=self.sel_cnt)
        attn = sv.sv_verify_attn_reused if (behind_own_layer and not self.anchors[layer]) else sv.sv_verify_attn
        attn(self.geom, q, self.kv[layer], draft_k, draft_v, self.parent, self.sel_idx, self.sel_cnt, out, lse=lse,
             workspace=self.workspace, status_word=self.status)

    def dense_layer(self, layer: int, q, draft_k, draft_v, out, lse=None) -> None:
        """Dense ("strict") verification attention over every cached block, for comparison."""
        if self.dense_workspace is None:
            n = max(16, sv.sv_workspace_bytes(self.geom, self.geom.max_blocks))
            self.dense_workspace = torch.empty(n, dtype=torch.uint8, device=self.workspace.device)
        sv.sv_verify_attn(self.geom, q, self.kv[layer], draft_k, draft_v, self.parent, None, None, out, lse=lse,
                          workspace=self.dense_workspace, status_word=self.status)

    def verify_step(self, q, draft_k, draft_v, out, refresh_tail: bool = False) -> None:
        """One verification step of the whole stack.  q/out: [layers][S][T][Hq][D]; draft_k/v: [layers][S][T][Hkv][D].

        refresh_tail: first recompute the representative of every sequence's last block (the block that
        grew when the previous step's accepted tokens were appended) -- one launch for all layers when the
        pools were given with set_kv_stack, else one per anchor layer."""
        if refresh_tail:
            if self._stack_kv is not None:
                self.refresh_tail_all()
            else:
                for l in range(self.n_layers):
                    if self.anchors[l]:
                        sv.sv_block_reps(self.geom, self.kv[l], self.reps[l], sv.SV_TAIL_BLOCK)
        for l in range(self.n_layers):
            self.verify_layer(l, q[l], draft_k[l], draft_v[l], out[l], behind_own_layer=l > 0)

    def verify_step_from_host(self, q_host, draft_k_host, draft_v_host, q, draft_k, draft_v, out, out_host,
                              layers_per_chunk=None, refresh_tail: bool = False) -> None:
        """verify_step with the step's inputs in pinned host memory and its outputs wanted there.  The copies go in chunks
        of a few layers (layers_per_chunk: one size, or a list of sizes) on two side streams: a chunk's layers start as soon as its inputs have arrived, its outputs leave
        while the next chunk computes, so only the first upload and the last download are not hidden behind kernels.
        q/draft_k/draft_v/out are the device staging tensors (shapes as for verify_step); the *_host tensors the pinned
        ones.  Returns with everything enqueued; the current stream ends behind the last download.  Capturable in a
        CUDA graph (the side streams fork from and join the current stream)."""
        main = torch.cuda.current_stream()
        if self._copy_streams is None:
            self._copy_streams = (torch.cuda.Stream(device=q.device), torch.cuda.Stream(device=q.device))
        s_in, s_out = self._copy_streams
        s_in.wait_stream(main)
        s_out.wait_stream(main)
        if layers_per_chunk is None:
            # two layers first and last (their upload / download is what nothing hides), the rest in two halves (every
            # chunk boundary costs the step a few microseconds): 32 layers measured 16.1 us/layer against 16.6 in chunks
            # of four and 18.5 with the copies whole
            mid = max(0, self.n_layers - 4)
            layers_per_chunk = [2, (mid + 1) // 2, mid // 2, 2] if self.n_layers > 4 else [self.n_layers]
        if isinstance(layers_per_chunk, int):
            sizes = [layers_per_chunk] * -(-self.n_layers // layers_per_chunk)
        else:   # a schedule: e.g. a small first and last chunk (their copies are the ones nothing hides), large ones between
            sizes = list(layers_per_chunk)
        chunks, c0 = [], 0
        for n in sizes:
            if c0 < self.n_layers and n > 0:
                chunks.append((c0, min(c0 + n, self.n_layers)))
                c0 += n
        if c0 < self.n_layers:
            chunks.append((c0, self.n_layers))
        arrived = []
        with torch.cuda.stream(s_in):
            for c0, c1 in chunks:
                q[c0:c1].copy_(q_host[c0:c1], non_blocking=True)
                draft_k[c0:c1].copy_(draft_k_host[c0:c1], non_blocking=True)
                draft_v[c0:c1].copy_(draft_v_host[c0:c1], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(s_in)
                arrived.append(ev)
        if refresh_tail:
            if self._stack_kv is not None:
                self.refresh_tail_all()
            else:
                for l in range(self.n_layers):
                    if self.anchors[l]:
                        sv.sv_block_reps(self.geom, self.kv[l], self.reps[l], sv.SV_TAIL_BLOCK)
        for (c0, c1), ev in zip(chunks, arrived):
            main.wait_event(ev)
            for l in range(c0, c1):
                # the kernel before a chunk's first layer is not this stream's previous layer alone (the upload joins there)
                self.verify_layer(l, q[l], draft_k[l], draft_v[l], out[l], behind_own_layer=l > c0)
            done = torch.cuda.Event()
            done.record(main)
            s_out.wait_event(done)
            with torch.cuda.stream(s_out):
                out_host[c0:c1].copy_(out[c0:c1], non_blocking=True)
        main.wait_stream(s_in)
        main.wait_stream(s_out)

    def accept(self, p_target, p_draft, tokens, u_accept, u_next):
        """Acceptance of the step's draft tokens (Eq. 2-3).  Returns (path [S][T], n_path [S], next_token [S]):
        the rows whose K/V enter the cache (root first) and the token drawn after the kept path."""
        S, T = int(self.geom.n_seq), int(self.geom.n_draft)
        dev = p_target.device
        path = torch.empty((S, T), dtype=torch.int32, device=dev)
        n_path = torch.empty((S,), dtype=torch.int32, device=dev)
        next_token = torch.empty((S,), dtype=torch.int32, device=dev)
        sv.sv_accept(p_target, p_draft, tokens, self.parent, u_accept, u_next, path, n_path, next_token)
        return path, n_path, next_token

    def commit(self, draft_k, draft_v, path, n_path) -> None:
        """Append the kept rows' K/V of every layer to the paged cache (sv_kv_append, which also refreshes the
        representatives of the blocks that grew: one launch for all layers when the pools were given with
        set_kv_stack, else one per layer) and advance the sequence lengths.  The block table
        must already hold pages for the blocks the sequences grow into.  draft_k/v: [layers][S][T][Hkv][D]."""
        if self._stack_kv is not None:   # one launch for all layers: (layer, sequence) is the batch dimension
            self.sync_block_table()
            L, g = self.n_layers, self.geom
            k_all, v_all = self._stack_pools
            new_len = torch.empty_like(self._stack_lens)
            sv.sv_kv_append(self._stack_geom, k_all.view(-1, *k_all.shape[2:]), v_all.view(-1, *v_all.shape[2:]),
                            self._stack_table, self._stack_lens, draft_k.reshape(L * g.n_seq, *draft_k.shape[2:]),
                            draft_v.reshape(L * g.n_seq, *draft_v.shape[2:]), path.repeat(L, 1), n_path.repeat(L), new_len,
                            self.reps.view(-1, *self.reps.shape[2:]))
            self._stack_lens.copy_(new_len)
            self.seq_lens.copy_(new_len[:g.n_seq])
            return
        new_len = torch.empty_like(self.seq_lens)
        for l in range(self.n_layers):
            k_pool, v_pool = self._pools[l]
            sv.sv_kv_append(self.geom, k_pool, v_pool, self.block_table, self.seq_lens, draft_k[l], draft_v[l], path,
                            n_path, new_len, self.reps[l])
        self.seq_lens.copy_(new_len)          # every layer has read the old lengths by now (same stream)

    def check_status(self) -> None:
        """Read the device status word back (this synchronises with the stream) and raise if a kernel gave up
        on a bounded wait, clamped a block index or page id, or met a list that block selection marked invalid
        (count -1).  The outputs written since the word was last zero are then invalid."""
        st = sv.sv_status_word_check(int(self.status.item()))
        if st == sv.SV_OK and int(self.sel_cnt.min().item()) < 0:
            st = 9   # SV_ERR_INDEX: a list marked invalid that no attention call has consumed yet
        if st != sv.SV_OK:
            raise sv.SvError(st, "SparseVerifier.check_status")

    def dense_step(self, q, draft_k, draft_v, out) -> None:
        for l in range(self.n_layers):
            self.dense_layer(l, q[l], draft_k[l], draft_v[l], out[l])

    def kernels_per_step(self, refresh_tail: bool = False, dense: bool = False) -> int:
        """Kernel launches of one step: tail refresh and select per anchor layer; attention (+ merge) per layer."""
        splits = sv.sv_verify_attn_splits(self.geom, self.geom.max_blocks if dense else self.max_sel)
        attn = self.n_layers * (2 if splits > 1 else 1)
        if dense:
            return attn
        refresh = 0 if not refresh_tail else (1 if self._stack_kv is not None else sum(self.anchors))
        return refresh + sum(self.anchors) + attn
