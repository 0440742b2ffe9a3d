"""Device buffers of one layer and the call sequence of one layer-step.

Plumbing only (allocation through PyTorch, streams, events); every computation is one
of the C-ABI calls in `binding`.
"""
from __future__ import annotations

from typing import Optional

import torch

from .binding import PulseInfer


class LayerBuffers:
    """Everything one layer keeps on the device for a batch of offloaded sequences."""

    def __init__(self, pi: PulseInfer, batch: int, device="cuda", keep_scores: bool = False):
        c = pi.cfg
        i32 = dict(dtype=torch.int32, device=device)
        self.batch = batch
        self.digest = torch.zeros((batch, c.max_blocks, 2, c.head_dim), dtype=torch.bfloat16, device=device)
        self.block_table = torch.full((batch, c.max_blocks), -1, **i32)
        self.slot_block = torch.full((batch, c.pool_slots), -1, **i32)
        self.slot_stamp = torch.zeros((batch, c.pool_slots), **i32)
        self.pool = torch.zeros((batch, c.pool_slots, c.n_kv_heads, 2, c.block_tokens, c.head_dim),
                                dtype=torch.bfloat16, device=device)
        self.sel_blocks = torch.full((batch, c.budget_blocks), -1, **i32)
        self.sel_count = torch.zeros((batch,), **i32)
        self.sel_slots = torch.full((batch, c.budget_blocks), -1, **i32)
        self.recall_list = torch.zeros((batch, c.budget_blocks, 4), **i32)
        self.recall_count = torch.zeros((batch,), **i32)
        self.scores = torch.zeros((batch, c.max_blocks), dtype=torch.float32, device=device) if keep_scores else None


class RecallPath:
    """score/select -> diff -> recall on a side stream, attention on the caller's stream."""

    def __init__(self, pi: PulseInfer):
        self.pi = pi
        self.side = torch.cuda.Stream()
        self._ev_in = torch.cuda.Event()
        self._ev_recall = torch.cuda.Event()

    def prepare_layer(self, layer: int, buf: LayerBuffers, host_kv: torch.Tensor, ctx_len: torch.Tensor,
                      resident: torch.Tensor, kv_for_digest: Optional[torch.Tensor] = None) -> None:
        """Digests from the keys, tables from the resident list, and the resident blocks
        pulled into the pool through the recall kernel (slot i <- block resident[i])."""
        pi = self.pi
        pi.build_digests(layer, host_kv if kv_for_digest is None else kv_for_digest, ctx_len, buf.digest)
        pi.table_init(resident, buf.block_table, buf.slot_block, buf.slot_stamp)
        C = pi.cfg.pool_slots
        fill = torch.zeros((buf.batch, C, 4), dtype=torch.int32, device=resident.device)
        valid = resident >= 0
        order = torch.argsort((~valid).to(torch.int8), dim=1, stable=True)        # occupied slots first
        n = valid.sum(dim=1).to(torch.int32)
        fill[:, :, 0] = torch.gather(resident, 1, order)
        fill[:, :, 1] = order.to(torch.int32)
        fill[:, :, 2] = 1
        fill[:, :, 3] = torch.arange(C, dtype=torch.int32, device=resident.device)
        pi.recall_gather_scatter(layer, host_kv, buf.pool, fill.contiguous(), n.contiguous())

    def select_and_recall(self, layer: int, step: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor,
                          host_kv: torch.Tensor, stream=None) -> None:
        pi = self.pi
        pi.score_select(layer, q, buf.digest, ctx_len, buf.sel_blocks, buf.sel_count, buf.scores, stream=stream)
        pi.diff_misses(layer, step, ctx_len, buf.sel_blocks, buf.sel_count, buf.block_table, buf.slot_block,
                       buf.slot_stamp, buf.sel_slots, buf.recall_list, buf.recall_count, stream=stream)
        pi.recall_gather_scatter(layer, host_kv, buf.pool, buf.recall_list, buf.recall_count, stream=stream)

    def attention(self, layer: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor, out: torch.Tensor,
                  lse: Optional[torch.Tensor] = None, stream=None) -> None:
        self.pi.sparse_decode_attn(layer, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx_len, out,
                                   lse, stream=stream)

    def layer_step(self, layer: int, step: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor,
                   host_kv: torch.Tensor, out: torch.Tensor, lse: Optional[torch.Tensor] = None) -> None:
        """Serial form: all four calls on the current stream."""
        self.select_and_recall(layer, step, buf, q, ctx_len, host_kv)
        self.attention(layer, buf, q, ctx_len, out, lse)

    def layer_step_overlapped(self, layer: int, step: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor,
                              host_kv: torch.Tensor, out: torch.Tensor, lse: Optional[torch.Tensor] = None) -> None:
        """Selection, diff and recall run on the side stream; attention waits for the
        recall event on the current stream, so the recall of the next call can overlap it."""
        main = torch.cuda.current_stream()
        self._ev_in.record(main)
        self.side.wait_event(self._ev_in)
        self.select_and_recall(layer, step, buf, q, ctx_len, host_kv, stream=self.side)
        ev = torch.cuda.Event()
        ev.record(self.side)
        main.wait_event(ev)
        self.attention(layer, buf, q, ctx_len, out, lse)
