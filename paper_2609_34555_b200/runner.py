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
                      resident: torch.Tensor, kv_for_digest: Optional[torch.Tensor] = None,
                      page_table: Optional[torch.Tensor] = None) -> None:
        """Digests from the keys, tables from the resident list, and the resident blocks
        pulled into the pool through the recall kernel (slot i <- block resident[i]).  A paged
        host store needs kv_for_digest (the keys in logical block order)."""
        if page_table is not None and kv_for_digest is None:
            raise ValueError("a paged host store cannot be read in block order: pass kv_for_digest")
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
        pi.recall_gather_scatter(layer, host_kv, buf.pool, fill.contiguous(), n.contiguous(), page_table=page_table)

    def select_and_recall(self, layer: int, step: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor,
                          host_kv: torch.Tensor, stream=None, fused: bool = True) -> None:
        """fused: selection and diff in one launch (pi_score_select_diff); else the two calls."""
        pi = self.pi
        if fused:
            pi.score_select_diff(layer, step, q, buf.digest, ctx_len, buf.sel_blocks, buf.sel_count, buf.block_table,
                                 buf.slot_block, buf.slot_stamp, buf.sel_slots, buf.recall_list, buf.recall_count,
                                 scores=buf.scores, stream=stream)
        else:
            pi.score_select(layer, q, buf.digest, ctx_len, buf.sel_blocks, buf.sel_count, buf.scores, stream=stream)
            pi.diff_misses(layer, step, ctx_len, buf.sel_blocks, buf.sel_count, buf.block_table, buf.slot_block,
                           buf.slot_stamp, buf.sel_slots, buf.recall_list, buf.recall_count, stream=stream)
        pi.recall_gather_scatter(layer, host_kv, buf.pool, buf.recall_list, buf.recall_count, stream=stream)

    def attention(self, layer: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor, out: torch.Tensor,
                  lse: Optional[torch.Tensor] = None, stream=None) -> None:
        self.pi.sparse_decode_attn(layer, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx_len, out,
                                   lse, stream=stream)

    def layer_step(self, layer: int, step: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor,
                   host_kv: torch.Tensor, out: torch.Tensor, lse: Optional[torch.Tensor] = None,
                   fused: bool = True) -> None:
        """Serial form: all calls on the current stream."""
        self.select_and_recall(layer, step, buf, q, ctx_len, host_kv, fused=fused)
        self.attention(layer, buf, q, ctx_len, out, lse)

    def layer_step_overlapped(self, layer: int, step: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor,
                              host_kv: torch.Tensor, out: torch.Tensor, lse: Optional[torch.Tensor] = None,
                              fused: bool = True) -> None:
        """Selection, diff and recall run on the side stream; attention waits for the
        recall event on the current stream, so the recall of the next call can overlap it."""
        main = torch.cuda.current_stream()
        self._ev_in.record(main)
        self.side.wait_event(self._ev_in)
        self.select_and_recall(layer, step, buf, q, ctx_len, host_kv, stream=self.side, fused=fused)
        ev = torch.cuda.Event()
        ev.record(self.side)
        main.wait_event(ev)
        self.attention(layer, buf, q, ctx_len, out, lse)


    def layer_step_split(self, layer: int, step: int, buf: LayerBuffers, q: torch.Tensor, ctx_len: torch.Tensor,
                         host_kv: torch.Tensor, out: torch.Tensor, state: torch.Tensor, fused: bool = True) -> None:
        """The layer's chain with the attention split around the recall: selection and diff on the current
        stream, the resident blocks' share of the attention beside the recall on the side stream, the recalled
        blocks' share on the current stream once the recall has landed."""
        pi = self.pi
        main = torch.cuda.current_stream()
        if fused:
            pi.score_select_diff(layer, step, q, buf.digest, ctx_len, buf.sel_blocks, buf.sel_count, buf.block_table,
                                 buf.slot_block, buf.slot_stamp, buf.sel_slots, buf.recall_list, buf.recall_count,
                                 scores=buf.scores)
        else:
            pi.score_select(layer, q, buf.digest, ctx_len, buf.sel_blocks, buf.sel_count, buf.scores)
            pi.diff_misses(layer, step, ctx_len, buf.sel_blocks, buf.sel_count, buf.block_table, buf.slot_block,
                           buf.slot_stamp, buf.sel_slots, buf.recall_list, buf.recall_count)
        self._ev_in.record(main)
        self.side.wait_event(self._ev_in)
        pi.sparse_decode_attn_resident(layer, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx_len,
                                       buf.recall_list, buf.recall_count, state, stream=self.side)
        self._ev_recall.record(self.side)
        pi.recall_gather_scatter(layer, host_kv, buf.pool, buf.recall_list, buf.recall_count)
        main.wait_event(self._ev_recall)
        pi.sparse_decode_attn_recalled(layer, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx_len,
                                       buf.recall_list, buf.recall_count, state, out)


class StageTimer:
    """CUDA events around each call of a decode step, on the stream the call runs on.

    `light=True` adds no event to any stream: the events the pipelined step records anyway to
    order its streams (selection+diff done, recall landed, attention done) are created with
    timing enabled and kept, and the stage intervals are reconstructed from their timestamps
    afterwards (`light_summary`).  Extra events between the kernels of the recall streams cost
    the pipelined step about 6 % of its rate, which is why the timed region uses this form."""

    STAGES = ("append", "select_diff", "score_select", "diff", "recall", "attn_resident", "attn")

    def __init__(self, stages=None, light: bool = False):
        self.stages = tuple(stages) if stages else self.STAGES
        self.pairs = {s: [] for s in self.stages}
        self.light = light
        self.records = []          # light form: (layer, recall stream index, ev_diff, ev_recall, ev_attn) in launch order

    def sync_events(self, layer: int, recall_stream: int):
        evs = tuple(torch.cuda.Event(enable_timing=True) for _ in range(3))
        self.records.append((layer, recall_stream) + evs)
        return evs

    def light_summary(self, base: torch.cuda.Event) -> dict:
        """Stage intervals of the light form on the clock of `base` (a timing event recorded before
        the first step; call after a synchronize).  A stage starts when its stream is free and its
        input event has fired: recall = max(diff done, previous recall of the same stream done) ->
        recall landed; attention = max(recall landed, previous attention done) -> attention done;
        select+diff = max(previous diff done, this layer's previous attention done) -> diff done.
        The first launch of each stream (no predecessor to bound its start) is left out."""
        last_recall, last_attn_of_layer = {}, {}
        prev_diff = prev_attn = None
        spans = {"recall": [], "attn": [], "select_diff": []}
        for layer, rs, evd, evr, eva in self.records:
            td, tr, ta = base.elapsed_time(evd), base.elapsed_time(evr), base.elapsed_time(eva)
            if rs in last_recall:
                spans["recall"].append((max(td, last_recall[rs]), tr))
            if prev_attn is not None:
                spans["attn"].append((max(tr, prev_attn), ta))
            if prev_diff is not None:
                spans["select_diff"].append((max(prev_diff, last_attn_of_layer.get(layer, 0.0)), td))
            last_recall[rs], last_attn_of_layer[layer] = tr, ta
            prev_diff, prev_attn = td, ta
        out = {}
        for name, lst in spans.items():
            ms = [b - a for a, b in lst]
            busy, end = 0.0, float("-inf")
            for a, b in sorted(lst):
                if a > end:
                    busy, end = busy + (b - a), b
                elif b > end:
                    busy, end = busy + (b - end), b
            out[name] = dict(launches=len(ms), total_ms=float(sum(ms)), mean_ms=float(sum(ms) / max(1, len(ms))),
                             busy_ms=float(busy))
        return out

    def wants(self, stage: str) -> bool:
        return stage in self.pairs

    def mark(self, stream) -> torch.cuda.Event:
        ev = torch.cuda.Event(enable_timing=True)
        ev.record(stream)
        return ev

    def add(self, stage: str, a: torch.cuda.Event, b: torch.cuda.Event) -> None:
        self.pairs[stage].append((a, b))

    def busy_ms(self, stage: str, base: torch.cuda.Event) -> float:
        """Milliseconds during which at least one launch of the stage was running: the union of the
        launches' intervals on the clock of `base` (a timing event recorded before all of them).
        Equals the summed durations when launches never overlap (call after a synchronize)."""
        spans = sorted((base.elapsed_time(a), base.elapsed_time(b)) for a, b in self.pairs[stage])
        busy, end = 0.0, float("-inf")
        for s0, s1 in spans:
            if s0 > end:
                busy += s1 - s0
                end = s1
            elif s1 > end:
                busy += s1 - end
                end = s1
        return busy

    def summary(self) -> dict:
        """Per stage: launches, mean and total milliseconds (call after a synchronize)."""
        out = {}
        for s, lst in self.pairs.items():
            ms = [a.elapsed_time(b) for a, b in lst]
            out[s] = dict(launches=len(ms), total_ms=float(sum(ms)), mean_ms=float(sum(ms) / max(1, len(ms))))
        return out


class DecodeSession:
    """All layers of one batch of offloaded sequences: per-layer device buffers, the pinned
    host store, and the pipelined decode step (selection + diff of every layer on one side
    stream, the recall pulls on a second, attention on the main stream as soon as that layer's
    recall has landed).

    `host_layers` < n_layers lets several layers share one region of the host store (layer l
    reads region l % host_layers) when host memory is short; digests, tables and pools stay
    per layer.

    `paged=True` scatters the blocks: each region becomes an arena of block-sized pages and a
    seeded random permutation (the region's page table, [batch][NB] int32 on the device) says
    which page holds block b of sequence s, so neighbouring blocks of a sequence are no longer
    neighbours in host memory and the pages of all sequences interleave.

    `recall_streams`: the recall launches of consecutive layers rotate over this many streams, so
    the fixed cost of one launch (launch gap, list scan, first round trip over the host link,
    drain) is covered by the transfer of the next."""

    def __init__(self, pi: PulseInfer, batch: int, n_layers: int, host_layers: Optional[int] = None,
                 device="cuda", keep_scores: bool = False, paged: bool = False, page_seed: int = 0,
                 recall_streams: int = 2, fused_select_diff: bool = True, split_attention: bool = False):
        c = pi.cfg
        # attention split around the recall: the resident blocks' share runs beside the recall (in the serial
        # form on a stream of its own), the recalled blocks' share after it
        self.split_attention = split_attention
        self.fused_select_diff = fused_select_diff     # selection + diff in one launch (pi_score_select_diff)
        self.pi, self.batch, self.n_layers = pi, batch, n_layers
        self.host_layers = n_layers if host_layers is None else max(1, min(host_layers, n_layers))
        self.device = torch.device(device)
        self.bufs = [LayerBuffers(pi, batch, device, keep_scores) for _ in range(n_layers)]
        shape = (batch, c.max_blocks, c.n_kv_heads, 2, c.block_tokens, c.head_dim)
        self.host_kv = [torch.empty(shape, dtype=torch.bfloat16, pin_memory=True) for _ in range(self.host_layers)]
        self.page_tables = None
        if paged:
            g = torch.Generator().manual_seed(page_seed)
            self.page_tables = [torch.randperm(batch * c.max_blocks, generator=g).to(torch.int32)
                                .view(batch, c.max_blocks).to(device) for _ in range(self.host_layers)]
        self.out = torch.zeros((n_layers, batch, c.n_q_heads, c.head_dim), dtype=torch.bfloat16, device=device)
        self.ctx_len = torch.zeros((batch,), dtype=torch.int32, device=device)
        self.ctx_prev = torch.zeros((batch,), dtype=torch.int32, device=device)     # length before the step's append
        self.step_dev = torch.zeros((1,), dtype=torch.int32, device=device)         # step number of graph replays
        self.main = torch.cuda.current_stream(self.device)
        self.side = torch.cuda.Stream(self.device)
        self.side2 = torch.cuda.Stream(self.device)
        self.recall_streams = [self.side2] + [torch.cuda.Stream(self.device) for _ in range(max(1, recall_streams) - 1)]
        self._ev_diff = [torch.cuda.Event() for _ in range(n_layers)]
        self._ev_recall = [torch.cuda.Event() for _ in range(n_layers)]
        self._ev_attn = [torch.cuda.Event() for _ in range(n_layers)]
        self._ev_res = [torch.cuda.Event() for _ in range(n_layers)]
        self._ev_start = torch.cuda.Event()
        self._path = RecallPath(pi)
        self._attn_state = pi.attn_state(batch, self.device) if split_attention else None
        self.step_count = 0
        self._copy_s = None                  # copy stream and double buffers of the end-to-end form (made on first use)
        self._host_graph = None
        self._step_dev_shadow = None

    def host_region(self, layer: int) -> torch.Tensor:
        """The layer's host store: [batch][NB] blocks in block order, or (paged) the arena of pages."""
        return self.host_kv[layer % self.host_layers]

    def page_table(self, layer: int) -> Optional[torch.Tensor]:
        return None if self.page_tables is None else self.page_tables[layer % self.host_layers]

    def logical_host(self, layer: int) -> torch.Tensor:
        """The layer's host store in logical block order (a copy when the store is paged)."""
        host = self.host_region(layer)
        pt = self.page_table(layer)
        if pt is None:
            return host
        pages = host.view((-1,) + tuple(host.shape[2:]))
        return pages[pt.cpu().view(-1).long()].view(host.shape)

    def load_layer(self, layer: int, kv_dev: Optional[torch.Tensor], resident: torch.Tensor, store: bool = True) -> None:
        """kv_dev (device copy of the layer's keys/values, logical block order) is stored into the
        host region when given (and `store`); digests are built from it, tables from `resident`,
        and the resident blocks are pulled back from the host store into the pool."""
        host = self.host_region(layer)
        pt = self.page_table(layer)
        if kv_dev is not None and store:
            if pt is None:
                host.copy_(kv_dev, non_blocking=False)
            else:
                scattered = torch.empty_like(kv_dev)
                scattered.view((-1,) + tuple(kv_dev.shape[2:]))[pt.view(-1).long()] = kv_dev.view((-1,) + tuple(kv_dev.shape[2:]))
                host.copy_(scattered, non_blocking=False)
                del scattered
        self._path.prepare_layer(layer, self.bufs[layer], host, self.ctx_len, resident,
                                 kv_for_digest=kv_dev, page_table=pt)

    def decode_step(self, q: torch.Tensor, overlapped: bool = True, timer: Optional[StageTimer] = None,
                    resident_script: Optional[torch.Tensor] = None, new_kv=None,
                    out: Optional[torch.Tensor] = None, capturing: bool = False) -> torch.Tensor:
        """q: device bf16 [n_layers][batch][Hq][D].  Returns `out` (default self.out, [n_layers][batch][Hq][D]);
        valid once the current stream has caught up.  resident_script (int32 [n_layers][batch][C]):
        workloads with scripted miss counts reset each layer's tables to these hot-set contents
        before the layer's diff (pool contents are not refreshed: timing runs only).
        new_kv = (k_new, v_new), each bf16 [n_layers][batch][Hkv][D]: the step's new token is appended
        to every layer first (pool slot, host store, digest) and the context grows by one.

        Overlapped form: selection and diff of every layer run ahead on one stream, the recall
        pulls follow on the recall streams in rotation (the host link stays busy back to back),
        and each layer's attention runs on the current stream once its recall landed."""
        pi = self.pi
        out = self.out if out is None else out
        self.step_count += 1
        step = self.step_count
        main = torch.cuda.current_stream(self.device)
        sel_s = self.side if overlapped else main
        if overlapped:
            self._ev_start.record(main)
            sel_s.wait_event(self._ev_start)
        if capturing:
            # inside a graph the step number lives on the device and advances with every replay
            with torch.cuda.stream(sel_s):
                self.step_dev += 1
            step = self.step_dev
        if new_kv is not None:
            with torch.cuda.stream(sel_s):
                self.ctx_prev.copy_(self.ctx_len)
                self.ctx_len += 1
        for l in range(self.n_layers):
            b, host, pt = self.bufs[l], self.host_region(l), self.page_table(l)
            rs_i = l % len(self.recall_streams)
            rec_s = self.recall_streams[rs_i] if overlapped else main
            tm = timer
            if overlapped and tm is not None and tm.light:
                # the ordering events double as timestamps: no extra work on any stream
                self._ev_diff[l], self._ev_recall[l], ev_attn_new = tm.sync_events(l, rs_i)
                tm = None
            else:
                ev_attn_new = None
            if overlapped and not capturing and self.step_count > 1:
                sel_s.wait_event(self._ev_attn[l])         # last step's attention still reads this layer's lists and pool
            if ev_attn_new is not None:
                self._ev_attn[l] = ev_attn_new
            if capturing:                                  # events of a capture live in the graph only
                evd, evr, eva = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()
            else:
                evd, evr, eva = self._ev_diff[l], self._ev_recall[l], self._ev_attn[l]
            if resident_script is not None:
                pi.table_init(resident_script[l], b.block_table, b.slot_block, b.slot_stamp, stream=sel_s)
            if new_kv is not None:
                ta = tm.mark(sel_s) if tm and tm.wants("append") else None
                pi.append_kv(l, step, new_kv[0][l], new_kv[1][l], self.ctx_prev, host, b.pool, b.block_table,
                             b.slot_block, b.slot_stamp, b.digest, page_table=pt, stream=sel_s)
                if ta is not None:
                    tm.add("append", ta, tm.mark(sel_s))
            if self.fused_select_diff:
                t0 = tm.mark(sel_s) if tm and tm.wants("select_diff") else None
                pi.score_select_diff(l, step, q[l], b.digest, self.ctx_len, b.sel_blocks, b.sel_count, b.block_table,
                                     b.slot_block, b.slot_stamp, b.sel_slots, b.recall_list, b.recall_count,
                                     scores=b.scores, stream=sel_s)
                if t0 is not None:
                    tm.add("select_diff", t0, tm.mark(sel_s))
                t0 = t1 = t2 = None
            else:
                t0 = tm.mark(sel_s) if tm and tm.wants("score_select") else None
                pi.score_select(l, q[l], b.digest, self.ctx_len, b.sel_blocks, b.sel_count, b.scores, stream=sel_s)
                t1 = tm.mark(sel_s) if tm and (tm.wants("score_select") or tm.wants("diff")) else None
                pi.diff_misses(l, step, self.ctx_len, b.sel_blocks, b.sel_count, b.block_table, b.slot_block,
                               b.slot_stamp, b.sel_slots, b.recall_list, b.recall_count, stream=sel_s)
                t2 = tm.mark(sel_s) if tm and tm.wants("diff") else None
            split = self.split_attention
            if split and self._attn_state is None:
                self._attn_state = pi.attn_state(self.batch, self.device)
            if overlapped or split:
                evd.record(sel_s)
            if overlapped:
                rec_s.wait_event(evd)
            # the resident blocks' share of a split attention runs beside the recall: on the attention stream in the
            # pipelined form; in the serial form on the side stream, so that the chain select -> recall -> rest of
            # the attention stays on one stream (dependent launches on a stream follow each other far more closely
            # than launches that wait for another stream's event)
            res_s = main if overlapped else self.side
            if split:
                res_s.wait_event(evd)
                ta0 = tm.mark(res_s) if tm and tm.wants("attn_resident") else None
                pi.sparse_decode_attn_resident(l, q[l], b.pool, b.sel_slots, b.sel_blocks, b.sel_count, self.ctx_len,
                                               b.recall_list, b.recall_count, self._attn_state, stream=res_s)
                if ta0 is not None:
                    tm.add("attn_resident", ta0, tm.mark(res_s))
                if not overlapped:
                    evs = torch.cuda.Event() if capturing else self._ev_res[l]
                    evs.record(res_s)
            t2r = tm.mark(rec_s) if tm and tm.wants("recall") else None
            pi.recall_gather_scatter(l, host, b.pool, b.recall_list, b.recall_count, page_table=pt, stream=rec_s)
            t3 = tm.mark(rec_s) if tm and tm.wants("recall") else None
            if overlapped:
                evr.record(rec_s)
                main.wait_event(evr)
            elif split:
                main.wait_event(evs)
            t4 = tm.mark(main) if tm and tm.wants("attn") else None
            if split:
                pi.sparse_decode_attn_recalled(l, q[l], b.pool, b.sel_slots, b.sel_blocks, b.sel_count, self.ctx_len,
                                               b.recall_list, b.recall_count, self._attn_state, out[l], stream=main)
            else:
                pi.sparse_decode_attn(l, q[l], b.pool, b.sel_slots, b.sel_blocks, b.sel_count, self.ctx_len,
                                      out[l], None, stream=main)
            t5 = tm.mark(main) if tm and tm.wants("attn") else None
            if overlapped:
                eva.record(main)
            if tm:
                if t0 is not None: tm.add("score_select", t0, t1)
                if t2 is not None: tm.add("diff", t1, t2)
                if t2r is not None: tm.add("recall", t2r, t3)
                if t4 is not None: tm.add("attn", t4, t5)
        return out

    def capture_step(self, q_static: torch.Tensor, out: Optional[torch.Tensor] = None,
                     new_kv_static=None) -> "torch.cuda.CUDAGraph":
        """Captures one pipelined decode step (all layers, all streams) into a CUDA graph that reads
        its queries from `q_static` and its step number from device memory.  Replays continue the
        session: call `replay_step(graph)` once per decode step after refreshing `q_static` (stream
        order serialises consecutive replays, as consecutive decode steps are anyway).  With
        new_kv_static = (k, v) buffers the graph also appends the step's token (refresh them too;
        the context lengths advance on the device).  Eager steps and replays may be mixed; steps
        that reset the tables from a script stay eager."""
        torch.cuda.synchronize(self.device)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.decode_step(q_static, overlapped=True, out=out, capturing=True, new_kv=new_kv_static)
        self.step_count -= 1                              # the capture itself ran nothing
        self._step_dev_shadow = None
        return graph

    def replay_step(self, graph: "torch.cuda.CUDAGraph") -> None:
        """One decode step by replaying a graph from capture_step on the current stream."""
        if self._step_dev_shadow != self.step_count:
            self.step_dev.fill_(self.step_count)          # eager steps ran in between: resynchronise the device counter
        self.step_count += 1
        self._step_dev_shadow = self.step_count           # the replay adds one on the device
        graph.replay()

    def prepare_host_graph(self) -> None:
        """Captures the graph decode_steps_from_host(use_graph=True) replays (synchronises; once)."""
        if self._host_graph is None:
            self._q_static = torch.empty(self.out.shape, dtype=torch.bfloat16, device=self.device)
            self._host_graph = self.capture_step(self._q_static)

    def decode_steps_from_host(self, q_hosts, out_hosts, resident_scripts=None, use_graph: bool = False) -> None:
        """End-to-end form over several steps with the copies off the critical path: step i's queries
        (pinned host, [n_layers][batch][Hq][D]) are uploaded on a copy stream while step i-1 computes,
        step i's outputs are downloaded to out_hosts[i % len(out_hosts)] (pinned host) while step i+1
        computes.  Queries and outputs are double-buffered on the device.  With use_graph the step
        itself is a replay of the graph from capture_step (device-to-device copies move the queries
        into, and the outputs out of, the graph's fixed buffers).  Returns once everything is
        enqueued; out_hosts are valid after a synchronize."""
        main = torch.cuda.current_stream(self.device)
        if self._copy_s is None:
            self._copy_s = torch.cuda.Stream(self.device)
            self._q2 = [torch.empty(self.out.shape, dtype=torch.bfloat16, device=self.device) for _ in range(2)]
            self._out2 = [torch.empty_like(self.out) for _ in range(2)]
        if use_graph and resident_scripts is not None:
            raise ValueError("steps that reset the tables from a script are not captured")
        if use_graph:
            self.prepare_host_graph()
        cp = self._copy_s
        n = len(q_hosts)
        ev_up = [torch.cuda.Event() for _ in range(n)]
        ev_done = [torch.cuda.Event() for _ in range(n)]
        ev_down = [torch.cuda.Event() for _ in range(n)]
        start = torch.cuda.Event()
        start.record(main)
        cp.wait_event(start)

        def upload(i):
            with torch.cuda.stream(cp):
                if i >= 2:
                    cp.wait_event(ev_done[i - 2])            # the step that last read this query buffer
                self._q2[i % 2].copy_(q_hosts[i], non_blocking=True)
                ev_up[i].record(cp)

        upload(0)
        for i in range(n):
            if i + 1 < n:
                upload(i + 1)
            main.wait_event(ev_up[i])
            if i >= 2:
                main.wait_event(ev_down[i - 2])              # the download that last read this output buffer
            if use_graph:
                self._q_static.copy_(self._q2[i % 2], non_blocking=True)
                self.replay_step(self._host_graph)
                self._out2[i % 2].copy_(self.out, non_blocking=True)
            else:
                self.decode_step(self._q2[i % 2], overlapped=True, out=self._out2[i % 2],
                                 resident_script=None if resident_scripts is None else resident_scripts[i])
            ev_done[i].record(main)
            with torch.cuda.stream(cp):
                cp.wait_event(ev_done[i])
                out_hosts[i % len(out_hosts)].copy_(self._out2[i % 2], non_blocking=True)
                ev_down[i].record(cp)
        main.wait_event(ev_down[n - 1])
        if n >= 2:
            main.wait_event(ev_down[n - 2])

    def decode_step_from_host(self, q_host: torch.Tensor, out_host: torch.Tensor, q_dev: torch.Tensor,
                              resident_script: Optional[torch.Tensor] = None) -> None:
        """End-to-end form: queries come from pinned host memory, results go back to pinned
        host memory; both copies are enqueued on the main stream around the step."""
        q_dev.copy_(q_host, non_blocking=True)
        self.decode_step(q_dev, overlapped=True, resident_script=resident_script)
        out_host.copy_(self.out, non_blocking=True)

    def miss_blocks(self) -> int:
        """Units recalled by the last step (synchronises; bookkeeping for reports)."""
        total = 0
        for b in self.bufs:
            cnt = b.recall_count
            lst = b.recall_list
            idx = torch.arange(lst.shape[1], device=lst.device)[None, :] < cnt[:, None]
            total += int((lst[:, :, 2] * idx).sum().item())
        return total
