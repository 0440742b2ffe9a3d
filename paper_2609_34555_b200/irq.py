"""Interruptible layer-wise scheduling (Sec. 4.2 of the paper): a thin host policy around the
recall path.

Two batches advance through their layers independently.  The offload batch, at layer m, runs
selection + diff and issues its recall, then yields; the normal batch (requests whose KV is
all on the GPU) runs layers until the recall has landed; the offload batch then runs attention
(+ FFN) of layer m, moves to m+1, issues the next recall and yields again.  The number of
normal layers executed during one recall wait is the overlap depth (not fixed: it follows the
actual I/O time).  Three ways of noticing the completion (Sec. 4.2.2):

  sync   the host synchronises on the whole normal layer before looking   (timely, drains the queue)
  async  the host never synchronises, it polls between enqueues           (busy GPU, late switch)
  semi   the host waits for the layer's attention only and decides while the FFN still runs

The scheduler talks to two small back ends (`issue_recall`, `compute`, `enqueue_attention`,
`enqueue_ffn`, events with query()/synchronize()); a simulated back end makes the policy
testable without a GPU, the CUDA back end drives the kernels of this library.

    python -m paper_2609_34555_b200.irq        # compares the three modes on the GPU
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys
import time
from dataclasses import dataclass, field
from pathlib import Path
from typing import Optional

MODES = ("sync", "async", "semi")


@dataclass
class IrqReport:
    mode: str
    offload_layers: int = 0
    normal_layers: int = 0
    depths: list = field(default_factory=list)           # normal layers per recall wait
    wall_s: float = 0.0
    resume_delay_us: list = field(default_factory=list)  # recall landed -> offload layer starts

    def summary(self) -> dict:
        return dict(mode=self.mode, offload_layers=self.offload_layers, normal_layers=self.normal_layers,
                    overlap_depth_mean=statistics.fmean(self.depths) if self.depths else 0.0,
                    overlap_depth_max=max(self.depths) if self.depths else 0,
                    resume_delay_us_mean=statistics.fmean(self.resume_delay_us) if self.resume_delay_us else None,
                    offload_layers_per_s=self.offload_layers / self.wall_s if self.wall_s else None,
                    normal_layers_per_s=self.normal_layers / self.wall_s if self.wall_s else None)


class IrqScheduler:
    """Inner (layer-granularity) scheduler.  `max_ahead` bounds how many normal layers the host
    may have queued without having seen them finish (the async mode's only brake)."""

    def __init__(self, offload, normal, mode: str = "semi", max_ahead: int = 4):
        assert mode in MODES
        self.offload, self.normal, self.mode, self.max_ahead = offload, normal, mode, max_ahead

    def run(self, offload_layers: int) -> IrqReport:
        rep = IrqReport(self.mode)
        off, nor = self.offload, self.normal
        t0 = off.now()
        layer, depth, nl = 0, 0, 0
        pending = []                                     # end-of-layer events of queued normal layers
        io = off.issue_recall(layer)
        while layer < offload_layers:
            if io.query():                               # recall landed: the offload batch resumes
                off.compute(layer, io)
                rep.depths.append(depth)
                rep.offload_layers += 1
                layer, depth = layer + 1, 0
                if layer < offload_layers:
                    io = off.issue_recall(layer)
                continue
            attn_done = nor.enqueue_attention(nl)
            layer_done = nor.enqueue_ffn(nl)
            nl, depth = nl + 1, depth + 1
            rep.normal_layers += 1
            pending.append(layer_done)
            if self.mode == "sync":
                layer_done.synchronize()
                pending.clear()
            elif self.mode == "semi":
                attn_done.synchronize()                  # the FFN is still queued or running: decide now
                pending = pending[-1:]
            elif len(pending) >= self.max_ahead:
                pending.pop(0).synchronize()
        off.drain()
        nor.drain()
        rep.wall_s = off.now() - t0
        rep.resume_delay_us = off.resume_delays_us()
        return rep


# ------------------------------------------------------------------------------ simulated back end
class SimClock:
    def __init__(self, launch_us: float = 4.0):
        self.host, self.compute, self.io, self.launch = 0.0, 0.0, 0.0, launch_us


class SimEvent:
    def __init__(self, clock: SimClock, t: float):
        self.clock, self.t = clock, t

    def query(self) -> bool:
        return self.t <= self.clock.host

    def synchronize(self) -> None:
        self.clock.host = max(self.clock.host, self.t)


class SimOffload:
    """Recall of `t_io` microseconds on an I/O stream, attention + FFN on the compute stream."""

    def __init__(self, clock: SimClock, t_io, t_attn: float = 30.0, t_ffn: float = 60.0):
        self.c, self.t_io, self.t_attn, self.t_ffn = clock, t_io, t_attn, t_ffn
        self.delays, self.idle_us = [], 0.0

    def now(self) -> float:
        return self.c.host * 1e-6

    def _launch(self, dur: float) -> float:
        c = self.c
        c.host += c.launch
        start = max(c.host, c.compute)
        self.idle_us += start - c.compute if c.compute > 0 else 0.0
        c.compute = start + dur
        return start

    def issue_recall(self, layer: int) -> SimEvent:
        c = self.c
        c.host += c.launch
        t = self.t_io(layer) if callable(self.t_io) else self.t_io
        c.io = max(c.host, c.io, c.compute) + t          # selection runs after the batch's previous layer
        return SimEvent(c, c.io)

    def compute(self, layer: int, io: SimEvent) -> None:
        start = self._launch(self.t_attn + self.t_ffn)
        self.delays.append(start - io.t)

    def drain(self) -> None:
        self.c.host = max(self.c.host, self.c.compute, self.c.io)

    def resume_delays_us(self):
        return self.delays


class SimNormal:
    def __init__(self, clock: SimClock, off: SimOffload, t_attn: float = 40.0, t_ffn: float = 80.0):
        self.c, self.off, self.t_attn, self.t_ffn = clock, off, t_attn, t_ffn

    def enqueue_attention(self, layer: int) -> SimEvent:
        self.off._launch(self.t_attn)
        return SimEvent(self.c, self.c.compute)

    def enqueue_ffn(self, layer: int) -> SimEvent:
        self.off._launch(self.t_ffn)
        return SimEvent(self.c, self.c.compute)

    def drain(self) -> None:
        self.c.host = max(self.c.host, self.c.compute)


def simulate(mode: str, offload_layers: int = 64, t_io=400.0, **kw):
    clock = SimClock(kw.pop("launch_us", 4.0))
    off = SimOffload(clock, t_io)
    nor = SimNormal(clock, off, **kw)
    rep = IrqScheduler(off, nor, mode).run(offload_layers)
    return rep, off.idle_us


# ------------------------------------------------------------------------------ CUDA back end
class CudaOffload:
    """The offload batch on the GPU: DecodeSession buffers, selection + diff on stream A, recall
    on stream B, attention (+ an FFN stand-in) on the compute stream.  split_attention: the resident
    blocks' share of the attention is issued with the recall (stream A, behind the diff) and only the
    recalled blocks' share is left for the moment the batch gets the GPU back."""

    def __init__(self, sess, q_all, ffn, split_attention: bool = False):
        import torch
        self.torch, self.sess, self.q_all, self.ffn = torch, sess, q_all, ffn
        self.split = split_attention
        self._state = sess.pi.attn_state(sess.batch, sess.device) if split_attention else None
        self._resident_done = None
        self.compute_stream = torch.cuda.current_stream(sess.device)
        self.step = 0
        self._marks = []

    def now(self) -> float:
        self.torch.cuda.synchronize()
        return time.perf_counter()

    def issue_recall(self, layer: int):
        s, pi = self.sess, self.sess.pi
        l = layer % s.n_layers
        if l == 0:
            self.step += 1
        b, q = s.bufs[l], self.q_all[(self.step - 1) % self.q_all.shape[0], l]
        ev = self.torch.cuda.Event()
        ev.record(self.compute_stream)                    # the layer's query exists once the previous layer is done
        s.side.wait_event(ev)
        pi.score_select_diff(l, self.step, q, b.digest, s.ctx_len, b.sel_blocks, b.sel_count, b.block_table, b.slot_block,
                             b.slot_stamp, b.sel_slots, b.recall_list, b.recall_count, stream=s.side)
        d = self.torch.cuda.Event(); d.record(s.side); s.side2.wait_event(d)
        pi.recall_gather_scatter(l, s.host_region(l), b.pool, b.recall_list, b.recall_count, stream=s.side2)
        io = self.torch.cuda.Event(enable_timing=True)
        io.record(s.side2)
        if self.split:
            pi.sparse_decode_attn_resident(l, q, b.pool, b.sel_slots, b.sel_blocks, b.sel_count, s.ctx_len,
                                           b.recall_list, b.recall_count, self._state, stream=s.side)
            self._resident_done = self.torch.cuda.Event()
            self._resident_done.record(s.side)
        return io

    def compute(self, layer: int, io) -> None:
        s, pi = self.sess, self.sess.pi
        l = layer % s.n_layers
        b, q = s.bufs[l], self.q_all[(self.step - 1) % self.q_all.shape[0], l]
        self.compute_stream.wait_event(io)
        start = self.torch.cuda.Event(enable_timing=True)
        start.record(self.compute_stream)
        self._marks.append((io, start))
        if self.split:
            self.compute_stream.wait_event(self._resident_done)
            pi.sparse_decode_attn_recalled(l, q, b.pool, b.sel_slots, b.sel_blocks, b.sel_count, s.ctx_len,
                                           b.recall_list, b.recall_count, self._state, s.out[l], stream=self.compute_stream)
        else:
            pi.sparse_decode_attn(l, q, b.pool, b.sel_slots, b.sel_blocks, b.sel_count, s.ctx_len, s.out[l], None,
                                  stream=self.compute_stream)
        self.ffn()

    def drain(self) -> None:
        self.torch.cuda.synchronize()

    def resume_delays_us(self):
        return [max(0.0, a.elapsed_time(b) * 1e3) for a, b in self._marks]


class CudaNormal:
    """The normal batch: short requests with all KV on the GPU.  Its attention is the same kernel
    over a selection that covers every block; its FFN is a bf16 matmul stand-in."""

    def __init__(self, pi, buf, q, ctx_len, out, ffn, n_layers: int):
        import torch
        self.torch, self.pi, self.buf, self.q, self.ctx, self.out, self.ffn, self.n_layers = torch, pi, buf, q, ctx_len, out, ffn, n_layers
        self.stream = torch.cuda.current_stream()

    def enqueue_attention(self, layer: int):
        b = self.buf
        self.pi.sparse_decode_attn(0, self.q, b.pool, b.sel_slots, b.sel_blocks, b.sel_count, self.ctx, self.out, None,
                                   stream=self.stream)
        ev = self.torch.cuda.Event(); ev.record(self.stream)
        return ev

    def enqueue_ffn(self, layer: int):
        self.ffn()
        ev = self.torch.cuda.Event(); ev.record(self.stream)
        return ev

    def drain(self) -> None:
        self.torch.cuda.synchronize()


def run_on_gpu(offload_layers: int = 256, normal_batch: int = 64, normal_ctx: int = 4096, layers: int = 8,
               recall_ctas: int = 0, split_attention: bool = False) -> list:
    import numpy as np
    import torch
    sys.path.insert(0, str(Path(__file__).resolve().parent.parent))
    from paper_2609_34555_b200 import PulseInfer
    from paper_2609_34555_b200.runner import DecodeSession, LayerBuffers
    from workloads import generate as gen, get_config

    dev = torch.device("cuda:0")
    cfg = get_config("c2").replace(n_layers=layers)
    pi = PulseInfer.from_workload(cfg, recall_ctas=recall_ctas)
    sess = DecodeSession(pi, cfg.batch, cfg.n_layers, host_layers=min(4, layers))
    sess.ctx_len.fill_(cfg.ctx)
    for l in range(cfg.n_layers):
        kv = gen.make_kv(cfg, l, device=dev) if l < sess.host_layers else None
        sess.load_layer(l, kv, torch.from_numpy(gen.initial_resident(cfg, l)).to(dev))
    q_all = torch.stack([gen.make_queries(cfg, l, 48, device=dev) for l in range(cfg.n_layers)], 1).contiguous()
    for t in range(16):                                    # settle the hot set
        sess.decode_step(q_all[t])
    torch.cuda.synchronize()
    # normal batch: every block selected, slot i holds block i
    ncfg = get_config("c2").replace(n_layers=1, batch=normal_batch, ctx=normal_ctx,
                                    budget_blocks=normal_ctx // 16, resident_frac=1.0)
    npi = PulseInfer.from_workload(ncfg)
    nbuf = LayerBuffers(npi, normal_batch, dev)
    nbuf.pool.copy_(torch.randn(nbuf.pool.shape, device=dev).to(torch.bfloat16))
    ident = torch.arange(ncfg.n_blocks, dtype=torch.int32, device=dev)[None, :].expand(normal_batch, -1).contiguous()
    nbuf.sel_slots.copy_(ident); nbuf.sel_blocks.copy_(ident); nbuf.sel_count.fill_(ncfg.n_blocks)
    nq = torch.randn((normal_batch, ncfg.n_q_heads, 128), device=dev).to(torch.bfloat16)
    nctx = torch.full((normal_batch,), normal_ctx, dtype=torch.int32, device=dev)
    nout = torch.zeros_like(nq)
    # FFN stand-ins (Llama-3-8B-shaped: 4096 -> 14336 -> 4096), plumbing only
    w1 = torch.randn((4096, 14336), device=dev, dtype=torch.bfloat16) * 0.01
    w2 = torch.randn((14336, 4096), device=dev, dtype=torch.bfloat16) * 0.01
    xn = torch.randn((normal_batch, 4096), device=dev, dtype=torch.bfloat16)
    xo = torch.randn((cfg.batch, 4096), device=dev, dtype=torch.bfloat16)
    ffn_n = lambda: torch.matmul(torch.matmul(xn, w1), w2)
    ffn_o = lambda: torch.matmul(torch.matmul(xo, w1), w2)
    out = []
    for mode in MODES:
        off = CudaOffload(sess, q_all, ffn_o, split_attention=split_attention)
        off.step = sess.step_count
        nor = CudaNormal(npi, nbuf, nq, nctx, nout, ffn_n, 32)
        rep = IrqScheduler(off, nor, mode).run(offload_layers)
        sess.step_count = off.step
        assert pi.status()[0] == 0 and npi.status()[0] == 0
        out.append(rep.summary())
    return out


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--offload-layers", type=int, default=256)
    ap.add_argument("--normal-batch", type=int, default=64)
    ap.add_argument("--normal-ctx", type=int, default=4096)
    ap.add_argument("--recall-ctas", type=int, default=10, help="one recall launch at a time here: 10 CTAs (the library default of 5 is sized for two launches side by side)")
    ap.add_argument("--split-attention", action="store_true",
                    help="the resident blocks' share of the offload batch's attention is issued with the recall")
    a = ap.parse_args()
    for r in run_on_gpu(a.offload_layers, a.normal_batch, a.normal_ctx, recall_ctas=a.recall_ctas,
                        split_attention=a.split_attention):
        print(json.dumps(r))
