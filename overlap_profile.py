"""Overlap-depth profile on the GPU (Sec. 4.3.2 of the paper): how many layers of the normal batch
fit into the recall I/O of one offload-batch layer, on a grid of batch sizes (B_o, B_n).

    python overlap_profile.py [--out FILE]

t_io(B_o)    time of selection + diff + recall of one layer for B_o offloaded sequences of the
             Llama-3-8B-shaped workload (32K context, 2048-token budget, settled hot set), measured
             with CUDA events per layer-step on one stream
t_layer(B_n) time of one layer of the normal batch: dense decode attention of B_n requests with
             all KV resident (the same attention kernel with every block selected) + an FFN
             stand-in (bf16 matmuls 4096 -> 14336 -> 4096)
m(B_o, B_n)  mean over the measured layer-steps of ceil(t_io / t_layer)  (Sec. 4.3.2)

The grid feeds `ioaa.OverlapDepthGrid` (bilinear interpolation at run time); the module ends with one
admission decision taken on the measured grid.  Plumbing and host policy only: every GPU step is a
call of the C ABI.
"""
from __future__ import annotations

import argparse
import json
import math
import sys
from pathlib import Path

import numpy as np
import torch

sys.path.insert(0, str(Path(__file__).resolve().parent))

from paper_2609_34555_b200 import PulseInfer  # noqa: E402
from paper_2609_34555_b200.ioaa import OverlapDepthGrid, ioaa_admit  # noqa: E402
from paper_2609_34555_b200.runner import DecodeSession, LayerBuffers  # noqa: E402
from workloads import generate as gen, get_config  # noqa: E402


def measure_t_io(bo_list, layers: int = 4, settle: int = 16, steps: int = 6, recall_ctas: int = 10):
    """{B_o: [microseconds of select + diff + recall per measured layer-step]}."""
    dev = torch.device("cuda:0")
    cfg = get_config("c2").replace(n_layers=layers, batch=max(bo_list))
    pi = PulseInfer.from_workload(cfg, recall_ctas=recall_ctas)
    sess = DecodeSession(pi, cfg.batch, cfg.n_layers, host_layers=min(2, layers))
    sess.ctx_len.fill_(cfg.ctx)
    for l in range(cfg.n_layers):
        kv = gen.make_kv(cfg, l, device=dev) if l < sess.host_layers else None
        sess.load_layer(l, kv, torch.from_numpy(gen.initial_resident(cfg, l)).to(dev))
    n_q = settle + steps * len(bo_list)
    q_all = torch.stack([gen.make_queries(cfg, l, n_q, device=dev) for l in range(cfg.n_layers)], 1).contiguous()
    t = 0
    for _ in range(settle):                                 # bring the hot sets to their steady state
        sess.decode_step(q_all[t]); t += 1
    torch.cuda.synchronize()
    out = {}
    step = sess.step_count
    # largest batch first: every smaller prefix then consists of sequences that were stepped at every
    # earlier measurement, so no sequence comes back with a stale hot set
    for bo in sorted(bo_list, reverse=True):
        pairs = []
        for _ in range(steps):
            step += 1
            for l in range(cfg.n_layers):
                b, host = sess.bufs[l], sess.host_region(l)
                a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                pi.score_select(l, q_all[t, l, :bo], b.digest[:bo], sess.ctx_len[:bo], b.sel_blocks[:bo], b.sel_count[:bo], None)
                pi.diff_misses(l, step, sess.ctx_len[:bo], b.sel_blocks[:bo], b.sel_count[:bo], b.block_table[:bo],
                               b.slot_block[:bo], b.slot_stamp[:bo], b.sel_slots[:bo], b.recall_list[:bo], b.recall_count[:bo])
                pi.recall_gather_scatter(l, host[:bo], b.pool[:bo], b.recall_list[:bo], b.recall_count[:bo])
                e.record()
                pairs.append((a, e))
            t += 1
        torch.cuda.synchronize()
        out[bo] = [a.elapsed_time(e) * 1e3 for a, e in pairs]
    sess.step_count = step
    assert pi.status()[0] == 0, pi.status()
    pi.close()
    return out


def measure_t_layer(bn_list, normal_ctx: int = 4096, reps: int = 12):
    """{B_n: microseconds of one normal-batch layer (dense decode attention + FFN stand-in)}."""
    dev = torch.device("cuda:0")
    bmax = max(bn_list)
    ncfg = get_config("c2").replace(n_layers=1, batch=bmax, ctx=normal_ctx, budget_blocks=normal_ctx // 16, resident_frac=1.0)
    pi = PulseInfer.from_workload(ncfg)
    buf = LayerBuffers(pi, bmax, dev)
    buf.pool.copy_(torch.randn(buf.pool.shape, device=dev).to(torch.bfloat16))
    ident = torch.arange(ncfg.n_blocks, dtype=torch.int32, device=dev)[None, :].expand(bmax, -1).contiguous()
    buf.sel_slots.copy_(ident); buf.sel_blocks.copy_(ident); buf.sel_count.fill_(ncfg.n_blocks)
    q = torch.randn((bmax, ncfg.n_q_heads, 128), device=dev).to(torch.bfloat16)
    ctx = torch.full((bmax,), normal_ctx, dtype=torch.int32, device=dev)
    o = torch.zeros_like(q)
    w1 = torch.randn((4096, 14336), device=dev, dtype=torch.bfloat16) * 0.01
    w2 = torch.randn((14336, 4096), device=dev, dtype=torch.bfloat16) * 0.01
    x = torch.randn((bmax, 4096), device=dev, dtype=torch.bfloat16)
    out = {}
    for bn in bn_list:
        def layer():
            pi.sparse_decode_attn(0, q[:bn], buf.pool[:bn], buf.sel_slots[:bn], buf.sel_blocks[:bn], buf.sel_count[:bn],
                                  ctx[:bn], o[:bn], None)
            torch.matmul(torch.matmul(x[:bn], w1), w2)
        for _ in range(3):
            layer()
        torch.cuda.synchronize()
        torch.cuda._sleep(2_000_000)                        # the train of layers queues up behind this
        a, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            layer()
        e.record()
        torch.cuda.synchronize()
        out[bn] = a.elapsed_time(e) * 1e3 / reps
    assert pi.status()[0] == 0, pi.status()
    pi.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--bo", default="2,4,8,16,32")
    ap.add_argument("--bn", default="8,16,32,64,128")
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    bo = [int(x) for x in args.bo.split(",")]
    bn = [int(x) for x in args.bn.split(",")]
    t_io = measure_t_io(bo)
    t_layer = measure_t_layer(bn)
    grid = OverlapDepthGrid.from_timings(bo, bn, [t_io[b] for b in bo], [t_layer[b] for b in bn])
    lines = ["t_io (select + diff + recall of one layer, us): " +
             ", ".join(f"B_o={b}: {np.mean(t_io[b]):.0f} (min {min(t_io[b]):.0f}, max {max(t_io[b]):.0f})" for b in bo),
             "t_layer (dense attention over 4096 tokens + FFN stand-in, us): " + ", ".join(f"B_n={b}: {t_layer[b]:.0f}" for b in bn),
             "", "overlap depth m = mean over layer-steps of ceil(t_io / t_layer):",
             "B_o \\ B_n " + " ".join(f"{b:>6d}" for b in bn)]
    for i, b in enumerate(bo):
        lines.append(f"{b:>9d} " + " ".join(f"{grid.m[i][j]:6.2f}" for j in range(len(bn))))
    # one admission decision on the measured grid: 30 waiting requests, truncated log-normal lengths
    rng = np.random.default_rng(0)
    lengths = np.clip(np.exp(rng.normal(math.log(16384), 1.0, size=30)), 1024, 131072).astype(int).tolist()
    adm = ioaa_admit(lengths, memory_budget=300_000, offload_budget_tokens=2048, depth=grid)
    lines += ["", f"admission example on this grid: 30 waiting requests (log-normal lengths, median 16K, 1K..128K), GPU budget 300K tokens "
                  f"of KV, 2048 tokens per offloaded request:",
              "  no complete assignment fits" if adm is None else
              f"  offload the {len(adm.offload)} longest (>= {min(lengths[i] for i in adm.offload) if adm.offload else 0} tokens), "
              f"{len(adm.normal)} normal; modelled throughput {adm.throughput:.1f} requests per layer time; "
              f"{adm.nodes_visited} tree nodes visited"]
    text = "\n".join(lines)
    print(text)
    if args.out:
        Path(args.out).write_text(text + "\n" + json.dumps(dict(bo=bo, bn=bn, m=grid.m, t_io_us={b: t_io[b] for b in bo},
                                                                  t_layer_us=t_layer)) + "\n")


if __name__ == "__main__":
    main()
