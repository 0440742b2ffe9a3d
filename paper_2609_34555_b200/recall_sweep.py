"""Recall-fragmentation sweep (the synthetic restatement of the paper's two bandwidth
figures: host-to-device bandwidth against transfer granularity, Sec. 3.4, and gather-scatter
against per-block copies, Sec. 4.4.2).

    python -m paper_2609_34555_b200.recall_sweep [--reps 8] [--out FILE]

One 8B-shaped layer (batch 32, context 32768).  For block sizes 16/32/64, miss totals
8..2048 per layer, uniform-random or clustered placement:
  coalesced   one list per sequence built by pi_diff_misses from a scripted selection
              (whole blocks, all KV heads; adjacent block/slot pairs merged into extents)
  per-head    eight lists per sequence with independently drawn blocks, one (block, head)
              fragment per extent, same total bytes
both moved by pi_recall_gather_scatter and timed with CUDA events (launches queued behind a
spin kernel so host latency is not in the number).  Context lines: one cudaMemcpyAsync per
block (copy engine), the paper's staged engine (the host gathers into pinned staging in 8 MB
chunks with torch.index_select on PyTorch's intra-op thread pool, each chunk is copied while the
next is gathered, GPU scatter at the end; best wall-clock time of a few runs on this machine's host
cores), and the pinned-copy peak
of the run.
"""
from __future__ import annotations

import argparse
import json
import sys
from pathlib import Path

import numpy as np
import torch

sys.path.insert(0, str(Path(__file__).resolve().parent.parent))

from paper_2609_34555_b200 import PulseInfer, h2d_copy_ms  # noqa: E402
from paper_2609_34555_b200.runner import LayerBuffers  # noqa: E402
from workloads import generate as gen, get_config  # noqa: E402


def timed(launches, reps: int) -> float:
    """Median milliseconds of `reps` queued executions of launches[i]() (i cycles)."""
    torch.cuda.synchronize()
    torch.cuda._sleep(3_000_000)
    evs = []
    for r in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); launches[r % len(launches)](); b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    return float(np.median([a.elapsed_time(b) for a, b in evs]))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=8)
    ap.add_argument("--out", default="")
    ap.add_argument("--recall-ctas", type=int, default=10,
                    help="CTAs of the one launch timed here (the library default of 5 is sized for two launches side by side)")
    ap.add_argument("--blocks", default="16,32,64")
    ap.add_argument("--misses", default="8,32,128,512,2048")
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    rows = []
    for B in [int(x) for x in args.blocks.split(",")]:
        cfg = get_config("c5").replace(block_tokens=B, budget_blocks=max(128 * 16 // B, 16))
        nb, C, Hkv = cfg.n_blocks, cfg.pool_slots, cfg.n_kv_heads
        pi = PulseInfer.from_workload(cfg, recall_ctas=args.recall_ctas)
        host = torch.empty((cfg.batch, nb, cfg.block_bytes // 2), dtype=torch.bfloat16, pin_memory=True)
        host.view(torch.int16).random_(0, 30000)
        buf = LayerBuffers(pi, cfg.batch, dev)
        pool_flat = buf.pool.view(cfg.batch, C, cfg.block_bytes // 2)
        ctx = torch.full((cfg.batch,), cfg.ctx, dtype=torch.int32, device=dev)
        probe = torch.empty(1 << 28, dtype=torch.bfloat16, device=dev)
        peak = (1 << 29) / (h2d_copy_ms(host.view(-1)[: 1 << 28], probe, 10) * 1e-3) / 1e9
        del probe
        pin = gen.pinned_blocks(cfg)
        K = cfg.budget_blocks
        for total in [int(x) for x in args.misses.split(",")]:
            if total > cfg.batch * cfg.k_mid:
                continue
            for clustered in (False, True):
                # ---- coalesced lists through the diff kernel: empty pool (only sink/local resident),
                # selection = sink/local + the scripted missing blocks
                res = np.full((cfg.batch, C), -1, np.int32)
                res[:, : len(pin)] = pin
                res_d = torch.from_numpy(res).to(dev)
                sels, lists = [], []
                for rep in range(2):
                    miss = gen.scripted_misses(cfg, total, clustered, extra=rep)
                    sel = np.full((cfg.batch, K), -1, np.int32)
                    cnt = np.zeros(cfg.batch, np.int32)
                    for s, m in enumerate(miss):
                        row = np.sort(np.concatenate([pin, m]))[:K]
                        sel[s, : len(row)] = row
                        cnt[s] = len(row)
                    sel_d, cnt_d = torch.from_numpy(sel).to(dev), torch.from_numpy(cnt).to(dev)
                    pi.table_init(res_d, buf.block_table, buf.slot_block, buf.slot_stamp)
                    lst = torch.zeros((cfg.batch, K, 4), dtype=torch.int32, device=dev)
                    lcnt = torch.zeros((cfg.batch,), dtype=torch.int32, device=dev)
                    pi.diff_misses(0, 1, ctx, sel_d, cnt_d, buf.block_table, buf.slot_block, buf.slot_stamp,
                                   buf.sel_slots, lst, lcnt)
                    lists.append((lst, lcnt))
                torch.cuda.synchronize()
                n_ext = int(lists[0][1].sum().item())
                moved = int((lists[0][0][:, :, 2] * (torch.arange(K, device=dev)[None, :] < lists[0][1][:, None])).sum().item())
                assert moved == total, (moved, total)
                ms = timed([lambda l=l: pi.recall_gather_scatter(0, host, pool_flat, l[0], l[1]) for l in lists], args.reps)
                bytes_ = total * cfg.block_bytes
                rows.append(dict(block=B, misses=total, placement="clustered" if clustered else "uniform",
                                 lists="coalesced", extents=n_ext, extent_kb=bytes_ / n_ext / 1024,
                                 us=ms * 1e3, gbs=bytes_ / (ms * 1e-3) / 1e9, frac_of_h2d_peak=bytes_ / (ms * 1e-3) / 1e9 / peak))
                # ---- per-head fragmented lists: independent draws per head, one fragment per extent
                per = max(1, -(-total // cfg.batch))
                hl = []
                for rep in range(2):
                    lst = torch.zeros((cfg.batch * Hkv, per, 4), dtype=torch.int32)
                    lcnt = torch.zeros((cfg.batch * Hkv,), dtype=torch.int32)
                    for h in range(Hkv):
                        miss = gen.scripted_misses(cfg, total, clustered, extra=100 + 10 * h + rep)
                        for s, m in enumerate(miss):
                            n = len(m)
                            e = torch.zeros((n, 4), dtype=torch.int32)
                            e[:, 0] = torch.from_numpy(m.astype(np.int32)) * Hkv + h
                            e[:, 1] = (torch.arange(n, dtype=torch.int32) + len(pin)) * Hkv + h
                            e[:, 2] = 1
                            e[:, 3] = torch.arange(n, dtype=torch.int32)
                            lst[s * Hkv + h, :n] = e
                            lcnt[s * Hkv + h] = n
                    hl.append((lst.to(dev), lcnt.to(dev)))
                ms = timed([lambda l=l: pi.recall_gather_scatter(0, host, pool_flat, l[0], l[1], lists_per_seq=Hkv,
                                                                 unit_bytes=cfg.frag_bytes) for l in hl], args.reps)
                rows.append(dict(block=B, misses=total, placement="clustered" if clustered else "uniform",
                                 lists="per-head", extents=total * Hkv, extent_kb=cfg.frag_bytes / 1024,
                                 us=ms * 1e3, gbs=bytes_ / (ms * 1e-3) / 1e9, frac_of_h2d_peak=bytes_ / (ms * 1e-3) / 1e9 / peak))
            # ---- context: the copy engine, one cudaMemcpyAsync per missing block (uniform placement)
            if total <= 512:
                miss = gen.scripted_misses(cfg, total, False, extra=7)
                pairs = [(s, int(b), len(pin) + i) for s, m in enumerate(miss) for i, b in enumerate(m)]
                def per_block():
                    for s, b, slot in pairs:
                        pool_flat[s, slot].copy_(host[s, b], non_blocking=True)
                torch.cuda.synchronize()
                a, bb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); per_block(); bb.record(); torch.cuda.synchronize()
                ms = a.elapsed_time(bb)
                rows.append(dict(block=B, misses=total, placement="uniform", lists="cudaMemcpyAsync per block",
                                 extents=total, extent_kb=cfg.block_bytes / 1024, us=ms * 1e3,
                                 gbs=total * cfg.block_bytes / (ms * 1e-3) / 1e9,
                                 frac_of_h2d_peak=total * cfg.block_bytes / (ms * 1e-3) / 1e9 / peak))
            # ---- context: the paper's staged engine (Sec. 4.4.2): the CPU gathers the scattered blocks
            # into one pinned staging buffer, ONE copy moves it to a device staging buffer, a GPU kernel
            # scatters it into the slots (here: the recall kernel reading device memory).  Wall clock,
            # because the host does part of the work; the lists are already on the host.
            miss = gen.scripted_misses(cfg, total, False, extra=7)
            flat = torch.from_numpy(np.concatenate([s * nb + m.astype(np.int64) for s, m in enumerate(miss)]))
            stage_host = torch.empty((total, cfg.block_bytes // 2), dtype=torch.bfloat16, pin_memory=True)
            stage_dev = torch.empty((total, cfg.block_bytes // 2), dtype=torch.bfloat16, device=dev)
            lst = torch.zeros((cfg.batch, 1, 4), dtype=torch.int32)
            lcnt = torch.zeros((cfg.batch,), dtype=torch.int32)
            off = 0
            for s, m in enumerate(miss):
                if len(m):
                    lst[s, 0] = torch.tensor([off, len(pin), len(m), 0], dtype=torch.int32)
                    lcnt[s] = 1
                off += len(m)
            lst_d, lcnt_d = lst.to(dev), lcnt.to(dev)
            host_pages = host.view(cfg.batch * nb, cfg.block_bytes // 2)
            import time as _time
            # chunks of about 8 MB: the copy of chunk i runs while the host threads gather chunk i + 1
            per_chunk = max(1, (8 << 20) // cfg.block_bytes)
            best = float("inf")
            for _ in range(max(3, args.reps // 2)):
                torch.cuda.synchronize()
                t0 = _time.perf_counter()
                for c0 in range(0, total, per_chunk):
                    c1 = min(total, c0 + per_chunk)
                    torch.index_select(host_pages, 0, flat[c0:c1], out=stage_host[c0:c1])
                    stage_dev[c0:c1].copy_(stage_host[c0:c1], non_blocking=True)
                pi.recall_gather_scatter(0, stage_dev, pool_flat, lst_d, lcnt_d, host_seq_stride=0)
                torch.cuda.synchronize()
                best = min(best, _time.perf_counter() - t0)
            rows.append(dict(block=B, misses=total, placement="uniform", lists="staged: CPU gather+DMA", extents=total,
                             extent_kb=cfg.block_bytes / 1024, us=best * 1e6, gbs=total * cfg.block_bytes / best / 1e9,
                             frac_of_h2d_peak=total * cfg.block_bytes / best / 1e9 / peak))
            del stage_host, stage_dev
        rows.append(dict(block=B, h2d_peak_gbs=peak))
        pi.close()
        del host, buf
    lines = [f"{'B':>3s} {'misses':>6s} {'placement':>10s} {'lists':>26s} {'extents':>8s} {'KB/ext':>8s} {'us':>9s} {'GB/s':>7s} {'of peak':>8s}"]
    for r in rows:
        if "h2d_peak_gbs" in r:
            lines.append(f"{r['block']:3d} pinned cudaMemcpyAsync peak of this run: {r['h2d_peak_gbs']:.2f} GB/s (512 MiB, best of 10)")
        else:
            lines.append(f"{r['block']:3d} {r['misses']:6d} {r['placement']:>10s} {r['lists']:>26s} {r['extents']:8d} {r['extent_kb']:8.1f} "
                         f"{r['us']:9.1f} {r['gbs']:7.2f} {r['frac_of_h2d_peak']:8.3f}")
    text = "\n".join(lines)
    print(text)
    if args.out:
        Path(args.out).write_text(text + "\n" + "\n".join(json.dumps(r) for r in rows) + "\n")


if __name__ == "__main__":
    main()
