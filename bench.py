#!/usr/bin/env python
"""Benchmark of the decode recall path (score -> select -> diff -> recall -> attention).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl reference]

One "step" is one decode step of the whole batch: every layer runs one layer-step of the
path.  The metric is layer-steps per second.  Rank 0 prints ONE JSON line.

  value        inputs (queries) already in HBM, the pipelined form (selection stream, two recall
               streams, attention stream)
  e2e          the same through DecodeSession with the queries coming from pinned host memory
               and the outputs copied back to pinned host memory inside the timed region
  roofline     the kernel that dominates the step (the recall pull, bound by the host link)
  rooflines    the HBM-bound kernels (attention, scoring) against the measured HBM copy rate
  cpu_baseline the CPU oracle timed on a bounded sample of the same workload

With --gpus N > 1 every rank runs its own batch of sequences (weak scaling, no collective
on the data path); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import numpy as np
import torch

METRIC = "decode layer-steps/s (select+recall+attn); recall GB/s vs measured H2D peak"
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (attn_kernel_c2.txt, score_select_kernel_c2.txt): same per-layer shapes as the bench
# (recall_kernel: its reads cross the host link and its 5 MB of writes stay in L2 during the launch,
# so DRAM sees next to nothing)
NCU_DRAM_TRAFFIC = {"c2": {"attn_kernel": 134.5e6 + 4.3e6, "score_select_kernel": 18.9e6, "recall_kernel": 21.0e3}}
FALLBACK_HBM_GBS = 6650.0


def measured_peaks() -> dict:
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, source="fallback")


def mem_available_bytes() -> int:
    for line in Path("/proc/meminfo").read_text().splitlines():
        if line.startswith("MemAvailable"):
            return int(line.split()[1]) * 1024
    return 0


class ClockSampler:
    """SM clocks and throttle reasons sampled (read-only, through NVML) every 10 ms while the
    timed region runs."""
    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20}

    def __init__(self, index: int):
        self.index, self.samples, self.max_mhz, self.reasons = index, [], None, set()
        self._stop, self._thread, self._err = None, None, None

    def _run(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            while not self._stop.is_set():
                self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                bits = int(pynvml.nvmlDeviceGetCurrentClocksEventReasons(h))
                for name, mask in self.REASONS.items():
                    if bits & mask:
                        self.reasons.add(name)
                self._stop.wait(0.01)
            pynvml.nvmlShutdown()
        except Exception as e:                       # noqa: BLE001 - reported in the JSON line
            self._err = repr(e)

    def start(self):
        import threading
        self._stop = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        self._thread.join(timeout=5)
        if self._err or not self.samples:
            return dict(sm_mhz=None, sm_max_mhz=self.max_mhz, samples=len(self.samples),
                        reasons=["clock sampling failed: " + str(self._err)])
        return dict(sm_mhz=statistics.median(self.samples), sm_max_mhz=self.max_mhz, samples=len(self.samples),
                    reasons=sorted(self.reasons))


def build_session(cfg, rank: int, host_layers_arg: int, world: int, recall_ctas: int = 0, ctx_start: int = 0,
                  paged: bool = False, recall_streams: int = 2, attn_ctas: int = 0):
    from paper_2609_34555_b200 import PulseInfer
    from paper_2609_34555_b200.runner import DecodeSession
    from workloads import generate as gen

    per_layer = cfg.batch * cfg.n_blocks * cfg.block_bytes
    if host_layers_arg > 0:
        R = min(host_layers_arg, cfg.n_layers)
    else:
        budget = 0.55 * mem_available_bytes() / max(1, world)
        R = int(max(1, min(cfg.n_layers, budget // per_layer)))
    pi = PulseInfer.from_workload(cfg, recall_ctas=recall_ctas, attn_ctas=attn_ctas)
    while True:                                  # pinning can fail below the MemAvailable estimate: halve and retry
        try:
            sess = DecodeSession(pi, cfg.batch, cfg.n_layers, host_layers=R, paged=paged, page_seed=cfg.seed,
                                 recall_streams=recall_streams)
            break
        except RuntimeError:
            if R == 1:
                raise
            R = max(1, R // 2)
            torch.cuda.empty_cache()
    ctx0 = ctx_start or cfg.ctx                 # runs that append tokens start short of the full context
    sess.ctx_len.fill_(ctx0)
    dev = sess.device
    short = cfg.replace(ctx=ctx0)
    for l in range(cfg.n_layers):
        # layers beyond the host regions share region l % R; a paged region cannot be read back in
        # block order, so its digests come from the regenerated keys of the layer that filled it
        kv = gen.make_kv(cfg, l % R, device=dev) if (l < R or paged) else None
        res_np = np.full((cfg.batch, cfg.pool_slots), -1, np.int32)
        r0 = gen.initial_resident(short, l)[:, :cfg.pool_slots]
        res_np[:, :r0.shape[1]] = r0
        res = torch.from_numpy(res_np).to(dev)
        sess.load_layer(l, kv, res, store=l < R)
        del kv
    torch.cuda.synchronize()
    return pi, sess, R


def make_all_queries(cfg, steps: int, device) -> torch.Tensor:
    """[steps][n_layers][batch][Hq][D] bf16 on `device`."""
    from workloads import generate as gen
    per_layer = [gen.make_queries(cfg, l, steps, device=device) for l in range(cfg.n_layers)]
    return torch.stack(per_layer, dim=1).contiguous()


def rank_config(base, rank: int):
    """Every rank runs the same shape on its own sequences: only the seed differs."""
    return base.replace(seed=base.seed + 7919 * rank)


def max_over_ranks(ms: float, world: int, device) -> float:
    if world <= 1:
        return ms
    import torch.distributed as dist
    tm = torch.tensor([ms], device=device)
    dist.all_reduce(tm, op=dist.ReduceOp.MAX)
    return float(tm.item())


def whole_job_value(world: int, steps: int, n_layers: int, ms: float) -> float:
    """Layer-steps per second of the whole job: every rank did steps * n_layers of them."""
    return world * steps * n_layers / (ms * 1e-3)


def parse_cpulist(text: str) -> set:
    """'0-3,8,10-11' -> {0, 1, 2, 3, 8, 10, 11} (the format of sysfs cpulist files)."""
    cpus = set()
    for part in text.strip().split(","):
        if not part:
            continue
        lo, _, hi = part.partition("-")
        cpus.update(range(int(lo), int(hi or lo) + 1))
    return cpus


def bind_near_gpu(index: int):
    """Multi-rank runs: keep this process (and so the pages of the pinned host store it is about to
    allocate, which land on the node of the allocating thread) on the NUMA node of its GPU, so that
    every rank's recall crosses only its own GPU's host link.  Best effort: returns the node or None."""
    try:
        bus = torch.cuda.get_device_properties(index).pci_bus_id
        dom = torch.cuda.get_device_properties(index).pci_domain_id
        dev_id = torch.cuda.get_device_properties(index).pci_device_id
        path = Path(f"/sys/bus/pci/devices/{dom:04x}:{bus:02x}:{dev_id:02x}.0/numa_node")
        node = int(path.read_text().strip())
        if node < 0:
            return None
        cpus = parse_cpulist(Path(f"/sys/devices/system/node/node{node}/cpulist").read_text())
        cpus &= os.sched_getaffinity(0)
        if not cpus:
            return None
        os.sched_setaffinity(0, cpus)
        return node
    except Exception:                                # noqa: BLE001 - placement hint only
        return None


def run_ours(args) -> dict:
    from paper_2609_34555_b200 import h2d_copy_ms
    from paper_2609_34555_b200.runner import StageTimer
    from workloads import get_config

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    numa_node = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        numa_node = bind_near_gpu(local)
    base = get_config(args.config)
    cfg = rank_config(base, rank)
    if args.layers > 0:                       # profiling only: fewer layers of the same shape
        cfg = cfg.replace(n_layers=min(args.layers, cfg.n_layers), name=f"{cfg.name}[{args.layers} layers only]")
    K, W = args.steps, max(3, args.warmup)

    t_setup = time.time()
    n_e2e = K if not args.no_e2e else 0
    n_serial = min(K, 4)
    n_graph = min(K, 16) if not args.no_graph else 0
    total_steps = args.settle + W + K + 4 * n_serial + n_e2e + n_graph + 1
    pi, sess, R = build_session(cfg, rank, args.host_layers, world, args.recall_ctas,
                                ctx_start=cfg.ctx - total_steps - 1 if args.append else 0, paged=args.paged,
                                recall_streams=args.recall_streams, attn_ctas=args.attn_ctas)
    q_all = make_all_queries(cfg, total_steps, dev)
    setup_s = time.time() - t_setup

    # pinned host -> device copy peak, measured in this run (1 GiB, best of 10)
    probe_bytes = min(1 << 30, sess.host_kv[0].numel() * 2)
    probe_src = sess.host_kv[0].view(-1)[: probe_bytes // 2]
    probe_dst = torch.empty(probe_bytes // 2, dtype=torch.bfloat16, device=dev)
    h2d_gbs = probe_bytes / (h2d_copy_ms(probe_src, probe_dst, reps=10) * 1e-3) / 1e9
    del probe_dst

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # scripted miss counts (config 3): a pre-pass computes every step's selections (they depend
    # on queries and digests only), then the hot-set contents of every (layer, step) are chosen so
    # that exactly the drawn heavy-tailed number of selected middle blocks is missing
    scripts = None
    if cfg.miss_script == "pareto":
        from workloads import generate as gen
        scripts = []
        b0 = sess.bufs[0]
        tmp_sel, tmp_cnt = torch.empty_like(b0.sel_blocks), torch.empty_like(b0.sel_count)
        for tt in range(q_all.shape[0]):
            per_layer = []
            for l in range(cfg.n_layers):
                pi.score_select(l, q_all[tt, l], sess.bufs[l].digest, sess.ctx_len, tmp_sel, tmp_cnt)
                m = gen.pareto_miss_counts(cfg, l, tt)
                per_layer.append(gen.scripted_resident_lists(cfg, tmp_sel, tmp_cnt, m, gen.seed_for(cfg, gen.T_PARETO, l, 7919 + tt)))
            scripts.append(torch.stack(per_layer))
        torch.cuda.synchronize()
    script = (lambda i: scripts[i]) if scripts is not None else (lambda i: None)
    new_kv = None
    if args.append:
        gk = torch.Generator(device=dev).manual_seed(cfg.seed * 7 + 1)
        shape = (cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.head_dim)
        new_kv = (torch.randn(shape, device=dev, generator=gk).to(torch.bfloat16),
                  torch.randn(shape, device=dev, generator=gk).to(torch.bfloat16))     # the same token values every step

    # settling steps (workload preparation, not warm-up): the hot set starts as a uniform
    # draw, so the first steps recall far more than the steady state does
    t = 0
    cold = None
    for i in range(args.settle):
        if i == 0:
            pi.stats(reset=True)
        sess.decode_step(q_all[t], resident_script=script(t), new_kv=new_kv); t += 1
        if i == 0:                                         # the cold first step, reported apart
            torch.cuda.synchronize()
            st0 = pi.stats(reset=True)
            cold = st0["missing_blocks"] / max(1, st0["sequences"])
    for _ in range(W):
        sess.decode_step(q_all[t], resident_script=script(t), new_kv=new_kv); t += 1
    barrier()
    pi.stats(reset=True)

    # ---------------- timed region: K pipelined decode steps, inputs resident in HBM
    sampler = ClockSampler(local)
    sampler.start()
    # the stage times of this region come from the events that order the streams anyway (no event
    # is added to any stream: extra events on the recall streams cost about 6 % of the rate)
    timer = StageTimer(light=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(K):
        sess.decode_step(q_all[t], timer=timer, resident_script=script(t), new_kv=new_kv); t += 1
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    stats = pi.stats(reset=True)
    stages = timer.light_summary(e0)
    status = pi.status()
    if status[0] != 0:
        raise RuntimeError(f"device status after the timed region: {status}")

    # ---------------- the same pipelined form with events around every call (per-call picture)
    det_timer = StageTimer()
    for _ in range(n_serial):
        sess.decode_step(q_all[t], timer=det_timer, resident_script=script(t), new_kv=new_kv); t += 1
    torch.cuda.synchronize()
    det = det_timer.summary()
    pi.stats(reset=True)

    # ---------------- serial form (one stream), a few steps, for the per-stage picture
    ser_timer = StageTimer()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(n_serial):
        sess.decode_step(q_all[t], overlapped=False, timer=ser_timer, resident_script=script(t), new_kv=new_kv); t += 1
    s1.record()
    torch.cuda.synchronize()
    serial_ms = s0.elapsed_time(s1) / max(1, n_serial)
    ser_stats = pi.stats(reset=True)
    ser = ser_timer.summary()
    # the same chain without events between the calls (events keep the dependent launches of the chain
    # from overlapping their predecessors)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for _ in range(n_serial):
        sess.decode_step(q_all[t], overlapped=False, resident_script=script(t), new_kv=new_kv); t += 1
    p1.record()
    torch.cuda.synchronize()
    serial_plain_ms = p0.elapsed_time(p1) / max(1, n_serial)
    pi.stats(reset=True)

    # ---------------- distribution of the miss counts: a few more steps, read back after each
    # (per sequence and layer-step: units of the recall lists)
    hist_edges = [0, 1, 3, 5, 9, 17, 33, 65, 1 << 30]
    hist = [0] * (len(hist_edges) - 1)
    for _ in range(n_serial):
        sess.decode_step(q_all[t], resident_script=script(t), new_kv=new_kv); t += 1
        torch.cuda.synchronize()
        for b in sess.bufs:
            idx = torch.arange(b.recall_list.shape[1], device=dev)[None, :] < b.recall_count[:, None]
            per_seq = (b.recall_list[:, :, 2] * idx).sum(dim=1).cpu().numpy()
            for k in range(len(hist)):
                hist[k] += int(((per_seq >= hist_edges[k]) & (per_seq < hist_edges[k + 1])).sum())
    pi.stats(reset=True)
    miss_hist = {("0" if k == 0 else f"{hist_edges[k]}-{hist_edges[k + 1] - 1}" if k < len(hist) - 1 else f"{hist_edges[k]}+"): hist[k]
                 for k in range(len(hist))}

    # ---------------- the pipelined step captured once into a CUDA graph and replayed (scripted-miss
    # workloads reset their tables from the host every step and stay eager)
    graph_leg = None
    if n_graph and scripts is None:
        q_static = q_all[t].clone()
        graph = sess.capture_step(q_static, new_kv_static=new_kv)
        q_static.copy_(q_all[t]); sess.replay_step(graph); t += 1          # one untimed replay
        barrier()
        pi.stats(reset=True)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(n_graph):
            q_static.copy_(q_all[t]); t += 1
            sess.replay_step(graph)
        g1.record()
        barrier()
        g_ms = max_over_ranks(g0.elapsed_time(g1), world, dev)
        g_stats = pi.stats(reset=True)
        graph_leg = dict(value=whole_job_value(world, n_graph, cfg.n_layers, g_ms), unit="layer-steps/s", steps=n_graph,
                         misses_per_seq_layer_step=g_stats["missing_blocks"] / max(1, g_stats["sequences"]),
                         note="one decode step (all layers, all streams) captured once, replayed per step; the step's "
                              "queries are copied into the graph's input buffer inside the timed region")
        del graph

    # ---------------- the two HBM-bound kernels back to back: one launch per layer (every layer has its
    # own pool / digests, so each launch reads data that left L2 long ago), ONE event pair around the
    # whole train of launches, so that the per-call cost of the events themselves is not in the number
    def back_to_back(fn) -> float:
        best = float("inf")
        for _ in range(3):
            torch.cuda.synchronize()
            b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda._sleep(5_000_000)                 # the launches queue up behind this
            b0.record(); fn(); b1.record()
            torch.cuda.synchronize()
            best = min(best, b0.elapsed_time(b1) / cfg.n_layers)
        return best
    qb = q_all[t - 1]
    def attn_train():
        for l in range(cfg.n_layers):
            b = sess.bufs[l]
            pi.sparse_decode_attn(l, qb[l], b.pool, b.sel_slots, b.sel_blocks, b.sel_count, sess.ctx_len, sess.out[l], None)
    def score_train():
        for l in range(cfg.n_layers):
            b = sess.bufs[l]
            pi.score_select(l, qb[l], b.digest, sess.ctx_len, b.sel_blocks, b.sel_count, None)
    b2b_attn_ms = back_to_back(attn_train)
    sel_keep = [(b.sel_blocks.clone(), b.sel_count.clone()) for b in sess.bufs]
    b2b_score_ms = back_to_back(score_train)            # rewrites the selections with those of query qb ...
    for b, (sb, sc) in zip(sess.bufs, sel_keep):        # ... so put the step's own selections back
        b.sel_blocks.copy_(sb); b.sel_count.copy_(sc)
    torch.cuda.synchronize()

    # ---------------- end to end: queries from pinned host memory, outputs back to it
    e2e = None
    if n_e2e:
        q_host = q_all[t:t + n_e2e].cpu().pin_memory()
        out_host = [torch.empty(sess.out.shape, dtype=torch.bfloat16, pin_memory=True) for _ in range(2)]
        e2e_graph = bool(n_graph) and scripts is None and not args.append
        if e2e_graph:
            sess.prepare_host_graph()                     # capture outside the timed region
        barrier()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        # every step: its queries come up from pinned host memory and its outputs go back to pinned host
        # memory; both copies are double-buffered so that they run beside the neighbouring steps
        sess.decode_steps_from_host([q_host[i] for i in range(n_e2e)], out_host,
                                    resident_scripts=None if scripts is None else [script(t + i) for i in range(n_e2e)],
                                    use_graph=e2e_graph)
        a1.record()
        barrier()
        e2e_ms = max_over_ranks(a0.elapsed_time(a1), world, dev)
        e2e_stats = pi.stats(reset=True)
        e2e = dict(value=whole_job_value(world, n_e2e, cfg.n_layers, e2e_ms), unit="layer-steps/s",
                   h2d_bytes_per_step=int(q_host[0].numel() * 2), d2h_bytes_per_step=int(out_host[0].numel() * 2),
                   misses_per_seq_layer_step=e2e_stats["missing_blocks"] / max(1, e2e_stats["sequences"]),
                   step_form="CUDA-graph replay" if e2e_graph else "eager launches",
                   note="host KV store is read by the recall kernel in both forms")

    peaks = measured_peaks()
    traffic = NCU_DRAM_TRAFFIC.get(base.name, {}) if args.layers == 0 else {}
    n_launch = K * cfg.n_layers
    recall_bytes = stats["missing_blocks"] * cfg.block_bytes
    # union of the launches' intervals (they overlap across the recall streams); the first launch of
    # each recall stream has no bounded start and is left out of bytes and time alike
    n_rec = stages["recall"]["launches"]
    recall_bytes = recall_bytes * n_rec / max(1, n_launch)
    recall_s = stages["recall"]["busy_ms"] * 1e-3
    attn_bytes_launch = stats["selected_blocks"] / max(1, n_launch) * cfg.block_bytes + 2 * cfg.batch * cfg.n_q_heads * 128 * 2
    score_bytes_launch = cfg.batch * cfg.n_blocks * 512 + cfg.batch * cfg.group * 128 * 2
    def hbm_entry(name, bytes_launch, st, traffic):
        ach = bytes_launch / (st["mean_ms"] * 1e-3) / 1e9
        return dict(kernel=name, bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=ach / peaks["hbm_gbs"], peak_source=peaks["source"], traffic=traffic,
                    bytes_per_launch=int(bytes_launch), mean_us=st["mean_ms"] * 1e3)
    ser_recall_gbs = ser_stats["missing_blocks"] * cfg.block_bytes / max(1e-9, ser["recall"]["total_ms"] * 1e-3) / 1e9
    recall_gbs = recall_bytes / max(1e-9, recall_s) / 1e9
    line = {
        "metric": METRIC, "value": whole_job_value(world, K, cfg.n_layers, ms), "unit": "layer-steps/s",
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms / K, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: {cfg.n_layers} layers x batch {cfg.batch} x ctx {cfg.ctx}, "
                               f"Hq/Hkv {cfg.n_q_heads}/{cfg.n_kv_heads}, block {cfg.block_tokens}, budget {cfg.budget_blocks} "
                               f"blocks, pool {cfg.pool_slots} slots/seq/layer, AR(1) queries a={cfg.ar1}",
                   "host_layout": "paged arena, random page order" if args.paged else "block-major per sequence",
                   "numa_node_of_rank0": numa_node,
                   "host_kv_layers": R, "host_kv_pinned_gb": R * cfg.batch * cfg.n_blocks * cfg.block_bytes / 2 ** 30,
                   "l2": f"inputs larger than L2 (pool reads {cfg.batch * cfg.budget_blocks * cfg.block_bytes / 2**20:.0f} MiB and digests "
                         f"{cfg.batch * cfg.n_blocks * 512 / 2**20:.0f} MiB per layer-step, {cfg.n_layers} distinct layers)",
                   "pipeline": f"select+diff on stream A, recall pulls rotating over {len(sess.recall_streams)} stream(s), attention on the main stream",
                   "sequence_layer_steps_per_s": world * K * cfg.n_layers * cfg.batch / (ms * 1e-3),
                   "misses_per_seq_layer_step": stats["missing_blocks"] / max(1, stats["sequences"]),
                   "misses_per_seq_layer_step_cold_first_step": cold,
                   "miss_histogram_per_seq_layer_step": miss_hist,
                   "miss_script": cfg.miss_script or "none (LRU)", "append": bool(args.append),
                   "settle_steps": args.settle, "setup_s": round(setup_s, 1)},
        "clocks": clocks, "e2e": e2e, "gpu_launches": 5 * n_launch,      # launches inside the timed region only
        "roofline": {"kernel": "recall_kernel", "bound": "host_link_h2d", "achieved": recall_gbs, "peak": h2d_gbs,
                     "unit": "GB/s", "frac": recall_gbs / h2d_gbs,
                     "peak_source": "pinned cudaMemcpyAsync H2D of 1 GiB, best of 10, this run (nominal 64 GB/s PCIe Gen5 x16)",
                     "traffic": traffic.get("recall_kernel"),
                     "traffic_note": "DRAM bytes per launch under ncu: the reads come over the host link, the writes stay in L2",
                     "bytes_per_launch": int(recall_bytes / max(1, n_rec)),
                     "mean_us": stages["recall"]["mean_ms"] * 1e3, "busy_us_per_launch": recall_s * 1e6 / max(1, n_rec),
                     "concurrent_streams": len(sess.recall_streams),
                     "achieved_is": "recalled bytes / time during which a recall launch was running (launches of consecutive "
                                    "layers overlap across the recall streams; with one stream this is bytes per launch / "
                                    "mean launch duration)",
                     "alone": {"achieved": ser_recall_gbs, "frac": ser_recall_gbs / h2d_gbs}},
        "rooflines": [hbm_entry("attn_kernel + attn_merge_kernel (timed region, recalls running beside it)", attn_bytes_launch, stages["attn"], traffic.get("attn_kernel")),
                      hbm_entry("score_select_kernel (pipelined form, events around every call)", score_bytes_launch, det["score_select"], traffic.get("score_select_kernel")),
                      hbm_entry("attn_kernel + attn_merge_kernel (serial form, nothing else running)", attn_bytes_launch, ser["attn"], traffic.get("attn_kernel")),
                      hbm_entry("score_select_kernel (serial form)", score_bytes_launch, ser["score_select"], traffic.get("score_select_kernel")),
                      hbm_entry("attn_kernel + attn_merge_kernel (one launch per layer back to back, one event pair around all)", attn_bytes_launch, dict(mean_ms=b2b_attn_ms), traffic.get("attn_kernel")),
                      hbm_entry("score_select_kernel (one launch per layer back to back, one event pair around all)", score_bytes_launch, dict(mean_ms=b2b_score_ms), traffic.get("score_select_kernel"))],
        "stages_us": {k: v["mean_ms"] * 1e3 for k, v in stages.items() if v["launches"]},
        "stages_us_events_around_every_call": {k: v["mean_ms"] * 1e3 for k, v in det.items() if v["launches"]},
        "graph_replay": graph_leg,
        "serial": {"layer_steps_per_s": cfg.n_layers / (serial_ms * 1e-3),
                   "layer_steps_per_s_without_events": cfg.n_layers / (serial_plain_ms * 1e-3),
                   "stages_us": {k: v["mean_ms"] * 1e3 for k, v in ser.items() if v["launches"]}},
        "h2d_peak_gbs": h2d_gbs,
    }
    if rank == 0 and not args.no_cpu and world == 1:
        line["cpu_baseline"] = cpu_baseline(cfg, sess, budget_s=args.cpu_seconds)
    return line if rank == 0 else {}


def oracle_state(cfg, sess, layers):
    """numpy state of the oracle for some layers, initialised like the GPU's was."""
    import oracle
    from workloads import generate as gen
    st = {}
    for l in layers:
        host = sess.host_region(l)
        kvb = oracle.bits(host)                              # view of the pinned store
        h = cfg.solo_head(l)
        dg = np.stack([oracle.build_digest(kvb[s], cfg.ctx, h) for s in range(cfg.batch)])
        res = gen.initial_resident(cfg, l)
        table = np.full((cfg.batch, cfg.n_blocks), -1, np.int32)
        pool = np.zeros((cfg.batch, cfg.pool_slots) + kvb.shape[2:], np.uint16)
        for s in range(cfg.batch):
            ok = res[s] >= 0
            table[s, res[s][ok]] = np.nonzero(ok)[0]
            pool[s, ok] = kvb[s, res[s][ok]]
        st[l] = dict(kvb=kvb, digest=dg, table=table, slot_block=res.copy(),
                     slot_stamp=np.zeros((cfg.batch, cfg.pool_slots), np.uint32), pool=pool, h=h)
    return st


def cpu_baseline(cfg, sess, budget_s: float) -> dict:
    """The oracle, as it stands, on a bounded sample: whole-batch layer-steps of the first
    layers with the same queries, until about `budget_s` seconds of CPU work are done."""
    import oracle
    from workloads import generate as gen
    layers = list(range(min(2, cfg.n_layers)))
    st = oracle_state(cfg, sess, layers)
    q = {l: oracle.bits(gen.make_queries(cfg, l, 64, device="cpu")) for l in layers}
    ctx_len = np.full(cfg.batch, cfg.ctx, np.int32)
    done, t0, step = 0, time.perf_counter(), 0
    while True:
        step += 1
        for l in layers:
            s = st[l]
            r = oracle.layer_step(ctx_len, cfg.n_blocks, cfg.block_tokens, cfg.n_kv_heads, s["h"], cfg.budget_blocks,
                                  cfg.n_sink_blocks, cfg.n_local_blocks, step, q[l][(step - 1) % 64], s["digest"],
                                  s["kvb"], s["table"], s["slot_block"], s["slot_stamp"], s["pool"])
            assert r["rc"] == 0
            done += 1
        el = time.perf_counter() - t0
        if el >= budget_s or step >= 4096:
            break
    cores = oracle.num_threads()
    # the same on one thread, two layer-steps (context: what the loop over sequences gains)
    oracle.set_num_threads(1)
    t1 = time.perf_counter()
    for l in layers:
        s = st[l]
        step += 1
        r = oracle.layer_step(ctx_len, cfg.n_blocks, cfg.block_tokens, cfg.n_kv_heads, s["h"], cfg.budget_blocks,
                              cfg.n_sink_blocks, cfg.n_local_blocks, step, q[l][(step - 1) % 64], s["digest"],
                              s["kvb"], s["table"], s["slot_block"], s["slot_stamp"], s["pool"])
        assert r["rc"] == 0
    single = len(layers) / (time.perf_counter() - t1)
    oracle.set_num_threads(cores)
    return dict(value=done / el, unit="layer-steps/s", cores=cores, kind="oracle", single_thread_value=single,
                sample=f"{done} whole-batch layer-steps (layers {layers}, {step - len(layers)} decode steps) in {el:.1f} s; "
                       f"host: {os.cpu_count()} cores")


def run_reference(args) -> dict:
    """The reference arm: the CPU oracle timed on bounded samples of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return {}
    import oracle
    from workloads import generate as gen, get_config
    cfg = get_config(args.config)
    K, W = args.steps, max(3, args.warmup)
    # a bounded sample: one layer of the model, the whole batch, one layer-step per bench step
    layer = 0
    kv = gen.make_kv(cfg, layer)
    kvb = oracle.bits(kv)
    h = cfg.solo_head(layer)
    dg = np.stack([oracle.build_digest(kvb[s], cfg.ctx, h) for s in range(cfg.batch)])
    res = gen.initial_resident(cfg, layer)
    table = np.full((cfg.batch, cfg.n_blocks), -1, np.int32)
    pool = np.zeros((cfg.batch, cfg.pool_slots) + kvb.shape[2:], np.uint16)
    for s in range(cfg.batch):
        ok = res[s] >= 0
        table[s, res[s][ok]] = np.nonzero(ok)[0]
        pool[s, ok] = kvb[s, res[s][ok]]
    sb, stmp = res.copy(), np.zeros((cfg.batch, cfg.pool_slots), np.uint32)
    q = oracle.bits(gen.make_queries(cfg, layer, W + K))
    ctx_len = np.full(cfg.batch, cfg.ctx, np.int32)
    per = max(1, min(cfg.n_layers, args.ref_layer_steps))

    def one(step):
        for _ in range(per):
            r = oracle.layer_step(ctx_len, cfg.n_blocks, cfg.block_tokens, cfg.n_kv_heads, h, cfg.budget_blocks,
                                  cfg.n_sink_blocks, cfg.n_local_blocks, step, q[step - 1], dg, kvb, table, sb, stmp, pool)
            assert r["rc"] == 0
    for t in range(W):
        one(t + 1)
    t0 = time.perf_counter()
    for t in range(W, W + K):
        one(t + 1)
    el = time.perf_counter() - t0
    value = K * per / el
    sample = (f"each step = {per} whole-batch layer-step(s) of layer 0 (of {cfg.n_layers} per decode step); "
              f"host: {os.cpu_count()} cores")
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": "layer-steps/s", "n_gpus": 1,
            "steps": K, "warmup": W, "ms_per_step": el / K * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{cfg.name}: CPU oracle, {sample}"},
            "cpu_baseline": dict(value=value, unit="layer-steps/s", cores=oracle.num_threads(), kind="oracle", sample=sample),
            "e2e": {"value": value, "unit": "layer-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c2")
    ap.add_argument("--host-layers", type=int, default=0, help="distinct host KV regions (0 = as many as fit)")
    ap.add_argument("--settle", type=int, default=24, help="untimed decode steps before the warm-up")
    ap.add_argument("--layers", type=int, default=0, help="cut the layer stack (for profiler captures only)")
    ap.add_argument("--recall-ctas", type=int, default=0, help="CTAs of the recall kernel (0 = library default)")
    ap.add_argument("--append", action="store_true", help="grow the context: append one synthetic token per step and layer")
    ap.add_argument("--attn-ctas", type=int, default=0, help="CTAs of the attention kernel (0 = library default)")
    ap.add_argument("--recall-streams", type=int, default=2, help="streams the recall launches rotate over")
    ap.add_argument("--paged", action="store_true", help="host store as an arena of pages in random order behind a page table")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay leg")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--ref-layer-steps", type=int, default=1)
    args = ap.parse_args()
    line = run_reference(args) if args.impl == "reference" else run_ours(args)
    if line:
        print(json.dumps(line), flush=True)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and args.impl != "reference":
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
