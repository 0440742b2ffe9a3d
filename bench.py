#!/usr/bin/env python
"""Benchmark of the decode recall path (score -> select -> diff -> recall -> attention).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2|c3|c4|c5] [--impl reference]

One "step" is one decode step of the whole batch: every layer runs one layer-step of the
path.  The metric is layer-steps per second.  Rank 0 prints ONE JSON line.

  value        inputs (queries) already in HBM, the pipelined form (selection stream, two recall
               streams, attention stream)
  e2e          the same through DecodeSession with the queries coming from pinned host memory
               and the outputs copied back to pinned host memory inside the timed region
  roofline     the kernel that dominates the step (the recall pull, bound by the host link)
  rooflines    the HBM-bound kernels (attention, scoring) against the measured HBM copy rate
  cpu_baseline the CPU oracle timed on a bounded sample of the same workload
  configs      (default run only) the other workloads in short form: the 70B-shaped stack c4 with
               its host store capped to a few regions, and c5 = scoring / attention at batch 32 for
               block sizes 16 / 32 / 64 plus a short recall-fragmentation sweep

--config c5 alone runs the full recall-fragmentation sweep and prints its table to stderr.
With --gpus N > 1 every rank runs its own batch of sequences (weak scaling, no collective
on the data path); the time is the maximum over ranks.  Started without torchrun, --gpus N
launches the N local ranks itself.
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
# profiles/ (attn_headmajor_kernel_c2.txt, score_select_cluster_kernel_c2.txt, recall_kernel_c2.txt): same
# per-layer shapes as the bench (recall_kernel: its reads cross the host link and its 5 MB of writes stay
# in L2 during the launch, so DRAM sees next to nothing; the attention's 4 MB of DRAM writes are write-backs
# of lines that were dirty in L2 when the capture started, the kernel itself writes 131 KB)
NCU_DRAM_TRAFFIC = {"c2": {"recall_kernel": 24.7e3, "attn_kernel": 134.42e6 + 4.2e6, "score_select_diff_kernel": 17.07e6}}
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


def launch_floor_us(reps: int = 40) -> float:
    """Mean time between two events around a kernel that does nothing: the floor under every per-call time."""
    from paper_2609_34555_b200 import empty_launch
    torch.cuda.synchronize()
    torch.cuda._sleep(2_000_000)                     # the launches queue up behind this
    evs = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); empty_launch(); b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    return float(np.mean([a.elapsed_time(b) for a, b in evs])) * 1e3


def hbm_entry(name: str, bytes_launch: float, mean_ms: float, peaks: dict, traffic=None) -> dict:
    ach = bytes_launch / (mean_ms * 1e-3) / 1e9
    return dict(kernel=name, bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s", frac=ach / peaks["hbm_gbs"],
                peak_source=peaks["source"], traffic=traffic, bytes_per_launch=int(bytes_launch), mean_us=mean_ms * 1e3)


def measure_path(args, cfg, rank: int, world: int, dev, *, K: int, W: int, settle: int, host_layers: int,
                 legs: set, base_name: str) -> dict:
    """Builds the workload of `cfg`, settles it, and measures the path.  legs: which of the optional
    measurements run ("e2e", "graph", "hist", "cpu").  Returns the fields of the JSON line."""
    from paper_2609_34555_b200 import h2d_copy_ms
    from paper_2609_34555_b200.runner import StageTimer

    local = dev.index
    t_setup = time.time()
    n_e2e = min(K, args.e2e_steps) if "e2e" in legs else 0
    n_serial = min(K, 4)
    n_graph = min(K, 16) if "graph" in legs else 0
    n_hist = n_serial if "hist" in legs else 0
    total_steps = settle + W + K + 8 * n_serial + n_e2e + n_graph + 4
    pi, sess, R = build_session(cfg, rank, host_layers, world, args.recall_ctas,
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
    floor_us = launch_floor_us()

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
    for i in range(settle):
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
    def serial_leg(with_events: bool):
        tm = StageTimer() if with_events else None
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        torch.cuda._sleep(2_000_000)                     # the launches queue up behind this
        nonlocal t
        a.record()
        for _ in range(n_serial):
            sess.decode_step(q_all[t], overlapped=False, timer=tm, resident_script=script(t), new_kv=new_kv); t += 1
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / max(1, n_serial), (tm.summary() if tm else None), pi.stats(reset=True)
    serial_ms, ser, ser_stats = serial_leg(True)
    # the same chain without events between the calls (events keep the dependent launches of the chain
    # from overlapping their predecessors)
    serial_plain_ms, _, _ = serial_leg(False)
    # and with selection and diff as two calls (pi_score_select, pi_diff_misses) instead of one
    sess.fused_select_diff = False
    serial2_ms, ser2, _ = serial_leg(True)
    serial2_plain_ms, _, _ = serial_leg(False)
    sess.fused_select_diff = True
    # and with the attention split around the recall: the recall on a stream of its own, the resident blocks'
    # share of the attention beside it, the recalled blocks' share once it has landed
    sess.split_attention = True
    serial3_ms, ser3, _ = serial_leg(True)
    serial3_plain_ms, _, _ = serial_leg(False)
    sess.split_attention = False

    # ---------------- distribution of the miss counts: a few more steps, read back after each
    # (per sequence and layer-step: units of the recall lists)
    miss_hist = None
    if n_hist:
        hist_edges = [0, 1, 3, 5, 9, 17, 33, 65, 1 << 30]
        hist = [0] * (len(hist_edges) - 1)
        for _ in range(n_hist):
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
        t += n_e2e
        e2e_ms = max_over_ranks(a0.elapsed_time(a1), world, dev)
        e2e_stats = pi.stats(reset=True)
        e2e = dict(value=whole_job_value(world, n_e2e, cfg.n_layers, e2e_ms), unit="layer-steps/s", steps=n_e2e,
                   h2d_bytes_per_step=int(q_host[0].numel() * 2), d2h_bytes_per_step=int(out_host[0].numel() * 2),
                   misses_per_seq_layer_step=e2e_stats["missing_blocks"] / max(1, e2e_stats["sequences"]),
                   step_form="CUDA-graph replay" if e2e_graph else "eager launches",
                   note="host KV store is read by the recall kernel in both forms")

    # ---------------- the HBM-bound kernels back to back: one launch per layer (every layer has its
    # own pool / digests, so each launch reads data that left L2 long ago), ONE event pair around the
    # whole train of launches, so that the per-call cost of the events themselves is not in the number.
    # Last, because the selection trains leave the tables of another query behind.
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
    def fused_train():
        sess.step_count += 1
        for l in range(cfg.n_layers):
            b = sess.bufs[l]
            pi.score_select_diff(l, sess.step_count, qb[l], b.digest, sess.ctx_len, b.sel_blocks, b.sel_count, b.block_table,
                                 b.slot_block, b.slot_stamp, b.sel_slots, b.recall_list, b.recall_count)
    b2b_attn_ms = back_to_back(attn_train)
    b2b_score_ms = back_to_back(score_train)
    b2b_fused_ms = back_to_back(fused_train)
    torch.cuda.synchronize()

    peaks = measured_peaks()
    traffic = NCU_DRAM_TRAFFIC.get(base_name, {}) if args.layers == 0 else {}
    n_launch = K * cfg.n_layers
    recall_bytes = stats["missing_blocks"] * cfg.block_bytes
    # union of the launches' intervals (they overlap across the recall streams); the first launch of
    # each recall stream has no bounded start and is left out of bytes and time alike
    n_rec = stages["recall"]["launches"]
    recall_bytes = recall_bytes * n_rec / max(1, n_launch)
    recall_s = stages["recall"]["busy_ms"] * 1e-3
    attn_bytes_launch = stats["selected_blocks"] / max(1, n_launch) * cfg.block_bytes + 2 * cfg.batch * cfg.n_q_heads * 128 * 2
    score_bytes_launch = cfg.batch * cfg.n_blocks * 512 + cfg.batch * cfg.group * 128 * 2
    ser_recall_gbs = ser_stats["missing_blocks"] * cfg.block_bytes / max(1e-9, ser["recall"]["total_ms"] * 1e-3) / 1e9
    recall_gbs = recall_bytes / max(1e-9, recall_s) / 1e9
    ta, tsd, tss = traffic.get("attn_kernel"), traffic.get("score_select_diff_kernel"), traffic.get("score_select_kernel")
    out = {
        "value": whole_job_value(world, K, cfg.n_layers, ms), "unit": "layer-steps/s",
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms / K,
        "config": {"workload": f"{cfg.name}: {cfg.n_layers} layers x batch {cfg.batch} x ctx {cfg.ctx}, "
                               f"Hq/Hkv {cfg.n_q_heads}/{cfg.n_kv_heads}, block {cfg.block_tokens}, budget {cfg.budget_blocks} "
                               f"blocks, pool {cfg.pool_slots} slots/seq/layer, AR(1) queries a={cfg.ar1}",
                   "host_layout": "paged arena, random page order" if args.paged else "block-major per sequence",
                   "host_kv_layers": R, "host_kv_pinned_gb": R * cfg.batch * cfg.n_blocks * cfg.block_bytes / 2 ** 30,
                   "l2": f"inputs larger than L2 (pool reads {cfg.batch * cfg.budget_blocks * cfg.block_bytes / 2**20:.0f} MiB and digests "
                         f"{cfg.batch * cfg.n_blocks * 512 / 2**20:.0f} MiB per layer-step, {cfg.n_layers} distinct layers)",
                   "pipeline": f"selection+diff (one launch) on stream A, recall pulls rotating over {len(sess.recall_streams)} stream(s), "
                               f"attention on the main stream",
                   "sequence_layer_steps_per_s": world * K * cfg.n_layers * cfg.batch / (ms * 1e-3),
                   "misses_per_seq_layer_step": stats["missing_blocks"] / max(1, stats["sequences"]),
                   "misses_per_seq_layer_step_cold_first_step": cold,
                   "miss_histogram_per_seq_layer_step": miss_hist,
                   "miss_script": cfg.miss_script or "none (LRU)", "append": bool(args.append),
                   "settle_steps": settle, "setup_s": round(setup_s, 1)},
        "clocks": clocks, "e2e": e2e,
        "gpu_launches": 3 * n_launch,      # select+diff, recall, attention (head-major: no merge kernel): launches inside the timed region only
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
        "rooflines": [hbm_entry("attention call, attn_headmajor_kernel (timed region, recalls running beside it)", attn_bytes_launch, stages["attn"]["mean_ms"], peaks, ta),
                      hbm_entry("attention call, attn_headmajor_kernel (serial form, nothing else running)", attn_bytes_launch, ser["attn"]["mean_ms"], peaks, ta),
                      hbm_entry("attention call, attn_headmajor_kernel (one launch per layer back to back, one event pair around all)", attn_bytes_launch, b2b_attn_ms, peaks, ta),
                      hbm_entry("score_select_cluster_kernel: score + select + diff in one launch (serial form)", score_bytes_launch, ser["select_diff"]["mean_ms"], peaks, tsd),
                      hbm_entry("score_select_cluster_kernel: score + select + diff (back to back)", score_bytes_launch, b2b_fused_ms, peaks, tsd),
                      hbm_entry("score_select_cluster_kernel: score + select as a call of its own (serial form)", score_bytes_launch, ser2["score_select"]["mean_ms"], peaks, tss),
                      hbm_entry("score_select_cluster_kernel: score + select as a call of its own (back to back)", score_bytes_launch, b2b_score_ms, peaks, tss)],
        "launch_floor_us": floor_us,
        "launch_floor_note": "mean time between two events around a kernel that does nothing (128 x 256 threads), this run: "
                             "part of every per-call (serial form) time above",
        "stages_us": {k: v["mean_ms"] * 1e3 for k, v in stages.items() if v["launches"]},
        "stages_us_events_around_every_call": {k: v["mean_ms"] * 1e3 for k, v in det.items() if v["launches"]},
        "graph_replay": graph_leg,
        "serial": {"layer_steps_per_s": cfg.n_layers / (serial_ms * 1e-3),
                   "layer_steps_per_s_without_events": cfg.n_layers / (serial_plain_ms * 1e-3),
                   "stages_us": {k: v["mean_ms"] * 1e3 for k, v in ser.items() if v["launches"]},
                   "attention_split_around_the_recall": {
                       "layer_steps_per_s": cfg.n_layers / (serial3_ms * 1e-3),
                       "layer_steps_per_s_without_events": cfg.n_layers / (serial3_plain_ms * 1e-3),
                       "stages_us": {k: v["mean_ms"] * 1e3 for k, v in ser3.items() if v["launches"]},
                       "note": "pi_sparse_decode_attn_resident runs beside the recall, pi_sparse_decode_attn_recalled ('attn') after it"},
                   "selection_and_diff_as_two_calls": {
                       "layer_steps_per_s": cfg.n_layers / (serial2_ms * 1e-3),
                       "layer_steps_per_s_without_events": cfg.n_layers / (serial2_plain_ms * 1e-3),
                       "stages_us": {k: v["mean_ms"] * 1e3 for k, v in ser2.items() if v["launches"]}}},
        "h2d_peak_gbs": h2d_gbs,
    }
    if "cpu" in legs:
        out["cpu_baseline"] = cpu_baseline(cfg, sess, budget_s=args.cpu_seconds)
    pi.close()
    del sess, q_all
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return out


def short_form(m: dict) -> dict:
    """The fields of a measure_path result that the `configs` entries of the default run keep."""
    keep = ("value", "unit", "steps", "warmup", "ms_per_step", "e2e", "stages_us", "launch_floor_us", "h2d_peak_gbs")
    out = {k: m[k] for k in keep if k in m}
    out["workload"] = m["config"]["workload"]
    out["host_kv_layers"] = m["config"]["host_kv_layers"]
    out["misses_per_seq_layer_step"] = m["config"]["misses_per_seq_layer_step"]
    out["setup_s"] = m["config"]["setup_s"]
    out["recall"] = {k: m["roofline"][k] for k in ("achieved", "peak", "frac", "bytes_per_launch", "alone")}
    out["rooflines"] = [{k: r[k] for k in ("kernel", "achieved", "frac", "mean_us", "bytes_per_launch")} for r in m["rooflines"]]
    out["serial"] = m["serial"]
    out["graph_replay"] = m["graph_replay"]
    return out


def per_call_ms(fn, reps: int, flush=None) -> float:
    """Mean milliseconds of fn(r) between two events, launches queued behind a spin kernel; `flush`
    (a buffer larger than L2) is read before every call so that the call starts cold."""
    for r in range(2):                                # untimed: the first launch of a kernel loads its module
        fn(r)
    torch.cuda.synchronize()
    torch.cuda._sleep(3_000_000)
    evs = []
    for r in range(reps):
        if flush is not None:
            flush.sum()                               # reading 256 MiB replaces L2's contents with clean lines (a write
                                                      # would leave dirty lines whose write-back overlaps the timed call)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(r); b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    return float(np.mean([a.elapsed_time(b) for a, b in evs]))


def measure_c5(args, dev, full: bool) -> dict:
    """Config 5: one 8B-shaped layer, batch 32, context 32768, block sizes 16 / 32 / 64.
    (i) scoring + selection and attention per call (256 MiB of other data read through L2 before every call) and
    back to back;
    (ii) the recall-fragmentation sweep: misses per layer x placement x list granularity, moved by
    pi_recall_gather_scatter, against the pinned-copy peak of the run (the synthetic restatement of the
    paper's bandwidth-against-granularity and gather-scatter figures, Sec. 3.4 and Sec. 4.4.2).
    full: every miss count and both placements, plus the two context lines (one cudaMemcpyAsync per
    block; the staged engine: host gather into pinned staging + copies + GPU scatter)."""
    from paper_2609_34555_b200 import PulseInfer, h2d_copy_ms
    from paper_2609_34555_b200.runner import LayerBuffers
    from workloads import generate as gen, get_config

    peaks = measured_peaks()
    flush = torch.zeros(64 << 20, dtype=torch.int32, device=dev)        # 256 MiB, read before every per-call measurement
    misses_list = [8, 32, 128, 512, 2048] if full else [32, 512, 2048]
    placements = (False, True) if full else (False,)
    reps = args.c5_reps
    out = {"workload": "c5: one 8B-shaped layer, batch 32, ctx 32768, Hq/Hkv 32/8", "blocks": {}, "recall_sweep": []}
    base = get_config("c5")
    host = torch.empty(base.batch * base.n_blocks * base.block_bytes // 2, dtype=torch.bfloat16, pin_memory=True)
    host.view(torch.int16).random_(0, 30000)
    probe = torch.empty(1 << 28, dtype=torch.bfloat16, device=dev)
    peak = (1 << 29) / (h2d_copy_ms(host[: 1 << 28], probe, 10) * 1e-3) / 1e9
    del probe
    out["h2d_peak_gbs"] = peak
    out["launch_floor_us"] = launch_floor_us()
    for B in (16, 32, 64):
        cfg = base.replace(block_tokens=B, budget_blocks=max(128 * 16 // B, 16))
        nb, C, Hkv, K = cfg.n_blocks, cfg.pool_slots, cfg.n_kv_heads, cfg.budget_blocks
        pi = PulseInfer.from_workload(cfg, recall_ctas=10)      # one launch at a time here (the default of 5 is sized for two side by side)
        buf = LayerBuffers(pi, cfg.batch, dev)
        g = torch.Generator(device=dev).manual_seed(cfg.seed + B)
        buf.digest.copy_(torch.randn(buf.digest.shape, device=dev, generator=g).to(torch.bfloat16))
        buf.pool.copy_(torch.randn(buf.pool.shape[:2] + (1,) * 4, device=dev, generator=g).to(torch.bfloat16).expand_as(buf.pool))
        ctx = torch.full((cfg.batch,), cfg.ctx, dtype=torch.int32, device=dev)
        res = torch.from_numpy(gen.initial_resident(cfg, 0)[:, :C]).contiguous().to(dev)
        pi.table_init(res, buf.block_table, buf.slot_block, buf.slot_stamp)
        q = gen.make_queries(cfg, 0, 8, device=dev)
        out_t = torch.empty((cfg.batch, cfg.n_q_heads, 128), dtype=torch.bfloat16, device=dev)
        # a valid selection with slots for the attention call (the pool bytes themselves do not matter for the timing)
        pi.score_select_diff(0, 1, q[0], buf.digest, ctx, buf.sel_blocks, buf.sel_count, buf.block_table, buf.slot_block,
                             buf.slot_stamp, buf.sel_slots, buf.recall_list, buf.recall_count)
        torch.cuda.synchronize()
        assert pi.status()[0] == 0, pi.status()
        score_bytes = cfg.batch * nb * 512 + cfg.batch * cfg.group * 256
        attn_bytes = int(buf.sel_count.sum().item()) * cfg.block_bytes + 2 * cfg.batch * cfg.n_q_heads * 256
        sc_ms = per_call_ms(lambda r: pi.score_select(0, q[r % 8], buf.digest, ctx, buf.sel_blocks, buf.sel_count, None), reps, flush)
        pi.score_select(0, q[0], buf.digest, ctx, buf.sel_blocks, buf.sel_count, None)      # the selection the slots belong to
        at_ms = per_call_ms(lambda r: pi.sparse_decode_attn(0, q[0], buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx, out_t, None), reps, flush)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda._sleep(3_000_000)
        t0.record()
        for _ in range(reps):
            pi.sparse_decode_attn(0, q[0], buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx, out_t, None)
        t1.record()
        torch.cuda.synchronize()
        at_b2b_ms = t0.elapsed_time(t1) / reps
        out["blocks"][str(B)] = {
            "n_blocks": nb, "budget_blocks": K, "pool_slots": C,
            "score_select": hbm_entry("score_select_cluster_kernel (per call, L2 refilled with other data before each)", score_bytes, sc_ms, peaks),
            "attention": hbm_entry("attention call, attn_headmajor_kernel (per call, L2 refilled with other data before each)", attn_bytes, at_ms, peaks),
            "attention_back_to_back": hbm_entry("attention call, attn_headmajor_kernel (back to back, pool reads 256 MiB > L2)", attn_bytes, at_b2b_ms, peaks)}

        # ---- recall-fragmentation sweep at this block size
        hostB = host.view(cfg.batch, nb, cfg.block_bytes // 2)
        pool_flat = buf.pool.view(cfg.batch, C, cfg.block_bytes // 2)
        pin = gen.pinned_blocks(cfg)

        def timed(launches) -> float:
            torch.cuda.synchronize()
            torch.cuda._sleep(3_000_000)
            evs = []
            for r in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); launches[r % len(launches)](); b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            return float(np.median([a.elapsed_time(b) for a, b in evs]))

        for total in misses_list:
            if total > cfg.batch * cfg.k_mid:
                continue
            for clustered in placements:
                place = "clustered" if clustered else "uniform"
                # coalesced lists through the diff kernel: empty pool (only sink/local resident),
                # selection = sink/local + the scripted missing blocks
                resn = np.full((cfg.batch, C), -1, np.int32)
                resn[:, : len(pin)] = pin
                res_d = torch.from_numpy(resn).to(dev)
                lists = []
                for rep in range(2):
                    miss = gen.scripted_misses(cfg, total, clustered, extra=rep)
                    sel = np.full((cfg.batch, K), -1, np.int32)
                    cnt = np.zeros(cfg.batch, np.int32)
                    for s_, m in enumerate(miss):
                        row = np.sort(np.concatenate([pin, m]))[:K]
                        sel[s_, : len(row)] = row
                        cnt[s_] = len(row)
                    sel_d, cnt_d = torch.from_numpy(sel).to(dev), torch.from_numpy(cnt).to(dev)
                    pi.table_init(res_d, buf.block_table, buf.slot_block, buf.slot_stamp)
                    lst = torch.zeros((cfg.batch, K, 4), dtype=torch.int32, device=dev)
                    lcnt = torch.zeros((cfg.batch,), dtype=torch.int32, device=dev)
                    pi.diff_misses(0, 1, ctx, sel_d, cnt_d, buf.block_table, buf.slot_block, buf.slot_stamp,
                                   buf.sel_slots, lst, lcnt)
                    lists.append((lst, lcnt))
                torch.cuda.synchronize()
                n_ext = int(lists[0][1].sum().item())
                ms_ = timed([lambda l=l: pi.recall_gather_scatter(0, hostB, pool_flat, l[0], l[1]) for l in lists])
                bytes_ = total * cfg.block_bytes
                out["recall_sweep"].append(dict(block=B, misses=total, placement=place, lists="coalesced", extents=n_ext,
                                                extent_kb=bytes_ / max(1, n_ext) / 1024, us=ms_ * 1e3, gbs=bytes_ / (ms_ * 1e-3) / 1e9,
                                                frac_of_h2d_peak=bytes_ / (ms_ * 1e-3) / 1e9 / peak))
                # per-head fragmented lists: independent draws per head, one fragment per extent
                per = max(1, -(-total // cfg.batch))
                hl = []
                for rep in range(2):
                    lst = torch.zeros((cfg.batch * Hkv, per, 4), dtype=torch.int32)
                    lcnt = torch.zeros((cfg.batch * Hkv,), dtype=torch.int32)
                    for h in range(Hkv):
                        miss = gen.scripted_misses(cfg, total, clustered, extra=100 + 10 * h + rep)
                        for s_, m in enumerate(miss):
                            n = len(m)
                            e = torch.zeros((n, 4), dtype=torch.int32)
                            e[:, 0] = torch.from_numpy(m.astype(np.int32)) * Hkv + h
                            e[:, 1] = (torch.arange(n, dtype=torch.int32) + len(pin)) * Hkv + h
                            e[:, 2] = 1
                            e[:, 3] = torch.arange(n, dtype=torch.int32)
                            lst[s_ * Hkv + h, :n] = e
                            lcnt[s_ * Hkv + h] = n
                    hl.append((lst.to(dev), lcnt.to(dev)))
                # per-head units are (block, head) fragments: the unit index is block * Hkv + head, frag_bytes apart
                ms_ = timed([lambda l=l: pi.recall_gather_scatter(0, hostB, pool_flat, l[0], l[1], lists_per_seq=Hkv,
                                                                   unit_bytes=cfg.frag_bytes) for l in hl])
                out["recall_sweep"].append(dict(block=B, misses=total, placement=place, lists="per-head", extents=total * Hkv,
                                                extent_kb=cfg.frag_bytes / 1024, us=ms_ * 1e3, gbs=bytes_ / (ms_ * 1e-3) / 1e9,
                                                frac_of_h2d_peak=bytes_ / (ms_ * 1e-3) / 1e9 / peak))
            if not full:
                continue
            # context: the copy engine, one cudaMemcpyAsync per missing block (uniform placement)
            if total <= 512:
                miss = gen.scripted_misses(cfg, total, False, extra=7)
                pairs = [(s_, int(b), len(pin) + i) for s_, m in enumerate(miss) for i, b in enumerate(m)]
                torch.cuda.synchronize()
                a, bb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                for s_, b, slot in pairs:
                    pool_flat[s_, slot].copy_(hostB[s_, b], non_blocking=True)
                bb.record(); torch.cuda.synchronize()
                ms_ = a.elapsed_time(bb)
                out["recall_sweep"].append(dict(block=B, misses=total, placement="uniform", lists="cudaMemcpyAsync per block",
                                                extents=total, extent_kb=cfg.block_bytes / 1024, us=ms_ * 1e3,
                                                gbs=total * cfg.block_bytes / (ms_ * 1e-3) / 1e9,
                                                frac_of_h2d_peak=total * cfg.block_bytes / (ms_ * 1e-3) / 1e9 / peak))
            # context: the paper's staged engine (Sec. 4.4.2): the CPU gathers the scattered blocks into pinned
            # staging in 8 MB chunks, each chunk is copied while the next is gathered, a GPU kernel scatters
            # (a context line written in the harness: the scatter is a library index copy).  Wall clock, the
            # host does part of the work.
            miss = gen.scripted_misses(cfg, total, False, extra=7)
            flat = torch.from_numpy(np.concatenate([s_ * nb + m.astype(np.int64) for s_, m in enumerate(miss)]))
            stage_host = torch.empty((total, cfg.block_bytes // 2), dtype=torch.bfloat16, pin_memory=True)
            stage_dev = torch.empty((total, cfg.block_bytes // 2), dtype=torch.bfloat16, device=dev)
            # destination of every staged block: slot len(pin) + i of its sequence
            dst_flat = torch.from_numpy(np.concatenate([s_ * C + len(pin) + np.arange(len(m), dtype=np.int64)
                                                        for s_, m in enumerate(miss)])).to(dev)
            pool_pages = pool_flat.view(cfg.batch * C, cfg.block_bytes // 2)
            host_pages = hostB.view(cfg.batch * nb, cfg.block_bytes // 2)
            per_chunk = max(1, (8 << 20) // cfg.block_bytes)
            best = float("inf")
            for _ in range(max(3, reps // 2)):
                torch.cuda.synchronize()
                t0_ = time.perf_counter()
                for c0 in range(0, total, per_chunk):
                    c1 = min(total, c0 + per_chunk)
                    torch.index_select(host_pages, 0, flat[c0:c1], out=stage_host[c0:c1])
                    stage_dev[c0:c1].copy_(stage_host[c0:c1], non_blocking=True)
                pool_pages.index_copy_(0, dst_flat, stage_dev)         # the scatter kernel of the staged engine
                torch.cuda.synchronize()
                best = min(best, time.perf_counter() - t0_)
            out["recall_sweep"].append(dict(block=B, misses=total, placement="uniform", lists="staged: CPU gather+DMA", extents=total,
                                            extent_kb=cfg.block_bytes / 1024, us=best * 1e6, gbs=total * cfg.block_bytes / best / 1e9,
                                            frac_of_h2d_peak=total * cfg.block_bytes / best / 1e9 / peak))
            del stage_host, stage_dev
        st = pi.status()
        out["blocks"][str(B)]["device_status"] = st[0]
        pi.close()
        del buf
        torch.cuda.empty_cache()
    return out


def c5_table(c5: dict) -> str:
    lines = [f"{'B':>3s} {'misses':>6s} {'placement':>10s} {'lists':>26s} {'extents':>8s} {'KB/ext':>8s} {'us':>9s} {'GB/s':>7s} {'of peak':>8s}"]
    for r in c5["recall_sweep"]:
        lines.append(f"{r['block']:3d} {r['misses']:6d} {r['placement']:>10s} {r['lists']:>26s} {r['extents']:8d} {r['extent_kb']:8.1f} "
                     f"{r['us']:9.1f} {r['gbs']:7.2f} {r['frac_of_h2d_peak']:8.3f}")
    lines.append(f"pinned cudaMemcpyAsync peak of this run: {c5['h2d_peak_gbs']:.2f} GB/s (512 MiB, best of 10)")
    for B, d in c5["blocks"].items():
        for k in ("score_select", "attention", "attention_back_to_back"):
            lines.append(f"B={B:>2s} {d[k]['kernel']}: {d[k]['mean_us']:.1f} us, {d[k]['achieved']:.0f} GB/s, {d[k]['frac']:.3f} of the measured HBM rate")
    return "\n".join(lines)


def run_ours(args) -> dict:
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
    if args.config == "c5":
        c5 = measure_c5(args, dev, full=True)
        if rank == 0:
            print(c5_table(c5), file=sys.stderr, flush=True)
            if args.out:
                Path(args.out).write_text(c5_table(c5) + "\n")
        best = max((r for r in c5["recall_sweep"] if r["lists"] in ("coalesced", "per-head")), key=lambda r: r["gbs"])
        line = {"metric": METRIC, "value": best["gbs"], "unit": "GB/s (best recall rate of the sweep; this config has no layer-step rate)",
                "n_gpus": world, "steps": args.c5_reps, "warmup": 0, "ms_per_step": best["us"] * 1e-3, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": c5["workload"] + ", block 16/32/64: recall-fragmentation sweep + scoring / attention per call"},
                "roofline": {"kernel": "recall_kernel", "bound": "host_link_h2d", "achieved": best["gbs"], "peak": c5["h2d_peak_gbs"],
                             "unit": "GB/s", "frac": best["frac_of_h2d_peak"], "traffic": None},
                "c5": c5}
        return line if rank == 0 else {}
    base = get_config(args.config)
    cfg = rank_config(base, rank)
    if args.layers > 0:                       # profiling only: fewer layers of the same shape
        cfg = cfg.replace(n_layers=min(args.layers, cfg.n_layers), name=f"{cfg.name}[{args.layers} layers only]")
    K, W = args.steps, max(3, args.warmup)
    legs = set()
    if not args.no_e2e: legs.add("e2e")
    if not args.no_graph: legs.add("graph")
    if not args.no_cpu and world == 1 and rank == 0: legs.add("cpu")
    legs.add("hist")
    m = measure_path(args, cfg, rank, world, dev, K=K, W=W, settle=args.settle, host_layers=args.host_layers, legs=legs,
                     base_name=base.name)
    line = {"metric": METRIC, "value": m["value"], "unit": m["unit"], "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic"}
    m["config"]["numa_node_of_rank0"] = numa_node
    line.update({k: v for k, v in m.items() if k not in line})
    # ---------------- the other workloads in short form (single GPU, default config only)
    if args.config == "c2" and world == 1 and not args.no_configs and args.layers == 0:
        c4 = get_config("c4")
        m4 = measure_path(args, c4, rank, world, dev, K=args.c4_steps, W=3, settle=args.c4_settle,
                          host_layers=args.c4_host_layers, legs={"e2e", "graph"}, base_name="c4")
        line["configs"] = {"c4": short_form(m4), "c5": measure_c5(args, dev, full=False)}
    return line if rank == 0 else {}


def self_launch(args) -> int:
    """--gpus N without torchrun's environment: start the N local ranks here (the same command under
    torch.distributed.run on 127.0.0.1) and pass their output through."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve())] + sys.argv[1:]
    return subprocess.call(cmd)


def launch_check(args) -> dict:
    """What the launcher produced, without touching a GPU (gloo): every rank reports itself, rank 0
    prints the roll call.  Used by the CPU test of the --gpus N launcher."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo", rank=rank, world_size=world)
        seen = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(seen, torch.tensor([rank], dtype=torch.int64))
        ranks = sorted(int(x) for x in seen)
        ms = max_over_ranks(float(rank + 1), world, device="cpu")
        dist.barrier()
        dist.destroy_process_group()
    else:
        ranks, ms = [0], 1.0
    return {"launch_check": True, "n_gpus": world, "ranks": ranks, "max_ms": ms,
            "local_rank": int(os.environ.get("LOCAL_RANK", "0"))} if rank == 0 else {}


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
    ap.add_argument("--config", default="c2", choices=["c2", "c3", "c4", "c5"])
    ap.add_argument("--host-layers", type=int, default=0, help="distinct host KV regions (0 = as many as fit)")
    ap.add_argument("--settle", type=int, default=24, help="untimed decode steps before the warm-up")
    ap.add_argument("--layers", type=int, default=0, help="cut the layer stack (for profiler captures only)")
    ap.add_argument("--recall-ctas", type=int, default=0, help="CTAs of the recall kernel (0 = library default)")
    ap.add_argument("--append", action="store_true", help="grow the context: append one synthetic token per step and layer")
    ap.add_argument("--attn-ctas", type=int, default=0, help="CTAs of the attention kernel (0 = library default)")
    ap.add_argument("--recall-streams", type=int, default=2, help="streams the recall launches rotate over")
    ap.add_argument("--paged", action="store_true", help="host store as an arena of pages in random order behind a page table")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=1 << 30, help="steps of the end-to-end leg (default: as many as --steps)")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay leg")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="headline workload only: skip the short forms of c4 and c5")
    ap.add_argument("--c4-steps", type=int, default=8, help="timed decode steps of the short c4 run (80 layer-steps each)")
    ap.add_argument("--c4-settle", type=int, default=16)
    ap.add_argument("--c4-host-layers", type=int, default=6, help="host KV regions of the short c4 run (2 GiB each, reused modulo)")
    ap.add_argument("--c5-reps", type=int, default=8)
    ap.add_argument("--out", default="", help="--config c5: also write the sweep table to this file")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--ref-layer-steps", type=int, default=1)
    ap.add_argument("--launch-check", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(self_launch(args))
    if args.launch_check:
        line = launch_check(args)
    else:
        line = run_reference(args) if args.impl == "reference" else run_ours(args)
    if line:
        print(json.dumps(line), flush=True)
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and args.impl != "reference" and not args.launch_check:
        import torch.distributed as dist
        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
