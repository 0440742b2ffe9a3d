"""Seeded tensors for the decode recall path: keys/values, queries, resident sets,
scripted miss lists.  Data only; the method's arithmetic lives elsewhere.

Layouts (all bf16 unless noted):
  kv      [batch][n_blocks][Hkv][2 = K,V][B][D]   one block of one kv head is a
                                                  contiguous 2*B*D*2-byte fragment
                                                  (8 KB at B=16, D=128: the paper's figure)
  q       [batch][Hq][D]
  resident int32 [batch][C]   block held by each pool slot at start, -1 = free

Recipe: K, V ~ N(0,1) rounded to bf16; four "outlier" channels per layer (same for
all heads and tokens of the layer) scaled by 8 in K and V; queries ~ N(0,1), either
independent per step or an AR(1) process per (seq, layer) whose coefficient sets the
step-to-step overlap of the selections.
"""
from __future__ import annotations

import math
from typing import Optional

import numpy as np
import torch

from .configs import PathConfig

T_KV, T_Q, T_RESIDENT, T_OUTLIER, T_PLANT, T_SCRIPT, T_PARETO = range(7)


def seed_for(cfg: PathConfig, tensor_id: int, layer: int = 0, extra: int = 0) -> int:
    return (cfg.seed * 1_000_003 + tensor_id) * 1_000_003 + layer * 4099 + extra


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def outlier_channels(cfg: PathConfig, layer: int) -> torch.Tensor:
    g = _gen("cpu", seed_for(cfg, T_OUTLIER, layer))
    return torch.randperm(cfg.head_dim, generator=g)[:4].sort().values


def make_kv(cfg: PathConfig, layer: int, device="cpu", seqs: Optional[range] = None) -> torch.Tensor:
    """Keys and values of `seqs` (default: the whole batch) for one layer."""
    seqs = range(cfg.batch) if seqs is None else seqs
    out = torch.empty((len(seqs), cfg.n_blocks, cfg.n_kv_heads, 2, cfg.block_tokens, cfg.head_dim),
                      dtype=torch.bfloat16, device=device)
    ch = outlier_channels(cfg, layer).to(device)
    for i, s in enumerate(seqs):
        g = _gen(device, seed_for(cfg, T_KV, layer, s))
        x = torch.randn(out.shape[1:], dtype=torch.float32, device=device, generator=g)
        x[..., ch] *= 8.0
        out[i] = x.to(torch.bfloat16)
    return out


def make_queries(cfg: PathConfig, layer: int, steps: int, device="cpu", ar1: Optional[float] = None) -> torch.Tensor:
    """[steps][batch][Hq][D] bf16.  AR(1) in fp32 along the step axis:
    x_{t+1} = a x_t + sqrt(1 - a^2) eps_t, each x_t rounded to bf16 on output."""
    a = cfg.ar1 if ar1 is None else ar1
    g = _gen(device, seed_for(cfg, T_Q, layer))
    shape = (cfg.batch, cfg.n_q_heads, cfg.head_dim)
    x = torch.randn(shape, dtype=torch.float32, device=device, generator=g)
    out = torch.empty((steps,) + shape, dtype=torch.bfloat16, device=device)
    out[0] = x.to(torch.bfloat16)
    b = math.sqrt(max(0.0, 1.0 - a * a))
    for t in range(1, steps):
        eps = torch.randn(shape, dtype=torch.float32, device=device, generator=g)
        x = a * x + b * eps
        out[t] = x.to(torch.bfloat16)
    return out


def pinned_blocks(cfg: PathConfig, n_blocks: Optional[int] = None) -> np.ndarray:
    n = cfg.n_blocks if n_blocks is None else n_blocks
    lo = np.arange(0, min(cfg.n_sink_blocks, n))
    hi = np.arange(max(n - cfg.n_local_blocks, 0), n)
    return np.union1d(lo, hi).astype(np.int32)


def initial_resident(cfg: PathConfig, layer: int, fill: float = 1.0) -> np.ndarray:
    """int32 [batch][C]: sink and local blocks first, then uniformly drawn middle
    blocks; `fill` < 1 leaves the tail of the slots free (-1)."""
    C = cfg.pool_slots
    out = np.full((cfg.batch, C), -1, dtype=np.int32)
    pin = pinned_blocks(cfg)
    mid = np.setdiff1d(np.arange(cfg.n_blocks, dtype=np.int32), pin)
    n_mid = max(0, min(len(mid), int(round(fill * (C - len(pin))))))
    for s in range(cfg.batch):
        rng = np.random.default_rng(seed_for(cfg, T_RESIDENT, layer, s))
        pick = np.sort(rng.choice(mid, size=n_mid, replace=False)) if n_mid else mid[:0]
        row = np.concatenate([pin, pick]).astype(np.int32)[:C]
        out[s, :len(row)] = row
    return out


def plant_hot_blocks(cfg: PathConfig, layer: int, kv: torch.Tensor, q: torch.Tensor,
                     resident: np.ndarray, n_hot: int = 16, mu: float = 16.0, lam: float = 1.0):
    """Make the query correlate with `n_hot` resident middle blocks: add mu * u_b
    (u_b a random sign vector) to the retrieval head's key of one token of block b,
    and lam * sum_b u_b / 4 to every query head of that head's group.
    Returns (kv, q, hot_blocks[batch][n_hot]); kv and q are modified in place."""
    h = cfg.solo_head(layer)
    G = cfg.group
    pin = set(pinned_blocks(cfg).tolist())
    hot = np.empty((cfg.batch, n_hot), dtype=np.int32)
    for s in range(cfg.batch):
        rng = np.random.default_rng(seed_for(cfg, T_PLANT, layer, s))
        cand = np.array([b for b in resident[s] if b >= 0 and b not in pin], dtype=np.int32)
        hot[s] = np.sort(rng.choice(cand, size=n_hot, replace=False))
        qs = q[s].float()
        for b in hot[s]:
            u = torch.from_numpy(rng.choice([-1.0, 1.0], size=cfg.head_dim).astype(np.float32))
            t = int(rng.integers(0, cfg.block_tokens))
            kv[s, b, h, 0, t] = (kv[s, b, h, 0, t].float() + mu * u).to(torch.bfloat16)
            qs[h * G:(h + 1) * G] += lam * u / 4.0
        q[s] = qs.to(torch.bfloat16)
    return kv, q, hot


def pareto_miss_counts(cfg: PathConfig, layer: int, step: int, alpha: float = 1.5, x_m: float = 4.0) -> np.ndarray:
    """Heavy-tailed number of misses per sequence: min(k_mid, floor(x_m (1-U)^(-1/alpha)))."""
    rng = np.random.default_rng(seed_for(cfg, T_PARETO, layer, step))
    u = rng.random(cfg.batch)
    m = np.floor(x_m * (1.0 - u) ** (-1.0 / alpha)).astype(np.int64)
    return np.minimum(m, cfg.k_mid).astype(np.int32)


def scripted_misses(cfg: PathConfig, total_misses: int, clustered: bool, extra: int = 0) -> list[np.ndarray]:
    """Missing middle blocks per sequence for the fragmentation sweep: `total_misses`
    spread evenly over the batch; uniform-random placement, or runs of consecutive
    blocks with geometric lengths (mean 8)."""
    per = [total_misses // cfg.batch + (1 if s < total_misses % cfg.batch else 0) for s in range(cfg.batch)]
    lo, hi = cfg.n_sink_blocks, cfg.n_blocks - cfg.n_local_blocks
    out = []
    for s, m in enumerate(per):
        rng = np.random.default_rng(seed_for(cfg, T_SCRIPT, int(clustered), s * 65537 + total_misses + extra))
        if not clustered:
            blocks = np.sort(rng.choice(np.arange(lo, hi), size=m, replace=False))
        else:
            chosen: set[int] = set()
            while len(chosen) < m:
                run = int(min(rng.geometric(1.0 / 8.0), m - len(chosen)))
                start = int(rng.integers(lo, hi - run + 1))
                chosen.update(range(start, start + run))
            blocks = np.sort(np.fromiter(chosen, dtype=np.int64))[:m]
        out.append(blocks.astype(np.int32))
    return out


def scripted_resident_lists(cfg: PathConfig, sel_blocks: torch.Tensor, sel_count: torch.Tensor,
                            miss_counts: np.ndarray, seed: int) -> torch.Tensor:
    """Hot-set contents that make exactly miss_counts[s] of the selected middle blocks of
    sequence s non-resident: int32 [batch][C] = sink/local blocks, the other selected middle
    blocks, then unselected filler blocks.  sel_blocks [batch][K] ascending (device or CPU)."""
    dev = sel_blocks.device
    batch, K = sel_blocks.shape
    C, nb = cfg.pool_slots, cfg.n_blocks
    g = _gen(dev, seed)
    pin = torch.from_numpy(pinned_blocks(cfg)).to(dev)
    is_pin = torch.zeros(nb, dtype=torch.bool, device=dev)
    is_pin[pin.long()] = True
    valid = torch.arange(K, device=dev)[None, :] < sel_count[:, None]
    sel = torch.where(valid, sel_blocks, torch.zeros_like(sel_blocks)).long()
    mid = valid & ~is_pin[sel]                                           # selected middle entries
    # drop `miss` of the middle entries per sequence: rank random keys among the middle entries
    keys = torch.rand((batch, K), device=dev, generator=g)
    keys = torch.where(mid, keys, torch.full_like(keys, 2.0))
    rank = keys.argsort(dim=1).argsort(dim=1)
    miss = torch.from_numpy(np.asarray(miss_counts, dtype=np.int64)).to(dev)
    dropped = mid & (rank < miss[:, None])
    keep = valid & ~dropped
    # priority per block: kept selected blocks first, then unselected non-pinned filler, never the dropped ones
    score = torch.rand((batch, nb), device=dev, generator=g)                # filler in random order
    rows = torch.arange(batch, device=dev)[:, None].expand(batch, K)
    score[rows[keep], sel[keep]] = 3.0
    score[rows[dropped], sel[dropped]] = -1.0
    score[:, pin.long()] = 4.0
    order = score.argsort(dim=1, descending=True)[:, :C]
    return order.to(torch.int32).contiguous()
