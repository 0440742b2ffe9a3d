"""Fits the AR(1) coefficient of the query process so that consecutive decode steps
select (on average) a given fraction of the same middle blocks.

    python -m workloads.calibrate_overlap c2 [--seqs 8] [--steps 24]

Bisection on the coefficient; the selections come from the CPU oracle (this script never
touches the CUDA library).  The fitted value is recorded by hand in workloads/configs.py.
"""
from __future__ import annotations

import argparse

import numpy as np

import oracle
from workloads import get_config
from workloads import generate as gen


def mean_overlap(cfg, digests, a: float, steps: int) -> float:
    q = oracle.bits(gen.make_queries(cfg, 0, steps, ar1=a))
    h = cfg.solo_head(0)
    pin = set(gen.pinned_blocks(cfg).tolist())
    tot, n = 0.0, 0
    for s in range(cfg.batch):
        prev = None
        for t in range(steps):
            sc = oracle.score(q[t, s], digests[s], cfg.n_blocks, cfg.n_kv_heads, h)
            sel, cnt = oracle.select(sc, cfg.n_sink_blocks, cfg.n_local_blocks, cfg.budget_blocks)
            mid = set(sel[:cnt].tolist()) - pin
            if prev is not None:
                tot += len(mid & prev) / max(1, len(mid))
                n += 1
            prev = mid
    return tot / n


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("config")
    ap.add_argument("--seqs", type=int, default=8)
    ap.add_argument("--steps", type=int, default=24)
    args = ap.parse_args()
    base = get_config(args.config)
    cfg = base.replace(batch=args.seqs, n_layers=1)
    kvb = oracle.bits(gen.make_kv(cfg, 0))
    digests = [oracle.build_digest(kvb[s], cfg.ctx, cfg.solo_head(0)) for s in range(cfg.batch)]
    lo, hi = 0.0, 1.0
    for _ in range(14):
        mid = 0.5 * (lo + hi)
        ov = mean_overlap(cfg, digests, mid, args.steps)
        print(f"a={mid:.5f} overlap={ov:.4f}", flush=True)
        if ov < base.overlap:
            lo = mid
        else:
            hi = mid
    a = 0.5 * (lo + hi)
    print(f"{args.config}: target {base.overlap} -> ar1 = {a:.4f} (overlap {mean_overlap(cfg, digests, a, args.steps):.4f})")


if __name__ == "__main__":
    main()
