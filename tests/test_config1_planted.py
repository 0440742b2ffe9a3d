"""Config 1 (the parity case): the query is planted to correlate with 16 resident middle blocks.
The recipe only means something if the oracle really ranks those 16 blocks inside the top-k, and
clearly so: every planted block must be selected and its score must exceed the best block left out
of the selection by at least 1 %."""
import numpy as np

import oracle
from workloads import generate as gen, get_config


def test_oracle_selects_all_planted_blocks_with_a_margin():
    cfg = get_config("c1")
    layer = 0
    kv = gen.make_kv(cfg, layer)
    q = gen.make_queries(cfg, layer, 1)[0].clone()
    res = gen.initial_resident(cfg, layer)
    _, _, hot = gen.plant_hot_blocks(cfg, layer, kv, q, res)
    assert hot.shape == (cfg.batch, 16)
    kvb, qb = oracle.bits(kv), oracle.bits(q)
    h = cfg.solo_head(layer)
    pinned = set(gen.pinned_blocks(cfg).tolist())
    for s in range(cfg.batch):
        assert not (set(hot[s].tolist()) & pinned) and set(hot[s].tolist()) <= set(res[s].tolist())
        dg = oracle.build_digest(kvb[s], cfg.ctx, h)
        sc = oracle.score(qb[s], dg, cfg.n_blocks, cfg.n_kv_heads, h)
        sel, cnt = oracle.select(sc, cfg.n_sink_blocks, cfg.n_local_blocks, cfg.budget_blocks)
        chosen = set(sel[:cnt].tolist())
        assert cnt == cfg.budget_blocks == 64 and cfg.k_mid == 55
        assert set(hot[s].tolist()) <= chosen, "a planted block was not selected"
        left_out = [b for b in range(cfg.n_blocks) if b not in chosen]
        best_out = max(sc[b] for b in left_out)
        worst_planted = min(sc[b] for b in hot[s])
        assert best_out > 0
        assert worst_planted >= 1.01 * best_out, (worst_planted, best_out)
        # the planted blocks are hits (resident), the rest of the top-k is mostly not
        middle_sel = [b for b in chosen if b not in pinned]
        hits = sum(b in set(res[s].tolist()) for b in middle_sel)
        assert 16 <= hits < len(middle_sel)
