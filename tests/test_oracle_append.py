"""Pins of the oracle's token append (KV store + pool + tables + digest) against rebuilds
from scratch and invariants.  The paper implies the operation but never describes it."""
import numpy as np
import torch

import oracle
from workloads import tiny_config
from workloads import generate as gen


def _state(cfg, ctx0, seed=0):
    rng = np.random.default_rng(seed)
    kv = oracle.bits(gen.make_kv(cfg.replace(batch=1), 0))[0].copy()        # [nb][Hkv][2][B][D]
    nb0 = -(-ctx0 // cfg.block_tokens)
    kv[nb0:] = 0x7fc0                                                       # beyond the context: poison (NaN pattern)
    kv[nb0 - 1, :, :, ctx0 - (nb0 - 1) * cfg.block_tokens:] = 0 if ctx0 % cfg.block_tokens else kv[nb0 - 1, :, :, :0].sum()
    h = cfg.solo_head(0)
    digest = np.zeros((cfg.n_blocks, 2, cfg.head_dim), np.uint16)
    digest[:nb0] = oracle.build_digest(kv, ctx0, h)[:nb0]
    C = cfg.pool_slots
    pin = gen.pinned_blocks(cfg, nb0).tolist()
    mid = [b for b in range(nb0) if b not in pin]
    res = pin + rng.choice(mid, size=min(len(mid), C - len(pin) - 2), replace=False).tolist()   # two free slots
    slot_block = np.full(C, -1, np.int32); slot_block[:len(res)] = res
    table = np.full(cfg.n_blocks, -1, np.int32); table[res] = np.arange(len(res))
    stamp = np.zeros(C, np.uint32); stamp[:len(res)] = rng.integers(1, 5, len(res))
    pool = np.zeros((C,) + kv.shape[1:], np.uint16)
    pool[:len(res)] = kv[res]
    return kv, digest, table, slot_block, stamp, pool, h, rng


def test_append_equals_rebuild_from_scratch_across_block_boundaries():
    cfg = tiny_config(batch=1, ctx=2000, budget_blocks=24, resident_frac=0.25)
    B, ctx0, T = cfg.block_tokens, 1003, 45                                  # crosses 3 block boundaries
    kv, digest, table, sb, st, pool, h, rng = _state(cfg, ctx0)
    toks = []
    for i in range(T):
        k = oracle.bits(torch.from_numpy(rng.standard_normal((cfg.n_kv_heads, 128)).astype(np.float32)).to(torch.bfloat16))
        v = oracle.bits(torch.from_numpy(rng.standard_normal((cfg.n_kv_heads, 128)).astype(np.float32)).to(torch.bfloat16))
        toks.append((k, v))
        ctx = ctx0 + i
        rc = oracle.append(k, v, ctx, B, h, cfg.n_sink_blocks, cfg.n_local_blocks, 10 + i, kv, pool, table, sb, st, digest)
        assert rc == 0
        b, t = divmod(ctx, B)
        # the token is where it belongs, in the host store and in the pool
        assert np.array_equal(kv[b, :, 0, t], k) and np.array_equal(kv[b, :, 1, t], v)
        assert table[b] >= 0 and np.array_equal(pool[table[b]], kv[b])
        # invariants of the tables
        nb = b + 1
        for s, blk in enumerate(sb):
            assert blk < 0 or table[blk] == s
        for pb in gen.pinned_blocks(cfg, nb):
            assert table[pb] >= 0, "sink and local blocks stay resident"
        assert st[table[b]] == 10 + i
        # digest == rebuild from scratch over the new length
        ref = oracle.build_digest(kv, ctx + 1, h)
        assert np.array_equal(digest[:nb], ref[:nb])
    # every resident block's pool bytes equal the host bytes
    for s, blk in enumerate(sb):
        if blk >= 0:
            assert np.array_equal(pool[s], kv[blk])
    # dense attention over the grown context sees the appended tokens
    ctx = ctx0 + T
    nb = -(-ctx // B)
    q = oracle.bits(torch.from_numpy(rng.standard_normal((cfg.n_q_heads, 128)).astype(np.float32)).to(torch.bfloat16))
    blocks = np.arange(nb, dtype=np.int32)
    out, _ = oracle.attention(q, kv, blocks, blocks, nb, ctx, B, cfg.n_kv_heads)
    out2, _ = oracle.attention(q, kv, blocks, blocks, nb, ctx - 1, B, cfg.n_kv_heads)
    assert np.all(np.isfinite(out)) and not np.allclose(out, out2)


def test_append_evicts_least_recently_selected_unpinned_slot_and_reports_full_pool():
    cfg = tiny_config(batch=1, ctx=2000, budget_blocks=24, resident_frac=0.0)     # C == K == 24
    B = cfg.block_tokens
    ctx0 = 64 * B                                                                  # next token opens block 64
    kv, digest, table, sb, st, pool, h, rng = _state(cfg, ctx0, seed=3)
    # fill the two free slots so that an eviction is needed; make slot 20 the oldest unpinned one
    free = np.nonzero(sb < 0)[0]
    unused = [b for b in range(1, 50) if table[b] < 0][:len(free)]
    for s, b in zip(free, unused):
        sb[s], table[b], st[s] = b, s, 4
    st[:] = 7
    st[20] = 2
    victim_block = sb[20]
    k = v = oracle.bits(torch.zeros((cfg.n_kv_heads, 128), dtype=torch.bfloat16))
    rc = oracle.append(k, v, ctx0, B, h, cfg.n_sink_blocks, cfg.n_local_blocks, 9, kv, pool, table, sb, st, digest)
    assert rc == 0 and table[64] == 20 and table[victim_block] == -1 and sb[20] == 64 and st[20] == 9
    assert not pool[20].any() and not kv[64].any()                                # a fresh block starts zeroed
    # a pool whose slots all hold sink/local blocks cannot take the new block
    sb2 = np.asarray([b for b in gen.pinned_blocks(cfg, 67).tolist() if b != 66], np.int32)   # sink + local under the new length
    t2 = np.full(cfg.n_blocks, -1, np.int32); t2[sb2] = np.arange(len(sb2))
    rc = oracle.append(k, v, 66 * B, B, h, cfg.n_sink_blocks, cfg.n_local_blocks, 9, kv,
                       np.zeros((len(sb2),) + kv.shape[1:], np.uint16), t2, sb2.copy(), np.zeros(len(sb2), np.uint32), digest)
    assert rc == oracle.POOL_TOO_SMALL
