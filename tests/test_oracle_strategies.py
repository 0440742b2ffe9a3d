"""Pins of the oracle's comparison strategies (Sec. 4.4.1: headwise, average) against the
single-head functions, closed forms and invariants."""
import numpy as np
import torch

import oracle
from tests.test_oracle_pins import _case, rand_bits


def test_all_head_digest_agrees_with_the_single_head_one():
    ctx, B, Hq, Hkv = 250, 16, 8, 4
    _, nb, kv, _ = _case(41, ctx, B, Hq, Hkv)
    da = oracle.build_digest_all(kv, ctx)
    for h in range(Hkv):
        assert np.array_equal(da[:nb, h], oracle.build_digest(kv, ctx, h)[:nb])


def test_one_head_of_the_set_score_is_the_single_head_score_and_sets_add_up():
    ctx, B, Hq, Hkv = 250, 16, 8, 4
    _, nb, kv, q = _case(42, ctx, B, Hq, Hkv)
    da = oracle.build_digest_all(kv, ctx)
    per_head = [oracle.score(q, oracle.build_digest(kv, ctx, h), nb, Hkv, h) for h in range(Hkv)]
    for h in range(Hkv):
        assert np.array_equal(oracle.score_heads(q, da, nb, h, h + 1), per_head[h])
    np.testing.assert_allclose(oracle.score_heads(q, da, nb, 0, Hkv), np.sum(per_head, axis=0), rtol=1e-13)
    # upper bound: the averaged score bounds the summed logits of all query heads for every token
    qf, kf = oracle.bf16_to_f64(q), oracle.bf16_to_f64(kv)[:, :, 0]              # [nb][Hkv][B][D]
    G = Hq // Hkv
    logits = sum(np.einsum("d,ntd->nt", qf[g], kf[:, g // G]) for g in range(Hq))
    avg = oracle.score_heads(q, da, nb, 0, Hkv)
    for b in range(nb):
        assert np.all(logits[b, :min(B, ctx - b * B)] <= avg[b] + 1e-9)


def test_identical_heads_make_every_strategy_select_the_same_blocks():
    ctx, B, Hq, Hkv = 400, 16, 8, 4
    rng, nb, kv, q = _case(43, ctx, B, Hq, Hkv)
    kv[:, 1:] = kv[:, :1]                                                       # all KV heads alike
    G = Hq // Hkv
    q = np.tile(q[:G], (Hkv, 1))                                                 # all query groups alike
    da = oracle.build_digest_all(kv, ctx)
    solo, n = oracle.select(oracle.score(q, oracle.build_digest(kv, ctx, 2), nb, Hkv, 2), 1, 2, 10)
    avg, _ = oracle.select(oracle.score_heads(q, da, nb, 0, Hkv), 1, 2, 10)
    assert np.array_equal(solo, avg)
    for h in range(Hkv):
        hw, _ = oracle.select(oracle.score_heads(q, da, nb, h, h + 1), 1, 2, 10)
        assert np.array_equal(solo, hw)


def test_single_kv_head_average_is_solohead():
    ctx, B, Hq, Hkv = 300, 16, 4, 1
    _, nb, kv, q = _case(44, ctx, B, Hq, Hkv)
    assert np.array_equal(oracle.score_heads(q, oracle.build_digest_all(kv, ctx), nb, 0, 1),
                          oracle.score(q, oracle.build_digest(kv, ctx, 0), nb, 1, 0))


def test_strided_recall_moves_one_head_fragment_and_nothing_else():
    rng = np.random.default_rng(3)
    Hkv, frag = 4, 256
    host = rng.integers(0, 256, size=(12, Hkv, frag), dtype=np.uint8)
    pool = rng.integers(0, 256, size=(6, Hkv, frag), dtype=np.uint8)
    snap = pool.copy()
    h = 2
    pairs = np.asarray([[3, 5], [9, 0]], np.int32)
    oracle.recall_strided(host.reshape(-1), pool.reshape(-1), pairs, frag, Hkv * frag, h * frag)
    for b, s in pairs:
        assert np.array_equal(pool[s, h], host[b, h])
    mask = np.ones(pool.shape[:2], bool)
    mask[pairs[:, 1], h] = False
    assert np.array_equal(pool[mask], snap[mask])


def test_paged_recall_reads_the_page_the_table_names_and_nothing_else():
    """Block b of a paged store is arena page page_table[b]: the pool must hold exactly what a
    recall from the block-major store (the arena gathered through the table) would give."""
    rng = np.random.default_rng(8)
    unit, nb, n_pages, C = 128, 20, 64, 9
    arena = rng.integers(0, 256, size=(n_pages, unit), dtype=np.uint8)
    table = rng.permutation(n_pages)[:nb].astype(np.int32)
    pairs = np.asarray([[2, 7], [3, 0], [19, 4]], np.int32)
    pool = rng.integers(0, 256, size=(C, unit), dtype=np.uint8)
    snap = pool.copy()
    oracle.recall_paged(arena, table, pool, pairs, unit)
    for b, s in pairs:
        assert np.array_equal(pool[s], arena[table[b]])            # written out, no call of the oracle
    untouched = np.setdiff1d(np.arange(C), pairs[:, 1])
    assert np.array_equal(pool[untouched], snap[untouched])
    # the identity table is the block-major store
    ref = snap.copy()
    oracle.recall(arena, ref, pairs, unit)
    ident = snap.copy()
    oracle.recall_paged(arena, np.arange(n_pages, dtype=np.int32), ident, pairs, unit)
    assert np.array_equal(ident, ref)
    # distinct pages per block: the page index, not the block index, picks the bytes
    assert not np.array_equal(pool[7], arena[2]) or table[2] == 2
