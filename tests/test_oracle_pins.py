"""Pins of the CPU oracle against things other than itself: a hand-worked example,
closed forms, invariants, special cases that reduce to library routines, and brute
force on small inputs.  No GPU needed."""
import json

import numpy as np
import pytest
import torch

import oracle
from workloads import tiny_config
from workloads import generate as gen


def to_bits(x) -> np.ndarray:
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    assert torch.equal(t.float(), torch.as_tensor(np.asarray(x, dtype=np.float32))), "not bf16-exact"
    return oracle.bits(t)


def rand_bits(rng, shape, scale=1.0) -> np.ndarray:
    t = torch.from_numpy(rng.standard_normal(shape).astype(np.float32) * scale).to(torch.bfloat16)
    return oracle.bits(t)


# ----------------------------------------------------------------- layout arithmetic
def test_layout_bytes_match_paper_figures():
    # Sec. 3.4 / 4.4.1: block 16, head_dim 128, bf16, K and V -> 8 KB per (block, head)
    cfg = tiny_config(block_tokens=16)
    assert cfg.frag_bytes == 8192
    # Sec. 5 Setup: 2048-token budget = 16 sink + 128 local + 1904 middle, block 16
    from workloads import get_config
    c2 = get_config("c2")
    assert (c2.n_sink_blocks, c2.n_local_blocks, c2.k_mid) == (1, 8, 119)
    assert c2.budget_blocks * c2.block_tokens == 2048 == 16 + 128 + 1904
    # Sec. 2.2: one 128K-token sequence of a 40-layer, 8-kv-head, head_dim-128 model = 20 GB
    per_token = 40 * 8 * 128 * 2 * 2
    assert per_token == 160 * 1024 and per_token * 128 * 1024 == 20 * 2 ** 30


# ----------------------------------------------------------------- hand-worked example
@pytest.fixture(scope="module")
def hand(golden_dir):
    return json.loads((golden_dir / "hand_example.json").read_text())


def _hand_kv(h):
    keys = np.asarray(h["keys"], dtype=np.float32)            # [nb][B][D]
    nb, B, D = keys.shape
    kv = np.zeros((nb, h["Hkv"], 2, B, D), dtype=np.float32)
    kv[:, 0, 0] = keys
    return to_bits(kv)


def test_hand_example_digest_score_select(hand):
    kv = _hand_kv(hand)
    dg = oracle.build_digest(kv, ctx=hand["n_blocks"] * hand["B"], h_star=0)
    assert np.array_equal(oracle.bf16_to_f64(dg[:, 0]), np.asarray(hand["digest_min"], float))
    assert np.array_equal(oracle.bf16_to_f64(dg[:, 1]), np.asarray(hand["digest_max"], float))
    sc = oracle.score(to_bits(hand["q"]), dg, hand["n_blocks"], hand["Hkv"], 0)
    assert sc.tolist() == hand["scores"]
    sel, cnt = oracle.select(sc, hand["n_sink"], hand["n_local"], hand["K"])
    assert cnt == 2 and sel.tolist() == hand["sel"]         # block 0 beats block 3 on the tie


def test_hand_example_diff(hand):
    d = hand["diff"]
    table = np.asarray(d["table_before"], np.int32)
    sb = np.asarray(d["slot_block_before"], np.int32)
    st = np.asarray(d["slot_stamp_before"], np.uint32)
    rc, slots, pairs = oracle.diff(np.asarray(hand["sel"], np.int32), 2, hand["n_blocks"], 0, 0,
                                   d["step"], table, sb, st)
    assert rc == 0
    assert pairs.tolist() == d["miss_pairs"]
    assert table.tolist() == d["table_after"]
    assert sb.tolist() == d["slot_block_after"]
    assert st.tolist() == d["slot_stamp_after"]
    assert slots.tolist() == d["sel_slots"]


# ----------------------------------------------------------------- O1 / O2 scoring
def _case(seed, ctx=250, B=16, Hq=8, Hkv=2, D=128):
    rng = np.random.default_rng(seed)
    nb = (ctx + B - 1) // B
    kv = rand_bits(rng, (nb, Hkv, 2, B, D))
    q = rand_bits(rng, (Hq, D))
    return rng, nb, kv, q


@pytest.mark.parametrize("seed,h_star", [(0, 0), (1, 1)])
def test_score_is_upper_bound_of_token_logits(seed, h_star):
    ctx, B, Hq, Hkv, D = 250, 16, 8, 2, 128
    _, nb, kv, q = _case(seed, ctx, B, Hq, Hkv, D)
    dg = oracle.build_digest(kv, ctx, h_star)
    sc = oracle.score(q, dg, nb, Hkv, h_star)
    G = Hq // Hkv
    qf = oracle.bf16_to_f64(q)[h_star * G:(h_star + 1) * G]          # [G][D]
    kf = oracle.bf16_to_f64(kv)[:, h_star, 0]                        # [nb][B][D]
    logits = np.einsum("gd,ntd->nt", qf, kf)                         # sum over the group
    for b in range(nb):
        valid = min(B, ctx - b * B)
        assert np.all(logits[b, :valid] <= sc[b] + 1e-9)
    # the bound is attained when all tokens of a block are identical
    kv2 = kv.copy()
    kv2[:, :, :, 1:] = kv2[:, :, :, :1]
    sc2 = oracle.score(q, oracle.build_digest(kv2, ctx, h_star), nb, Hkv, h_star)
    l2 = np.einsum("gd,nd->n", qf, oracle.bf16_to_f64(kv2)[:, h_star, 0, 0])
    np.testing.assert_allclose(sc2, l2, rtol=1e-12, atol=1e-12)


def test_digest_ignores_tokens_beyond_ctx_and_other_heads():
    ctx, B, Hkv = 250, 16, 2
    rng, nb, kv, _ = _case(3, ctx, B, 8, Hkv)
    dg = oracle.build_digest(kv, ctx, 1)
    kv2 = kv.copy()
    kv2[nb - 1, :, :, ctx - (nb - 1) * B:] = to_bits(np.float32(1000.0))     # past the end
    kv2[:, 0] = rand_bits(rng, kv2[:, 0].shape)                                # the other head
    kv2[:, 1, 1] = rand_bits(rng, kv2[:, 1, 1].shape)                          # V plane
    assert np.array_equal(dg, oracle.build_digest(kv2, ctx, 1))
    kf = oracle.bf16_to_f64(kv)[:, 1, 0]
    assert np.array_equal(oracle.bf16_to_f64(dg[0, 0]), kf[0].min(axis=0))
    assert np.array_equal(oracle.bf16_to_f64(dg[nb - 1, 1]), kf[nb - 1, :ctx - (nb - 1) * B].max(axis=0))


def test_block_of_one_token_reduces_to_gemv():
    ctx, B, Hq, Hkv, D = 37, 1, 8, 2, 128
    _, nb, kv, q = _case(5, ctx, B, Hq, Hkv, D)
    dg = oracle.build_digest(kv, ctx, 1)
    sc = oracle.score(q, dg, nb, Hkv, 1)
    G = Hq // Hkv
    ref = oracle.bf16_to_f64(kv)[:, 1, 0, 0] @ oracle.bf16_to_f64(q)[G:2 * G].sum(axis=0)
    np.testing.assert_allclose(sc, ref, rtol=1e-12, atol=1e-12)


def test_score_equals_qplus_qminus_form():
    _, nb, kv, q = _case(6)
    dg = oracle.build_digest(kv, 250, 0)
    sc = oracle.score(q, dg, nb, 2, 0)
    qf = oracle.bf16_to_f64(q)[:4]
    qp, qm = np.maximum(qf, 0).sum(0), np.minimum(qf, 0).sum(0)
    d = oracle.bf16_to_f64(dg)
    np.testing.assert_allclose(sc, d[:, 1] @ qp + d[:, 0] @ qm, rtol=1e-12, atol=1e-12)


def test_selection_invariant_to_positive_query_scale():
    _, nb, kv, q = _case(7)
    dg = oracle.build_digest(kv, 250, 0)
    q4 = oracle.bits((torch.from_numpy(oracle.bf16_to_f64(q)).float() * 4).to(torch.bfloat16))
    a, _ = oracle.select(oracle.score(q, dg, nb, 2, 0), 1, 2, 8)
    b, _ = oracle.select(oracle.score(q4, dg, nb, 2, 0), 1, 2, 8)
    assert np.array_equal(a, b)


# ----------------------------------------------------------------- O3 selection
def _brute_select(score, n_sink, n_local, K):
    n = len(score)
    pinned = [b for b in range(n) if b < n_sink or b >= n - n_local]
    mid = [b for b in range(n) if b not in pinned]
    order = sorted(mid, key=lambda b: (-score[b], b))
    return sorted(pinned + order[:max(0, K - n_sink - n_local)])


@pytest.mark.parametrize("n,n_sink,n_local,K,levels", [
    (40, 1, 2, 10, 0), (40, 1, 2, 10, 3), (64, 0, 0, 7, 2), (33, 2, 4, 20, 0), (9, 1, 8, 12, 0),
    (5, 1, 8, 12, 0), (50, 1, 2, 60, 0)])
def test_select_matches_brute_force(n, n_sink, n_local, K, levels):
    rng = np.random.default_rng(n * 31 + K)
    for _ in range(20):
        sc = rng.standard_normal(n)
        if levels:                      # few distinct values: many ties
            sc = np.round(sc * levels) / levels
        sel, cnt = oracle.select(sc, n_sink, n_local, K)
        want = _brute_select(sc, n_sink, n_local, K)[:K]
        assert cnt == len(want) and sel[:cnt].tolist() == want
        assert np.all(sel[cnt:] == -1)


def test_select_all_when_budget_covers_middle_and_permutation():
    rng = np.random.default_rng(0)
    sc = rng.standard_normal(30)
    sel, cnt = oracle.select(sc, 1, 2, 64)
    assert cnt == 30 and sel[:30].tolist() == list(range(30))
    # permuting the middle scores permutes the chosen middle blocks
    mid = np.arange(1, 28)
    perm = rng.permutation(mid)
    sc2 = sc.copy()
    sc2[mid] = sc[perm]                 # block mid[i] now has the score of block perm[i]
    a, ca = oracle.select(sc, 1, 2, 10)
    b, cb = oracle.select(sc2, 1, 2, 10)
    inv = {int(p): int(m) for m, p in zip(mid, perm)}
    moved = sorted(inv.get(int(x), int(x)) for x in a[:ca])
    assert moved == b[:cb].tolist()
    for s in (a, b):
        assert {0, 28, 29} <= set(s.tolist())


# ----------------------------------------------------------------- O4 diff
def _brute_diff(sel, n_blocks, n_sink, n_local, step, table, slot_block, stamp):
    selset = {int(b) for b in sel if b >= 0}
    where = {int(b): s for s, b in enumerate(slot_block) if b >= 0}
    miss = sorted(selset - set(where))
    pinned = {b for b in range(n_blocks) if b < n_sink or b >= n_blocks - n_local}
    cand = sorted((int(stamp[s]), s) for s, b in enumerate(slot_block)
                  if b < 0 or (int(b) not in selset and int(b) not in pinned))
    if len(cand) < len(miss):
        return None
    pairs = []
    for b, (_, s) in zip(miss, cand):
        if slot_block[s] >= 0:
            table[slot_block[s]] = -1
        table[b], slot_block[s] = s, b
        pairs.append([b, s])
    for b in selset:
        stamp[table[b]] = step
    return pairs


def test_diff_matches_set_brute_force_over_many_steps():
    n_blocks, n_sink, n_local, K, C = 96, 1, 3, 24, 40
    rng = np.random.default_rng(11)
    table = np.full(n_blocks, -1, np.int32)
    sb = np.full(C, -1, np.int32)
    st = np.zeros(C, np.uint32)
    for i, b in enumerate([0, 93, 94, 95] + rng.choice(np.arange(1, 93), 20, replace=False).tolist()):
        table[b], sb[i] = i, b
    t2, sb2, st2 = table.copy(), sb.copy(), st.copy()
    base = rng.standard_normal(n_blocks)
    for step in range(1, 40):
        base = 0.8 * base + 0.6 * rng.standard_normal(n_blocks)
        sel, cnt = oracle.select(base, n_sink, n_local, K)
        before = sb.copy()
        rc, slots, pairs = oracle.diff(sel, cnt, n_blocks, n_sink, n_local, step, table, sb, st)
        want = _brute_diff(sel, n_blocks, n_sink, n_local, step, t2, sb2, st2)
        assert rc == 0 and pairs.tolist() == want
        assert np.array_equal(table, t2) and np.array_equal(sb, sb2) and np.array_equal(st, st2)
        # invariants
        hits = [b for b in sel[:cnt] if b in set(before[before >= 0].tolist())]
        assert len(hits) + len(pairs) == cnt
        assert all(not (b < n_sink or b >= n_blocks - n_local) for b, _ in pairs)
        for s, b in enumerate(sb):
            assert b < 0 or table[b] == s                    # mutual inverses
        assert (table >= 0).sum() == (sb >= 0).sum() <= C
        assert all(table[b] >= 0 and slots[j] == table[b] for j, b in enumerate(sel[:cnt]))
        assert len(set(slots[:cnt].tolist())) == cnt
        assert np.all(st[slots[:cnt]] == step)


def test_diff_reports_pool_too_small_and_leaves_tables_alone():
    n_blocks, C = 10, 3
    table = np.full(n_blocks, -1, np.int32)
    sb = np.asarray([0, 9, 4], np.int32)
    st = np.asarray([1, 1, 1], np.uint32)
    table[[0, 9, 4]] = [0, 1, 2]
    snap = (table.copy(), sb.copy(), st.copy())
    sel = np.asarray([0, 2, 3, 9], np.int32)                   # 2 misses, 1 evictable slot
    rc, slots, pairs = oracle.diff(sel, 4, n_blocks, 1, 1, 2, table, sb, st)
    assert rc == oracle.POOL_TOO_SMALL and len(pairs) == 0
    assert all(np.array_equal(a, b) for a, b in zip(snap, (table, sb, st)))
    assert slots.tolist() == [0, -1, -1, 1]


# ----------------------------------------------------------------- O5 recall
def test_recall_copies_exact_bytes_and_nothing_else():
    rng = np.random.default_rng(2)
    unit = 512
    host = rng.integers(0, 256, size=(20, unit), dtype=np.uint8)
    pool = rng.integers(0, 256, size=(8, unit), dtype=np.uint8)
    snap = pool.copy()
    pairs = np.asarray([[3, 5], [4, 0], [17, 6]], np.int32)
    oracle.recall(host, pool, pairs, unit)
    for b, s in pairs:
        assert pool[s].tobytes() == host[b].tobytes()
    untouched = [s for s in range(8) if s not in pairs[:, 1]]
    assert np.array_equal(pool[untouched], snap[untouched])


# ----------------------------------------------------------------- O6 attention
def _dense_reference(q, kv, ctx, B, Hkv):
    """Dense attention over all ctx tokens through a library routine, in fp64."""
    qf = torch.from_numpy(oracle.bf16_to_f64(q))                        # [Hq][D]
    kvf = torch.from_numpy(oracle.bf16_to_f64(kv))                      # [nb][Hkv][2][B][D]
    Hq, D = qf.shape
    k = kvf[:, :, 0].permute(1, 0, 2, 3).reshape(Hkv, -1, D)[:, :ctx]
    v = kvf[:, :, 1].permute(1, 0, 2, 3).reshape(Hkv, -1, D)[:, :ctx]
    G = Hq // Hkv
    out = torch.nn.functional.scaled_dot_product_attention(
        qf.view(Hkv, G, D), k, v)                                        # [Hkv][G][D]
    return out.reshape(Hq, D).numpy()


@pytest.mark.parametrize("ctx", [256, 250, 17])
def test_sparse_equals_dense_when_everything_is_selected(ctx):
    B, Hq, Hkv = 16, 8, 2
    _, nb, kv, q = _case(21, ctx, B, Hq, Hkv)
    blocks = np.arange(nb, dtype=np.int32)
    out, lse = oracle.attention(q, kv, blocks, blocks, nb, ctx, B, Hkv)
    np.testing.assert_allclose(out, _dense_reference(q, kv, ctx, B, Hkv), rtol=1e-9, atol=1e-12)
    # lse against a direct logsumexp
    qf, kf = oracle.bf16_to_f64(q), oracle.bf16_to_f64(kv)[:, :, 0]
    for g in range(Hq):
        s = (kf[:, g // (Hq // Hkv)].reshape(-1, 128)[:ctx] @ qf[g]) / np.sqrt(128.0)
        np.testing.assert_allclose(lse[g], np.log(np.exp(s - s.max()).sum()) + s.max(), rtol=1e-12)


def test_sparse_subset_matches_library_attention_on_gathered_tokens_and_order():
    ctx, B, Hq, Hkv = 400, 16, 8, 2
    rng, nb, kv, q = _case(22, ctx, B, Hq, Hkv)
    sel = np.sort(rng.choice(nb - 1, 9, replace=False)).astype(np.int32)
    sel = np.append(sel, nb - 1).astype(np.int32)            # includes the ragged last block
    out, _ = oracle.attention(q, kv, sel, sel, len(sel), ctx, B, Hkv)
    gathered = kv[sel]
    n_tok = (len(sel) - 1) * B + (ctx - (nb - 1) * B)
    ref = _dense_reference(q, gathered, n_tok, B, Hkv)
    np.testing.assert_allclose(out, ref, rtol=1e-9, atol=1e-12)
    perm = rng.permutation(len(sel))
    out2, _ = oracle.attention(q, kv, sel[perm], sel[perm], len(sel), ctx, B, Hkv)
    np.testing.assert_allclose(out2, out, rtol=1e-12, atol=1e-14)


def test_attention_special_cases():
    ctx, B, Hq, Hkv, D = 64, 16, 4, 2, 128
    rng, nb, kv, q = _case(23, ctx, B, Hq, Hkv, D)
    blocks = np.arange(nb, dtype=np.int32)
    # identical keys -> uniform weights -> mean of the values
    kv1 = kv.copy()
    kv1[:, :, 0] = kv1[0, 0, 0, 0]
    out, _ = oracle.attention(q, kv1, blocks, blocks, nb, ctx, B, Hkv)
    vmean = oracle.bf16_to_f64(kv1)[:, :, 1].transpose(1, 0, 2, 3).reshape(Hkv, -1, D).mean(axis=1)
    np.testing.assert_allclose(out, np.repeat(vmean, Hq // Hkv, axis=0), rtol=1e-12, atol=1e-13)
    # one dominant logit -> that token's value row
    kv2 = kv.copy()
    kv2[:, :, 0] = 0
    big = oracle.bits((torch.from_numpy(oracle.bf16_to_f64(q[0])).float() * 64).to(torch.bfloat16))
    kv2[2, 0, 0, 5] = big
    out, _ = oracle.attention(q, kv2, blocks, blocks, nb, ctx, B, Hkv)
    np.testing.assert_allclose(out[0], oracle.bf16_to_f64(kv2[2, 0, 1, 5]), atol=1e-9)


def test_attention_through_pool_slots_equals_attention_on_host_copy():
    ctx, B, Hq, Hkv = 400, 16, 8, 2
    rng, nb, kv, q = _case(24, ctx, B, Hq, Hkv)
    sel = np.sort(rng.choice(nb, 10, replace=False)).astype(np.int32)
    slots = rng.permutation(16)[:10].astype(np.int32)
    pool = rand_bits(rng, (16,) + kv.shape[1:])
    unit = kv[0].nbytes
    oracle.recall(kv.view(np.uint8).reshape(nb, unit), pool.view(np.uint8).reshape(16, unit),
                  np.stack([sel, slots], 1), unit)
    a, la = oracle.attention(q, pool, slots, sel, 10, ctx, B, Hkv)
    b, lb = oracle.attention(q, kv, sel, sel, 10, ctx, B, Hkv)
    assert np.array_equal(a, b) and np.array_equal(la, lb)


# ----------------------------------------------------------------- whole layer-step
def test_layer_step_is_the_composition_of_its_stages():
    cfg = tiny_config()
    kv = gen.make_kv(cfg, 0)
    q = gen.make_queries(cfg, 0, 3, ar1=0.9)
    res = gen.initial_resident(cfg, 0)
    h = cfg.solo_head(0)
    nb, C, K = cfg.n_blocks, cfg.pool_slots, cfg.budget_blocks
    kvb = oracle.bits(kv)
    dg = np.stack([oracle.build_digest(kvb[s], cfg.ctx, h) for s in range(cfg.batch)])
    table = np.full((cfg.batch, nb), -1, np.int32)
    sb = res.copy()
    st = np.zeros((cfg.batch, C), np.uint32)
    pool = np.zeros((cfg.batch, C) + kvb.shape[2:], np.uint16)
    for s in range(cfg.batch):
        for i, b in enumerate(res[s]):
            if b >= 0:
                table[s, b] = i
                pool[s, i] = kvb[s, b]
    t2, sb2, st2, pool2 = table.copy(), sb.copy(), st.copy(), pool.copy()
    ctx_len = np.full(cfg.batch, cfg.ctx, np.int32)
    for step in range(1, 4):
        qb = oracle.bits(q[step - 1])
        r = oracle.layer_step(ctx_len, nb, cfg.block_tokens, cfg.n_kv_heads, h, K, cfg.n_sink_blocks,
                              cfg.n_local_blocks, step, qb, dg, kvb, table, sb, st, pool)
        assert r["rc"] == 0
        for s in range(cfg.batch):
            sc = oracle.score(qb[s], dg[s], nb, cfg.n_kv_heads, h)
            sel, cnt = oracle.select(sc, cfg.n_sink_blocks, cfg.n_local_blocks, K)
            rc, slots, pairs = oracle.diff(sel, cnt, nb, cfg.n_sink_blocks, cfg.n_local_blocks, step,
                                           t2[s], sb2[s], st2[s])
            unit = kvb[s, 0].nbytes
            oracle.recall(kvb[s].view(np.uint8).reshape(nb, unit),
                          pool2[s].view(np.uint8).reshape(C, unit), pairs, unit)
            out, lse = oracle.attention(qb[s], pool2[s], slots, sel, cnt, cfg.ctx, cfg.block_tokens,
                                        cfg.n_kv_heads)
            assert np.array_equal(sc, r["score"][s]) and np.array_equal(sel, r["sel"][s])
            assert np.array_equal(slots, r["sel_slots"][s]) and len(pairs) == r["n_miss"][s]
            assert np.array_equal(out, r["out"][s]) and np.array_equal(lse, r["lse"][s])
            # byte invariant: every selected block's pool bytes equal the host bytes
            for j in range(cnt):
                assert np.array_equal(pool[s, slots[j]], kvb[s, sel[j]])
        assert np.array_equal(pool, pool2) and np.array_equal(table, t2)


# ----------------------------------------------------------------- Middle Attention Mass (Eq. 2)
def test_attention_mass_of_a_token_set_from_two_logsumexps():
    """sum_{i in S} A(i) = exp(lse_S - lse_all): the identity the MAM helper relies on, checked
    against the softmax weights written out."""
    ctx, B, Hq, Hkv = 400, 16, 8, 2
    _, nb, kv, q = _case(31, ctx, B, Hq, Hkv)
    allb = np.arange(nb, dtype=np.int32)
    mid = np.arange(1, nb - 8, dtype=np.int32)
    _, lse_all = oracle.attention(q, kv, allb, allb, nb, ctx, B, Hkv)
    _, lse_mid = oracle.attention(q, kv, mid, mid, len(mid), ctx, B, Hkv)
    qf, kf = oracle.bf16_to_f64(q), oracle.bf16_to_f64(kv)[:, :, 0]
    for g in range(Hq):
        s = (kf[:, g // (Hq // Hkv)].reshape(-1, 128)[:ctx] @ qf[g]) / np.sqrt(128.0)
        w = np.exp(s - s.max()); w /= w.sum()
        np.testing.assert_allclose(np.exp(lse_mid[g] - lse_all[g]), w[B:(nb - 8) * B].sum(), rtol=1e-10)
