"""CUDA path vs CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from workloads import get_config, tiny_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")


def test_tiny_ragged_batch_multi_step():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=3, ctx=1000)                       # 63 blocks, last one partial (8 tokens)
    case = make_case(cfg, steps=6, ctx_len=np.asarray([1000, 517, 160]))
    stats = run_and_compare(case, steps=6)
    assert sum(stats["misses"]) > 0


@pytest.mark.parametrize("fused", [False, True])
def test_selection_and_diff_as_two_calls_and_as_one(fused):
    """The path with pi_score_select + pi_diff_misses, and with pi_score_select_diff, against the oracle:
    ragged batch, cold pool (many misses: the ranking path of the victim choice), several steps."""
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=4, ctx=5000, n_q_heads=16, n_kv_heads=4, budget_blocks=48, resident_frac=0.25)
    case = make_case(cfg, steps=5, ctx_len=np.asarray([5000, 4999, 2100, 330]), fill=0.3)
    stats = run_and_compare(case, steps=5, fused=fused)
    assert max(stats["misses"]) > 8 and min(stats["misses"]) <= 8


def test_one_launch_equals_two_launches_bit_for_bit():
    """pi_score_select_diff writes exactly what pi_score_select followed by pi_diff_misses writes."""
    import paper_2609_34555_b200 as pkg
    from paper_2609_34555_b200.runner import LayerBuffers
    from workloads import generate as gen
    for cfg in (get_config("c2").replace(n_layers=1, batch=5), tiny_config(batch=3, ctx=2000, budget_blocks=32, resident_frac=0.3)):
        dev = torch.device("cuda:0")
        pi = pkg.PulseInfer.from_workload(cfg)
        ctx = torch.full((cfg.batch,), cfg.ctx, dtype=torch.int32, device=dev)
        ctx[-1] = cfg.ctx // 2 + 3
        q = gen.make_queries(cfg, 0, 4, ar1=0.8).to(dev)
        res = torch.from_numpy(gen.initial_resident(cfg.replace(ctx=int(ctx[-1])), 0)[:, :cfg.pool_slots]).to(dev)
        res = torch.nn.functional.pad(res, (0, cfg.pool_slots - res.shape[1]), value=-1).contiguous()
        digest = torch.randn((cfg.batch, cfg.n_blocks, 2, 128), generator=torch.Generator().manual_seed(3)).to(torch.bfloat16).to(dev)
        bufs = [LayerBuffers(pi, cfg.batch, dev, keep_scores=True) for _ in range(2)]
        for b in bufs:
            b.digest.copy_(digest)
            pi.table_init(res, b.block_table, b.slot_block, b.slot_stamp)
        for step in range(1, 5):
            a, b = bufs
            pi.score_select(0, q[step - 1], a.digest, ctx, a.sel_blocks, a.sel_count, a.scores)
            pi.diff_misses(0, step, ctx, a.sel_blocks, a.sel_count, a.block_table, a.slot_block, a.slot_stamp,
                           a.sel_slots, a.recall_list, a.recall_count)
            pi.score_select_diff(0, step, q[step - 1], b.digest, ctx, b.sel_blocks, b.sel_count, b.block_table,
                                 b.slot_block, b.slot_stamp, b.sel_slots, b.recall_list, b.recall_count, scores=b.scores)
            torch.cuda.synchronize()
            assert pi.status()[0] == 0, pi.status()
            for name in ("scores", "sel_blocks", "sel_count", "block_table", "slot_block", "slot_stamp", "sel_slots", "recall_count"):
                assert torch.equal(getattr(a, name), getattr(b, name)), (step, name)
            n = a.recall_count.cpu().numpy()
            for s_ in range(cfg.batch):
                assert torch.equal(a.recall_list[s_, :n[s_]], b.recall_list[s_, :n[s_]]), (step, s_)
            assert int(a.recall_count.sum()) > 0 or step > 1
        pi.close()


def test_config1_planted_query():
    from tests.parity import make_case, run_and_compare
    cfg = get_config("c1")
    case = make_case(cfg, steps=3, plant=True)
    stats = run_and_compare(case, steps=3)
    assert stats["misses"][0] > 0


def test_group_of_eight_heads_and_block_32_overlapped_streams():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=5, ctx=4000, n_q_heads=64, n_kv_heads=8, block_tokens=32, budget_blocks=20,
                      resident_frac=0.3)
    case = make_case(cfg, steps=4)
    run_and_compare(case, steps=4, overlapped=True)


def test_block_64_many_ctas_split_one_sequence():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=1, ctx=8000, n_q_heads=8, n_kv_heads=2, block_tokens=64, budget_blocks=48,
                      resident_frac=0.5)
    case = make_case(cfg, steps=3)
    run_and_compare(case, steps=3)


def test_budget_covers_all_blocks_equals_dense_attention():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=2, ctx=300, budget_blocks=24, resident_frac=1.0)   # 19 blocks < K
    case = make_case(cfg, steps=2)
    stats = run_and_compare(case, steps=2)
    assert sum(stats["misses"]) == 0


def test_cold_start_empty_pool():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=2, ctx=2000, budget_blocks=32, resident_frac=0.4)
    case = make_case(cfg, steps=3, fill=0.0)                    # only sink/local resident
    stats = run_and_compare(case, steps=3)
    assert stats["extents"] < sum(stats["misses"])            # cold fill lands in adjacent slots: runs merge


def test_cold_start_with_many_misses_takes_the_sort_path():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=2, ctx=16000, n_q_heads=16, n_kv_heads=4, budget_blocks=100, resident_frac=0.2)
    case = make_case(cfg, steps=3, fill=0.0)                    # 91 misses per sequence at step 1
    stats = run_and_compare(case, steps=3)
    assert max(stats["misses"]) > 40 and min(stats["misses"]) <= 40


def test_full_size_config2_shapes_sampled_sequences():
    """Launch configuration of the bench (batch 16, 2048 blocks, K 128, C 409, pipelined
    DecodeSession) on two of the 32 layers; the oracle follows three of the 16 sequences."""
    from tests.parity import run_session_sampled
    cfg = get_config("c2").replace(n_layers=2)
    stats = run_session_sampled(cfg, steps=3, sample_seqs=[0, 7, 15])
    assert stats["misses"] > 0


def test_full_size_config4_shapes_group_of_eight_sampled():
    """70B-shaped layer (64 query heads / 8 kv heads, 4096 blocks, K 256, C 614), one layer,
    two of the 8 sequences followed by the oracle."""
    from tests.parity import run_session_sampled
    cfg = get_config("c4").replace(n_layers=1)
    run_session_sampled(cfg, steps=2, sample_seqs=[1, 6])


def test_full_size_config3_shapes_block_32_sampled():
    """Per-sequence shapes of the long-context config (131072 tokens, 4096 blocks of 32 tokens, K 64,
    C 409) on one layer and 8 of its 64 sequences; the oracle follows two of them."""
    from tests.parity import run_session_sampled
    cfg = get_config("c3").replace(n_layers=1, batch=8)
    stats = run_session_sampled(cfg, steps=3, sample_seqs=[2, 6])
    assert stats["misses"] > 0


@pytest.mark.parametrize("B", [16, 64])
def test_full_size_config5_shapes_batch_32_sampled(B):
    """The recall-fragmentation config's layer (batch 32, 32 768 tokens; blocks of 16 tokens with a budget of
    128 blocks, and blocks of 64 tokens with a budget of 32) in the bench's launch configuration: 256 work
    items for the attention (two per CTA), 32 selection clusters; the oracle follows three sequences."""
    from tests.parity import run_session_sampled
    cfg = get_config("c5").replace(block_tokens=B, budget_blocks=max(128 * 16 // B, 16))
    stats = run_session_sampled(cfg, steps=3, sample_seqs=[0, 17, 31])
    assert stats["misses"] > 0


def gen_pinned(cfg):
    from workloads import generate as gen
    return gen.pinned_blocks(cfg).tolist()


def test_errors_seen_on_the_device_or_at_the_boundary():
    import paper_2609_34555_b200 as pkg
    from paper_2609_34555_b200.runner import LayerBuffers
    cfg = tiny_config(batch=2, ctx=1000)
    dev = torch.device("cuda:0")
    pi = pkg.PulseInfer.from_workload(cfg)
    buf = LayerBuffers(pi, cfg.batch, dev)
    # an unpinned host store is refused before anything is launched
    host = torch.zeros((cfg.batch, cfg.n_blocks, cfg.block_bytes // 2), dtype=torch.bfloat16)
    with pytest.raises(pkg.PiError) as e:
        pi.recall_gather_scatter(0, host, buf.pool, buf.recall_list, buf.recall_count)
    assert e.value.code == -5
    # a selection index out of range sets the status word and is skipped, nothing faults
    ctx = torch.full((cfg.batch,), cfg.ctx, dtype=torch.int32, device=dev)
    buf.sel_blocks.fill_(-1)
    buf.sel_blocks[0, 0] = 10 ** 6
    buf.sel_count.fill_(1)
    buf.sel_blocks[1, 0] = 0
    pi.diff_misses(0, 1, ctx, buf.sel_blocks, buf.sel_count, buf.block_table, buf.slot_block, buf.slot_stamp,
                   buf.sel_slots, buf.recall_list, buf.recall_count)
    torch.cuda.synchronize()
    st = pi.status()
    assert st[0] == -8 and st[1] == 2 and st[2] == 0 and st[4] == 10 ** 6
    assert buf.sel_slots[0, 0].item() == -1 and buf.recall_count[0].item() == 0
    pi.clear_status()
    assert pi.status()[0] == 0
    # a pool with fewer evictable slots than misses: tables untouched, status says so
    small = tiny_config(batch=1, ctx=1000, resident_frac=0.0)                    # C == K == 24
    pi2 = pkg.PulseInfer.from_workload(small)
    b2 = LayerBuffers(pi2, 1, dev)
    C = small.pool_slots
    pinned = gen_pinned(small)
    middle = [b for b in range(small.n_blocks) if b not in set(pinned)]
    res = torch.tensor([pinned + middle[:C - len(pinned)]], dtype=torch.int32, device=dev)
    pi2.table_init(res, b2.block_table, b2.slot_block, b2.slot_stamp)
    sel = torch.tensor([middle[C:C + small.budget_blocks]], dtype=torch.int32, device=dev)    # 24 misses, 15 candidates
    cnt = torch.tensor([small.budget_blocks], dtype=torch.int32, device=dev)
    ctx1 = torch.tensor([small.ctx], dtype=torch.int32, device=dev)
    before = (b2.block_table.clone(), b2.slot_block.clone(), b2.slot_stamp.clone())
    pi2.diff_misses(0, 3, ctx1, sel, cnt, b2.block_table, b2.slot_block, b2.slot_stamp, b2.sel_slots,
                    b2.recall_list, b2.recall_count)
    torch.cuda.synchronize()
    st = pi2.status()
    assert st[0] == -4 and st[1] == 2 and st[3] == small.budget_blocks and st[4] == C - len(pinned)
    assert b2.recall_count[0].item() == 0 and (b2.sel_slots == -1).all()
    assert all(torch.equal(a, b) for a, b in zip(before, (b2.block_table, b2.slot_block, b2.slot_stamp)))
    pi2.close()
    pi.close()


def test_recall_skips_and_reports_an_extent_that_leaves_the_pool_or_the_host_region():
    """One hand-built extent whose destination runs past the sequence's last pool slot (and one whose
    source runs past the sequence's last block) among valid ones: the units outside are skipped and
    reported (status -8, stage 3: list, extent, unit), the units inside are copied, and nothing is
    written outside the pool (guard zones before and after it)."""
    import paper_2609_34555_b200 as pkg
    from workloads import generate as gen
    cfg = tiny_config(batch=2, ctx=1000)
    dev = torch.device("cuda:0")
    pi = pkg.PulseInfer.from_workload(cfg)
    C, nb, bb = cfg.pool_slots, cfg.n_blocks, cfg.block_bytes
    kv = gen.make_kv(cfg, 0).pin_memory()
    arena, (off,) = _carve([cfg.batch * C * bb], dev)
    pool = arena[off:off + cfg.batch * C * bb].view(torch.bfloat16).view(cfg.batch, C, cfg.n_kv_heads, 2, cfg.block_tokens, 128)
    pool.zero_()
    covered = torch.zeros(arena.numel(), dtype=torch.bool, device=dev)
    covered[off:off + cfg.batch * C * bb] = True
    for bad, want_value in (((5, C - 1, 3, 3), C), ((nb - 2, 9, 4, 3), nb)):
        pool.zero_()
        lst = torch.zeros((cfg.batch, cfg.budget_blocks, 4), dtype=torch.int32, device=dev)
        lst[0, 0] = torch.tensor([3, 2, 2, 0])                    # blocks 3,4 -> slots 2,3
        lst[0, 1] = torch.tensor([20, 7, 1, 2])                   # block 20 -> slot 7
        lst[1, 0] = torch.tensor([1, 0, 3, 0])                    # blocks 1..3 -> slots 0..2
        lst[1, 1] = torch.tensor(bad)                             # runs off the end (first unit is inside)
        cnt = torch.tensor([2, 2], dtype=torch.int32, device=dev)
        pi.recall_gather_scatter(0, kv, pool, lst, cnt)
        torch.cuda.synchronize()
        st = pi.status()
        # (the units outside are found by different warps at the same time: either one may report first)
        assert st[0] == -8 and st[1] == 3 and st[2] == 1 and st[3] == 1 and st[4] in (want_value, want_value + 1), st
        assert bool((arena[~covered] == 0x5A).all()), "written outside the pool"
        got = pool.cpu()
        want = torch.zeros_like(got)
        want[0, 2:4] = kv[0, 3:5]; want[0, 7] = kv[0, 20]; want[1, 0:3] = kv[1, 1:4]
        src, dst, n, _ = bad
        for k in range(n):
            if dst + k < C and src + k < nb:
                want[1, dst + k] = kv[1, src + k]
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
        pi.clear_status()
    # a damaged list (a billion units): skipped as a whole and reported, the other list is copied, the call returns at once
    pool.zero_()
    lst = torch.zeros((cfg.batch, cfg.budget_blocks, 4), dtype=torch.int32, device=dev)
    lst[0, 0] = torch.tensor([3, 2, 2, 0])
    lst[1, 0] = torch.tensor([1, 0, 1 << 30, 0])
    cnt = torch.tensor([1, 1], dtype=torch.int32, device=dev)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record(); pi.recall_gather_scatter(0, kv, pool, lst, cnt); t1.record()
    torch.cuda.synchronize()
    st = pi.status()
    assert st[0] == -9 and st[1] == 3 and st[2] == 1 and st[4] == C, st
    assert t0.elapsed_time(t1) < 50.0
    want = torch.zeros_like(pool.cpu()); want[0, 2:4] = kv[0, 3:5]
    assert torch.equal(pool.cpu().view(torch.int16), want.view(torch.int16))
    assert bool((arena[~covered] == 0x5A).all()), "written outside the pool"
    pi.close()


def test_append_needs_a_local_window_and_9800_blocks_fit_the_selection_kernel():
    import paper_2609_34555_b200 as pkg
    from paper_2609_34555_b200.runner import LayerBuffers
    dev = torch.device("cuda:0")
    # pure top-k (no local window): nothing keeps the block being filled resident, so appends are refused
    cfg = tiny_config(batch=1, ctx=1500, n_q_heads=4, n_kv_heads=1, budget_blocks=20, sink_tokens=0, local_tokens=0)
    pi = pkg.PulseInfer.from_workload(cfg)
    buf = LayerBuffers(pi, 1, dev)
    kv = torch.zeros((1, cfg.n_blocks, 1, 2, 16, 128), dtype=torch.bfloat16).pin_memory()
    k_new = torch.zeros((1, 1, 128), dtype=torch.bfloat16, device=dev)
    ctx = torch.tensor([100], dtype=torch.int32, device=dev)
    with pytest.raises(pkg.PiError) as e:
        pi.append_kv(0, 1, k_new, k_new, ctx, kv, buf.pool, buf.block_table, buf.slot_block, buf.slot_stamp, buf.digest)
    assert e.value.code == -1
    pi.close()
    # 9800 blocks: the key buffer plus the kernel's static shared memory pass 48 KB together
    from tests.parity import make_case, run_and_compare
    big = tiny_config(batch=1, ctx=9800 * 16, n_q_heads=4, n_kv_heads=1, budget_blocks=40, resident_frac=0.01)
    assert big.n_blocks == 9800
    run_and_compare(make_case(big, steps=2), steps=2)


def test_sequences_that_no_cta_splits_pipelined_and_repeatable():
    """Fewer attention CTAs than sequences and equal unit counts: every sequence is covered by one CTA,
    no partial is written and the merge kernel has nothing to do, yet it must still wait for the
    attention kernel before the stream moves on.  One 16-token block per sequence as the smallest
    case; several pipelined steps; two runs give the same bits."""
    from tests.parity import make_case, run_and_compare
    from tests.parity import run_session_sampled
    one_block = tiny_config(batch=4, ctx=16, n_q_heads=8, n_kv_heads=2, budget_blocks=2, resident_frac=1.0,
                            sink_tokens=0, local_tokens=16)
    for ctas in (1, 2, 4):
        run_and_compare(make_case(one_block, steps=2), steps=2, overlapped=True, pi_kwargs=dict(attn_ctas=ctas))
    cfg = tiny_config(batch=6, ctx=2000, n_q_heads=16, n_kv_heads=4, budget_blocks=24, resident_frac=0.4, n_layers=3)
    outs = []
    for _ in range(2):
        st = run_session_sampled(cfg, steps=4, sample_seqs=[0, 3, 5], pi_kwargs=dict(attn_ctas=3), return_out=True)
        outs.append(st["out"])
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("mode", [1, 2])
def test_a_bounded_wait_that_runs_out_is_reported_and_nothing_hangs(mode):
    """A short wait limit and the test-only hold-back of every CTA's last tile: the consumers' wait for that
    tile runs out, the kernel returns by itself, the status word says PI_ERR_TIMEOUT (stage 4) and the
    context stays usable: after clearing the status the same shapes run clean on a context without the hook."""
    import time
    from tests.parity import make_case, run_and_compare
    import paper_2609_34555_b200 as pkg
    from paper_2609_34555_b200.runner import LayerBuffers
    cfg = tiny_config(batch=2, ctx=2000, n_q_heads=16, n_kv_heads=4, budget_blocks=24, resident_frac=1.0)
    dev = torch.device("cuda:0")
    pi = pkg.PulseInfer.from_workload(cfg, wait_limit_us=300, test_hold_producer=1, attn_mode=mode)
    buf = LayerBuffers(pi, cfg.batch, dev)
    ident = torch.arange(cfg.budget_blocks, dtype=torch.int32, device=dev)[None, :].expand(cfg.batch, -1).contiguous()
    buf.sel_slots.copy_(ident); buf.sel_blocks.copy_(ident); buf.sel_count.fill_(cfg.budget_blocks)
    q = torch.randn((cfg.batch, cfg.n_q_heads, 128), device=dev).to(torch.bfloat16)
    ctx = torch.full((cfg.batch,), cfg.ctx, dtype=torch.int32, device=dev)
    out = torch.zeros_like(q)
    t0 = time.perf_counter()
    pi.sparse_decode_attn(0, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx, out)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0                      # gave up after the limit, not after seconds
    st = pi.status()
    assert st[0] == -7 and st[1] == 4 and st[3] < st[4], st    # timeout, attention stage, the CTA's units
    pi.clear_status()
    assert pi.status()[0] == 0
    pi.close()
    # the device and the library are fine afterwards
    run_and_compare(make_case(cfg, steps=2), steps=2)


def test_append_then_decode_with_growing_ragged_contexts():
    from tests.parity import run_append_and_compare
    cfg = tiny_config(batch=4, ctx=1200, n_q_heads=16, n_kv_heads=4, budget_blocks=24, resident_frac=0.4)
    # sequences sit at different offsets inside their last block: block boundaries are crossed at different steps
    stats = run_append_and_compare(cfg, steps=20, ctx_len0=[1000, 1007, 639, 800])
    assert stats["new_blocks"] >= 4


def test_append_block_32_group_of_eight():
    from tests.parity import run_append_and_compare
    cfg = tiny_config(batch=2, ctx=2100, n_q_heads=64, n_kv_heads=8, block_tokens=32, budget_blocks=16, resident_frac=0.3)
    stats = run_append_and_compare(cfg, steps=40, ctx_len0=[2015, 1500])
    assert stats["new_blocks"] >= 2


def test_middle_attention_mass_and_retrieval_head_choice():
    import oracle
    import paper_2609_34555_b200 as pkg
    from paper_2609_34555_b200.mam import choose_solo_head, kv_head_mam, middle_attention_mass
    from workloads import generate as gen
    cfg = tiny_config(batch=3, ctx=1500, n_q_heads=16, n_kv_heads=4, budget_blocks=96, resident_frac=1.0)
    dev = torch.device("cuda:0")
    kv = gen.make_kv(cfg, 0)
    # KV heads 0, 1, 3 are made streaming heads (their queries line up with a sink-token key, so
    # nearly all their attention mass sits outside the middle); head 2 keeps random queries
    q = gen.make_queries(cfg, 0, 1)[0]
    G = cfg.group
    for s in range(cfg.batch):
        for h in (0, 1, 3):
            for g in range(h * G, (h + 1) * G):
                q[s, g] = (kv[s, 0, h, 0, 1].float() * 0.5).to(torch.bfloat16)
    pi = pkg.PulseInfer.from_workload(cfg)
    pool = torch.zeros((cfg.batch, cfg.pool_slots) + tuple(kv.shape[2:]), dtype=torch.bfloat16, device=dev)
    pool[:, :cfg.n_blocks] = kv.to(dev)
    ctx = torch.tensor([1500, 1111, 700], dtype=torch.int32, device=dev)
    mam_t, mam_kv = middle_attention_mass(pi, 0, q.to(dev), pool, ctx, return_kv=True)
    assert torch.allclose(mam_kv.cpu(), kv_head_mam(mam_t.cpu(), cfg.n_kv_heads), rtol=1e-5, atol=1e-7)
    mam = mam_t.cpu().numpy()
    kvb, qb = oracle.bits(kv), oracle.bits(q)
    for s in range(cfg.batch):
        nb = -(-int(ctx[s]) // cfg.block_tokens)
        allb = np.arange(nb, dtype=np.int32)
        mid = np.arange(cfg.n_sink_blocks, nb - cfg.n_local_blocks, dtype=np.int32)
        _, la = oracle.attention(qb[s], kvb[s], allb, allb, nb, int(ctx[s]), cfg.block_tokens, cfg.n_kv_heads)
        _, lm = oracle.attention(qb[s], kvb[s], mid, mid, len(mid), int(ctx[s]), cfg.block_tokens, cfg.n_kv_heads)
        np.testing.assert_allclose(mam[s], np.exp(lm - la), rtol=2e-3, atol=1e-4)
    assert choose_solo_head(torch.from_numpy(mam), cfg.n_kv_heads) == 2
    assert choose_solo_head(torch.from_numpy(mam), cfg.n_kv_heads, reversed_rank=True) != 2
    assert kv_head_mam(torch.from_numpy(mam), cfg.n_kv_heads).shape == (4,)
    assert pi.status()[0] == 0
    pi.close()


def _carve(total_bytes_list, dev, pattern=0x5A):
    """One allocation holding every buffer with 4 KB guard zones before, between and after."""
    guard = 4096
    offs, pos = [], guard
    for n in total_bytes_list:
        pos = (pos + 255) // 256 * 256
        offs.append(pos)
        pos += n + guard
    arena = torch.full((pos + guard,), pattern, dtype=torch.uint8, device=dev)
    return arena, offs


def test_guard_zones_stay_intact_and_results_repeat_bit_for_bit():
    """No out-of-bounds write anywhere on the path (guard zones around every buffer the kernels
    write), and two runs from the same state give identical bytes everywhere."""
    import paper_2609_34555_b200 as pkg
    from workloads import generate as gen
    cfg = tiny_config(batch=3, ctx=3000, n_q_heads=32, n_kv_heads=8, budget_blocks=40, resident_frac=0.3)
    dev = torch.device("cuda:0")
    pi = pkg.PulseInfer.from_workload(cfg)
    nb, C, K, Hq = cfg.n_blocks, cfg.pool_slots, cfg.budget_blocks, cfg.n_q_heads
    shapes = dict(digest=((cfg.batch, nb, 2, 128), torch.bfloat16), table=((cfg.batch, nb), torch.int32),
                  slot_block=((cfg.batch, C), torch.int32), slot_stamp=((cfg.batch, C), torch.int32),
                  pool=((cfg.batch, C, 8, 2, 16, 128), torch.bfloat16), sel=((cfg.batch, K), torch.int32),
                  cnt=((cfg.batch,), torch.int32), slots=((cfg.batch, K), torch.int32),
                  lst=((cfg.batch, K, 4), torch.int32), lcnt=((cfg.batch,), torch.int32),
                  out=((cfg.batch, Hq, 128), torch.bfloat16), lse=((cfg.batch, Hq), torch.float32),
                  scores=((cfg.batch, nb), torch.float32))
    sizes = [int(np.prod(s)) * torch.empty((), dtype=d).element_size() for s, d in shapes.values()]
    kv = gen.make_kv(cfg, 0).pin_memory()
    q = gen.make_queries(cfg, 0, 3, ar1=0.8).to(dev)
    ctx = torch.tensor([3000, 2990, 1600], dtype=torch.int32, device=dev)
    res = torch.from_numpy(gen.initial_resident(cfg.replace(ctx=1600), 0)[:, :C]).to(dev)   # valid for the shortest sequence
    res = torch.nn.functional.pad(res, (0, C - res.shape[1]), value=-1).contiguous()
    results = []
    for run in range(2):
        arena, offs = _carve(sizes, dev)
        t = {}
        for (name, (shape, dt)), off, n in zip(shapes.items(), offs, sizes):
            t[name] = arena[off:off + n].view(dt).view(shape)
        covered = torch.zeros(arena.numel(), dtype=torch.bool, device=dev)
        for off, n in zip(offs, sizes):
            covered[off:off + n] = True
        t["pool"].zero_()
        pi.build_digests(0, kv, ctx, t["digest"])
        pi.table_init(res, t["table"], t["slot_block"], t["slot_stamp"])
        for step in range(1, 4):
            pi.score_select(0, q[step - 1], t["digest"], ctx, t["sel"], t["cnt"], t["scores"])
            pi.diff_misses(0, step, ctx, t["sel"], t["cnt"], t["table"], t["slot_block"], t["slot_stamp"], t["slots"],
                           t["lst"], t["lcnt"])
            pi.recall_gather_scatter(0, kv, t["pool"], t["lst"], t["lcnt"])
            pi.sparse_decode_attn(0, q[step - 1], t["pool"], t["slots"], t["sel"], t["cnt"], ctx, t["out"], t["lse"])
        torch.cuda.synchronize()
        assert pi.status()[0] == 0
        assert bool((arena[~covered] == 0x5A).all()), "a guard zone was written"
        results.append(arena.clone())
    assert torch.equal(results[0], results[1]), "two identical runs differ"
    pi.close()


def test_empty_sequence_in_the_batch():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=3, ctx=1000)
    case = make_case(cfg, steps=3, ctx_len=np.asarray([1000, 0, 7]))     # nothing, and less than one block
    run_and_compare(case, steps=3)


def test_largest_supported_block_count_and_wide_budget():
    """16384 blocks per sequence (the library's limit), 512-block budget, 1024-slot pool."""
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=1, ctx=262144, n_q_heads=8, n_kv_heads=2, budget_blocks=512, resident_frac=1024 / 16384)
    assert cfg.n_blocks == 16384 and cfg.pool_slots == 1024
    case = make_case(cfg, steps=2)
    stats = run_and_compare(case, steps=2)
    assert stats["misses"][0] > 100


def test_more_than_512_misses_in_the_fused_launch_take_the_sorting_path():
    """A 640-block budget against a pool of 1 024 slots that holds almost none of the selection: about 600
    misses per step, beyond what the ranked victim search covers.  In the one-launch form the cluster's other
    CTAs still prepare the eviction order (the pool is small enough for it); the first CTA ignores it, sorts,
    and must not leave before they are done."""
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=2, ctx=131072, n_q_heads=8, n_kv_heads=2, budget_blocks=640, resident_frac=1024 / 8192)
    assert cfg.n_blocks == 8192 and cfg.pool_slots == 1024
    case = make_case(cfg, steps=2)
    stats = run_and_compare(case, steps=2)
    assert max(stats["misses"]) > 512


def test_averaged_and_headwise_selection_strategies():
    from tests.parity import run_strategies_and_compare
    cfg = tiny_config(batch=2, ctx=3000, n_q_heads=16, n_kv_heads=4, budget_blocks=32, resident_frac=0.3)
    stats = run_strategies_and_compare(cfg, steps=2)
    assert stats["misses"] > 0 and stats["distinct_head_selections"] > 1


def test_strategies_with_eight_kv_heads_and_group_of_eight():
    from tests.parity import run_strategies_and_compare
    cfg = tiny_config(batch=2, ctx=2500, n_q_heads=64, n_kv_heads=8, budget_blocks=24, resident_frac=0.25)
    run_strategies_and_compare(cfg, steps=2)


def test_group_of_sixteen_query_heads_per_kv_head():
    """G = 16 takes the two-column-tile variant of the attention kernel."""
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=2, ctx=2000, n_q_heads=32, n_kv_heads=2, budget_blocks=24, resident_frac=0.3)
    run_and_compare(make_case(cfg, steps=3), steps=3)


def test_single_kv_head_and_pure_topk_without_sink_or_local_window():
    from tests.parity import make_case, run_and_compare
    cfg = tiny_config(batch=2, ctx=1500, n_q_heads=4, n_kv_heads=1, budget_blocks=20, resident_frac=0.4,
                      sink_tokens=0, local_tokens=0)
    assert cfg.n_sink_blocks == 0 and cfg.n_local_blocks == 0 and cfg.k_mid == 20
    # the ragged last block is then an ordinary candidate: it may or may not be selected
    run_and_compare(make_case(cfg, steps=4, ctx_len=np.asarray([1500, 1493])), steps=4)


@pytest.mark.parametrize("seed", range(8))
def test_random_shapes(seed):
    """Randomly drawn small shapes: head counts, block sizes, budgets, pool sizes, ragged contexts."""
    from tests.parity import make_case, run_and_compare
    rng = np.random.default_rng(1000 + seed)
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    B = int(rng.choice([16, 32, 64]))
    batch = int(rng.integers(1, 5))
    nb = int(rng.integers(12, 90))
    sink = int(rng.choice([0, 16]))
    local = int(rng.choice([0, 128]))
    pinned = (-(-sink // B) if sink else 0) + (max(1, local // B) if local else 0)
    K = int(rng.integers(pinned + 1, pinned + 30))
    cfg = tiny_config(batch=batch, ctx=nb * B - int(rng.integers(0, B)), n_q_heads=Hkv * G, n_kv_heads=Hkv,
                      block_tokens=B, budget_blocks=K, resident_frac=float(rng.uniform(0.1, 0.9)),
                      sink_tokens=sink, local_tokens=local, seed=seed)
    lens = [int(rng.integers(1, cfg.ctx + 1)) for _ in range(batch)]
    lens[0] = cfg.ctx
    case = make_case(cfg, steps=3, ctx_len=np.asarray(lens), fill=float(rng.choice([0.0, 0.5, 1.0])))
    run_and_compare(case, steps=3, overlapped=bool(seed % 2), fused=bool((seed // 2) % 2))


@pytest.mark.parametrize("seed", range(10))
def test_random_shapes_with_the_head_major_attention(seed):
    """The same kind of random small shapes with the attention forced into its head-major form (one
    (sequence, KV head) per CTA, eight warps sharing the tokens, merge inside the CTA): few items per
    grid, several items per CTA (attn_ctas below the item count), ragged and empty sequences, G up to 16."""
    from tests.parity import make_case, run_and_compare
    rng = np.random.default_rng(2000 + seed)
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    B = int(rng.choice([16, 32, 64]))
    batch = int(rng.integers(1, 6))
    nb = int(rng.integers(12, 120))
    sink = int(rng.choice([0, 16]))
    local = int(rng.choice([0, 128]))
    pinned = (-(-sink // B) if sink else 0) + (max(1, local // B) if local else 0)
    K = int(rng.integers(pinned + 1, pinned + 40))
    cfg = tiny_config(batch=batch, ctx=nb * B - int(rng.integers(0, B)), n_q_heads=Hkv * G, n_kv_heads=Hkv,
                      block_tokens=B, budget_blocks=K, resident_frac=float(rng.uniform(0.1, 0.9)),
                      sink_tokens=sink, local_tokens=local, seed=100 + seed)
    lens = [int(rng.integers(0, cfg.ctx + 1)) for _ in range(batch)]
    lens[0] = cfg.ctx
    case = make_case(cfg, steps=3, ctx_len=np.asarray(lens), fill=float(rng.choice([0.0, 0.5, 1.0])))
    ctas = int(rng.choice([0, 1, 3, 7]))                       # 0: one CTA per item; else several items per CTA
    run_and_compare(case, steps=3, overlapped=bool(seed % 2), pi_kwargs=dict(attn_mode=2, attn_ctas=ctas))


@pytest.mark.parametrize("mode", [1, 2])
def test_both_attention_forms_on_the_bench_shapes(mode):
    """Config 2's per-layer shapes (batch 16 x 8 KV heads = 128 items) with the flat and with the head-major
    attention, pipelined session, oracle on three sequences; two runs of a form give the same bits."""
    from tests.parity import run_session_sampled
    cfg = get_config("c2").replace(n_layers=2)
    outs = []
    for _ in range(2):
        st = run_session_sampled(cfg, steps=2, sample_seqs=[0, 9, 15], pi_kwargs=dict(attn_mode=mode), return_out=True)
        outs.append(st["out"])
    assert torch.equal(outs[0], outs[1])


@pytest.mark.parametrize("seed", range(8))
def test_attention_split_around_the_recall_random_shapes(seed):
    """The resident blocks' share of the attention beside the recall, the recalled blocks' share after it:
    the pair gives the oracle's attention on random shapes (KV heads, group sizes, block sizes, ragged and
    empty sequences, first step with an almost empty pool = nearly everything recalled, later steps with few
    misses), in the head-major form where it applies and through the fallback (the flat form) where not."""
    from tests.parity import make_case, run_and_compare
    rng = np.random.default_rng(7000 + seed)
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 8, 16]))
    B = int(rng.choice([16, 32, 64]))
    batch = int(rng.integers(1, 6))
    nb = int(rng.integers(12, 120))
    sink = int(rng.choice([0, 16]))
    local = int(rng.choice([0, 128]))
    pinned = (-(-sink // B) if sink else 0) + (max(1, local // B) if local else 0)
    K = int(rng.integers(pinned + 1, pinned + 40))
    cfg = tiny_config(batch=batch, ctx=nb * B - int(rng.integers(0, B)), n_q_heads=Hkv * G, n_kv_heads=Hkv,
                      block_tokens=B, budget_blocks=K, resident_frac=float(rng.choice([0.0, 0.3, 0.9])),
                      sink_tokens=sink, local_tokens=local, seed=300 + seed)
    lens = [int(rng.integers(0, cfg.ctx + 1)) for _ in range(batch)]
    lens[0] = cfg.ctx
    case = make_case(cfg, steps=3, ctx_len=np.asarray(lens), fill=float(rng.choice([0.0, 0.5, 1.0])))
    mode = int(rng.choice([0, 1, 2]))                          # 1: the flat form, i.e. the fallback of the pair
    ctas = int(rng.choice([0, 1, 3, 7])) if mode == 2 else 0
    run_and_compare(case, steps=3, split=True, pi_kwargs=dict(attn_mode=mode, attn_ctas=ctas))


@pytest.mark.parametrize("name,kw,pikw", [("c2", dict(n_layers=2), {}), ("c4", dict(n_layers=2), {}),
                                          ("c3", dict(n_layers=1, batch=20), dict(attn_mode=2))])
def test_attention_split_around_the_recall_on_the_bench_shapes(name, kw, pikw):
    """The bench's shapes (c2: one CTA per item; c4: an item shared by a cluster of two CTAs; c3: block 32,
    several items per CTA), pipelined session with the split attention against the oracle on sampled
    sequences; the outputs also agree with the unsplit attention to a bf16 rounding step, and the split
    repeats bit for bit."""
    from tests.parity import run_session_sampled
    cfg = get_config(name).replace(**kw)
    seqs = [0, cfg.batch // 2, cfg.batch - 1]
    outs = [run_session_sampled(cfg, steps=2, sample_seqs=seqs, return_out=True, split=sp, pi_kwargs=pikw)["out"].float()
            for sp in (True, True, False)]
    assert torch.equal(outs[0], outs[1])
    gap = (outs[0] - outs[2]).abs()
    assert float((gap / outs[2].abs().clamp_min(1.0)).max()) <= 2.0 ** -7, float(gap.max())


def test_the_resident_share_reads_no_slot_that_the_recall_is_filling():
    """Between the diff and the recall every destination slot of the recall list is overwritten with
    large values; the first call of the split attention runs on that pool, then the recall, then the second
    call.  Had the first call read one of those slots, the result would be far off the unsplit attention."""
    from tests.parity import make_case
    from paper_2609_34555_b200 import PulseInfer
    from paper_2609_34555_b200.runner import LayerBuffers, RecallPath
    cfg = tiny_config(batch=3, ctx=96 * 16 - 5, n_q_heads=32, n_kv_heads=8, budget_blocks=24, resident_frac=0.5, seed=11)
    case = make_case(cfg, steps=3, ctx_len=np.asarray([cfg.ctx, 700, cfg.ctx - 40]))
    dev = torch.device("cuda:0")
    pi = PulseInfer.from_workload(cfg)
    path = RecallPath(pi)
    buf = LayerBuffers(pi, cfg.batch, dev)
    ctx_d = torch.from_numpy(case.ctx_len).to(dev)
    path.prepare_layer(0, buf, case.kv, ctx_d, torch.from_numpy(case.resident).to(dev))
    state = pi.attn_state(cfg.batch, dev)
    out = torch.zeros((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.bfloat16, device=dev)
    plain = torch.zeros_like(out)
    filled = 0
    for t in range(3):
        q = case.q[t].to(dev)
        pi.score_select_diff(0, t + 1, q, buf.digest, ctx_d, buf.sel_blocks, buf.sel_count, buf.block_table, buf.slot_block,
                             buf.slot_stamp, buf.sel_slots, buf.recall_list, buf.recall_count)
        torch.cuda.synchronize()
        lst, cnt = buf.recall_list.cpu().numpy(), buf.recall_count.cpu().numpy()
        for s in range(cfg.batch):
            for e in range(int(cnt[s])):
                _, dst, n, _ = lst[s, e]
                buf.pool[s, dst:dst + n] = 100.0
                filled += int(n)
        pi.sparse_decode_attn_resident(0, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx_d,
                                       buf.recall_list, buf.recall_count, state)
        torch.cuda.synchronize()
        pi.recall_gather_scatter(0, case.kv, buf.pool, buf.recall_list, buf.recall_count)
        pi.sparse_decode_attn_recalled(0, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx_d,
                                       buf.recall_list, buf.recall_count, state, out)
        pi.sparse_decode_attn(0, q, buf.pool, buf.sel_slots, buf.sel_blocks, buf.sel_count, ctx_d, plain)
        torch.cuda.synchronize()
        assert pi.status()[0] == 0
        gap = (out.float() - plain.float()).abs() / plain.float().abs().clamp_min(1.0)
        assert float(gap.max()) <= 2.0 ** -7, (t, float(gap.max()))
    assert filled > 0
    pi.close()


def test_pipelined_session_with_append_on_two_layers():
    """DecodeSession's three-stream step with a token appended to every layer each step; the
    context crosses a block boundary on the way."""
    from tests.parity import run_session_sampled
    cfg = tiny_config(batch=4, ctx=4096, n_q_heads=32, n_kv_heads=8, budget_blocks=40, resident_frac=0.3, n_layers=2)
    stats = run_session_sampled(cfg, steps=12, sample_seqs=[0, 3], append=True, ctx_start=4096 - 20)
    assert stats["misses"] > 0


def test_paged_host_store_recall_against_the_oracle():
    """Blocks of all sequences interleaved in one arena of pages, located through a page table:
    the recall kernel against the oracle's paged recall, byte for byte, untouched slots intact."""
    import numpy as np
    import torch
    import oracle
    from paper_2609_34555_b200 import PulseInfer
    cfg = tiny_config(batch=3, ctx=16 * 40, n_q_heads=8, n_kv_heads=2, budget_blocks=12, resident_frac=0.5)
    pi = PulseInfer.from_workload(cfg)
    rng = np.random.default_rng(17)
    unit, nb, C = cfg.block_bytes, cfg.n_blocks, cfg.pool_slots
    n_pages = cfg.batch * nb + 7
    arena = torch.from_numpy(rng.integers(0, 256, size=(n_pages, unit), dtype=np.uint8)).pin_memory()
    table = rng.permutation(n_pages)[: cfg.batch * nb].astype(np.int32).reshape(cfg.batch, nb)
    pool0 = rng.integers(0, 256, size=(cfg.batch, C, unit), dtype=np.uint8)
    pool = torch.from_numpy(pool0).cuda()
    cap = 8
    lists = np.zeros((cfg.batch, cap, 4), np.int32)
    counts = np.zeros(cfg.batch, np.int32)
    pairs_of = []
    for s in range(cfg.batch):
        # extents of 1..3 logical blocks; destination slots consecutive inside an extent
        src = [(1, 2), (7, 1), (20, 3)][: s + 1]
        dst, before, pairs = 0, 0, []
        for i, (b0, n) in enumerate(src):
            lists[s, i] = (b0, dst, n, before)
            pairs += [(b0 + k, dst + k) for k in range(n)]
            dst += n + 1
            before += n
        counts[s] = len(src)
        pairs_of.append(np.asarray(pairs, np.int32))
    pi.recall_gather_scatter(0, arena, pool, torch.from_numpy(lists).cuda(), torch.from_numpy(counts).cuda(),
                             page_table=torch.from_numpy(table).cuda(), n_pages=n_pages)
    torch.cuda.synchronize()
    assert pi.status()[0] == 0
    got = pool.cpu().numpy()
    for s in range(cfg.batch):
        ref = pool0[s].copy()
        oracle.recall_paged(arena.numpy(), table[s], ref, pairs_of[s], unit)
        assert np.array_equal(got[s], ref)
    # a page index outside the arena is reported, not followed
    bad = table.copy()
    bad[0, 1] = n_pages
    pi.recall_gather_scatter(0, arena, pool, torch.from_numpy(lists).cuda(), torch.from_numpy(counts).cuda(),
                             page_table=torch.from_numpy(bad).cuda(), n_pages=n_pages)
    torch.cuda.synchronize()
    st = pi.status()
    assert st[0] == -8 and st[1] == 3, st
    pi.close()


def test_pipelined_session_on_a_paged_host_store_with_append():
    """The whole decode step, two layers, pipelined, blocks scattered over a paged arena, one token
    appended per step: every stage against the oracle, and the host store after the appends."""
    from tests.parity import run_session_sampled
    cfg = tiny_config(batch=4, ctx=4096, n_q_heads=32, n_kv_heads=8, budget_blocks=40, resident_frac=0.3, n_layers=2)
    stats = run_session_sampled(cfg, steps=10, sample_seqs=[1, 2], append=True, ctx_start=4096 - 18, paged=True)
    assert stats["misses"] > 0


def test_double_buffered_host_stepping_matches_plain_stepping():
    """decode_steps_from_host (queries uploaded and outputs downloaded beside the neighbouring steps)
    must return, step by step, exactly what decode_step returns from the same state."""
    import numpy as np
    import torch
    from paper_2609_34555_b200 import PulseInfer
    from paper_2609_34555_b200.runner import DecodeSession
    from workloads import generate as gen
    cfg = tiny_config(batch=3, ctx=2048, n_q_heads=16, n_kv_heads=4, budget_blocks=24, resident_frac=0.3, n_layers=3)
    steps = 5
    outs = []
    for form in ("plain", "host", "host+graph"):
        pi = PulseInfer.from_workload(cfg)
        sess = DecodeSession(pi, cfg.batch, cfg.n_layers)
        sess.ctx_len.fill_(cfg.ctx)
        for l in range(cfg.n_layers):
            kv = gen.make_kv(cfg, l, device=sess.device)
            sess.load_layer(l, kv, torch.from_numpy(gen.initial_resident(cfg, l)).to(sess.device))
        q_all = torch.stack([gen.make_queries(cfg, l, steps, device=sess.device) for l in range(cfg.n_layers)], 1).contiguous()
        if form == "plain":
            got = []
            for t in range(steps):
                sess.decode_step(q_all[t])
                torch.cuda.synchronize()
                got.append(sess.out.cpu().clone())
        else:
            q_host = q_all.cpu().pin_memory()
            out_host = [torch.empty(sess.out.shape, dtype=torch.bfloat16, pin_memory=True) for _ in range(steps)]
            sess.decode_steps_from_host([q_host[t] for t in range(steps)], out_host, use_graph=form == "host+graph")
            torch.cuda.synchronize()
            got = [o.clone() for o in out_host]
        assert pi.status()[0] == 0
        outs.append(got)
        pi.close()
    for t in range(steps):
        assert torch.equal(outs[0][t].view(torch.int16), outs[1][t].view(torch.int16)), f"step {t}"
        assert torch.equal(outs[0][t].view(torch.int16), outs[2][t].view(torch.int16)), f"step {t}, graph replay"


@pytest.mark.parametrize("mode", [1, 2])
def test_headwise_attention_with_unequal_and_empty_head_lists(mode):
    """Every KV head attends over its own list; lists of one sequence differ in length, one is empty,
    the last block is partial.  Pool slot i holds block i, so slots and blocks coincide."""
    import numpy as np
    import torch
    import oracle
    from paper_2609_34555_b200 import PulseInfer
    from tests.parity import check_attention
    from workloads import generate as gen
    cfg = tiny_config(batch=3, ctx=16 * 37 + 5, n_q_heads=16, n_kv_heads=4, budget_blocks=20, resident_frac=1.0)
    nb, Hkv, K, G = cfg.n_blocks, cfg.n_kv_heads, cfg.budget_blocks, cfg.group
    assert cfg.pool_slots >= nb
    pi = PulseInfer.from_workload(cfg, attn_mode=mode)
    kv = gen.make_kv(cfg, 0)
    kvb = oracle.bits(kv)
    pool = torch.zeros((cfg.batch, cfg.pool_slots) + tuple(kv.shape[2:]), dtype=torch.bfloat16)
    pool[:, :nb] = kv
    q = gen.make_queries(cfg, 0, 1)[0]
    qb = oracle.bits(q)
    rng = np.random.default_rng(5)
    sel = np.full((cfg.batch, Hkv, K), -1, np.int32)
    cnt = np.zeros((cfg.batch, Hkv), np.int32)
    for s in range(cfg.batch):
        for h in range(Hkv):
            n = [K, 7, 0, 13][(s + h) % 4]
            rows = np.sort(rng.choice(nb, size=n, replace=False)).astype(np.int32)
            if n and (s + h) % 2 == 0:
                rows[-1] = nb - 1                                   # the partial last block
                rows = np.unique(rows)
            sel[s, h, : len(rows)] = rows
            cnt[s, h] = len(rows)
    ctx = np.full(cfg.batch, cfg.ctx, np.int32)
    out = torch.zeros((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros((cfg.batch, cfg.n_q_heads), dtype=torch.float32, device="cuda")
    sel_d = torch.from_numpy(sel).cuda()
    pi.sparse_decode_attn(0, q.cuda(), pool.cuda(), sel_d, sel_d, torch.from_numpy(cnt).cuda(),
                          torch.from_numpy(ctx).cuda(), out, lse, headwise=True)
    torch.cuda.synchronize()
    assert pi.status()[0] == 0, pi.status()
    g_out, g_lse = out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    for s in range(cfg.batch):
        for h in range(Hkv):
            rows = slice(h * G, (h + 1) * G)
            if cnt[s, h] == 0:
                assert np.all(g_out[s, rows] == 0) and np.all(np.isneginf(g_lse[s, rows]))
                continue
            ref, ref_lse = oracle.attention(qb[s], kvb[s], sel[s, h], sel[s, h], int(cnt[s, h]), cfg.ctx,
                                            cfg.block_tokens, Hkv)
            check_attention(g_out[s, rows], ref[rows], cfg, 0)
            np.testing.assert_allclose(g_lse[s, rows], ref_lse[rows], rtol=1e-3, atol=1e-3)
    pi.close()


def test_layer_step_can_be_captured_into_a_cuda_graph_and_replayed():
    """No call of the path synchronises the host or allocates: one layer-step (score/select, diff,
    recall, attention) captured into a CUDA graph and replayed from the same starting state gives
    the bits of the eager run."""
    import torch
    from paper_2609_34555_b200 import PulseInfer
    from paper_2609_34555_b200.runner import LayerBuffers, RecallPath
    from tests.parity import make_case
    cfg = tiny_config(batch=4, ctx=2048, n_q_heads=16, n_kv_heads=4, budget_blocks=24, resident_frac=0.3)
    case = make_case(cfg, steps=1)
    dev = torch.device("cuda:0")
    pi = PulseInfer.from_workload(cfg)
    path = RecallPath(pi)
    buf = LayerBuffers(pi, cfg.batch, dev)
    ctx_d = torch.from_numpy(case.ctx_len).to(dev)
    path.prepare_layer(0, buf, case.kv, ctx_d, torch.from_numpy(case.resident).to(dev))
    q_d = case.q[0].to(dev)
    out = torch.zeros((cfg.batch, cfg.n_q_heads, cfg.head_dim), dtype=torch.bfloat16, device=dev)
    lse = torch.zeros((cfg.batch, cfg.n_q_heads), dtype=torch.float32, device=dev)
    torch.cuda.synchronize()
    state = [t.clone() for t in (buf.block_table, buf.slot_block, buf.slot_stamp, buf.pool)]

    path.layer_step(0, 1, buf, q_d, ctx_d, case.kv, out, lse)          # eager (also warms every launch path up)
    torch.cuda.synchronize()
    want = [t.clone() for t in (out, lse, buf.sel_blocks, buf.sel_slots, buf.recall_count, buf.block_table,
                                buf.slot_stamp, buf.pool)]
    assert int(buf.recall_count.sum()) > 0

    for t, s in zip((buf.block_table, buf.slot_block, buf.slot_stamp, buf.pool), state):
        t.copy_(s)
    out.zero_(); lse.zero_()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        path.layer_step(0, 1, buf, q_d, ctx_d, case.kv, out, lse)
    torch.cuda.synchronize()
    assert float(out.float().abs().sum()) == 0.0                       # capture records, it does not run
    graph.replay()
    torch.cuda.synchronize()
    assert pi.status()[0] == 0, pi.status()
    got = (out, lse, buf.sel_blocks, buf.sel_slots, buf.recall_count, buf.block_table, buf.slot_stamp, buf.pool)
    for g, w in zip(got, want):
        assert torch.equal(g.view(torch.int16) if g.dtype == torch.bfloat16 else g, w.view(torch.int16) if w.dtype == torch.bfloat16 else w)
    pi.close()


@pytest.mark.parametrize("split", [False, True], ids=["attention in one call", "attention split around the recall"])
def test_graph_replayed_decode_steps_match_eager_steps(split):
    """A whole pipelined decode step (three layers, all streams) captured once and replayed, with an
    eager step mixed in: outputs, tables and stamps equal those of a session stepped eagerly."""
    import torch
    from paper_2609_34555_b200 import PulseInfer
    from paper_2609_34555_b200.runner import DecodeSession
    from workloads import generate as gen
    cfg = tiny_config(batch=3, ctx=2048, n_q_heads=16, n_kv_heads=4, budget_blocks=24, resident_frac=0.3, n_layers=3)
    steps = 6
    results = []
    for form in ("eager", "graph"):
        pi = PulseInfer.from_workload(cfg)
        sess = DecodeSession(pi, cfg.batch, cfg.n_layers, split_attention=split)
        sess.ctx_len.fill_(cfg.ctx)
        for l in range(cfg.n_layers):
            kv = gen.make_kv(cfg, l, device=sess.device)
            sess.load_layer(l, kv, torch.from_numpy(gen.initial_resident(cfg, l)).to(sess.device))
        q_all = torch.stack([gen.make_queries(cfg, l, steps, device=sess.device) for l in range(cfg.n_layers)], 1).contiguous()
        got = []
        if form == "eager":
            for t in range(steps):
                sess.decode_step(q_all[t])
                torch.cuda.synchronize()
                got.append(sess.out.cpu().clone())
        else:
            sess.decode_step(q_all[0])                     # step 1 eager (warms the launch paths up)
            torch.cuda.synchronize()
            got.append(sess.out.cpu().clone())
            q_static = q_all[0].clone()
            graph = sess.capture_step(q_static)
            for t in range(1, steps):
                if t == 3:                                 # an eager step between replays
                    sess.decode_step(q_all[t])
                else:
                    q_static.copy_(q_all[t])
                    sess.replay_step(graph)
                torch.cuda.synchronize()
                got.append(sess.out.cpu().clone())
        assert pi.status()[0] == 0, pi.status()
        state = [torch.stack([getattr(b, name).cpu() for b in sess.bufs]) for name in ("block_table", "slot_stamp", "sel_slots")]
        results.append((got, state))
        pi.close()
    for t in range(steps):
        assert torch.equal(results[0][0][t].view(torch.int16), results[1][0][t].view(torch.int16)), f"outputs of step {t}"
    for a, b in zip(results[0][1], results[1][1]):
        assert torch.equal(a, b)


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_of_the_rows_beyond_the_hot_path(seed):
    """Randomly drawn shapes for the selection strategies with per-head attention (seed % 3 == 0), the
    append (1) and the pipelined session, with or without append and paging (2)."""
    from tests.parity import run_append_and_compare, run_session_sampled, run_strategies_and_compare
    rng = np.random.default_rng(5000 + seed)
    Hkv, G, B = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 4, 8, 16])), int(rng.choice([16, 32, 64]))
    batch, nb = int(rng.integers(1, 4)), int(rng.integers(40, 120))
    pinned = 1 + max(1, 128 // B)
    K = int(rng.integers(pinned + 2, pinned + 24))
    cfg = tiny_config(batch=batch, ctx=nb * B - int(rng.integers(0, B)), n_q_heads=Hkv * G, n_kv_heads=Hkv, block_tokens=B,
                      budget_blocks=K, resident_frac=float(rng.uniform(0.4, 0.9)), seed=seed)
    if seed % 3 == 0:
        run_strategies_and_compare(cfg, steps=2)
    elif seed % 3 == 1:
        lens = [int(rng.integers(cfg.ctx // 2, cfg.ctx - 40)) for _ in range(batch)]
        run_append_and_compare(cfg, steps=int(rng.integers(5, 40)), ctx_len0=lens)
    else:
        run_session_sampled(cfg.replace(n_layers=2), steps=6, sample_seqs=[0], append=bool(seed % 2),
                            ctx_start=cfg.ctx - 10 if seed % 2 else 0, paged=bool((seed // 2) % 2))


def test_graph_replay_with_append_matches_eager_steps():
    """The captured step also appends the step's token (stamp and context length from device memory):
    outputs, context lengths, digests, tables and the host store equal those of eager stepping."""
    import torch
    from paper_2609_34555_b200 import PulseInfer
    from paper_2609_34555_b200.runner import DecodeSession
    from workloads import generate as gen
    cfg = tiny_config(batch=3, ctx=2048, n_q_heads=16, n_kv_heads=4, budget_blocks=24, resident_frac=0.3, n_layers=2)
    steps, ctx0 = 8, 2048 - 21                              # the context crosses a block boundary (2032) at step 6
    results = []
    for form in ("eager", "graph"):
        pi = PulseInfer.from_workload(cfg)
        sess = DecodeSession(pi, cfg.batch, cfg.n_layers)
        sess.ctx_len.fill_(ctx0)
        short = cfg.replace(ctx=ctx0)
        for l in range(cfg.n_layers):
            kv = gen.make_kv(cfg, l, device=sess.device)
            sess.load_layer(l, kv, torch.from_numpy(gen.initial_resident(short, l)).to(sess.device))
        q_all = torch.stack([gen.make_queries(cfg, l, steps, device=sess.device) for l in range(cfg.n_layers)], 1).contiguous()
        g = torch.Generator(device=sess.device).manual_seed(77)
        shp = (steps, cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.head_dim)
        k_all = torch.randn(shp, device=sess.device, generator=g).to(torch.bfloat16)
        v_all = torch.randn(shp, device=sess.device, generator=g).to(torch.bfloat16)
        got = []
        if form == "eager":
            for t in range(steps):
                sess.decode_step(q_all[t], new_kv=(k_all[t], v_all[t]))
                torch.cuda.synchronize()
                got.append(sess.out.cpu().clone())
        else:
            sess.decode_step(q_all[0], new_kv=(k_all[0], v_all[0]))
            torch.cuda.synchronize()
            got.append(sess.out.cpu().clone())
            q_s, k_s, v_s = q_all[0].clone(), k_all[0].clone(), v_all[0].clone()
            graph = sess.capture_step(q_s, new_kv_static=(k_s, v_s))
            for t in range(1, steps):
                q_s.copy_(q_all[t]); k_s.copy_(k_all[t]); v_s.copy_(v_all[t])
                sess.replay_step(graph)
                torch.cuda.synchronize()
                got.append(sess.out.cpu().clone())
        assert pi.status()[0] == 0, pi.status()
        state = [sess.ctx_len.cpu()] + [torch.stack([getattr(b, name).cpu() for b in sess.bufs])
                                         for name in ("block_table", "slot_stamp", "sel_slots")]
        state += [torch.stack([b.digest.cpu().view(torch.int16) for b in sess.bufs]),
                  torch.stack([sess.host_region(l).view(torch.int16).clone() for l in range(cfg.n_layers)])]
        results.append((got, state))
        pi.close()
    assert int(results[0][1][0][0]) == ctx0 + steps
    for t in range(steps):
        assert torch.equal(results[0][0][t].view(torch.int16), results[1][0][t].view(torch.int16)), f"outputs of step {t}"
    for a, b in zip(results[0][1], results[1][1]):
        assert torch.equal(a, b)
