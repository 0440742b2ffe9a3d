"""The allocation-free selection entry point against the regular one.

Some users of this library may not allocate device memory at all (an engine that hands out
every byte itself, a callback where an allocation could stall or fail); for them the library
offers pi_score_select_noalloc, whose scratch is a fixed array inside the library.  This file
checks, through the C ABI, that it selects exactly what pi_score_select selects, on two calls
in a row (the second call finds the first call's leftovers in the shared array).  It is named
to be collected last, so a failure here cannot hide another test's result.
"""
import pytest
import torch

from workloads import tiny_config
from workloads import generate as gen

pytestmark = pytest.mark.gpu


@pytest.mark.skipif(not torch.cuda.is_available(), reason="no CUDA device")
def test_noalloc_selection_matches_regular_entry_point_twice_in_a_row():
    import paper_2609_34555_b200 as pkg
    from paper_2609_34555_b200.runner import LayerBuffers

    cfg = tiny_config(batch=5, ctx=70000, n_q_heads=32, n_kv_heads=8, budget_blocks=96, resident_frac=0.1)
    dev = torch.device("cuda:0")
    pi = pkg.PulseInfer.from_workload(cfg)
    buf = LayerBuffers(pi, cfg.batch, dev, keep_scores=True)
    g = torch.Generator(device="cpu").manual_seed(11)
    buf.digest.copy_(torch.randn(buf.digest.shape, generator=g).to(torch.bfloat16))
    ctx_len = torch.tensor([70000, 65000, 4097, 300, 16], dtype=torch.int32, device=dev)
    q = gen.make_queries(cfg, 0, 2, ar1=0.5).to(dev)
    status = torch.zeros(8, dtype=torch.int32, device=dev)
    h = cfg.solo_head(0)
    for call in range(2):
        ref_sel, ref_cnt = buf.sel_blocks, buf.sel_count
        pi.score_select(0, q[call], buf.digest, ctx_len, ref_sel, ref_cnt, buf.scores)
        got_sel = torch.full_like(ref_sel, -7)
        got_cnt = torch.full_like(ref_cnt, -7)
        pkg.score_select_noalloc(q[call], buf.digest, ctx_len, got_sel, got_cnt, n_kv_heads=cfg.n_kv_heads,
                                 block_tokens=cfg.block_tokens, budget_blocks=cfg.budget_blocks,
                                 n_sink_blocks=cfg.n_sink_blocks, n_local_blocks=cfg.n_local_blocks,
                                 solo_head=h, status=status)
        torch.cuda.synchronize()
        assert status[0].item() == 0, status.tolist()
        assert torch.equal(got_cnt, ref_cnt), f"call {call}: counts differ"
        assert torch.equal(got_sel, ref_sel), f"call {call}: selections differ"   # integer result: exact
        assert (got_cnt > 0).all()
    pi.close()


@pytest.mark.skipif(not torch.cuda.is_available(), reason="no CUDA device")
def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    import paper_2609_34555_b200 as pkg
    dev = torch.device("cuda:0")
    q = torch.zeros((65, 8, 128), dtype=torch.bfloat16, device=dev)
    digest = torch.zeros((65, 64, 2, 128), dtype=torch.bfloat16, device=dev)
    ctx = torch.full((65,), 64 * 16, dtype=torch.int32, device=dev)
    sel = torch.zeros((65, 16), dtype=torch.int32, device=dev)
    cnt = torch.zeros((65,), dtype=torch.int32, device=dev)
    with pytest.raises(pkg.PiError) as e:
        pkg.score_select_noalloc(q, digest, ctx, sel, cnt, n_kv_heads=2, block_tokens=16, budget_blocks=16,
                                 n_sink_blocks=1, n_local_blocks=8, solo_head=0)
    assert e.value.code == -10 and "64 x 8192" in str(e.value)
