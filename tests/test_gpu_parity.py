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
