"""The C-ABI library loads without a GPU and exports every symbol the header declares;
argument checks that need no device return their codes."""
import ctypes
import re
from pathlib import Path

import pytest

import paper_2609_34555_b200 as pkg
from paper_2609_34555_b200.binding import PiConfig

ROOT = Path(__file__).resolve().parent.parent


def declared_functions():
    hdr = (ROOT / "include" / "pulseinfer.h").read_text()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    return sorted(set(re.findall(r"\b(pi_[a-z0-9_]+)\s*\(", hdr)))


def test_library_exports_every_declared_symbol():
    lib = pkg.load_library()
    names = declared_functions()
    assert {"pi_score_select", "pi_diff_misses", "pi_recall_gather_scatter", "pi_sparse_decode_attn"} <= set(names)
    for n in names:
        assert getattr(lib, n) is not None
    assert sorted(pkg.EXPORTS) == names


def test_error_strings():
    assert pkg.strerror(0) == "ok"
    for code in range(-10, 0):
        assert pkg.strerror(code) not in ("ok", "unknown error")


def _cfg(**kw):
    base = dict(n_layers=1, n_q_heads=32, n_kv_heads=8, head_dim=128, block_tokens=16, budget_blocks=64,
                n_sink_blocks=1, n_local_blocks=8, pool_slots=128, max_batch=4, max_blocks=512,
                recall_ctas=0, attn_ctas=0, attn_mode=0, wait_limit_us=0, test_hold_producer=0)
    base.update(kw)
    heads = (ctypes.c_int32 * base["n_layers"])(*([0] * base["n_layers"]))
    return PiConfig(*[base[f] for f, _ in PiConfig._fields_[:-1]], heads), heads


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=64), -3), (dict(block_tokens=8), -3), (dict(n_kv_heads=3, n_q_heads=3), -3),
    (dict(n_q_heads=36), -3), (dict(pool_slots=32), -4), (dict(budget_blocks=4), -1),
    (dict(max_blocks=1 << 20), -3), (dict(max_batch=0), -1), (dict(wait_limit_us=-5), -1), (dict(test_hold_producer=7), -1), (dict(attn_mode=3), -1)])
def test_create_rejects_bad_configs_before_touching_the_device(kw, code):
    lib = pkg.load_library()
    cfg, _keep = _cfg(**kw)
    out = ctypes.c_void_p()
    assert lib.pi_create(ctypes.byref(cfg), ctypes.byref(out)) == code
    assert not out.value


def test_null_arguments_are_rejected():
    lib = pkg.load_library()
    assert lib.pi_create(None, None) == -1
    assert lib.pi_destroy(None) == -1
    assert lib.pi_score_select(None, 0, 1, None, None, None, None, None, None, None) == -1
    assert lib.pi_get_status(None, None) == -1
    assert lib.pi_sparse_decode_attn_resident(None, 0, 1, None, None, None, None, None, None, None, 1, None, None, None) == -1
    assert lib.pi_sparse_decode_attn_recalled(None, 0, 1, None, None, None, None, None, None, None, 1, None, None, None, None) == -1
    assert lib.pi_attn_state_bytes(None, 1) == -1
