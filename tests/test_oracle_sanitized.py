"""The oracle's C code under AddressSanitizer + UndefinedBehaviorSanitizer: the hand-worked example
and whole layer-steps of a ragged batch run in a child process that loads the instrumented build;
any out-of-bounds access, use of an uninitialised size, signed overflow or misaligned access ends
the child with a non-zero exit code."""
import os
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

CHILD = r"""
import json, sys
import numpy as np, torch
sys.path.insert(0, sys.argv[1])
import oracle
from workloads import generate as gen, tiny_config

def bf16(a):
    return oracle.bits(torch.tensor(a, dtype=torch.float32).to(torch.bfloat16))

g = json.load(open(sys.argv[2]))
B, D, nb = g["B"], g["D"], g["n_blocks"]
kv = np.zeros((nb, 1, 2, B, D), np.uint16)
kv[:, 0, 0] = bf16(g["keys"])
dg = oracle.build_digest(kv, nb * B, 0)
sc = oracle.score(bf16(g["q"]), dg, nb, 1, 0)
assert sc.tolist() == g["scores"]
sel, cnt = oracle.select(sc, 0, 0, g["K"])
assert sel.tolist() == g["sel"]
d = g["diff"]
table, sb = np.asarray(d["table_before"], np.int32), np.asarray(d["slot_block_before"], np.int32)
stamp = np.asarray(d["slot_stamp_before"], np.uint32)
rc, slots, pairs = oracle.diff(sel, cnt, nb, 0, 0, d["step"], table, sb, stamp)
assert rc == 0 and slots.tolist() == d["sel_slots"] and table.tolist() == d["table_after"]

# whole layer-steps of a ragged batch (last block partial, one short sequence)
cfg = tiny_config(batch=3, ctx=1000, n_q_heads=8, n_kv_heads=2, budget_blocks=24, resident_frac=0.5)
kvb = oracle.bits(gen.make_kv(cfg, 0))
ctx = np.asarray([1000, 517, 160], np.int32)
h = cfg.solo_head(0)
dgs = np.zeros((cfg.batch, cfg.n_blocks, 2, cfg.head_dim), np.uint16)
table = np.full((cfg.batch, cfg.n_blocks), -1, np.int32)
sb = np.full((cfg.batch, cfg.pool_slots), -1, np.int32)
stamp = np.zeros((cfg.batch, cfg.pool_slots), np.uint32)
pool = np.zeros((cfg.batch, cfg.pool_slots) + kvb.shape[2:], np.uint16)
for s in range(cfg.batch):
    n_s = -(-int(ctx[s]) // cfg.block_tokens)
    dgs[s, :n_s] = oracle.build_digest(kvb[s], int(ctx[s]), h)[:n_s]
    pin = gen.pinned_blocks(cfg, n_s)
    sb[s, :len(pin)] = pin
    table[s, pin] = np.arange(len(pin))
    pool[s, :len(pin)] = kvb[s, pin]
q = oracle.bits(gen.make_queries(cfg, 0, 3))
for t in range(3):
    r = oracle.layer_step(ctx, cfg.n_blocks, cfg.block_tokens, cfg.n_kv_heads, h, cfg.budget_blocks,
                          cfg.n_sink_blocks, cfg.n_local_blocks, t + 1, q[t], dgs, kvb, table, sb, stamp, pool)
    assert r["rc"] == 0 and np.isfinite(r["out"]).all()
# the append step as well: a token that opens a new block
k_new = oracle.bits(torch.randn((cfg.n_kv_heads, cfg.head_dim), generator=torch.Generator().manual_seed(1)).to(torch.bfloat16))
host0 = kvb[1].copy()
rc = oracle.append(k_new, k_new, 528, cfg.block_tokens, h, cfg.n_sink_blocks, cfg.n_local_blocks, 9, host0, pool[1],
                   table[1], sb[1], stamp[1], dgs[1])
assert rc == 0
print("sanitized oracle ok")
"""


def test_oracle_runs_clean_under_address_and_undefined_behaviour_sanitizers(tmp_path):
    import oracle
    lib = oracle.build_sanitized()
    asan = subprocess.check_output(["gcc", "-print-file-name=libasan.so"], text=True).strip()
    ubsan = subprocess.check_output(["gcc", "-print-file-name=libubsan.so"], text=True).strip()
    script = tmp_path / "child.py"
    script.write_text(CHILD)
    env = dict(os.environ, PI_ORACLE_LIB=str(lib), LD_PRELOAD=f"{asan} {ubsan}",
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=0:exitcode=23", UBSAN_OPTIONS="halt_on_error=1:exitcode=24",
               OMP_NUM_THREADS="2")
    r = subprocess.run([sys.executable, str(script), str(ROOT), str(ROOT / "tests" / "golden" / "hand_example.json")],
                       env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, f"exit {r.returncode}\n{r.stdout[-2000:]}\n{r.stderr[-4000:]}"
    assert "sanitized oracle ok" in r.stdout
    assert "ERROR: AddressSanitizer" not in r.stderr and "runtime error" not in r.stderr
