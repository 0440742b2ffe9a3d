"""ctypes front end of the CPU oracle (pi_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU
baseline leg of the benchmark.  The CUDA package never imports this module and this
module never imports the CUDA package.

bf16 tensors cross this boundary as uint16 numpy arrays holding the raw bits.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "pi_oracle.c"
_LIB = _HERE / "libpi_oracle.so"

POOL_TOO_SMALL = -4


def build(force: bool = False) -> Path:
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                               "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def build_sanitized() -> Path:
    """The same source with AddressSanitizer and UndefinedBehaviorSanitizer (a test loads it in a
    child process through PI_ORACLE_LIB, with the sanitizer runtime preloaded)."""
    out = _HERE / "libpi_oracle_asan.so"
    if not out.exists() or out.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = out.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["gcc", "-O1", "-g", "-std=c11", "-fopenmp", "-fsanitize=address,undefined",
                               "-fno-sanitize-recover=undefined", "-fno-omit-frame-pointer", "-shared", "-fPIC",
                               "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, out)
    return out


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(os.environ.get("PI_ORACLE_LIB") or str(build()))
        _lib.pio_num_threads.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be contiguous"
    return a.ctypes.data_as(ctypes.c_void_p)


def bits(t) -> np.ndarray:
    """torch bf16 tensor (CPU) -> uint16 numpy array sharing its memory."""
    import torch
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bf16_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def num_threads() -> int:
    return int(lib().pio_num_threads())


def set_num_threads(n: int) -> None:
    """Threads of the loop over sequences in layer_step (timing only)."""
    lib().pio_set_num_threads(int(n))


def build_digest(kv_seq: np.ndarray, ctx: int, h_star: int) -> np.ndarray:
    """kv_seq uint16 [n_blocks][Hkv][2][B][D] -> digest uint16 [n_blocks][2][D]."""
    nb, Hkv, _, B, D = kv_seq.shape
    assert nb >= (ctx + B - 1) // B
    out = np.zeros((nb, 2, D), dtype=np.uint16)
    lib().pio_build_digest(_p(kv_seq), ctx, B, Hkv, D, h_star, _p(out))
    return out


def score(q: np.ndarray, digest: np.ndarray, n_blocks: int, Hkv: int, h_star: int) -> np.ndarray:
    Hq, D = q.shape
    out = np.zeros(n_blocks, dtype=np.float64)
    lib().pio_score(_p(q), _p(digest), n_blocks, Hq, Hkv, D, h_star, _p(out))
    return out


def select(score_: np.ndarray, n_sink: int, n_local: int, K: int):
    score_ = np.ascontiguousarray(score_, dtype=np.float64)
    sel = np.full(K, -1, dtype=np.int32)
    cnt = ctypes.c_int32(0)
    lib().pio_select(_p(score_), len(score_), n_sink, n_local, K, _p(sel), ctypes.byref(cnt))
    return sel, int(cnt.value)


def diff(sel: np.ndarray, sel_count: int, n_blocks: int, n_sink: int, n_local: int, step: int,
         table: np.ndarray, slot_block: np.ndarray, slot_stamp: np.ndarray):
    """Updates table / slot_block / slot_stamp in place.
    Returns (rc, sel_slots[K], miss_pairs[n_miss][2])."""
    K, C = len(sel), len(slot_block)
    assert table.dtype == np.int32 and slot_block.dtype == np.int32 and slot_stamp.dtype == np.uint32
    sel = np.ascontiguousarray(sel, dtype=np.int32)
    sel_slots = np.full(K, -1, dtype=np.int32)
    pairs = np.full((K, 2), -1, dtype=np.int32)
    n = ctypes.c_int32(0)
    rc = lib().pio_diff(_p(sel), sel_count, n_blocks, C, n_sink, n_local, ctypes.c_uint32(step),
                        _p(table), _p(slot_block), _p(slot_stamp), _p(sel_slots), K, _p(pairs),
                        ctypes.byref(n))
    return int(rc), sel_slots, pairs[: n.value].copy()


def recall(host_seq: np.ndarray, pool_seq: np.ndarray, pairs: np.ndarray, unit_bytes: int) -> None:
    pairs = np.ascontiguousarray(pairs, dtype=np.int32)
    lib().pio_recall(_p(host_seq), _p(pool_seq), _p(pairs), len(pairs), ctypes.c_int64(unit_bytes))


def attention(q: np.ndarray, store: np.ndarray, where: np.ndarray, blocks: np.ndarray, count: int,
              ctx: int, B: int, Hkv: int):
    """q uint16 [Hq][D]; store uint16 [...][Hkv][2][B][D] -> (out f64 [Hq][D], lse f64 [Hq])."""
    Hq, D = q.shape
    where = np.ascontiguousarray(where, dtype=np.int32)
    blocks = np.ascontiguousarray(blocks, dtype=np.int32)
    out = np.zeros((Hq, D), dtype=np.float64)
    lse = np.zeros(Hq, dtype=np.float64)
    lib().pio_attention(_p(q), _p(store), _p(where), _p(blocks), count, ctx, B, Hq, Hkv, D,
                        _p(out), _p(lse))
    return out, lse


def layer_step(ctx_len: np.ndarray, max_blocks: int, B: int, Hkv: int, h_star: int, K: int,
               n_sink: int, n_local: int, step: int, q: np.ndarray, digest: np.ndarray,
               host_kv: np.ndarray, table: np.ndarray, slot_block: np.ndarray,
               slot_stamp: np.ndarray, pool: np.ndarray):
    """One layer-step of a whole batch; tables and pool are updated in place.
    q uint16 [batch][Hq][D]; digest uint16 [batch][max_blocks][2][D]; host_kv / pool uint8 or
    uint16 arrays of [batch][max_blocks | C] blocks.  Returns a dict of the stage outputs."""
    batch, Hq, D = q.shape
    C = slot_block.shape[1]
    r = dict(score=np.zeros((batch, max_blocks)), sel=np.full((batch, K), -1, np.int32),
             sel_count=np.zeros(batch, np.int32), sel_slots=np.full((batch, K), -1, np.int32),
             miss_pairs=np.full((batch, K, 2), -1, np.int32), n_miss=np.zeros(batch, np.int32),
             out=np.zeros((batch, Hq, D)), lse=np.zeros((batch, Hq)))
    ctx_len = np.ascontiguousarray(ctx_len, dtype=np.int32)
    r["rc"] = int(lib().pio_layer_step(
        batch, _p(ctx_len), max_blocks, B, Hq, Hkv, D, h_star, K, n_sink, n_local, C,
        ctypes.c_uint32(step), _p(q), _p(digest), _p(host_kv), _p(table), _p(slot_block),
        _p(slot_stamp), _p(pool), _p(r["score"]), _p(r["sel"]), _p(r["sel_count"]),
        _p(r["sel_slots"]), _p(r["miss_pairs"]), _p(r["n_miss"]), _p(r["out"]), _p(r["lse"])))
    return r


def append(k_new: np.ndarray, v_new: np.ndarray, ctx: int, B: int, h_star: int, n_sink: int, n_local: int,
           step: int, host_seq: np.ndarray, pool_seq: np.ndarray, table: np.ndarray, slot_block: np.ndarray,
           slot_stamp: np.ndarray, digest: np.ndarray) -> int:
    """Appends one token (k_new, v_new uint16 [Hkv][D]) at position ctx; host store, pool, tables
    and the digest are updated in place.  Returns the oracle's status code."""
    Hkv, D = k_new.shape
    return int(lib().pio_append(_p(np.ascontiguousarray(k_new)), _p(np.ascontiguousarray(v_new)), ctx, B, Hkv, D,
                                h_star, n_sink, n_local, len(slot_block), ctypes.c_uint32(step), _p(host_seq),
                                _p(pool_seq), _p(table), _p(slot_block), _p(slot_stamp), _p(digest)))


def build_digest_all(kv_seq: np.ndarray, ctx: int) -> np.ndarray:
    """kv_seq uint16 [n_blocks][Hkv][2][B][D] -> digests of every KV head, uint16 [n_blocks][Hkv][2][D]."""
    nb, Hkv, _, B, D = kv_seq.shape
    out = np.zeros((nb, Hkv, 2, D), dtype=np.uint16)
    lib().pio_build_digest_all(_p(kv_seq), ctx, B, Hkv, D, _p(out))
    return out


def score_heads(q: np.ndarray, digest_all: np.ndarray, n_blocks: int, h_lo: int, h_hi: int) -> np.ndarray:
    """Sum of the per-head query-digest scores of KV heads [h_lo, h_hi)."""
    Hq, D = q.shape
    Hkv = digest_all.shape[1]
    out = np.zeros(n_blocks, dtype=np.float64)
    lib().pio_score_heads(_p(q), _p(digest_all), n_blocks, Hq, Hkv, D, h_lo, h_hi, _p(out))
    return out


def recall_strided(host_seq: np.ndarray, pool_seq: np.ndarray, pairs: np.ndarray, unit_bytes: int,
                   unit_stride: int, offset: int) -> None:
    pairs = np.ascontiguousarray(pairs, dtype=np.int32)
    lib().pio_recall_strided(_p(host_seq), _p(pool_seq), _p(pairs), len(pairs), ctypes.c_int64(unit_bytes),
                             ctypes.c_int64(unit_stride), ctypes.c_int64(offset))


def recall_paged(arena: np.ndarray, page_table: np.ndarray, pool_seq: np.ndarray, pairs: np.ndarray, unit_bytes: int) -> None:
    """arena uint8 [n_pages][unit_bytes]; page_table int32 [n_blocks] (logical block -> page)."""
    pairs = np.ascontiguousarray(pairs, dtype=np.int32)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    lib().pio_recall_paged(_p(arena), _p(page_table), _p(pool_seq), _p(pairs), len(pairs), ctypes.c_int64(unit_bytes))
