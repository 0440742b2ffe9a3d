"""Thin ctypes binding of the C ABI in include/pulseinfer.h.

Argument marshalling only: tensors are checked (dtype, device, contiguity) and handed
over as raw pointers; every step of the path runs in the CUDA library.  There is no
fallback: a missing library or a failing call raises.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, c_char_p, c_float, c_int, c_int32, c_int64, c_uint32, c_void_p
from typing import Optional, Sequence

import torch

from .build import LIB, build

OK = 0
ERR_NAMES = {
    -1: "PI_ERR_INVALID_ARG", -2: "PI_ERR_BAD_ALIGN", -3: "PI_ERR_UNSUPPORTED_DIM",
    -4: "PI_ERR_POOL_TOO_SMALL", -5: "PI_ERR_NOT_PINNED", -6: "PI_ERR_CUDA", -7: "PI_ERR_TIMEOUT",
    -8: "PI_ERR_INDEX_RANGE", -9: "PI_ERR_CAPACITY", -10: "PI_ERR_STATIC_LIMIT",
}
EXTENT_DTYPE = torch.int32      # a pi_extent is four int32: src_unit, dst_unit, n_units, units_before

EXPORTS = ["pi_create", "pi_destroy", "pi_score_select", "pi_score_select_diff", "pi_score_select_diff_devstep", "pi_score_select_noalloc", "pi_score_select_strategy", "pi_diff_misses", "pi_diff_misses_devstep", "pi_recall_gather_scatter",
           "pi_recall_gather_scatter_paged", "pi_sparse_decode_attn", "pi_sparse_decode_attn_headwise", "pi_sparse_decode_attn_resident", "pi_sparse_decode_attn_recalled", "pi_attn_state_bytes", "pi_append_kv", "pi_append_kv_paged", "pi_append_kv_devstep", "pi_build_digests", "pi_build_digests_all", "pi_table_init", "pi_h2d_copy_ms", "pi_empty_launch", "pi_middle_attention_mass",
           "pi_get_status", "pi_get_stats", "pi_clear_status", "pi_strerror"]


class PiConfig(ctypes.Structure):
    _fields_ = [("n_layers", c_int32), ("n_q_heads", c_int32), ("n_kv_heads", c_int32), ("head_dim", c_int32),
                ("block_tokens", c_int32), ("budget_blocks", c_int32), ("n_sink_blocks", c_int32),
                ("n_local_blocks", c_int32), ("pool_slots", c_int32), ("max_batch", c_int32),
                ("max_blocks", c_int32), ("recall_ctas", c_int32), ("attn_ctas", c_int32),
                ("attn_mode", c_int32), ("wait_limit_us", c_int32), ("test_hold_producer", c_int32), ("solo_head", POINTER(c_int32))]


class PiError(RuntimeError):
    def __init__(self, call: str, code: int, text: str):
        super().__init__(f"{call} failed: {ERR_NAMES.get(code, code)} ({text})")
        self.code = code


_lib = None


def load_library(rebuild: bool = False) -> ctypes.CDLL:
    """Loads (building first if the sources are newer) the CUDA library.  Raises if it
    cannot be built or loaded: there is no other implementation to fall back to."""
    global _lib
    if _lib is not None and not rebuild:
        return _lib
    path = build(force=rebuild)
    lib = ctypes.CDLL(str(path))
    vp, i32p, u32p = c_void_p, c_void_p, c_void_p
    lib.pi_create.argtypes = [POINTER(PiConfig), POINTER(c_void_p)]
    lib.pi_destroy.argtypes = [c_void_p]
    lib.pi_score_select.argtypes = [c_void_p, c_int, c_int, vp, vp, i32p, i32p, i32p, vp, vp]
    lib.pi_score_select_noalloc.argtypes = [c_int] * 9 + [vp, vp, i32p, i32p, i32p, i32p, vp]
    lib.pi_score_select_diff.argtypes = [c_void_p, c_int, c_int, c_uint32, vp, vp, i32p, i32p, i32p, vp, i32p, i32p, u32p, i32p, vp, i32p, vp]
    lib.pi_score_select_diff_devstep.argtypes = [c_void_p, c_int, c_int, u32p, vp, vp, i32p, i32p, i32p, vp, i32p, i32p, u32p, i32p, vp, i32p, vp]
    lib.pi_diff_misses.argtypes = [c_void_p, c_int, c_int, c_uint32, i32p, i32p, i32p, i32p, i32p, u32p, i32p, vp, i32p, vp]
    lib.pi_diff_misses_devstep.argtypes = [c_void_p, c_int, c_int, u32p, i32p, i32p, i32p, i32p, i32p, u32p, i32p, vp, i32p, vp]
    lib.pi_recall_gather_scatter.argtypes = [c_void_p, c_int, c_int, c_int, vp, c_int64, vp, c_int64, vp, c_int32, i32p,
                                             c_int64, c_int64, c_int64, vp]
    lib.pi_recall_gather_scatter_paged.argtypes = [c_void_p, c_int, c_int, c_int, vp, i32p, c_int64, c_int32, vp, c_int64, vp,
                                                   c_int32, i32p, c_int64, c_int64, c_int64, vp]
    lib.pi_append_kv_paged.argtypes = [c_void_p, c_int, c_int, c_uint32, vp, vp, i32p, vp, i32p, c_int64, c_int32, vp, i32p,
                                       i32p, u32p, vp, vp]
    lib.pi_append_kv_devstep.argtypes = [c_void_p, c_int, c_int, u32p, vp, vp, i32p, vp, c_int64, i32p, c_int64, c_int32, vp,
                                         i32p, i32p, u32p, vp, vp]
    lib.pi_score_select_strategy.argtypes = [c_void_p, c_int, c_int, c_int, vp, vp, i32p, i32p, i32p, vp, vp]
    lib.pi_build_digests_all.argtypes = [c_void_p, c_int, vp, c_int64, i32p, vp, vp]
    lib.pi_sparse_decode_attn.argtypes = [c_void_p, c_int, c_int, vp, vp, i32p, i32p, i32p, i32p, vp, vp, vp]
    lib.pi_sparse_decode_attn_headwise.argtypes = [c_void_p, c_int, c_int, vp, vp, i32p, i32p, i32p, i32p, vp, vp, vp]
    lib.pi_sparse_decode_attn_resident.argtypes = [c_void_p, c_int, c_int, vp, vp, i32p, i32p, i32p, i32p, vp, c_int32, i32p, vp, vp]
    lib.pi_sparse_decode_attn_recalled.argtypes = [c_void_p, c_int, c_int, vp, vp, i32p, i32p, i32p, i32p, vp, c_int32, i32p, vp, vp, vp]
    lib.pi_attn_state_bytes.argtypes = [c_void_p, c_int]
    lib.pi_append_kv.argtypes = [c_void_p, c_int, c_int, c_uint32, vp, vp, i32p, vp, c_int64, vp, i32p, i32p, u32p, vp, vp]
    lib.pi_build_digests.argtypes = [c_void_p, c_int, c_int, vp, c_int64, i32p, vp, vp]
    lib.pi_table_init.argtypes = [c_void_p, c_int, i32p, i32p, i32p, u32p, vp]
    lib.pi_h2d_copy_ms.argtypes = [vp, vp, c_int64, c_int, POINTER(c_float)]
    lib.pi_empty_launch.argtypes = [c_int, c_int, vp]
    lib.pi_middle_attention_mass.argtypes = [c_void_p, c_int, vp, vp, vp, vp, vp]
    lib.pi_get_status.argtypes = [c_void_p, POINTER(c_int32 * 8)]
    lib.pi_get_stats.argtypes = [c_void_p, POINTER(c_int64 * 4), c_int]
    lib.pi_clear_status.argtypes = [c_void_p]
    lib.pi_strerror.argtypes = [c_int]
    lib.pi_strerror.restype = c_char_p
    for name in EXPORTS:
        if name != "pi_strerror":
            getattr(lib, name).restype = c_int
    lib.pi_attn_state_bytes.restype = c_int64
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().pi_strerror(code).decode()


def _check(call: str, rc: int) -> None:
    if rc != OK:
        raise PiError(call, rc, strerror(rc))


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def h2d_copy_ms(host_pinned: torch.Tensor, dev: torch.Tensor, reps: int = 10) -> float:
    """Best time (ms) of a pinned host -> device copy of the whole tensor."""
    if not host_pinned.is_pinned() or not dev.is_cuda:
        raise TypeError("h2d_copy_ms: need a pinned host tensor and a CUDA tensor")
    nbytes = host_pinned.numel() * host_pinned.element_size()
    assert dev.numel() * dev.element_size() >= nbytes
    ms = c_float(0)
    _check("pi_h2d_copy_ms", load_library().pi_h2d_copy_ms(host_pinned.data_ptr(), dev.data_ptr(), nbytes, reps, ctypes.byref(ms)))
    return float(ms.value)


def empty_launch(n_ctas: int = 128, n_threads: int = 256, stream=None) -> None:
    """A kernel that does nothing: between two events it measures the launch floor of the box."""
    _check("pi_empty_launch", load_library().pi_empty_launch(n_ctas, n_threads, _stream(stream)))


def score_select_noalloc(q, digest, ctx_len, sel_blocks, sel_count, *, n_kv_heads: int, block_tokens: int,
                         budget_blocks: int, n_sink_blocks: int, n_local_blocks: int, solo_head: int,
                         status=None, stream=None) -> None:
    """Selection without a context and without any device allocation, for callers that are not
    allowed to allocate (an engine that owns all device memory, a callback on a hot path).
    Same results as PulseInfer.score_select.  batch <= 64 and max_blocks <= 8192; calls on one
    device share a fixed scratch array inside the library, so do not let two of them overlap."""
    batch, n_q_heads = q.shape[0], q.shape[1]
    max_blocks = digest.shape[1]
    _check("pi_score_select_noalloc", load_library().pi_score_select_noalloc(
        batch, n_q_heads, n_kv_heads, block_tokens, budget_blocks, n_sink_blocks, n_local_blocks, max_blocks,
        solo_head, _dev(q, torch.bfloat16, "q"), _dev(digest, torch.bfloat16, "digest"),
        _dev(ctx_len, torch.int32, "ctx_len"), _dev(sel_blocks, torch.int32, "sel_blocks"),
        _dev(sel_count, torch.int32, "sel_count"),
        None if status is None else _dev(status, torch.int32, "status"), _stream(stream)))


class PulseInfer:
    """One context = one model shape on the current CUDA device."""

    def __init__(self, *, n_layers: int, n_q_heads: int, n_kv_heads: int, block_tokens: int, budget_blocks: int,
                 n_sink_blocks: int, n_local_blocks: int, pool_slots: int, max_batch: int, max_blocks: int,
                 solo_head: Sequence[int], head_dim: int = 128, recall_ctas: int = 0, attn_ctas: int = 0,
                 attn_mode: int = 0, wait_limit_us: int = 0, test_hold_producer: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2609_34555_b200 needs a CUDA device; there is no CPU path")
        self._lib = load_library()
        heads = (c_int32 * n_layers)(*[int(h) for h in solo_head])
        self.cfg = PiConfig(n_layers, n_q_heads, n_kv_heads, head_dim, block_tokens, budget_blocks, n_sink_blocks,
                            n_local_blocks, pool_slots, max_batch, max_blocks, recall_ctas, attn_ctas, attn_mode, wait_limit_us,
                            test_hold_producer, heads)
        self._ctx = c_void_p()
        _check("pi_create", self._lib.pi_create(ctypes.byref(self.cfg), ctypes.byref(self._ctx)))
        self.frag_bytes = block_tokens * head_dim * 2 * 2
        self.block_bytes = self.frag_bytes * n_kv_heads

    @classmethod
    def from_workload(cls, cfg, max_batch: Optional[int] = None, **kw) -> "PulseInfer":
        return cls(n_layers=cfg.n_layers, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads,
                   block_tokens=cfg.block_tokens, budget_blocks=cfg.budget_blocks,
                   n_sink_blocks=cfg.n_sink_blocks, n_local_blocks=cfg.n_local_blocks, pool_slots=cfg.pool_slots,
                   max_batch=max_batch or cfg.batch, max_blocks=cfg.n_blocks,
                   solo_head=[cfg.solo_head(l) for l in range(cfg.n_layers)], head_dim=cfg.head_dim, **kw)

    def close(self) -> None:
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self._lib.pi_destroy(self._ctx)
            self._ctx = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ the four path calls
    def score_select(self, layer: int, q, digest, ctx_len, sel_blocks, sel_count, scores=None, stream=None) -> None:
        batch = q.shape[0]
        _check("pi_score_select", self._lib.pi_score_select(
            self._ctx, layer, batch, _dev(q, torch.bfloat16, "q"), _dev(digest, torch.bfloat16, "digest"),
            _dev(ctx_len, torch.int32, "ctx_len"), _dev(sel_blocks, torch.int32, "sel_blocks"),
            _dev(sel_count, torch.int32, "sel_count"),
            None if scores is None else _dev(scores, torch.float32, "scores"), _stream(stream)))

    def score_select_diff(self, layer: int, step, q, digest, ctx_len, sel_blocks, sel_count, block_table, slot_block,
                          slot_stamp, sel_slots, recall_list, recall_count, scores=None, stream=None) -> None:
        """score_select and diff_misses in one launch (same results).  step: a positive int, or a
        one-element int32 CUDA tensor read when the kernel runs (calls captured into a CUDA graph)."""
        batch = q.shape[0]
        dev_step = isinstance(step, torch.Tensor)
        fn = self._lib.pi_score_select_diff_devstep if dev_step else self._lib.pi_score_select_diff
        _check("pi_score_select_diff_devstep" if dev_step else "pi_score_select_diff", fn(
            self._ctx, layer, batch, _dev(step, torch.int32, "step") if dev_step else step,
            _dev(q, torch.bfloat16, "q"), _dev(digest, torch.bfloat16, "digest"), _dev(ctx_len, torch.int32, "ctx_len"),
            _dev(sel_blocks, torch.int32, "sel_blocks"), _dev(sel_count, torch.int32, "sel_count"),
            None if scores is None else _dev(scores, torch.float32, "scores"),
            _dev(block_table, torch.int32, "block_table"), _dev(slot_block, torch.int32, "slot_block"),
            _dev(slot_stamp, torch.int32, "slot_stamp"), _dev(sel_slots, torch.int32, "sel_slots"),
            _dev(recall_list, EXTENT_DTYPE, "recall_list"), _dev(recall_count, torch.int32, "recall_count"),
            _stream(stream)))

    AVERAGE, HEADWISE = 1, 2

    def score_select_strategy(self, strategy: int, layer: int, q, digest_all, ctx_len, sel_blocks, sel_count,
                              scores=None, stream=None) -> None:
        """Averaged (shared) or headwise (per KV head) selection over digests of every KV head."""
        batch = q.shape[0]
        _check("pi_score_select_strategy", self._lib.pi_score_select_strategy(
            self._ctx, strategy, layer, batch, _dev(q, torch.bfloat16, "q"), _dev(digest_all, torch.bfloat16, "digest_all"),
            _dev(ctx_len, torch.int32, "ctx_len"), _dev(sel_blocks, torch.int32, "sel_blocks"),
            _dev(sel_count, torch.int32, "sel_count"),
            None if scores is None else _dev(scores, torch.float32, "scores"), _stream(stream)))

    def build_digests_all(self, kv, ctx_len, digest_all, kv_seq_stride: Optional[int] = None, stream=None) -> None:
        batch = ctx_len.shape[0]
        stride = kv_seq_stride if kv_seq_stride is not None else kv.stride(0) * kv.element_size()
        _check("pi_build_digests_all", self._lib.pi_build_digests_all(
            self._ctx, batch, kv.data_ptr(), stride, _dev(ctx_len, torch.int32, "ctx_len"),
            _dev(digest_all, torch.bfloat16, "digest_all"), _stream(stream)))

    def diff_misses(self, layer: int, step, ctx_len, sel_blocks, sel_count, block_table, slot_block, slot_stamp,
                    sel_slots, recall_list, recall_count, stream=None) -> None:
        """step: a positive int, or a one-element int32 CUDA tensor the kernel reads when it runs
        (for calls captured into a CUDA graph)."""
        batch = sel_count.shape[0]
        if isinstance(step, torch.Tensor):
            _check("pi_diff_misses_devstep", self._lib.pi_diff_misses_devstep(
                self._ctx, layer, batch, _dev(step, torch.int32, "step"), _dev(ctx_len, torch.int32, "ctx_len"),
                _dev(sel_blocks, torch.int32, "sel_blocks"), _dev(sel_count, torch.int32, "sel_count"),
                _dev(block_table, torch.int32, "block_table"), _dev(slot_block, torch.int32, "slot_block"),
                _dev(slot_stamp, torch.int32, "slot_stamp"), _dev(sel_slots, torch.int32, "sel_slots"),
                _dev(recall_list, EXTENT_DTYPE, "recall_list"), _dev(recall_count, torch.int32, "recall_count"),
                _stream(stream)))
            return
        _check("pi_diff_misses", self._lib.pi_diff_misses(
            self._ctx, layer, batch, step, _dev(ctx_len, torch.int32, "ctx_len"),
            _dev(sel_blocks, torch.int32, "sel_blocks"), _dev(sel_count, torch.int32, "sel_count"),
            _dev(block_table, torch.int32, "block_table"), _dev(slot_block, torch.int32, "slot_block"),
            _dev(slot_stamp, torch.int32, "slot_stamp"), _dev(sel_slots, torch.int32, "sel_slots"),
            _dev(recall_list, EXTENT_DTYPE, "recall_list"), _dev(recall_count, torch.int32, "recall_count"),
            _stream(stream)))

    def recall_gather_scatter(self, layer: int, host_kv, pool, recall_list, recall_count, *, lists_per_seq: int = 1,
                              unit_bytes: Optional[int] = None, host_seq_stride: Optional[int] = None,
                              pool_seq_stride: Optional[int] = None, unit_stride: int = 0, list_offset: int = 0,
                              page_table=None, n_pages: Optional[int] = None, stream=None) -> None:
        """host_kv: pinned host tensor [batch][NB] blocks; pool: CUDA tensor [batch][C] blocks;
        recall_list: int32 [n_lists][capacity][4].  With page_table (int32 CUDA tensor [batch][NB]) the
        host tensor is an arena of pages and block b of sequence s is page page_table[s][b]."""
        n_lists, cap = recall_list.shape[0], recall_list.shape[1]
        if not host_kv.is_cuda and not host_kv.is_pinned():
            raise PiError("pi_recall_gather_scatter", -5, strerror(-5))
        ps = pool_seq_stride if pool_seq_stride is not None else pool.stride(0) * pool.element_size()
        if page_table is not None:
            ub = unit_bytes or self.block_bytes
            pages = n_pages if n_pages is not None else host_kv.numel() * host_kv.element_size() // (unit_stride or ub)
            _check("pi_recall_gather_scatter_paged", self._lib.pi_recall_gather_scatter_paged(
                self._ctx, layer, n_lists, lists_per_seq, host_kv.data_ptr(), _dev(page_table, torch.int32, "page_table"),
                page_table.stride(0), pages, pool.data_ptr(), ps, _dev(recall_list, EXTENT_DTYPE, "recall_list"), cap,
                _dev(recall_count, torch.int32, "recall_count"), ub, unit_stride, list_offset, _stream(stream)))
            return
        hs = host_seq_stride if host_seq_stride is not None else host_kv.stride(0) * host_kv.element_size()
        _check("pi_recall_gather_scatter", self._lib.pi_recall_gather_scatter(
            self._ctx, layer, n_lists, lists_per_seq, host_kv.data_ptr(), hs, pool.data_ptr(), ps,
            _dev(recall_list, EXTENT_DTYPE, "recall_list"), cap, _dev(recall_count, torch.int32, "recall_count"),
            unit_bytes or self.block_bytes, unit_stride, list_offset, _stream(stream)))

    def sparse_decode_attn(self, layer: int, q, pool, sel_slots, sel_blocks, sel_count, ctx_len, out, lse=None,
                           stream=None, headwise: bool = False) -> None:
        """headwise=True: sel_slots / sel_blocks are [batch][Hkv][K] (or [batch*Hkv][K]) and sel_count
        [batch][Hkv]: every KV head attends over its own selection."""
        batch = q.shape[0]
        if not pool.is_cuda or not pool.is_contiguous():
            raise TypeError("pool: expected a contiguous CUDA tensor")
        fn = self._lib.pi_sparse_decode_attn_headwise if headwise else self._lib.pi_sparse_decode_attn
        _check("pi_sparse_decode_attn_headwise" if headwise else "pi_sparse_decode_attn", fn(
            self._ctx, layer, batch, _dev(q, torch.bfloat16, "q"), pool.data_ptr(),
            _dev(sel_slots, torch.int32, "sel_slots"), _dev(sel_blocks, torch.int32, "sel_blocks"),
            _dev(sel_count, torch.int32, "sel_count"), _dev(ctx_len, torch.int32, "ctx_len"),
            _dev(out, torch.bfloat16, "out"), None if lse is None else _dev(lse, torch.float32, "lse"),
            _stream(stream)))

    def attn_state(self, batch: int, device=None) -> torch.Tensor:
        """Scratch for the attention split around the recall (sparse_decode_attn_resident / _recalled)."""
        n = self._lib.pi_attn_state_bytes(self._ctx, batch)
        if n < 0:
            raise PiError("pi_attn_state_bytes", int(n), strerror(int(n)))
        return torch.empty(n // 4, dtype=torch.float32, device=device or torch.device("cuda"))

    def sparse_decode_attn_resident(self, layer: int, q, pool, sel_slots, sel_blocks, sel_count, ctx_len, recall_list,
                                    recall_count, state, stream=None) -> None:
        """First half of the attention split around the recall: the selected blocks the step's recall list
        does not touch; may run beside recall_gather_scatter.  Leaves its softmax state in `state`."""
        batch = q.shape[0]
        if not pool.is_cuda or not pool.is_contiguous():
            raise TypeError("pool: expected a contiguous CUDA tensor")
        _check("pi_sparse_decode_attn_resident", self._lib.pi_sparse_decode_attn_resident(
            self._ctx, layer, batch, _dev(q, torch.bfloat16, "q"), pool.data_ptr(),
            _dev(sel_slots, torch.int32, "sel_slots"), _dev(sel_blocks, torch.int32, "sel_blocks"),
            _dev(sel_count, torch.int32, "sel_count"), _dev(ctx_len, torch.int32, "ctx_len"),
            _dev(recall_list, torch.int32, "recall_list"), recall_list.shape[-2],
            _dev(recall_count, torch.int32, "recall_count"), _dev(state, torch.float32, "state"), _stream(stream)))

    def sparse_decode_attn_recalled(self, layer: int, q, pool, sel_slots, sel_blocks, sel_count, ctx_len, recall_list,
                                    recall_count, state, out, stream=None) -> None:
        """Second half: the blocks the recall brought in, merged with `state`; writes `out`.  The caller
        orders it after the first half and after the recall."""
        batch = q.shape[0]
        if not pool.is_cuda or not pool.is_contiguous():
            raise TypeError("pool: expected a contiguous CUDA tensor")
        _check("pi_sparse_decode_attn_recalled", self._lib.pi_sparse_decode_attn_recalled(
            self._ctx, layer, batch, _dev(q, torch.bfloat16, "q"), pool.data_ptr(),
            _dev(sel_slots, torch.int32, "sel_slots"), _dev(sel_blocks, torch.int32, "sel_blocks"),
            _dev(sel_count, torch.int32, "sel_count"), _dev(ctx_len, torch.int32, "ctx_len"),
            _dev(recall_list, torch.int32, "recall_list"), recall_list.shape[-2],
            _dev(recall_count, torch.int32, "recall_count"), _dev(state, torch.float32, "state"),
            _dev(out, torch.bfloat16, "out"), _stream(stream)))

    def append_kv(self, layer: int, step: int, k_new, v_new, ctx_len, host_kv, pool, block_table, slot_block,
                  slot_stamp, digest, host_seq_stride: Optional[int] = None, page_table=None,
                  n_pages: Optional[int] = None, stream=None) -> None:
        """The step's new token (k_new, v_new: [batch][Hkv][D] bf16) joins block ctx_len // B of every
        sequence: pool slot, host store, running digest; ctx_len is the length before the append.
        With page_table the host tensor is an arena of block-sized pages (see recall_gather_scatter)."""
        batch = ctx_len.shape[0]
        if not host_kv.is_cuda and not host_kv.is_pinned():
            raise PiError("pi_append_kv", -5, strerror(-5))
        if isinstance(step, torch.Tensor):               # the step number lives on the device (graph replay)
            pages = 0
            if page_table is not None:
                pages = n_pages if n_pages is not None else host_kv.numel() * host_kv.element_size() // self.block_bytes
            hs = host_seq_stride if host_seq_stride is not None else host_kv.stride(0) * host_kv.element_size()
            _check("pi_append_kv_devstep", self._lib.pi_append_kv_devstep(
                self._ctx, layer, batch, _dev(step, torch.int32, "step"), _dev(k_new, torch.bfloat16, "k_new"),
                _dev(v_new, torch.bfloat16, "v_new"), _dev(ctx_len, torch.int32, "ctx_len"), host_kv.data_ptr(), hs,
                None if page_table is None else _dev(page_table, torch.int32, "page_table"),
                0 if page_table is None else page_table.stride(0), pages, pool.data_ptr(),
                _dev(block_table, torch.int32, "block_table"), _dev(slot_block, torch.int32, "slot_block"),
                _dev(slot_stamp, torch.int32, "slot_stamp"), _dev(digest, torch.bfloat16, "digest"), _stream(stream)))
            return
        if page_table is not None:
            pages = n_pages if n_pages is not None else host_kv.numel() * host_kv.element_size() // self.block_bytes
            _check("pi_append_kv_paged", self._lib.pi_append_kv_paged(
                self._ctx, layer, batch, step, _dev(k_new, torch.bfloat16, "k_new"), _dev(v_new, torch.bfloat16, "v_new"),
                _dev(ctx_len, torch.int32, "ctx_len"), host_kv.data_ptr(), _dev(page_table, torch.int32, "page_table"),
                page_table.stride(0), pages, pool.data_ptr(), _dev(block_table, torch.int32, "block_table"),
                _dev(slot_block, torch.int32, "slot_block"), _dev(slot_stamp, torch.int32, "slot_stamp"),
                _dev(digest, torch.bfloat16, "digest"), _stream(stream)))
            return
        hs = host_seq_stride if host_seq_stride is not None else host_kv.stride(0) * host_kv.element_size()
        _check("pi_append_kv", self._lib.pi_append_kv(
            self._ctx, layer, batch, step, _dev(k_new, torch.bfloat16, "k_new"), _dev(v_new, torch.bfloat16, "v_new"),
            _dev(ctx_len, torch.int32, "ctx_len"), host_kv.data_ptr(), hs, pool.data_ptr(),
            _dev(block_table, torch.int32, "block_table"), _dev(slot_block, torch.int32, "slot_block"),
            _dev(slot_stamp, torch.int32, "slot_stamp"), _dev(digest, torch.bfloat16, "digest"), _stream(stream)))

    # ------------------------------------------------------------------ helpers
    def build_digests(self, layer: int, kv, ctx_len, digest, kv_seq_stride: Optional[int] = None, stream=None) -> None:
        batch = ctx_len.shape[0]
        stride = kv_seq_stride if kv_seq_stride is not None else kv.stride(0) * kv.element_size()
        _check("pi_build_digests", self._lib.pi_build_digests(
            self._ctx, layer, batch, kv.data_ptr(), stride, _dev(ctx_len, torch.int32, "ctx_len"),
            _dev(digest, torch.bfloat16, "digest"), _stream(stream)))

    def table_init(self, resident, block_table, slot_block, slot_stamp, stream=None) -> None:
        batch = resident.shape[0]
        _check("pi_table_init", self._lib.pi_table_init(
            self._ctx, batch, _dev(resident, torch.int32, "resident"), _dev(block_table, torch.int32, "block_table"),
            _dev(slot_block, torch.int32, "slot_block"), _dev(slot_stamp, torch.int32, "slot_stamp"), _stream(stream)))

    def middle_attention_mass(self, lse_mid, lse_all, mam_q, mam_kv, stream=None) -> None:
        """Eq. 2 from two log-sum-exps: mam_q [batch][Hq] = exp(lse_mid - lse_all), mam_kv [Hkv] = its mean
        over the batch and over each KV head's query heads."""
        _check("pi_middle_attention_mass", self._lib.pi_middle_attention_mass(
            self._ctx, lse_all.shape[0], _dev(lse_mid, torch.float32, "lse_mid"), _dev(lse_all, torch.float32, "lse_all"),
            _dev(mam_q, torch.float32, "mam_q"), _dev(mam_kv, torch.float32, "mam_kv"), _stream(stream)))

    def status(self) -> list[int]:
        out = (c_int32 * 8)()
        _check("pi_get_status", self._lib.pi_get_status(self._ctx, ctypes.byref(out)))
        return list(out)

    def stats(self, reset: bool = False) -> dict:
        out = (c_int64 * 4)()
        _check("pi_get_stats", self._lib.pi_get_stats(self._ctx, ctypes.byref(out), int(reset)))
        return dict(sequences=out[0], selected_blocks=out[1], missing_blocks=out[2], extents=out[3])

    def clear_status(self) -> None:
        _check("pi_clear_status", self._lib.pi_clear_status(self._ctx))
