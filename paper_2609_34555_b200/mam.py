"""Middle Attention Mass (Eq. 2 of the paper) and the choice of the retrieval head.

MAM_q = sum over middle positions i of the attention weight A_q(i); the MAM of a KV head is the
mean over the query heads that GQA maps to it; the KV head with the highest MAM of a layer is
its retrieval ("SoloHead") head (Sec. 4.4.1).  With lse_S the log-sum-exp of the logits over a
token set S,  sum_{i in S} A(i) = exp(lse_S - lse_all): two calls of pi_sparse_decode_attn (all
blocks, middle blocks only) and pi_middle_attention_mass give the mass and its per-KV-head mean;
picking the arg-max of Hkv numbers is left to the host.  "Middle" is
block-granular here, like the path's sink and local blocks.  The sample sequences must be fully
resident in the pool (slot i = block i); this is an offline profiling helper, not a hot call.
"""
from __future__ import annotations

import torch

from .binding import PulseInfer


def middle_attention_mass(pi: PulseInfer, layer: int, q: torch.Tensor, pool: torch.Tensor, ctx_len: torch.Tensor,
                          return_kv: bool = False):
    """q [batch][Hq][D] bf16, pool [batch][C >= n_blocks] blocks with slot i = block i.
    Returns MAM per query head, float32 [batch][Hq]; with return_kv also the per-KV-head mean [Hkv]
    (both from pi_middle_attention_mass)."""
    c = pi.cfg
    batch, dev = q.shape[0], q.device
    K, B = c.budget_blocks, c.block_tokens
    n_blocks = (ctx_len + B - 1) // B
    if int(n_blocks.max()) > K:
        raise ValueError("the context must fit the budget: build the context with budget_blocks >= n_blocks")
    idx = torch.arange(K, dtype=torch.int32, device=dev)[None, :].expand(batch, -1)
    out = torch.empty_like(q)
    lse_all = torch.empty((batch, c.n_q_heads), dtype=torch.float32, device=dev)
    lse_mid = torch.empty_like(lse_all)
    # all blocks
    cnt = n_blocks.to(torch.int32).contiguous()
    sel = torch.where(idx < cnt[:, None], idx, torch.full_like(idx, -1)).contiguous()
    pi.sparse_decode_attn(layer, q, pool, sel, sel, cnt, ctx_len, out, lse_all)
    # middle blocks only: [n_sink, n_blocks - n_local)
    lo = torch.minimum(torch.full_like(cnt, c.n_sink_blocks), cnt)
    hi = torch.maximum(cnt - c.n_local_blocks, lo)
    mcnt = (hi - lo).contiguous()
    msel = torch.where(idx < mcnt[:, None], idx + lo[:, None], torch.full_like(idx, -1)).contiguous()
    pi.sparse_decode_attn(layer, q, pool, msel, msel, mcnt, ctx_len, out, lse_mid)
    mam_q = torch.empty_like(lse_all)
    mam_kv = torch.empty((c.n_kv_heads,), dtype=torch.float32, device=dev)
    pi.middle_attention_mass(lse_mid, lse_all, mam_q, mam_kv)
    return (mam_q, mam_kv) if return_kv else mam_q


def kv_head_mam(mam_q: torch.Tensor, n_kv_heads: int) -> torch.Tensor:
    """Mean over samples and over each KV head's query heads: [Hkv] (host-side regrouping of masses
    that pi_middle_attention_mass has computed, for samples collected over several calls)."""
    batch, Hq = mam_q.shape
    return mam_q.view(batch, n_kv_heads, Hq // n_kv_heads).mean(dim=(0, 2))


def choose_solo_head(mam_q: torch.Tensor, n_kv_heads: int, reversed_rank: bool = False) -> int:
    """The KV head with the highest (or, for the paper's control experiment, lowest) MAM."""
    m = kv_head_mam(mam_q, n_kv_heads)
    return int(torch.argmin(m) if reversed_rank else torch.argmax(m))
