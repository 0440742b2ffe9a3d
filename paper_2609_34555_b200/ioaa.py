"""IO-Adaptive Offloading Admission (Sec. 4.3 of the paper): a thin host policy.

For the requests waiting at a decode-step boundary it picks who joins the normal batch (full
KV on the GPU, no recall I/O) and who joins the offload batch (fixed GPU budget, recall I/O),
by evaluating the paper's throughput model

    throughput  ~  m/(m+1) * B_n  +  1/(m+1) * B_o                                  (Eq. 1)

on the leaves of a binary tree (one level per request, branches = normal / offload) with the
two pruning rules of Sec. 4.3.1, the overlap depth m(B_o, B_n) being interpolated from a grid
profiled offline (Sec. 4.3.2; m = ceil(t_io / t_layer) averaged over layers, so it need not be
an integer).  Pure host code: nothing here touches the GPU.
"""
from __future__ import annotations

import bisect
import math
from dataclasses import dataclass, field
from typing import Optional, Sequence


def throughput_model(m: float, b_n: int, b_o: int) -> float:
    """Eq. 1: one offload-batch layer is overlapped with m normal-batch layers."""
    m = max(1.0, m)
    return m / (m + 1.0) * b_n + 1.0 / (m + 1.0) * b_o


def overlap_depth(t_io: float, t_layer: float) -> int:
    """m = ceil(t_io / t_layer), at least 1 (Sec. 4.3.2)."""
    return max(1, math.ceil(t_io / t_layer))


@dataclass
class OverlapDepthGrid:
    """Overlap depth profiled on a grid of (B_o, B_n); bilinear interpolation in between,
    clamped at the edges, never below 1."""
    bo: Sequence[float]
    bn: Sequence[float]
    m: Sequence[Sequence[float]]            # m[i][j] for bo[i], bn[j]

    def __call__(self, b_o: float, b_n: float) -> float:
        def bracket(xs, x):
            if x <= xs[0]:
                return 0, 0, 0.0
            if x >= xs[-1]:
                return len(xs) - 1, len(xs) - 1, 0.0
            hi = bisect.bisect_right(xs, x)
            lo = hi - 1
            return lo, hi, (x - xs[lo]) / (xs[hi] - xs[lo])
        i0, i1, u = bracket(self.bo, b_o)
        j0, j1, v = bracket(self.bn, b_n)
        a = self.m[i0][j0] * (1 - v) + self.m[i0][j1] * v
        b = self.m[i1][j0] * (1 - v) + self.m[i1][j1] * v
        return max(1.0, a * (1 - u) + b * u)

    @classmethod
    def from_timings(cls, bo: Sequence[float], bn: Sequence[float], t_io, t_layer) -> "OverlapDepthGrid":
        """t_io[i][l]: recall latency of layer l at offload batch bo[i]; t_layer[j]: time of one
        normal-batch layer at bn[j].  m is the mean over layers of ceil(t_io / t_layer)."""
        m = [[sum(overlap_depth(t, t_layer[j]) for t in t_io[i]) / len(t_io[i]) for j in range(len(bn))]
             for i in range(len(bo))]
        return cls(list(bo), list(bn), m)


@dataclass
class Admission:
    normal: list[int] = field(default_factory=list)      # indices into the waiting list
    offload: list[int] = field(default_factory=list)
    throughput: float = 0.0
    nodes_visited: int = 0


def ioaa_admit(lengths: Sequence[int], memory_budget: int, offload_budget_tokens: int, depth: OverlapDepthGrid,
               running_normal: int = 0, running_offload: int = 0) -> Optional[Admission]:
    """Best complete assignment of the waiting requests (token lengths `lengths`) under the GPU
    memory budget (in tokens of KV): a normal request costs its length, an offloaded one the fixed
    `offload_budget_tokens`.  Returns None when no complete assignment fits.

    Search: requests in order of decreasing length; at each level try offload, then normal.
    Pruning rule 1: a branch whose memory exceeds the budget is cut.  Pruning rule 2 (length
    monotonicity): once a request went to the normal batch, every shorter one goes there too, so
    below a `normal` branch the tree is a single path."""
    order = sorted(range(len(lengths)), key=lambda i: (-lengths[i], i))
    suffix = [0] * (len(order) + 1)                      # tokens of all requests from position i on
    for i in range(len(order) - 1, -1, -1):
        suffix[i] = suffix[i + 1] + lengths[order[i]]
    best = Admission(throughput=-1.0)
    visited = 0

    def leaf(n_off: int) -> None:
        nonlocal best
        b_o = running_offload + n_off
        b_n = running_normal + len(order) - n_off
        thr = throughput_model(depth(b_o, b_n), b_n, b_o)
        if thr > best.throughput:
            best = Admission(normal=sorted(order[n_off:]), offload=sorted(order[:n_off]), throughput=thr)

    def descend(level: int, used: int) -> None:
        nonlocal visited
        visited += 1
        if level == len(order):
            leaf(level)
            return
        # branch "normal": everything shorter follows (rule 2) -- one leaf, if it fits (rule 1)
        if used + suffix[level] <= memory_budget:
            visited += 1
            leaf(level)
        # branch "offload"
        if used + offload_budget_tokens <= memory_budget:
            descend(level + 1, used + offload_budget_tokens)

    descend(0, 0)
    if best.throughput < 0:
        return None
    best.nodes_visited = visited
    return best


def admit_fcfs(lengths: Sequence[int], memory_budget: int, offload_budget_tokens: int, depth: OverlapDepthGrid,
               running_normal: int = 0, running_offload: int = 0) -> Admission:
    """Admits the longest arrival-order prefix of the waiting queue for which a complete
    assignment fits; the rest keeps waiting."""
    for n in range(len(lengths), 0, -1):
        a = ioaa_admit(lengths[:n], memory_budget, offload_budget_tokens, depth, running_normal, running_offload)
        if a is not None:
            return a
    return Admission()
