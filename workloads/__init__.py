"""Seeded synthetic inputs for the decode recall path.

This package only *creates data* (keys, values, queries, resident sets, scripted
recall lists).  It holds none of the method's arithmetic: digests, scores,
selections, diffs and attention are computed by the CUDA library and, separately,
by the CPU oracle, each from the tensors produced here.
"""
from .configs import PathConfig, CONFIGS, get_config, tiny_config  # noqa: F401
