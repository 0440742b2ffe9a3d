"""B200 (sm_100a) decode recall path of sparse KV-cache offloading:
score -> top-k select -> miss diff -> gather-scatter recall -> sparse GQA attention.

The work is done by the CUDA library built from csrc/ behind the C ABI declared in
include/pulseinfer.h; `binding` is its ctypes front end.
"""
from .binding import PulseInfer, PiError, score_select_noalloc, load_library, h2d_copy_ms, empty_launch, strerror, EXPORTS  # noqa: F401
