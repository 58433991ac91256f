"""B200-native planner for G10's compile-time tensor-migration analysis (vitality, pressure timeline,
greedy eviction planner) behind the C ABI of include/g10.h.  `traces` builds the synthetic inputs,
`binding` calls the CUDA library, `build` compiles it."""
from . import traces  # noqa: F401

__all__ = ["traces", "binding", "build"]
