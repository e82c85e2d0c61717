"""B200 (sm_100a) library for the GAD training epoch (arXiv 2110.02987): CUDA kernels behind a C ABI
(``include/gad.h``, built into ``libgad.so``) and a thin ctypes binding."""
from .binding import (  # noqa: F401
    Gad, GadError, Augmenter, augment, default_params, gad_workspace_bytes, from_workload, launch_count, load, subgraph_weights_static, LIB_PATH, SYMBOLS,
)
from .multi import ShardedEpoch, RoundsEpoch, shard_subgraphs  # noqa: F401
