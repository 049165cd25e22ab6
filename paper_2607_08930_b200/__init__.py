"""B200-native (sm_100a) mixed-state block-denoising engine: CUDA library + thin ctypes binding."""
from . import binding  # noqa: F401
from .binding import Engine, engine_for_workload, make_config, query_sizes  # noqa: F401
