"""B200-native KVMem recall step: Mean-K block scoring, selection, execution-view assembly and
GQA decode attention as hand-written sm_100a CUDA behind a C ABI (``include/kvmem.h``)."""
from .kvmem import (  # noqa: F401
    KvmemError,
    Pool,
    PoolConfig,
    SelectParams,
    View,
    budget_blocks,
    load_library,
    set_option,
)
