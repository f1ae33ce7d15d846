"""B200-native link-prediction GNN training step (C-ABI library + thin ctypes binding)."""
from .binding import (  # noqa: F401
    Context,
    LpError,
    ModelDesc,
    Stats,
    load_library,
    weight_grad_static,
    EXPORTS,
    PROF_CATEGORIES,
    LP_GCN,
    LP_SAGE_MEAN,
    LP_FP32,
    LP_BF16,
    LP_NEG_PER_SOURCE,
    LP_NEG_GLOBAL_PAIR,
)
