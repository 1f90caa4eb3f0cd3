"""B200-native fused DSA indexer top-k (C-ABI CUDA library + thin ctypes binding).

Importing the package does not load the CUDA library; the first call through
`binding` does, and fails loudly if the library has not been built.
"""
from . import binding  # noqa: F401
from .binding import (  # noqa: F401
    LT_DTYPE_BF16,
    LT_DTYPE_E4M3,
    LT_DTYPE_F32,
    LT_PATH_AUTO,
    LT_PATH_FUSED,
    LT_PATH_GENERIC,
    LtError,
    Tunables,
    lt_indexer_scores,
    lt_indexer_topk,
    lt_indexer_topk_ex,
    lt_indexer_topk_static,
    lt_indexer_topk_workspace_bytes,
    lt_read_status,
    lt_unfused_topk,
)
