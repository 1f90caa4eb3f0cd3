"""Seeded synthetic inputs for the DSA indexer top-k path.

This package only *produces inputs* (random draws, storage-format encoding,
planted structure).  It holds none of the scoring or selection arithmetic, and
is the one module the CPU oracle's tests and the CUDA path's tests both use.
"""
from .gen import (  # noqa: F401
    CONFIGS,
    KNN_CONFIGS,
    KnnInputs,
    IndexerInputs,
    bf16_encode,
    e4m3_encode,
    make_config,
    make_inputs,
    make_knn,
    quantize_e4m3_per_token,
)
