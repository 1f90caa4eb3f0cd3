"""CPU oracle (test infrastructure; never imported by the product path)."""
from .indexer_topk import (  # noqa: F401
    OracleResult,
    decode,
    decode_bf16,
    decode_e4m3,
    indexer_scores,
    indexer_topk,
    oracle_topk,
    score_row,
    select_topk,
    visible_keys,
)
from .sampler import frequent_positions, position_counts  # noqa: F401,E402
from .litedsa import pack_mask_words, union_and_masks  # noqa: F401,E402
from .knn import knn_scores, knn_topk  # noqa: F401,E402
