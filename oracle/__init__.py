"""CPU oracle for the Stream hot path. Test infrastructure only: the CUDA library never imports it."""
from .stream_oracle import (  # noqa: F401
    OracleProblem,
    build,
    build_mask_rows,
    mask_difference,
    num_query_blocks,
    num_rows,
    sparse_attention_rows,
    threads,
    tile_score,
    vertical_scores,
)
