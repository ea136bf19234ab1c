"""fp64 CPU oracle for the attention forward+backward path.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline / reference legs of the benchmark.  The CUDA library and its
Python binding never import this package, and this package imports neither.
"""
from .attention import (  # noqa: F401
    build,
    num_threads,
    attn_fwd_bwd,
    attn_fwd_bwd_gqa,
    attn_head_full,
    attn_rows,
    attn_cols,
)
from .decode import decode_attn  # noqa: F401,E402
from .block import (  # noqa: F401,E402
    rmsnorm_fwd_bwd, gated_mlp_fwd_bwd, gated_mlp_bwd_from_saved, gemm, transformer_block_fwd_bwd,
)
