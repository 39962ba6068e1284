"""Tree verification for staged speculative decoding on B200: Python binding of libssd.

The binding only marshals arguments; every step of the hot path runs in the CUDA
kernels of ``libssd.so`` (built in-tree by ``paper_2308_04623_b200.build``).  Importing
this package without the built library raises: there is no CPU fallback.
"""
from .binding import (  # noqa: F401
    SSD_OK, SSD_ERR_BAD_ARG, SSD_ERR_NOT_LOADED, SSD_ERR_INVALID_TREE, SSD_ERR_CTX_OVERFLOW, SSD_ERR_BAD_PATH,
    SSD_ERR_CUDA, SSD_ERR_TIMEOUT, SSD_ERR_NOMEM, SSD_ERR_UNSUPPORTED, SSD_GREEDY, SSD_SAMPLING,
    SSD_DTYPE_F32, SSD_DTYPE_BF16, SSD_DTYPE_BF16_W8,
    SSD_TUNE_LOW_PLANE, SSD_TUNE_DEPENDENT_LAUNCH, SSD_TUNE_GRAPH, SSD_TUNE_GEMM_CTAS, SSD_TUNE_CLUSTER_REDUCE, SSD_TUNE_CLUSTER_MAX, SSD_TUNE_ATTN_LOW_PLANE, SSD_TUNE_HEAD_CTAS, SSD_TUNE_KERNEL_TRACE, SSD_TUNE_HEAD_STATS, SSD_TUNE_W8_PLANES, SSD_TUNE_STAGE_KV_FROM, SSD_TUNE_ATTN_SPLITS, SSD_TUNE_NODE_GROUPS, SSD_TUNE_FUSED_GELU, SSD_TUNE_ATTN_STAGED_WARPS,
    SsdError, Context, KV, Trigram, lib, library_path, EXPORTS,
)
