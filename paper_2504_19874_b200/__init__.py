"""TurboQuant hot path for B200: thin Python binding over the C-ABI CUDA library libtq.so.

Every computation runs inside the library's CUDA kernels; this package only marshals
arguments (torch tensors supply device memory and streams).  There is no CPU fallback: a
missing library or a missing GPU raises.
"""
from .binding import (  # noqa: F401
    TQ_BF16, TQ_F32, TQ_GAUSSIAN, TQ_MSE, TQ_OP_DEQUANTIZE, TQ_OP_QUANTIZE, TQ_OP_SCORE, TQ_OP_TOPK, TQ_OP_WSUM,
    TQ_ORTHOGONAL, TQ_PROD, Plan, TqError, lib, tq_codebook, tq_dequantize, tq_idx_row_bytes, tq_launch_count, tq_plan_status, tq_qjl_row_bytes,
    tq_quantize_mse, tq_quantize_prod, tq_rotation, tq_score, tq_score_static, tq_select_topk, tq_softmax, tq_topk, TQ_STATIC_SCRATCH_BYTES, tq_workspace_bytes, tq_wsum,
    TQ_LAYOUT_CANONICAL, TQ_LAYOUT_NIBBLE, tq_convert_layout, tq_query_bytes, tq_query_prepare, tq_score_prepared,
    tq_score_static_max_queries, tq_selftest_wait_timeout, tq_entropy_lengths, tq_entropy_pack, tq_entropy_unpack,
    KvGroup, tq_attend_decode, tq_attend_decode_workspace_bytes, tq_kv_append,
)
