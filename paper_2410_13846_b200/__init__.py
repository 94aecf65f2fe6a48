"""B200-native hybrid decode attention (LightTransfer hot path).

The work is done by liblt.so (hand-written CUDA for sm_100a behind a C ABI,
declared in include/lt.h).  This package is the thin Python binding: argument
marshalling only.  There is no CPU or PyTorch fallback: calls raise when the
library is missing or a CUDA device is absent.
"""
from .binding import (  # noqa: F401
    LT_BF16, LT_F32, LayerTables, LtError, Shape, check, decode_step, decode_step_host, decode_step_layers, hybrid_decode_attn, hybrid_decode_attn_static, kv_append, lazy_scores, lazy_scores_lse, lazy_scores_with_lse, lib, lib_path,
    ring_slot, select_lazy, select_lazy_frequency, select_lazy_per_seq, select_lazy_push, status_string, stream_init, stream_init_layer, version, workspace_bytes, workspace_bytes_layers, workspace_init,
)
