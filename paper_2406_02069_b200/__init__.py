"""B200-native PyramidKV prefill KV-cache compression (budget schedule, window scores,
pool + top-k, gather) behind a C-ABI CUDA library; see include/pyramidkv.h."""
from . import workloads  # noqa: F401
from .binding import (PkvConfig, PkvError, PkvTensor, attention_recall, check_status, decode_attention, compress_layer, config_of,  # noqa: F401
                      gather_compact, kept_count, layer_budgets, library_path, make_config, new_workspace, profile_layer,
                      score_window, score_window_static, check_status_static, select_topk, strerror, total_rows, workspace_bytes,
                      compress_layer_paged, decode_attention_paged, gather_paged, pages_needed, memory_kind, Lanes, compress_model_lanes,
                      attend_window, attend_compress_layer)
