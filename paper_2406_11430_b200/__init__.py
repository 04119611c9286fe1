"""l2kv: L2-norm KV-cache compression and decode attention on B200 (sm_100a).

Thin Python front end of the C library ``libl2kv.so``: the functions here only
marshal torch tensors into pointers and sizes; every step runs in the library's
CUDA kernels.  There is no CPU fallback -- a missing library is an ImportError.
"""
from .binding import (L2KVError, Layout, Rows, key_norms, select_compact, decode_attention,  # noqa: F401
                      append_evict, decode_attention_static, select_compact_per_head,
                      decode_attention_per_head, append_evict_per_head, prefix_attention_per_head, prefix_attention_workspace, prefix_attention_causal, prefix_attention_flags, PREFIX_CAUSAL, PREFIX_LEN_PER_HEAD, PREFIX_SPLIT_WEIGHTS, attention_loss, prefix_attention, keep_count, workspace_bytes, new_workspace,
                      read_device_status, workspace_reset, selftest_wait_timeout,
                      decode_attention_static_status, status_string, library_path, lib,
                      KEEP_LOWEST_NORM, KEEP_HIGHEST_NORM, KEEP_RANDOM)
