"""B200-native Dynamic Depth Decoding draft-tree path: thin ctypes binding over libddd.so.

Every step of the path runs in the CUDA kernels behind the C ABI of include/ddd.h; this
package only marshals arguments.  PyTorch supplies device memory and streams.
"""
from .binding import (  # noqa: F401
    DDD_DTYPE_BF16, DDD_DTYPE_FP32, DDD_LAUNCH_FUSED, DDD_LAUNCH_GRAPH, DDD_LAUNCH_PLAIN, DDD_LAUNCH_STREAM, DDD_LM_HEAD_AUTO,
    DDD_LM_HEAD_SIMT, DDD_LM_HEAD_TCGEN05, DddConfig, DddError, DddOutput, DddTrace, DddVerifyOutput, DraftEngine,
    ddd_create, ddd_destroy, ddd_draft, ddd_draft_host, ddd_draft_host_gated, ddd_launches_per_draft, ddd_lm_head_blocks, ddd_fused_pass_kind,
    ddd_lm_head_pass, ddd_lm_head_topk_noalloc, ddd_shard_begin, ddd_shard_lm_head, ddd_shard_records_bytes, ddd_shard_select,
    ddd_strerror, ddd_verify_greedy, ddd_workspace_bytes, exported_symbols, library_path, load_library, vocab_slice,
)
