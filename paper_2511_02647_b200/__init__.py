"""FedAttn attention hot path for NVIDIA B200 (sm_100a): thin Python binding over the C-ABI
library ``lib/libfedattn.so`` (hand-written CUDA).  Argument marshalling only: every step of
the path runs in the library's kernels.  There is no CPU fallback; importing the binding
raises if the library has not been built or cannot be loaded."""
from .binding import (  # noqa: F401
    AGG_CONCAT, AGG_INDEXED, AGG_TOPK_KNORM, AGG_TOPK_TOKEN, BF16, DECODE_LOCAL, DECODE_SYNC, F32,
    FedAttnError, Context, PreparedCall, Shape, exported_symbols, fedattn_aggregate_kv, fedattn_decode,
    fedattn_decode_noalloc, fedattn_local, fedattn_merge, fedattn_sync, fedattn_sync_remote, fedattn_workspace_bytes,
    library_path, prepare_aggregate_kv, prepare_decode, prepare_local, prepare_merge, prepare_sync, prepare_sync_remote,
    status_string,
)
