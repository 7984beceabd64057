"""B200-native LightKV vision-token compression step: thin Python binding over liblightkv.so.

The hot path lives entirely in the CUDA library (csrc/); this package only marshals arguments.
Importing the package does not load the library; the first call does and fails loudly if the
shared object has not been built (see __graft_entry__.build)."""
from .lightkv import (  # noqa: F401
    BF16, FP32, XI_GIVEN, XI_ATTN_FULL, XI_ATTN_LSE, XI_UNIFORM, KV_MERGE, KV_GATHER,
    ENGINE_AUTO, ENGINE_SIMT, FD_COSINE, FD_L2SQ, FD_L2, DIR_A2B, DIR_B2A, MAX_TEXT_RANGES, LightKVError, Plan, StageBuffers, compress_layer, compress_layer_builtin_ws, BUILTIN_WS_BYTES, compact_kv,
    library, library_path, status_string, version, TRACE_EVENTS, TRACE_NAMES,
)
