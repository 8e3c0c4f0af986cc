"""B200-native declared-reference (fold) softmax attention decode: CUDA library + thin binding."""
from .binding import (  # noqa: F401
    FoldArgs, FoldKV, FoldPartials, FoldWsHeader, FoldError, KVCache, DecodeBuffers,
    Z_ESTIMATE, Z_GIVEN, Z_EXACT_MAX, Z_ZERO, ROW_RANGE, ROW_NONFINITE, ROW_EMPTY,
    FOLD_OK, FOLD_EINVAL, FOLD_EUNSUPPORTED, FOLD_EWORKSPACE, FOLD_ECUDA, FOLD_ETOOLARGE, STATIC_SCRATCH_BYTES, INPUTS_SETTLED, SEPARATE_LAUNCHES, ONE_LAUNCH, CascadeSide,
    make_args, alloc_buffers, decode, decode_certified, slots_view, lib,
    fold_workspace_bytes, fold_chunk_keys, fold_num_chunks, fold_estimate_z, fold_decode_split,
    fold_cascade_merge, fold_decode, fold_decode_launches, fold_decode_cascade, fold_host_staging_bytes, fold_decode_host, fold_decode_static, fold_block_means, fold_running_means,
    fold_quantize_keys, fold_quantize_values, fold_probe_read,
)
