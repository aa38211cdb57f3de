"""IsoQuant compressed-space decode attention for B200 (sm_100a).

A thin Python binding over the C-ABI CUDA library `libisoquant.so` (declared in include/isoquant.h). Every
step of the path runs in the library's kernels; this package only marshals arguments (torch tensors ->
device pointers, the current torch stream -> cudaStream_t). There is no CPU fallback: if the compiled
library is missing or fails to load, importing `paper_2608_08081_b200.binding` raises.
"""
from .binding import (  # noqa: F401
    IQError,
    Cache,
    Codebook,
    Shape,
    iq_combine_splits,
    iq_combine_splits_sharded,
    iq_decode_attention,
    iq_decode_attention_static,
    iq_static_scratch_bytes,
    iq_default_codebook,
    iq_int8_codebook,
    iq_lloyd_max_codebook,
    iq_codebook_set_v,
    iq_row_bytes_bits,
    iq_make_rotation,
    iq_quantize_append,
    iq_rotation_floats,
    iq_row_bytes,
    iq_strerror,
    iq_decode_step_host,
    iq_decode_step_fused,
    iq_decode_step_workspace_bytes,
    iq_fit_codebook,
    iq_reconstruct_rows,
    iq_rotated_histogram,
    iq_suggest_splits,
    iq_fit_rotation,
    iq_format_version,
    iq_selftest_bounded_wait,
    iq_version,
    iq_wht_coordinates,
    lib_path,
    new_cache,
    new_paged_cache,
    DecodeWorkspace,
    HostStepper,
    decode_step,
)
