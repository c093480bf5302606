"""huffllm: Huffman-compressed bf16 weights decoded on the fly inside GPU matrix products.

The Python layer only marshals arguments into the C-ABI library (``libhuffllm.so``); every
step of the method runs in that library.  Importing this package fails loudly when the
library has not been built — there is no fallback path.
"""
from .binding import (  # noqa: F401
    BF16, FP16, SPLIT_PAPER, SPLIT_WHOLE_EXPONENT, HuffllmError, Codebook, Desc, lib, build_codebook, encode_bound, encode, validate_blob,
    workspace_bytes, workspace_control_bytes, decode_smem_plan, decode_launch_plan, decode, decode_gemv, decode_gemm, decode_gemm_host, decode_gemm_multi, decode_gemm_multi_host, PreparedMulti, decode_gemm_static, STATIC_MAX_BATCH, plain_gemv, plain_gemv_multi, PreparedPlainMulti, last_error, exported_symbols,
    stage_copy, split_counts_size, split_histogram, split_entropy, build_codebook_from_counts, encode_device_scratch_bytes, encode_device,
)
