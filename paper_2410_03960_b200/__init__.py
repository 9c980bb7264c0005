"""SwiftKV prefill for NVIDIA B200: a thin Python binding over the C-ABI CUDA library (libswiftkv.so).

Every step of the prefill runs in the library's kernels; this package only marshals arguments.
PyTorch is used for device memory and streams.
"""
from .binding import (  # noqa: F401
    ACT_BF16,
    DISTILL_FP32,
    DISTILL_TF32,
    DISTILL_TF32X3,
    ACT_F16,
    ACT_F16_SPLIT,
    SPLIT_ATTN_OUT,
    SPLIT_MLP_ACT,
    SPLIT_MLP_INPUT,
    SPLIT_QKV_INPUT,
    SPLIT_SCORES,
    KC_NAMES,
    KV_FP8,
    KV_MODEL_DTYPE,
    SwiftKVError,
    SwiftKVModel,
    adamw_update,
    attention_prefill,
    attention_prefill_split,
    gemm_tc_split,
    gemm_tc,
    gemm_tf32,
    library_path,
    load_library,
    quantize_rows_fp8,
    tail_attention,
    tail_attention_fp8,
    tail_attention_noalloc,
    workspace_bytes,
)
from .flops import prefill_flops  # noqa: F401
