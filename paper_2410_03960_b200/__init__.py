"""SwiftKV prefill for NVIDIA B200: a thin Python binding over the C-ABI CUDA library (libswiftkv.so).

Every step of the prefill runs in the library's kernels; this package only marshals arguments.
PyTorch is used for device memory and streams.
"""
from .binding import (  # noqa: F401
    ACT_BF16,
    ACT_F16,
    KC_NAMES,
    SwiftKVError,
    SwiftKVModel,
    attention_prefill,
    gemm_tc,
    library_path,
    load_library,
    tail_attention,
    tail_attention_noalloc,
    workspace_bytes,
)
from .flops import prefill_flops  # noqa: F401
