"""Skip-FFN decoder sublayer for NVIDIA B200 (sm_100a).

Python binding of ``libskipffn.so``: argument marshalling only.  PyTorch supplies device memory
and the CUDA stream; every step of the path (mask compaction, row routing, the five GEMM kinds
with their fused epilogues) runs in the library's own kernels.  There is no CPU or PyTorch
fallback: if the library is missing, or no CUDA device is present, calls raise.
"""
from .binding import (SkipFFNError, SkipFFN, load_library, skipffn_workspace_bytes, skipffn_flops,
                      skipffn_strerror, skipffn_compact_static, skipffn_schedule, skipffn_schedule_plan, summary_forward, summary_backward, token_merge, STATIC_MAX_TOKENS, BF16, FP32, PATH_DEFAULT, PATH_SIMT, EXPORTS)

__all__ = ["SkipFFNError", "SkipFFN", "load_library", "skipffn_workspace_bytes", "skipffn_flops",
           "skipffn_strerror", "skipffn_compact_static", "skipffn_schedule", "skipffn_schedule_plan", "summary_forward", "summary_backward", "token_merge", "STATIC_MAX_TOKENS", "BF16", "FP32", "PATH_DEFAULT", "PATH_SIMT", "EXPORTS"]
