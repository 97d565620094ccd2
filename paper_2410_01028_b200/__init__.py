"""Adaptive self-speculative decoding (arXiv 2410.01028) on one B200: thin Python binding of ``libasd.so``.

Every step of the method runs in the CUDA library; this package only marshals arguments.
PyTorch is used for device memory and the CUDA stream, nothing else.
"""
from .binding import (  # noqa: F401
    ADMG_ALL, EPI_PLAIN, EPI_RESIDUAL, EPI_SWIGLU, MODE_AR, MODE_SPEC, MODE_SPEC_MANUAL_MASK, PREFILL_AUTO, PREFILL_GEMM,
    PREFILL_ROWS, RUNNING_C, USE_CS, USE_CS_MLP, USE_RULE1, USE_RULE2, AsdError, Decoder, admg, admg_ext, fused_gemv, fused_gemv_scratch_bytes, fused_gemv_static,
    gemm_bf16, lib, workspace_bytes,
)
