"""vitint: integerized ViT matmul path for NVIDIA B200 (thin ctypes binding over libvitint.so).

Every function here only marshals arguments: all arithmetic of the path runs in the CUDA
kernels of the C-ABI library declared in include/vitint.h.  PyTorch supplies device memory
and streams.  There is no CPU fallback: a missing library raises at import of the binding.
"""
from .binding import (  # noqa: F401
    Codes, Epilogue, Slabs, AttentionWeights, VitintError, fold_layernorm_references, fold_requant, vitint_fold_layernorm_references, vitint_fold_requant, lib, packed_pitch,
    vitint_attention_block, vitint_attention_block_workspace_bytes, vitint_attention_core,
    vitint_attention_core_noalloc, vitint_attention_core_shift, vitint_attention_core_shift_workspace_bytes, vitint_attention_core_prepared, vitint_attention_core_workspace_bytes,
    vitint_attention_exp_table, vitint_device_status, vitint_selftest_wait_timeout,
    vitint_layernorm_compare_quantize, vitint_layernorm_quantize, vitint_linear, vitint_linear_e2m1, vitint_linear_qkv_norm, vitint_pv, vitint_qk, vitint_quantize,
    vitint_softmax_quantize, vitint_softmax_quantize_bounded, vitint_softmax_table_workspace_bytes, vitint_softmax_shift_quantize, vitint_status_string, vitint_version, vitint_widen, EPI_ACC_I32, EPI_DEQUANT_F32, EPI_REQUANT,
)
