"""B200-native MXFP4 weight-only linear layer (the draft-model hot path of ML-SpecQD).

The CUDA library is loaded on first use, not at import, so that the input
generators in :mod:`paper_2503_13565_b200.synth` can be used on a machine
without the built extension.  There is no CPU fallback: every operation raises
if ``libmxq.so`` is missing.
"""
from .binding import (MAX_M, MAX_T, MXQ_BF16, MXQ_F32, MxqError, mxq_accept_workspace_bytes, mxq_codes_bytes,  # noqa: F401
                      mxq_dequantize, mxq_greedy_accept, mxq_greedy_accept_static,
                      mxq_greedy_accept_static_max_bytes, mxq_greedy_accept_tokens, mxq_linear, mxq_linear_host,
                      KERNELS, mxq_linear_device_status, mxq_linear_plan_info, mxq_linear_workspace_bytes,
                      mxq_set_linear_kernel, mxq_linear_bf16, mxq_linear_fused_workspace_bytes, mxq_linear_residual, mxq_linear_swiglu, interleave_gate_up, mxq_lm_head_accept, mxq_lm_head_accept_workspace_bytes, mxq_quantize, mxq_scales_bytes, mxq_set_pdl, mxq_version,
                      new_workspace, status_string, LinearBatch, IndependentBatches, mxq_linear_batch, mxq_set_linear_layout,
                      mxq_debug_batch_fault, mxq_debug_bounds_report, mxq_debug_bounds_selftest)
