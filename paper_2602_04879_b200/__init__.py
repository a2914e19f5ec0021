"""DPPO per-token loss path for NVIDIA B200: a C-ABI CUDA library (include/dppo.h, csrc/) and this
thin ctypes binding.  The library is loaded on first use; there is no CPU or PyTorch fallback."""
from . import binding  # noqa: F401
from .binding import (BF16, BINARY_KL, BINARY_TV, F32, KERNEL_AUTO, KERNEL_GENERIC, KERNEL_RING, GIVEN_D, MINIMAL_MASK, PPO_CLIP, TOPK_KL, TOPK_TV,  # noqa: F401
                      DppoError, dppo_exact_divergence, dppo_host_staging_bytes, dppo_fused_lmhead_fwd_bwd, dppo_fused_workspace_bytes, dppo_gemm_nn_bf16, dppo_gemm_tn_bf16, dppo_loss_fwd_bwd,
                      dppo_loss_fwd_bwd_host, dppo_loss_fwd_bwd_static_ws,
                      dppo_workspace_bytes, error_string, version)
