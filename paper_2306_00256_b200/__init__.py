"""DSGD-CECA hot path on one NVIDIA B200: thin Python binding of the C-ABI library.

Every function here only marshals arguments (pointers, sizes, the current CUDA stream) into
``libceca_b200.so``; all arithmetic runs in the library's CUDA kernels.  There is no CPU
fallback: if the library is missing it is built with nvcc, and if that fails the import
of the symbol fails loudly.
"""
from .binding import (CECA_1P, CECA_2P, FUSED_AUTO, FUSED_BLOCK, FUSED_SMEM, FUSED_TMEM, UNFUSED, CecaError, Round, WS_CONSENSUS_FUSED, WS_CONSENSUS_UNFUSED,
                      WS_LOGREG_GRAD, WS_STEP_HOST, ceca_consensus_rounds, ceca_gossip_sgd_step,
                      ceca_fused_wait_selftest, ceca_gossip_sgd_step_bf16, ceca_gossip_sgd_step_host, ceca_read_status, ceca_schedule, ceca_status_string,
                      ceca_workspace_bytes, dsgd_grad_shard_apply, dsgd_grad_shard_dots, dsgd_grad_shard_sum, dsgd_logreg_grad, dsgd_logreg_grad_static, shard_columns,
                      dsgd_logreg_grad_static_capacity, dsgd_lsq_grad, library, library_path)

__all__ = ["CECA_1P", "CECA_2P", "FUSED_AUTO", "FUSED_BLOCK", "FUSED_SMEM", "FUSED_TMEM", "UNFUSED", "ceca_fused_wait_selftest", "ceca_gossip_sgd_step_bf16", "CecaError", "Round", "WS_CONSENSUS_FUSED", "WS_CONSENSUS_UNFUSED",
           "WS_LOGREG_GRAD", "WS_STEP_HOST", "ceca_consensus_rounds", "ceca_gossip_sgd_step",
           "ceca_gossip_sgd_step_host", "ceca_read_status", "ceca_schedule", "ceca_status_string",
           "ceca_workspace_bytes", "dsgd_grad_shard_apply", "dsgd_grad_shard_dots", "dsgd_grad_shard_sum", "shard_columns", "dsgd_logreg_grad", "dsgd_logreg_grad_static",
           "dsgd_logreg_grad_static_capacity", "dsgd_lsq_grad", "library", "library_path"]
