"""B200 (sm_100a) kernels for the sampled-GNN training pass of E2E-GRec, behind a C ABI.

``binding`` mirrors the entry points of ``include/e2egrec.h`` one to one; it only
marshals arguments (torch tensors supply device memory and the stream).
"""
from .binding import (  # noqa: F401
    csr_transpose, edge_cumulate, graph_from_coo, lightgcn_backward, lightgcn_forward, lightgcn_sampled_backward, lightgcn_sampled_forward,
    aggregate_backward, aggregate_forward, aggregate_forward_static, aggregate_forward_static_limit,
    BF16, F32, Blocks, JointStep, E2EGrecError, launch_count, lib, profile_tap, sample_join, sample_khop, blocks_transpose, sample_khop_workspace, sampler_scratch_init, sampler_set_step,
    sage_backward, sage_backward_multi, sage_ctx_views, sage_forward, status_string, ssl_loss, gradient_norm, gradient_norms, gradnorm_update, gate_fusion_forward, gate_fusion_backward,
)
