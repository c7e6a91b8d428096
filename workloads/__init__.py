"""Synthetic parameter sets and seeded gradient generators.

This package serves both the CPU oracle's tests and the CUDA path's tests and
benchmark.  It holds tensor shapes and random-number recipes only: none of the
optimizer's arithmetic lives here, and it imports neither the oracle nor the
CUDA binding.
"""
from .shapes import (  # noqa: F401
    ROLE_EMBED, ROLE_Q, ROLE_K, ROLE_V, ROLE_QKV_FUSED, ROLE_ATTN_OUT, ROLE_MLP,
    ROLE_LM_HEAD, ROLE_VECTOR, ROLE_OTHER, Tensor, Workload, get_workload,
    WORKLOAD_NAMES,
)
from .gen import init_params, grad_for_tensor, to_grad_dtype, GradPool, bf16_bits_to_f32, round_to_bf16_bits  # noqa: F401
