"""Seeded synthetic inputs and workload shapes shared by the CPU oracle and the CUDA library.

This package holds no arithmetic of the method: only random draws, tensor shapes and
network descriptions.  Neither the oracle nor the CUDA library lives here.
"""
from .workloads import (  # noqa: F401
    Net,
    config_net,
    gaussian_like_int8,
    gemm_operands,
    gemm_grad_operands,
    he_like_exponent,
    make_net_inputs,
    make_step_batch,
    uniform_int8,
    GEMM_SWEEP_DIMS,
)
