"""Seeded synthetic inputs shared by the CPU oracle and the CUDA path.

This package holds model shapes, workload descriptions and the seeded
generators of weights and prompts.  It contains none of the method's
arithmetic: no layer math, no sampling, no scheduling.  Both sides load
the same arrays from here and share nothing else.
"""
from .configs import ModelShape, Workload, CONFIGS, WORKLOADS, get_config  # noqa: F401
from .gen import bf16_round, make_weights, make_prompt, weight_order  # noqa: F401
