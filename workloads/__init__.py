"""Seeded synthetic inputs shared by the tests, the bench and the CPU oracle's callers.

This module holds no arithmetic of the method itself (no packing, no RoPE, no
attention): it only draws prompt lengths and N(0,1) Q/K/V tensors for the five
workload shapes, so that the CUDA path and the oracle can be fed identical values
without sharing any code.
"""
from .configs import (CONFIGS, WorkloadConfig, get_config, prompt_lengths,
                      draw_lengths, make_qkv, split_by_prompt)

__all__ = ["CONFIGS", "WorkloadConfig", "get_config", "prompt_lengths",
           "draw_lengths", "make_qkv", "split_by_prompt"]
