"""Seeded synthetic inputs for one verification step of speculative decoding.

This module only draws random tensors and lays them out (paged KV pool, page
table, draft tokens and draft distributions).  It holds none of the arithmetic
of the verification step itself; both the CPU oracle's tests and the CUDA
path's tests feed from it so that the two sides see identical bytes.
"""
from .configs import CONFIGS, VerifyConfig, get_config
from .gen import generate, kv_bytes, PAGE_SIZE

__all__ = ["CONFIGS", "VerifyConfig", "get_config", "generate", "kv_bytes", "PAGE_SIZE"]
