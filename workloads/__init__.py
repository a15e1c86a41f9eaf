"""Seeded synthetic input generators shared by the CPU oracle's tests and the CUDA path's tests/bench.

This package holds input generation only: no table logic, no tree growth, no attention, no acceptance.
Every random value is a pure function of (seed, tensor id, flat index) through a counter-based integer
hash, so any element can be materialised on its own, on the host (numpy, here) or on the device (the
fill kernel in ``workloads/fill.cu`` implements the same integer arithmetic).
"""
from .rng import mix64, normal_i32, normal_f32, normal_bf16_bits, bf16_bits_to_f32, f32_to_bf16_bits, uniform_f64
from .configs import CbConfig, CONFIGS, get_config
from .streams import make_stream, make_streams
from .trees import random_tree
from .tensors import (TID, make_block_table, ctx_lens, pool_slice_kv, pool_pages_bits, pool_full_bits, seq_bits,
                      full_bits, tree_kv, queries, logits_rows, plant_logits)

__all__ = [
    "mix64", "normal_i32", "normal_f32", "normal_bf16_bits", "bf16_bits_to_f32", "f32_to_bf16_bits",
    "uniform_f64", "CbConfig", "CONFIGS", "get_config", "make_stream", "make_streams", "random_tree",
    "TID", "make_block_table", "ctx_lens", "pool_slice_kv", "tree_kv", "queries",
    "logits_rows", "plant_logits", "pool_pages_bits", "pool_full_bits", "seq_bits", "full_bits",
]
