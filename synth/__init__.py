"""Seeded synthetic KV caches shaped like the paper's Llama-class workloads.

This package only draws numbers: it holds none of the method's arithmetic and
is used, unchanged, to feed both the GPU library and the CPU oracle (the same
bytes go to both -- a tensor is generated once and then copied).
"""
from .rng import normal, uniform, hash_u64          # noqa: F401
from .workloads import (Workload, WORKLOADS, make_kv_slab, make_cache, make_query,  # noqa: F401
                        make_new_kv, planted_positions, ragged_lengths, to_numpy, packing,
                        pack_rows, unpack_rows, make_cache_packed)
