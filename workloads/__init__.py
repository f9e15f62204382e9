"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke run.

Holds the workload definitions (shapes, placements, block tables) and the
counter-based value streams.  It contains none of the re-layout arithmetic and
imports neither the CUDA package nor the CPU oracle.
"""
from .configs import (MASTER_SEED, KIND_ATTN, KIND_EXPERTS, KIND_KV, ParallelConfig, Shape,
                      Workload, WORKLOAD_NAMES, EXTRA_WORKLOAD_NAMES, arena_key, make_block_table, make_seq_lens,
                      make_exchange_workload, make_workload, place_contiguous, place_hot_replicated, place_round_robin,
                      small_variant, with_shared, zipf_load)
from . import rng

__all__ = [n for n in dir() if not n.startswith("_")]
