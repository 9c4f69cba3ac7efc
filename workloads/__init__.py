"""Seeded synthetic inputs for the tree-verification step.

This module only *draws inputs*: trees (parent arrays), candidate-path rows,
tokens, Q/K/V and logits with the shapes of the paper's workloads (node
budgets 16-256 and depth 4-16 of Table 2, accepted lengths like Table 1's
accept_L row).  It holds none of the method's arithmetic - no mask, no
ancestor table, no attention, no argmax, no acceptance - and is the only code
shared by the CPU oracle's tests and the CUDA path's tests and bench.
"""
from .configs import CONFIGS, VerifyConfig, get_config
from .trees import (random_parent_tree, topk_expansion_tree, spine_tree, covering_chains_tree, chain_tree, star_tree, leaf_paths,
                    capped_paths)
from .cases import make_case, case_to_numpy, bf16_bits, bits_to_f32, randn_bf16

__all__ = [
    "CONFIGS", "VerifyConfig", "get_config",
    "random_parent_tree", "topk_expansion_tree", "spine_tree", "covering_chains_tree", "chain_tree", "star_tree",
    "leaf_paths", "capped_paths", "make_case", "case_to_numpy", "bf16_bits", "bits_to_f32", "randn_bf16",
]
