"""Seeded synthetic inputs for the tree-verification path.

This package only *draws* numbers (weights, audio-embedding vectors, token ids,
tree topologies) and converts storage formats.  It contains none of the
decoder's arithmetic, and it is the only code shared by the CPU oracle and the
CUDA path: both are fed the very same arrays.
"""
from .configs import ModelConfig, CONFIGS, get_config
from .bf16 import f32_to_bf16_bits, bf16_bits_to_f32, bf16_bits_to_f64
from .weights import WeightStore, LAYER_TENSORS, GLOBAL_TENSORS
from .inputs import audio_prefix, prompt_tokens, uniform_tokens
from .proposals import CorruptedGreedyProposer
from .trees import (
    chain_tree,
    complete_binary_tree,
    sparse_tree,
    trunk_tree,
    main_path,
    fill_tree_tokens,
    relabel_tree,
)

__all__ = [
    "ModelConfig", "CONFIGS", "get_config",
    "f32_to_bf16_bits", "bf16_bits_to_f32", "bf16_bits_to_f64",
    "WeightStore", "LAYER_TENSORS", "GLOBAL_TENSORS",
    "audio_prefix", "prompt_tokens", "uniform_tokens",
    "chain_tree", "complete_binary_tree", "sparse_tree", "trunk_tree",
    "main_path", "fill_tree_tokens", "relabel_tree",
    "CorruptedGreedyProposer",
]
