"""Seeded synthetic inputs: weights, prompts, candidate trees, planting schedules.

This package only *generates inputs* (random tensors, token ids, tree topologies).  It holds none
of the decoding arithmetic, and both the CPU oracle's tests and the CUDA path's harness draw their
inputs from it so that the two sides see identical data.
"""
from .rng import hash_u64, uniform_ids, normal_
from .configs import CONFIGS, ModelCfg, HeadCfg, get_config
from .trees import grow_tree, load_tree, chain_tree, star_tree, node_score, rank_paths, ALPHA, BETA
from .weights import make_weights, make_tensor, weight_names
from .prompts import make_prompts
from .plant import plant_row, planted_length
