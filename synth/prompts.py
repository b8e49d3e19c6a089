"""Synthetic prompts: token ids uniform in [0, vocab), one random stream per sequence."""
from typing import List
import torch
from .rng import uniform_ids


def make_prompts(seed: int, lens: List[int], vocab: int) -> List[torch.Tensor]:
    return [uniform_ids(seed, 5000 + b, n, vocab) for b, n in enumerate(lens)]
