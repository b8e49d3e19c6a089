"""The five benchmark shapes (model, heads, tree, batch, prompt lengths, decode steps)."""
from dataclasses import dataclass, field, asdict
from typing import List


@dataclass
class ModelCfg:
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-6
    rope_theta: float = 1e4
    dtype: str = "bf16"            # "fp32" | "bf16": storage type of the weights
    kv_planes: int = 2             # bf16 path: float16 planes of q and the KV caches (2: hi + lo, 1: hi only)


@dataclass
class HeadCfg:
    n_heads: int                   # K: number of Hydra heads = tree depth
    n_mlp_layers: int              # m: MLP layers per head
    prefix_attn: bool              # Hydra++ extra decoder layer
    has_bias: bool = True
    medusa: bool = False           # sequentially independent heads: head i sees the hidden state only (the Medusa baseline)


@dataclass
class RunCfg:
    name: str
    model: ModelCfg
    head: HeadCfg
    tree: str                      # name of a committed tree file
    batch: int
    prompt_lens: List[int]
    steps: int
    seed: int
    max_seq: int


def _ragged(seed, batch, lo, hi):
    from .rng import uniform_ids
    return [int(lo + v) for v in uniform_ids(seed, 9000 + batch, batch, hi - lo + 1)]


_7B = dict(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ffn=11008, vocab=32000)
_13B = dict(n_layers=40, d_model=5120, n_heads=40, head_dim=128, d_ffn=13824, vocab=32000)
_33B = dict(n_layers=60, d_model=6656, n_heads=52, head_dim=128, d_ffn=17920, vocab=32000)
_PP = dict(n_heads=4, n_mlp_layers=4, prefix_attn=True)


def get_config(name: str) -> RunCfg:
    if name == "c1":
        return RunCfg("c1", ModelCfg(2, 256, 4, 64, 688, 1024, dtype="fp32"), HeadCfg(3, 1, False),
                      "tree15_d3", 1, [32], 8, 0, 128)
    if name == "c2":
        return RunCfg("c2", ModelCfg(**_7B), HeadCfg(**_PP), "tree63_d4", 1, [512], 128, 1, 512 + 128 * 5 + 64)
    if name == "c2s":          # c2 cut to 4 layers (1.9 GB of weights): the small case for profiler captures
        return RunCfg("c2s", ModelCfg(**dict(_7B, n_layers=4)), HeadCfg(**_PP), "tree63_d4", 1, [512], 16, 1, 512 + 16 * 5 + 64)
    if name.startswith("c3"):
        small = name.endswith("s")                         # "c3b8s": cut to 4 layers, the small case for profiler captures
        b = int(name[3:].rstrip("s")) if len(name) > 2 else 8          # "c3b1", "c3b2", "c3b4", "c3b8"
        return RunCfg(name, ModelCfg(**dict(_7B, n_layers=4 if small else 32)), HeadCfg(**_PP), "tree63_d4", b, _ragged(2, b, 128, 1024),
                      16 if small else 64, 2, 1024 + 64 * 5 + 64)
    if name == "c4s":          # c4 cut to 4 layers: the small case for profiler captures of the long-cache attention
        return RunCfg("c4s", ModelCfg(**dict(_13B, n_layers=4)), HeadCfg(**_PP), "tree63_d4", 1, [2048], 16, 3, 2048 + 16 * 5 + 64)
    if name == "c4":
        return RunCfg("c4", ModelCfg(**_13B), HeadCfg(**_PP), "tree63_d4", 1, [2048], 64, 3, 2048 + 64 * 5 + 64)
    if name == "c5":
        return RunCfg("c5", ModelCfg(**_33B), HeadCfg(**_PP), "tree63_d4", 4, [1024] * 4, 64, 4, 1024 + 64 * 5 + 64)
    raise KeyError(name)


CONFIGS = ["c1", "c2", "c3b1", "c3b2", "c3b4", "c3b8", "c4", "c5"]
