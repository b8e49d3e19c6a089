"""Random-initialised weights: every linear, embedding and bias entry ~ N(0, 0.02), norm gains 1 (or, on request, random).

Each tensor is its own random stream (keyed by its name), so single tensors or layers can be
regenerated on demand without holding a whole model.  All matrices are row-major [out][in].
"""
import zlib
from typing import Dict, List, Optional
import torch
from .configs import ModelCfg, HeadCfg
from .rng import normal_

STD = 0.02


def _layer_shapes(prefix: str, m: ModelCfg) -> Dict[str, tuple]:
    d, f = m.d_model, m.d_ffn
    return {
        prefix + "attn_norm": (d,), prefix + "wqkv": (3 * d, d), prefix + "wo": (d, d),
        prefix + "ffn_norm": (d,), prefix + "w_gate_up": (2 * f, d), prefix + "w_down": (d, f),
    }


def weight_shapes(m: ModelCfg, h: HeadCfg) -> Dict[str, tuple]:
    """Name -> shape of every tensor of the base model, the prefix layer and the Hydra heads."""
    d = m.d_model
    s = {"embed": (m.vocab, d), "lm_head": (m.vocab, d), "final_norm": (d,)}
    for l in range(m.n_layers):
        s.update(_layer_shapes(f"L{l}.", m))
    if h.prefix_attn:
        s.update(_layer_shapes("P.", m))
    for i in range(1, h.n_heads + 1):
        # input = [hidden ; E(x_t) ; E of the i-1 speculated tokens], or the hidden state alone for sequentially independent heads
        s[f"H{i}.w1"] = (d, d if h.medusa else (i + 1) * d)
        s[f"H{i}.b1"] = (d,)
        if h.n_mlp_layers > 1:
            s[f"H{i}.wr"] = (h.n_mlp_layers - 1, d, d)
            s[f"H{i}.br"] = (h.n_mlp_layers - 1, d)
    return s


def weight_names(m: ModelCfg, h: HeadCfg) -> List[str]:
    return list(weight_shapes(m, h).keys())


def make_tensor(m: ModelCfg, h: HeadCfg, seed: int, name: str, device="cpu", norm_gain_std: float = 0.0) -> torch.Tensor:
    """norm_gain_std > 0 draws every norm gain as 1 + norm_gain_std * N(0,1) from the tensor's own stream (parity
    tests use it so that each norm's gain vector is distinguishable); the benchmark shapes keep gains of 1."""
    shape = weight_shapes(m, h)[name]
    dtype = torch.float32 if m.dtype == "fp32" else torch.bfloat16
    if name.endswith("norm"):
        if norm_gain_std > 0.0:
            g = normal_(torch.empty(shape, dtype=torch.float64, device=device), seed, zlib.crc32(name.encode()), norm_gain_std)
            return (1.0 + g).to(dtype)
        return torch.ones(shape, dtype=dtype, device=device)
    out = torch.empty(shape, dtype=dtype, device=device)
    if not h.has_bias and (name.endswith(".b1") or name.endswith(".br")):
        return out.zero_()
    return normal_(out, seed, zlib.crc32(name.encode()), STD)


def make_weights(m: ModelCfg, h: HeadCfg, seed: int, device="cpu", names: Optional[List[str]] = None,
                 norm_gain_std: float = 0.0):
    names = weight_names(m, h) if names is None else names
    return {n: make_tensor(m, h, seed, n, device, norm_gain_std) for n in names}
