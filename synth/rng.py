"""Stateless counter-based random numbers built from torch integer ops.

value(seed, stream, index) depends on nothing else, so any tensor (or any slice of one) can be
regenerated on demand, on the CPU or on a CUDA device, with identical integer results.  Normal
variates use the Box-Muller transform evaluated in float64; after rounding to float32 or bfloat16
CPU and CUDA agree except when a float64 result sits within an ulp of a rounding boundary
(probability ~1e-8 per element for float32, ~1e-13 for bfloat16).
"""
import math
import torch

_MASK = (1 << 64) - 1


def _to_i64(x: int) -> int:
    x &= _MASK
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLD = _to_i64(0x9E3779B97F4A7C15)
_M1 = _to_i64(0xBF58476D1CE4E5B9)
_M2 = _to_i64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, n: int) -> torch.Tensor:
    """Logical right shift of int64 lanes (torch's >> is arithmetic)."""
    return (z >> n) & ((1 << (64 - n)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output function (Steele, Lea, Flood 2014) on wrapping int64 lanes."""
    z = z + _GOLD
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _mix64_int(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def stream_key(seed: int, stream: int) -> int:
    """64-bit key of one random stream (one tensor, one prompt, ...)."""
    return _mix64_int(_mix64_int(seed & _MASK) ^ ((stream * 0xD6E8FEB86659FD93) & _MASK))


def hash_u64(seed: int, stream: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """int64 tensor holding the 64 hash bits of elements start..start+count-1 of a stream."""
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix64(idx * _M2 + _to_i64(stream_key(seed, stream)))


def uniform_ids(seed: int, stream: int, count: int, high: int, device="cpu") -> torch.Tensor:
    """count integers uniform in [0, high) (int32).  high <= 2**31."""
    bits = _lsr(hash_u64(seed, stream, 0, count, device), 33)          # 31 random bits
    return ((bits * high) >> 31).to(torch.int32)


def normal_(out: torch.Tensor, seed: int, stream: int, std: float, chunk: int = 0) -> torch.Tensor:
    """Fill `out` (any float dtype, contiguous) with std * N(0,1), element i = f(seed, stream, i)."""
    flat = out.view(-1)
    n = flat.numel()
    if chunk <= 0:
        chunk = (1 << 25) if out.is_cuda else (1 << 22)
    two_pi = 2.0 * math.pi
    for s in range(0, n, chunk):
        c = min(chunk, n - s)
        bits = hash_u64(seed, stream, s, c, out.device)
        u1 = (_lsr(bits, 32).to(torch.float64) + 1.0) * (1.0 / 4294967296.0)      # (0, 1]
        u2 = (bits & 0xFFFFFFFF).to(torch.float64) * (1.0 / 4294967296.0)         # [0, 1)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(two_pi * u2)
        flat[s:s + c] = (std * z).to(out.dtype)
    return out
