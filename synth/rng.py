"""Counter-based random numbers built from plain torch integer ops.

value(seed, stream, i) depends only on its three arguments, so any slab of any
tensor can be drawn on its own, on any device, in any order.  The integer hash
is bit-identical on CPU and GPU; the float transforms (log, cos) may differ in
the last bit between devices, which is why a tensor is always generated once
and copied to wherever else it is needed.
"""
import math

import torch

_MASK = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _signed(x):
    x &= _MASK
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_int(x):
    """splitmix64 finaliser (Steele, Lea, Flood 2014) on a Python int."""
    x &= _MASK
    x = ((x ^ (x >> 30)) * _C1) & _MASK
    x = ((x ^ (x >> 27)) * _C2) & _MASK
    return x ^ (x >> 31)


def _lsr(x, s):
    """Logical shift right of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x):
    """The same finaliser on an int64 tensor (two's-complement arithmetic wraps)."""
    x = (x ^ _lsr(x, 30)) * _signed(_C1)
    x = (x ^ _lsr(x, 27)) * _signed(_C2)
    return x ^ _lsr(x, 31)


def hash_u64(seed, stream, start, count, device):
    """64 hashed bits (as int64) for counters start .. start+count-1 of one stream."""
    key = _mix_int(_mix_int(seed) ^ ((stream + 1) * _GOLD))
    i = torch.arange(start, start + count, dtype=torch.int64, device=device)
    return _mix(i * _signed(_GOLD) + _signed(key))


def uniform(seed, stream, start, count, device):
    """Uniforms in (0, 1), fp32, from the top 24 hashed bits."""
    h = hash_u64(seed, stream, start, count, device)
    return (_lsr(h, 40).to(torch.float32) + 0.5) * (1.0 / (1 << 24))


def normal(seed, stream, start, count, device):
    """Standard normals, fp32, by Box-Muller from two 24-bit uniforms of one hash."""
    h = hash_u64(seed, stream, start, count, device)
    u1 = (_lsr(h, 40).to(torch.float32) + 0.5) * (1.0 / (1 << 24))
    u2 = ((_lsr(h, 16) & 0xFFFFFF).to(torch.float32) + 0.5) * (1.0 / (1 << 24))
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
