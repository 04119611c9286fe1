"""The five benchmark workloads and the recipe that fills them.

Recipe (stated once, used everywhere):
  K[b,l,h,t,d] = round_dtype( z * c_K[l,h,d] * a[b,l,h,t] ),   z ~ N(0,1)
  V[b,l,h,t,d] = round_dtype( z' * c_V[l,h,d] ),               z' ~ N(0,1)
  c = exp(0.5 * N(0,1)) per (l,h,d) channel                     (lognormal(0, 0.5))
  a = 0.1 for t = 0 and for a Bernoulli(1 %) draw per token     (low-norm keys),
      `planted_scale` for `planted` seeded positions per head,  (must survive)
      1 otherwise
  q ~ N(0,1) per (step, b, l, hq); appended K/V rows follow the same law.
The low-norm first token and sprinkling of low-norm tokens mirror what the
paper reports for real key caches (Section 3: the start-of-sequence and
punctuation keys have a much lower norm); peaked per-channel scales mirror its
Section 6 observation of a few dominant key dimensions.
"""
from dataclasses import dataclass, replace

import numpy as np
import torch

from . import rng

_TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16}

# stream ids of the counter-based generator
_S_K, _S_V, _S_CK, _S_CV, _S_LOW, _S_PLANT, _S_LEN = 0, 1, 2, 3, 4, 5, 6
_S_Q, _S_KNEW, _S_VNEW, _S_LOWNEW = 100, 101, 102, 103   # + 8 * step


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    L: int
    Hkv: int
    Hq: int
    D: int
    T: int                      # context length (maximum, when ragged)
    dtype: str                  # "f32" | "bf16"
    keep_ratio: float
    uncompressed: tuple = ()
    decode_steps: int = 1
    seed: int = 0
    planted: int = 0
    planted_scale: float = 0.05
    ragged_lo: int = 0          # > 0: lengths uniform in [ragged_lo, T]
    append_steps: int = 0       # > 0: budget-maintained serving loop

    @property
    def torch_dtype(self):
        return _TORCH_DT[self.dtype]

    @property
    def elem_bytes(self):
        return 2 if self.dtype == "bf16" else 4

    def scaled(self, **kw):
        return replace(self, **kw)


WORKLOADS = (
    Workload("tiny", 1, 1, 4, 4, 64, 1024, "f32", 0.5, (), 1, seed=0),
    Workload("llama2-7b-4k", 1, 32, 32, 32, 128, 4096, "bf16", 0.5, (), 1, seed=1),
    Workload("llama3-8b-32k", 4, 32, 8, 32, 128, 32768, "bf16", 0.5, (0, 1), 64, seed=2),
    Workload("extreme-128k", 1, 32, 8, 32, 128, 131072, "bf16", 0.1, (0, 1), 64, seed=3,
             planted=50),
    Workload("serving-ragged", 64, 32, 8, 32, 128, 16384, "bf16", 0.5, (0, 1), 256, seed=4,
             ragged_lo=1024, append_steps=256),
)


def ragged_lengths(w: Workload):
    """Per-sequence context lengths (host int32 array)."""
    if w.ragged_lo <= 0:
        return np.full(w.B, w.T, dtype=np.int32)
    u = rng.uniform(w.seed, _S_LEN, 0, w.B, "cpu").double().numpy()
    return (w.ragged_lo + np.floor(u * (w.T - w.ragged_lo + 1))).astype(np.int32)


def _channel_scale(w, stream, l, device):
    n = w.Hkv * w.D
    z = rng.normal(w.seed, stream, l * n, n, device)
    return torch.exp(0.5 * z).view(w.Hkv, 1, w.D)


def planted_positions(w: Workload, b, l, device="cpu"):
    """[Hkv, planted] distinct seeded positions per head (one per stratum of T // planted)."""
    if w.planted <= 0:
        return torch.zeros((w.Hkv, 0), dtype=torch.int64, device=device)
    stride = w.T // w.planted
    n = w.Hkv * w.planted
    h = rng.hash_u64(w.seed, _S_PLANT, (b * w.L + l) * n, n, device)
    off = (h & 0x7FFFFFFF) % stride
    base = torch.arange(w.planted, dtype=torch.int64, device=device) * stride
    return off.view(w.Hkv, w.planted) + base


def _token_scale(w, b, l, device):
    n = w.Hkv * w.T
    u = rng.uniform(w.seed, _S_LOW, (b * w.L + l) * n, n, device).view(w.Hkv, w.T)
    a = torch.where(u < 0.01, 0.1, 1.0).to(torch.float32)
    a[:, 0] = 0.1
    if w.planted > 0:
        a.scatter_(1, planted_positions(w, b, l, device),
                   torch.full((w.Hkv, w.planted), w.planted_scale, device=device))
    return a.view(w.Hkv, w.T, 1)


def make_kv_slab(w: Workload, which, b, l, device):
    """One (b, l) slab [Hkv, T, D] of K (which='K') or V (which='V')."""
    n = w.Hkv * w.T * w.D
    start = (b * w.L + l) * n
    z = rng.normal(w.seed, _S_K if which == "K" else _S_V, start, n, device).view(w.Hkv, w.T, w.D)
    z = z * _channel_scale(w, _S_CK if which == "K" else _S_CV, l, device)
    if which == "K":
        z = z * _token_scale(w, b, l, device)
    return z.to(w.torch_dtype)


def make_cache(w: Workload, device, t_cap=None):
    """K, V as [B, L, Hkv, t_cap, D]; rows past T are zero."""
    t_cap = w.T if t_cap is None else t_cap
    shape = (w.B, w.L, w.Hkv, t_cap, w.D)
    K = torch.zeros(shape, dtype=w.torch_dtype, device=device)
    V = torch.zeros(shape, dtype=w.torch_dtype, device=device)
    for b in range(w.B):
        for l in range(w.L):
            K[b, l, :, : w.T] = make_kv_slab(w, "K", b, l, device)
            V[b, l, :, : w.T] = make_kv_slab(w, "V", b, l, device)
    return K, V


def make_query(w: Workload, step, device):
    """One decode query per head: [B, L, Hq, D]."""
    n = w.B * w.L * w.Hq * w.D
    z = rng.normal(w.seed, _S_Q + 8 * step, 0, n, device)
    return z.view(w.B, w.L, w.Hq, w.D).to(w.torch_dtype)


def make_new_kv(w: Workload, step, device):
    """The K and V rows appended at a decode step: each [B, L, Hkv, D]."""
    n = w.B * w.L * w.Hkv
    shape = (w.B, w.L, w.Hkv, w.D)
    ck = torch.stack([_channel_scale(w, _S_CK, l, device).view(w.Hkv, w.D) for l in range(w.L)])
    cv = torch.stack([_channel_scale(w, _S_CV, l, device).view(w.Hkv, w.D) for l in range(w.L)])
    a = torch.where(rng.uniform(w.seed, _S_LOWNEW + 8 * step, 0, n, device) < 0.01, 0.1, 1.0)
    k = rng.normal(w.seed, _S_KNEW + 8 * step, 0, n * w.D, device).view(shape)
    v = rng.normal(w.seed, _S_VNEW + 8 * step, 0, n * w.D, device).view(shape)
    k = k * ck.unsqueeze(0) * a.view(w.B, w.L, w.Hkv, 1)
    v = v * cv.unsqueeze(0)
    return k.to(w.torch_dtype), v.to(w.torch_dtype)


def packing(caps):
    """Row ranges of a packed (unpadded) cache.  caps [B, L]: rows that (b, l) may hold.  The
    ranges lie back to back in (b, l) order on one row axis shared by all sequences and layers:
    returns (row_off int64 [B, L], row_cap int32 [B, L], total_rows)."""
    caps = np.asarray(caps, dtype=np.int64)
    flat = caps.reshape(-1)
    off = np.concatenate([[0], np.cumsum(flat)[:-1]]).reshape(caps.shape)
    return off.astype(np.int64), caps.astype(np.int32), int(flat.sum())


def pack_rows(dense, rows, n_rows=None):
    """Dense [B, L, H, T, ...] (numpy or torch) -> packed [H, total_rows, ...]: the first
    n_rows[b, l] (default: the capacity) rows of every (b, l) copied to its range."""
    off, cap, total = rows
    B, L, H = dense.shape[:3]
    n_rows = cap if n_rows is None else np.broadcast_to(np.asarray(n_rows), (B, L))
    if torch.is_tensor(dense):
        out = torch.zeros((H, total) + tuple(dense.shape[4:]), dtype=dense.dtype, device=dense.device)
    else:
        out = np.zeros((H, total) + tuple(dense.shape[4:]), dtype=dense.dtype)
    for b in range(B):
        for l in range(L):
            n = int(n_rows[b, l])
            out[:, int(off[b, l]):int(off[b, l]) + n] = dense[b, l, :, :n]
    return out


def unpack_rows(packed, rows, B, L, t_cap):
    """Packed [H, total_rows, ...] -> dense [B, L, H, t_cap, ...] (rows past a range's capacity
    stay zero)."""
    off, cap, total = rows
    H = packed.shape[0]
    if torch.is_tensor(packed):
        out = torch.zeros((B, L, H, t_cap) + tuple(packed.shape[2:]), dtype=packed.dtype,
                          device=packed.device)
    else:
        out = np.zeros((B, L, H, t_cap) + tuple(packed.shape[2:]), dtype=packed.dtype)
    for b in range(B):
        for l in range(L):
            n = min(int(cap[b, l]), t_cap)
            out[b, l, :, :n] = packed[:, int(off[b, l]):int(off[b, l]) + n]
    return out


def make_cache_packed(w: Workload, lens, device):
    """K, V of a ragged batch without padding: [Hkv, total_rows, D], the rows of (b, l) being the
    first lens[b] tokens of the slab make_cache would give it.  Returns (K, V, rows)."""
    rows = packing(np.repeat(np.asarray(lens, dtype=np.int64)[:, None], w.L, axis=1))
    off, _, total = rows
    K = torch.zeros((w.Hkv, total, w.D), dtype=w.torch_dtype, device=device)
    V = torch.zeros_like(K)
    for b in range(w.B):
        n = int(lens[b])
        for l in range(w.L):
            o = int(off[b, l])
            K[:, o:o + n] = make_kv_slab(w, "K", b, l, device)[:, :n]
            V[:, o:o + n] = make_kv_slab(w, "V", b, l, device)[:, :n]
    return K, V, rows


def to_numpy(t):
    """Host copy of a tensor as the oracle wants it: bf16 becomes its uint16 bit pattern."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()
