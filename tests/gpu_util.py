"""Helpers shared by the GPU parity tests: run the library through its C ABI on
torch tensors and bring everything back as numpy for comparison with the oracle."""
import numpy as np
import torch

import synth

DEV = "cuda:0"


def i32(x, device=DEV):
    return torch.tensor(np.asarray(x, dtype=np.int32), dtype=torch.int32, device=device)


def gpu_compress(l2, K, V, lens, keep, unc=(), policy=0, t_cap_out=None, max_len=None, seed=0,
                 sumsq_in=None):
    """K, V: device tensors [B, L, H, T_cap, D].  Returns (device dict, numpy dict)."""
    B, L, H, T_cap, D = K.shape
    t_cap_out = T_cap if t_cap_out is None else t_cap_out
    max_len = int(max(lens)) if max_len is None else max_len
    K_c = torch.zeros((B, L, H, t_cap_out, D), dtype=K.dtype, device=K.device)
    V_c = torch.zeros_like(K_c)
    idx = torch.full((B, L, H, t_cap_out), -1, dtype=torch.int32, device=K.device)
    sumsq = torch.full((B, L, H, t_cap_out), float("nan"), dtype=torch.float32, device=K.device)
    kept_len = torch.zeros((B, L), dtype=torch.int32, device=K.device)
    ws = l2.new_workspace(l2.Layout(K), max_len, K.device)
    l2.select_compact(K, V, i32(lens), i32(keep), max_len, unc, K_c, V_c, idx, sumsq,
                      kept_len, ws, policy=policy, seed=seed, sumsq_in=sumsq_in)
    torch.cuda.synchronize()
    dev = dict(K_c=K_c, V_c=V_c, idx=idx, sumsq=sumsq, kept_len=kept_len)
    host = {k: synth.to_numpy(v) for k, v in dev.items()}
    return dev, host


def gpu_attention(l2, q, K_c, V_c, cur_len, max_len=None, scale=0.0):
    B, L, H, T_cap, D = K_c.shape
    cur = cur_len if torch.is_tensor(cur_len) else i32(np.asarray(cur_len).reshape(B, L))
    max_len = T_cap if max_len is None else max_len
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=q.device)
    ws = l2.new_workspace(l2.Layout(K_c, q_heads=q.shape[2]), max_len, q.device)
    l2.decode_attention(q, K_c, V_c, cur, max_len, out, ws, scale=scale)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def assert_attention_close(got, want, atol=2e-3, rtol=1e-2):
    """|got - want| <= 2e-3 + 1e-2 |want| element-wise (bf16 inputs, fp32 accumulation)."""
    err = np.abs(got.astype(np.float64) - want)
    bound = atol + rtol * np.abs(want)
    assert np.all(err <= bound), f"max err {err.max():.3e}, worst excess {(err - bound).max():.3e}"
    return float(err.max())


def compare_with_band(got_idx, want_idx, key64, keep, band=1e-6):
    """Kept sets must agree except for tokens whose fp64 norm lies within `band`
    (relative) of the oracle's threshold norm.  Returns the number of swaps."""
    got, want = set(got_idx.tolist()), set(want_idx.tolist())
    assert len(got) == keep == len(want)
    if got == want:
        return 0
    norm = np.sqrt(key64)
    thr = np.sort(norm)[keep - 1]
    for t in got ^ want:
        assert abs(norm[t] - thr) <= band * thr, f"token {t} differs outside the tie band"
    return len(got - want)
