"""GPU parity of the per-head calls: a keep count per (b, l, h) in compression and a cache
length per (b, l, kv head) in decode attention, against the CPU oracle on the same bytes.
Bars as in the per-sequence tests: index maps, rows and stored keys bit-exact against the
oracle on the fp32 key order; attention within |err| <= 2e-3 + 1e-2 |ref|."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import DEV, i32, assert_attention_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def l2():
    import paper_2406_11430_b200 as lib
    lib.lib()
    return lib


def gpu_compress_per_head(l2, K, V, lens, keep, unc=(), policy=0, t_cap_out=None, seed=0):
    B, L, H, T_cap, D = K.shape
    t_cap_out = T_cap if t_cap_out is None else t_cap_out
    max_len = int(max(lens))
    K_c = torch.zeros((B, L, H, t_cap_out, D), dtype=K.dtype, device=K.device)
    V_c = torch.zeros_like(K_c)
    idx = torch.full((B, L, H, t_cap_out), -1, dtype=torch.int32, device=K.device)
    sumsq = torch.full((B, L, H, t_cap_out), float("nan"), dtype=torch.float32, device=K.device)
    kept = torch.full((B, L, H), -7, dtype=torch.int32, device=K.device)
    ws = l2.new_workspace(l2.Layout(K), max_len, K.device)
    l2.select_compact_per_head(K, V, i32(lens), i32(keep), max_len, unc, K_c, V_c, idx, sumsq,
                               kept, ws, policy=policy, seed=seed)
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    dev = dict(K_c=K_c, V_c=V_c, idx=idx, sumsq=sumsq, kept_len=kept)
    return dev, {k: synth.to_numpy(v) for k, v in dev.items()}


def random_keep(rng, lens, L, H):
    keep = np.stack([rng.integers(0, n + 1, size=(L, H)) for n in lens]).astype(np.int32)
    return keep


@pytest.mark.parametrize("dtype,D,policy", [("bf16", 128, 0), ("f32", 64, 0), ("bf16", 64, 1),
                                            ("bf16", 128, 2)])
def test_compress_per_head_counts(l2, dtype, D, policy):
    w = synth.WORKLOADS[2].scaled(dtype=dtype, D=D, B=2, L=3, Hkv=4, Hq=8, T=2100)
    K, V = synth.make_cache(w, DEV)
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    lens = [2100, 613]
    keep = random_keep(np.random.default_rng(5), lens, w.L, w.Hkv)
    keep[0, 0, 0], keep[0, 0, 1], keep[1, 2, 3], keep[0, 2, 2] = 0, 2100, 613, 1
    _, got = gpu_compress_per_head(l2, K, V, lens, keep, unc=(1,), policy=policy, seed=99)
    want = oracle.compress(Kn, Vn, dtype, lens, keep, (1,), key_mode=1, policy=policy,
                           nthreads=8, seed=99)
    assert np.array_equal(got["kept_len"], want["kept_len"])
    assert np.array_equal(got["idx"], want["idx"])
    assert np.array_equal(got["K_c"], want["K_c"])
    assert np.array_equal(got["V_c"], want["V_c"])
    assert np.array_equal(got["sumsq"].astype(np.float64), want["key"], equal_nan=True)


def test_compress_per_head_output_shorter_than_input(l2):
    w = synth.WORKLOADS[2].scaled(B=1, L=2, Hkv=2, Hq=8, T=1500)
    K, V = synth.make_cache(w, DEV)
    keep = np.array([[[700, 1], [350, 699]]], dtype=np.int32)
    _, got = gpu_compress_per_head(l2, K, V, [1500], keep, t_cap_out=704)
    want = oracle.compress(synth.to_numpy(K), synth.to_numpy(V), "bf16", [1500], keep,
                           key_mode=1, t_cap_out=704, nthreads=8)
    for k in ("kept_len", "idx", "K_c", "V_c"):
        assert np.array_equal(got[k], want[k])


@pytest.mark.parametrize("dtype,D,Hkv,Hq", [("bf16", 128, 2, 8), ("bf16", 128, 4, 4),
                                            ("f32", 64, 2, 4), ("bf16", 64, 1, 8)])
def test_attention_with_a_length_per_head(l2, dtype, D, Hkv, Hq):
    w = synth.WORKLOADS[2].scaled(dtype=dtype, D=D, Hkv=Hkv, Hq=Hq, B=2, L=2, T=2600)
    K, V = synth.make_cache(w, DEV)
    q = synth.make_query(w, 0, DEV)
    rng = np.random.default_rng(3)
    cur = rng.integers(0, 2601, size=(2, 2, Hkv)).astype(np.int32)
    cur.flat[0], cur.flat[-1] = 2600, 0
    if Hkv > 1:
        cur[0, 1, 1], cur[1, 0, 0] = 1, 1025
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    ws = l2.new_workspace(l2.Layout(K, q_heads=Hq), 2600, DEV)
    l2.decode_attention_per_head(q, K, V, i32(cur), 2600, out, ws)
    torch.cuda.synchronize()
    want = oracle.attention(synth.to_numpy(q), synth.to_numpy(K), synth.to_numpy(V), dtype, cur,
                            nthreads=8)
    got = out.cpu().numpy()
    assert_attention_close(got, want)
    G = Hq // Hkv
    assert not got[1, 1, (Hkv - 1) * G:].any()           # empty head -> zeros


def test_per_head_pipeline_compress_then_attend(l2):
    """Per-head lengths written by the compression feed the attention call directly."""
    w = synth.WORKLOADS[2].scaled(B=1, L=2, Hkv=2, Hq=8, T=3000)
    K, V = synth.make_cache(w, DEV)
    q = synth.make_query(w, 0, DEV)
    keep = np.array([[[3000, 40], [1500, 2999]]], dtype=np.int32)
    dev, got = gpu_compress_per_head(l2, K, V, [3000], keep)
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    ws = l2.new_workspace(l2.Layout(K, q_heads=8), 3000, DEV)
    l2.decode_attention_per_head(q, dev["K_c"], dev["V_c"], dev["kept_len"], 3000, out, ws)
    torch.cuda.synchronize()
    ref = oracle.compress(synth.to_numpy(K), synth.to_numpy(V), "bf16", [3000], keep, key_mode=1,
                          nthreads=8)
    want = oracle.attention(synth.to_numpy(q), ref["K_c"], ref["V_c"], "bf16", ref["kept_len"],
                            nthreads=8)
    assert_attention_close(out.cpu().numpy(), want)
