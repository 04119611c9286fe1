"""GPU parity of the attention-loss analysis (Eqs. 5-7) against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import DEV, i32

pytestmark = pytest.mark.gpu


def run(l2, q, K, cur, max_len, curves=True):
    B, L, Hkv, T_cap, D = K.shape
    Hq = q.shape[2]
    lens = i32(np.full(B, T_cap))
    sumsq = torch.zeros((B, L, Hkv, T_cap), dtype=torch.float32, device=DEV)
    l2.key_norms(K, lens, T_cap, sumsq)
    alr = torch.full((B, L, Hq), float("nan"), dtype=torch.float32, device=DEV)
    loss = torch.full((B, L, Hq, T_cap), float("nan"), dtype=torch.float32, device=DEV) if curves else None
    ref = torch.full((B, L, Hq, T_cap), float("nan"), dtype=torch.float32, device=DEV) if curves else None
    l2.attention_loss(q, K, i32(np.asarray(cur).reshape(B, L)), max_len, sumsq, alr, loss, ref)
    torch.cuda.synchronize()
    return alr.cpu().numpy(), (loss.cpu().numpy() if curves else None), (ref.cpu().numpy() if curves else None)


@pytest.mark.parametrize("dtype,D,Hkv,Hq,T", [("bf16", 128, 2, 8, 5000), ("f32", 64, 4, 4, 1024),
                                             ("bf16", 64, 2, 2, 4097), ("f32", 128, 1, 2, 700),
                                             ("bf16", 128, 1, 2, 20000), ("bf16", 128, 1, 1, 70000),
                                             ("bf16", 128, 1, 12, 3000), ("f32", 64, 2, 6, 2500),
                                             ("bf16", 128, 1, 3, 33000), ("bf16", 128, 2, 4, 32768)])
def test_attention_loss_matches_oracle(dtype, D, Hkv, Hq, T):
    import paper_2406_11430_b200 as l2
    w = synth.WORKLOADS[2].scaled(dtype=dtype, D=D, Hkv=Hkv, Hq=Hq, B=2, L=2, T=T)
    K, _ = synth.make_cache(w, DEV)
    q = synth.make_query(w, 0, DEV)
    cur = np.array([[T, 1], [0, max(2, T // 3)]], dtype=np.int32)
    alr, loss, ref = run(l2, q, K, cur, T)
    want, wloss, wref = oracle.attention_loss(synth.to_numpy(q), synth.to_numpy(K), dtype, cur,
                                              key_mode=1, curves=True, nthreads=8)
    for b in range(2):
        for l in range(2):
            n = cur[b, l]
            np.testing.assert_allclose(loss[b, l, :, :n], wloss[b, l, :, :n], rtol=0, atol=3e-5)
            np.testing.assert_allclose(ref[b, l, :, :n], wref[b, l, :, :n], rtol=0, atol=3e-5)
            assert np.isnan(loss[b, l, :, n:]).all()                 # untouched past n
            np.testing.assert_allclose(alr[b, l], want[b, l], rtol=2e-4, atol=1e-4 * max(n, 1))
    assert np.all(alr[1, 0] == 0.0) and np.all(alr[0, 1] == 0.0)      # empty / one-token caches
    assert np.all(alr >= -1e-3)


def test_attention_loss_planted_structure():
    # Keys whose norm falls exactly as their score rises lose nothing against the ideal.
    import paper_2406_11430_b200 as l2
    n, D = 3000, 128
    K = torch.zeros((1, 1, 1, n, D), dtype=torch.float32, device=DEV)
    K[0, 0, 0, :, 0] = torch.linspace(1.0, 0.0, n, device=DEV)      # score falls with position
    K[0, 0, 0, :, 1] = torch.linspace(1.0, 9.0, n, device=DEV)      # norm rises with position
    q = torch.zeros((1, 1, 1, D), dtype=torch.float32, device=DEV)
    q[..., 0] = 30.0
    alr, _, _ = run(l2, q, K, [[n]], n, curves=False)
    assert abs(alr[0, 0, 0]) < 1e-2
    alr2, _, _ = run(l2, q, K.flip(3).contiguous(), [[n]], n, curves=False)   # same set, other slots
    assert abs(alr2[0, 0, 0]) < 1e-2
    # the opposite pairing (highest norm = highest score) is the worst case: loss well above 0
    K[0, 0, 0, :, 1] = torch.linspace(9.0, 1.0, n, device=DEV)
    alr3, _, _ = run(l2, q, K, [[n]], n, curves=False)
    assert alr3[0, 0, 0] > 100.0


def test_attention_loss_per_head_lengths_and_packed_cache():
    """A length per (b, l, kv head), and a packed cache: each unit against the oracle run on that
    unit alone (its rows, its length, its query heads)."""
    import paper_2406_11430_b200 as l2
    B, L, Hkv, Hq, D, T = 2, 2, 2, 8, 128, 900
    G = Hq // Hkv
    w = synth.WORKLOADS[2].scaled(B=B, L=L, Hkv=Hkv, Hq=Hq, T=T)
    K, _ = synth.make_cache(w, DEV)
    q = synth.make_query(w, 3, DEV)
    Kn, qn = synth.to_numpy(K), synth.to_numpy(q)

    def unit_oracle(rows, n, qs):
        return oracle.attention_loss(np.ascontiguousarray(qs[None, None]), np.ascontiguousarray(rows[None, None, None]),
                                     "bf16", [[n]], key_mode=1)[0, 0]

    # per-head lengths on the dense cache
    cur = np.array([[[900, 333], [1, 0]], [[512, 777], [64, 899]]], dtype=np.int32)
    lens = i32(np.full(B, T))
    sumsq = torch.zeros((B, L, Hkv, T), dtype=torch.float32, device=DEV)
    l2.key_norms(K, lens, T, sumsq)
    alr = torch.full((B, L, Hq), float("nan"), dtype=torch.float32, device=DEV)
    l2.attention_loss(q, K, i32(cur), T, sumsq, alr, per_head=True)
    torch.cuda.synchronize()
    got = alr.cpu().numpy()
    for b in range(B):
        for l in range(L):
            for h in range(Hkv):
                n = int(cur[b, l, h])
                want = unit_oracle(Kn[b, l, h, :max(n, 1)], n, qn[b, l, h * G:(h + 1) * G])
                np.testing.assert_allclose(got[b, l, h * G:(h + 1) * G], want, rtol=2e-4, atol=1e-4 * max(n, 1))

    # the same cache packed: (b, l) ranges of different sizes on one row axis
    caps = [[900, 400], [64, 700]]
    cur_bl = np.array([[900, 350], [0, 700]], dtype=np.int32)
    off, cap, total = synth.packing(caps)
    rows = l2.Rows(off, cap, total, DEV)
    Kp = torch.zeros((Hkv, total, D), dtype=K.dtype, device=DEV)
    for b in range(B):
        for l in range(L):
            o, c = int(off[b, l]), int(cap[b, l])
            Kp[:, o:o + c] = K[b, l, :, :c]
    ss = torch.zeros((Hkv, total), dtype=torch.float32, device=DEV)
    l2.key_norms(Kp, i32([900, 700]), 900, ss, rows=rows)
    alr2 = torch.full((B, L, Hq), float("nan"), dtype=torch.float32, device=DEV)
    l2.attention_loss(q, Kp, i32(cur_bl), 900, ss, alr2, rows=rows)
    torch.cuda.synchronize()
    got2 = alr2.cpu().numpy()
    for b in range(B):
        for l in range(L):
            n = int(cur_bl[b, l])
            for h in range(Hkv):
                want = unit_oracle(Kn[b, l, h, :max(n, 1)], n, qn[b, l, h * G:(h + 1) * G])
                np.testing.assert_allclose(got2[b, l, h * G:(h + 1) * G], want, rtol=2e-4, atol=1e-4 * max(n, 1))
