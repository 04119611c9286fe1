"""GPU parity of prefix attention (several new queries over the compressed cache; tensor-core
contractions) against the oracle's single-query attention applied query by query.

Two forms of the weights are tested in every case.  "split": each softmax weight multiplies V
as two bf16 terms (16 significant bits) -- held to the decode path's bound
|err| <= 2e-3 + 1e-2 |ref|.  "single": one rounded bf16 weight (relative error up to 2^-9 per
weight, the usual arrangement of fused attention kernels) -- a documented reading with the
absolute term 4e-3 (the error is largest for caches of a few hundred tokens, where few
weights carry the sum); the RMS error is bounded separately."""
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle
import synth
from gpu_util import DEV, i32, assert_attention_close, gpu_attention

pytestmark = pytest.mark.gpu


def make_queries(w, n_q, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn((w.B, w.L, n_q, w.Hq, w.D), generator=g).to(torch.bfloat16).to(DEV)


WEIGHTS = ["split", "single"]
ATOL = {"split": 2e-3, "single": 4e-3}


def call(l2, weights, q, K, V, cur_dev, max_len, out, lse, scale=0.0, workspace=None, causal=False):
    """Both forms go through the general entry point; "single" without flags is what the plain
    l2kv_prefix_attention / _causal calls do (test_plain_entry_points_are_the_flagless_call)."""
    flags = (l2.PREFIX_SPLIT_WEIGHTS if weights == "split" else 0) | (l2.PREFIX_CAUSAL if causal else 0)
    l2.prefix_attention_flags(q, K, V, cur_dev, max_len, out, flags, lse_out=lse, scale=scale,
                              workspace=workspace)


def run(l2, q, K, V, cur, max_len, scale=0.0, weights="single"):
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full(q.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.zeros(256, dtype=torch.uint8, device=DEV)
    if os.environ.get("L2KV_PREFIX_KERNEL") == "persistent":      # that kernel needs room for cut items
        ws = l2.prefix_attention_workspace(K, q, max_len)
    call(l2, weights, q, K, V, i32(np.asarray(cur)), max_len, out, lse, scale=scale, workspace=ws)
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    return out.cpu().numpy(), lse.cpu().numpy()


# the three kernels, and the library's own choice between them
KERNELS = ["pipelined", "basic", "persistent", "auto"]


def test_plain_entry_points_are_the_flagless_call():
    import paper_2406_11430_b200 as l2
    w = synth.WORKLOADS[2].scaled(B=1, L=2, Hkv=2, Hq=8, T=500)
    K, V = synth.make_cache(w, DEV)
    q = make_queries(w, 33, 5)
    cur = i32(np.array([[500, 77]]))
    for causal, plain in ((False, l2.prefix_attention), (True, l2.prefix_attention_causal)):
        a = torch.empty(q.shape, dtype=torch.float32, device=DEV)
        b = torch.empty_like(a)
        plain(q, K, V, cur, 500, a)
        l2.prefix_attention_flags(q, K, V, cur, 500, b, l2.PREFIX_CAUSAL if causal else 0)
        torch.cuda.synchronize()
        assert torch.equal(a, b)
    with pytest.raises(l2.L2KVError) as e:
        l2.prefix_attention_flags(q, K, V, cur, 500, a, 8)
    assert e.value.status == -1


def choose(monkeypatch, kernel):
    if kernel == "auto":
        monkeypatch.delenv("L2KV_PREFIX_KERNEL", raising=False)
    else:
        monkeypatch.setenv("L2KV_PREFIX_KERNEL", kernel)


@pytest.mark.parametrize("weights", WEIGHTS)
@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("Hkv,Hq,n_q,T", [(2, 8, 40, 300), (2, 2, 130, 257), (1, 8, 1, 1000),
                                          (2, 4, 64, 128), (2, 8, 70, 200)])
def test_prefix_attention_matches_oracle(Hkv, Hq, n_q, T, kernel, weights, monkeypatch):
    import paper_2406_11430_b200 as l2
    choose(monkeypatch, kernel)
    w = synth.WORKLOADS[2].scaled(B=2, L=2, Hkv=Hkv, Hq=Hq, T=T)
    K, V = synth.make_cache(w, DEV)
    q = make_queries(w, n_q, 3)
    cur = np.array([[T, 128], [0, min(T, 129)]], dtype=np.int32)
    out, lse = run(l2, q, K, V, cur, T, weights=weights)
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    G = Hq // Hkv
    rms_bound = 3e-3 if weights == "single" else 2e-4
    for s in range(n_q):
        want = oracle.attention(synth.to_numpy(q[:, :, s].contiguous()), Kn, Vn, "bf16", cur, nthreads=8)
        assert_attention_close(out[:, :, s], want, atol=ATOL[weights])
        assert np.sqrt(np.mean((out[:, :, s] - want) ** 2)) <= rms_bound * max(np.sqrt(np.mean(want ** 2)), 0.05)
    assert not out[1, 0].any() and np.all(np.isneginf(lse[1, 0]))          # empty cache
    # log-sum-exp against a library routine on a few rows
    qf, Kf = q.float().cpu().numpy().astype(np.float64), K.float().cpu().numpy().astype(np.float64)
    for (b, l, s, j) in [(0, 0, 0, 0), (0, 1, n_q - 1, Hq - 1), (1, 1, n_q // 2, Hq // 2)]:
        z = Kf[b, l, j // G, :cur[b, l]] @ qf[b, l, s, j] / np.sqrt(w.D)
        np.testing.assert_allclose(lse[b, l, s, j], scipy.special.logsumexp(z), rtol=1e-5, atol=1e-4)


@pytest.mark.parametrize("kernel", KERNELS)
def test_prefix_attention_agrees_with_decode_and_ignores_rows_past_the_length(kernel, monkeypatch):
    import paper_2406_11430_b200 as l2
    choose(monkeypatch, kernel)
    w = synth.WORKLOADS[2].scaled(B=1, L=2, T=700)
    K, V = synth.make_cache(w, DEV)
    q = make_queries(w, 5, 9)
    cur = np.array([[700, 333]], dtype=np.int32)
    out, _ = run(l2, q, K, V, cur, 700, scale=0.07)
    for s in range(5):
        dec = gpu_attention(l2, q[:, :, s].contiguous(), K, V, cur, scale=0.07)
        np.testing.assert_allclose(out[:, :, s], dec, rtol=1e-2, atol=2e-3)
    Kp, Vp = K.clone(), V.clone()
    Kp[0, 1, :, 333:] = float("nan")
    Vp[0, 1, :, 333:] = float("inf")
    out2, _ = run(l2, q, Kp, Vp, cur, 700, scale=0.07)
    assert np.array_equal(out, out2)


@pytest.mark.parametrize("weights", WEIGHTS)
@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("direction", [1, -1])
def test_prefix_attention_with_drifting_maxima(kernel, direction, weights, monkeypatch):
    """Scores that grow (or fall) steadily along the cache: the running maximum moves by far
    more than the range one reference maximum can cover, so the accumulated output is rescaled
    several times (growing), or later weights underflow to zero (falling)."""
    import paper_2406_11430_b200 as l2
    choose(monkeypatch, kernel)
    T = 900
    w = synth.WORKLOADS[2].scaled(B=1, L=1, Hkv=2, Hq=4, T=T)
    K, V = synth.make_cache(w, DEV)
    ramp = torch.arange(T, device=DEV, dtype=torch.float32) * (0.25 * direction)
    K[0, 0, :, :, 0] = ramp.to(torch.bfloat16)
    q = make_queries(w, 7, 21)
    q[..., 0] = 4.0
    cur = np.array([[T]], dtype=np.int32)
    out, lse = run(l2, q, K, V, cur, T, weights=weights)
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    for s in range(7):
        want = oracle.attention(synth.to_numpy(q[:, :, s].contiguous()), Kn, Vn, "bf16", cur, nthreads=8)
        assert_attention_close(out[:, :, s], want, atol=ATOL[weights])
    z = K[0, 0, 1].double().cpu().numpy() @ q[0, 0, 3, 2].double().cpu().numpy() / np.sqrt(w.D)
    np.testing.assert_allclose(lse[0, 0, 3, 2], scipy.special.logsumexp(z), rtol=1e-5, atol=1e-4)


@pytest.mark.parametrize("weights", WEIGHTS)
@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("lens", [[9000, 4700], [4608, 0], [4609, 8999]])
def test_prefix_attention_split_over_the_cache(kernel, lens, weights, monkeypatch):
    """Few KV heads and queries, long cache: with the workspace the library asks for, the cache
    is split into chunks (multiples of 128 tokens) whose results are merged; lengths that end
    inside a chunk, at a chunk's edge, just past it, and an empty cache."""
    import paper_2406_11430_b200 as l2
    choose(monkeypatch, kernel)
    T = 9000
    w = synth.WORKLOADS[2].scaled(B=1, L=2, Hkv=2, Hq=8, T=T)
    K, V = synth.make_cache(w, DEV)
    q = make_queries(w, 24, 11)
    cur = np.array([lens], dtype=np.int32)
    ws = l2.prefix_attention_workspace(K, q, T)
    assert ws.numel() > 256                                   # room for a split was asked for
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full(q.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
    call(l2, weights, q, K, V, i32(cur), T, out, lse, workspace=ws)
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    got, got_lse = out.cpu().numpy(), lse.cpu().numpy()
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    for s in range(0, 24, 5):
        want = oracle.attention(synth.to_numpy(q[:, :, s].contiguous()), Kn, Vn, "bf16", cur, nthreads=8)
        assert_attention_close(got[:, :, s], want, atol=ATOL[weights])
    # the unsplit launch (no room for partial results): same rows up to the bf16 rounding of the
    # weights, which are taken against per-chunk maxima in the split launch; same log-sum-exps
    out1, lse1 = run(l2, q, K, V, cur, T, weights=weights)
    np.testing.assert_allclose(got, out1, rtol=1e-2, atol=2e-3)
    np.testing.assert_allclose(got_lse, lse1, rtol=1e-5, atol=1e-5)
    for l in range(2):
        if lens[l] == 0:
            assert not got[0, l].any() and np.all(np.isneginf(got_lse[0, l]))


@pytest.mark.parametrize("weights", WEIGHTS)
@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("T,lens,n_q,split", [(700, [700, 333], 40, False), (300, [130, 17], 24, False),
                                               (9000, [9000, 4620], 40, True)])
def test_prefix_attention_causal(kernel, T, lens, n_q, split, weights, monkeypatch):
    """The chunk's own keys are the last n_q cached rows: query s sees rows < len - n_q + s + 1.
    Checked query by query against the oracle with that length; a cache shorter than the chunk
    (17 rows for 24 queries) leaves the first queries with nothing to see: zeros, lse = -inf."""
    import paper_2406_11430_b200 as l2
    choose(monkeypatch, kernel)
    w = synth.WORKLOADS[2].scaled(B=1, L=2, Hkv=2, Hq=8, T=T)
    K, V = synth.make_cache(w, DEV)
    q = make_queries(w, n_q, 13)
    cur = np.array([lens], dtype=np.int32)
    if kernel == "persistent":
        ws = l2.prefix_attention_workspace(K, q, T)
    else:
        ws = l2.prefix_attention_workspace(K, q, T) if split else torch.zeros(256, dtype=torch.uint8, device=DEV)
        assert (ws.numel() > 256) == split
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full(q.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
    call(l2, weights, q, K, V, i32(cur), T, out, lse, workspace=ws, causal=True)
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    got, got_lse = out.cpu().numpy(), lse.cpu().numpy()
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    Kf, qf = K.float().cpu().numpy().astype(np.float64), q.float().cpu().numpy().astype(np.float64)
    for s in sorted(set(list(range(0, n_q, 7)) + [n_q - 1])):
        see = np.maximum(cur - n_q + s + 1, 0).astype(np.int32)
        want = oracle.attention(synth.to_numpy(q[:, :, s].contiguous()), Kn, Vn, "bf16", see, nthreads=8)
        assert_attention_close(got[:, :, s], want, atol=ATOL[weights])
        for l in range(2):
            if see[0, l] == 0:
                assert not got[0, l, s].any() and np.all(np.isneginf(got_lse[0, l, s]))
            else:
                z = Kf[0, l, 1, :see[0, l]] @ qf[0, l, s, 5] / np.sqrt(w.D)
                np.testing.assert_allclose(got_lse[0, l, s, 5], scipy.special.logsumexp(z), rtol=1e-5, atol=1e-4)


@pytest.mark.parametrize("seed", range(8))
def test_prefix_attention_random_shapes(seed, monkeypatch):
    """Seeded random cases: group size, query count, cache lengths (empty ones included), scale,
    causal or not, either form of the weights, with or without room to split the cache; a sample
    of the queries is compared with the oracle run at the length that query may see."""
    import paper_2406_11430_b200 as l2
    monkeypatch.delenv("L2KV_PREFIX_KERNEL", raising=False)
    rng = np.random.default_rng(1000 + seed)
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.integers(1, 4))
    B, L = int(rng.integers(1, 3)), int(rng.integers(1, 4))
    T = int(rng.choice([65, 200, 777, 1500, 5000]))
    n_q = int(rng.integers(1, 150))
    causal = bool(rng.integers(0, 2))
    weights = WEIGHTS[int(rng.integers(0, 2))]
    split = bool(rng.integers(0, 2))
    scale = float(rng.choice([0.0, 0.05, 0.2]))
    w = synth.WORKLOADS[2].scaled(B=B, L=L, Hkv=Hkv, Hq=Hkv * G, T=T, seed=77 + seed)
    K, V = synth.make_cache(w, DEV)
    q = make_queries(w, n_q, 100 + seed)
    cur = rng.integers(0, T + 1, size=(B, L)).astype(np.int32)
    cur[0, 0] = T
    if B * L > 1:
        cur[-1, -1] = int(rng.choice([0, 1, min(T, n_q - 1) if n_q > 1 else 0]))
    ws = l2.prefix_attention_workspace(K, q, T) if split else torch.zeros(256, dtype=torch.uint8, device=DEV)
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full(q.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
    call(l2, weights, q, K, V, i32(cur), T, out, lse, scale=scale, workspace=ws, causal=causal)
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    got, got_lse = out.cpu().numpy(), lse.cpu().numpy()
    assert not np.isnan(got).any() and not np.isnan(got_lse).any()
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    for s in sorted(set(rng.integers(0, n_q, size=5).tolist() + [0, n_q - 1])):
        see = (np.maximum(cur - n_q + s + 1, 0) if causal else cur).astype(np.int32)
        want = oracle.attention(synth.to_numpy(q[:, :, s].contiguous()), Kn, Vn, "bf16", see, scale=scale,
                                nthreads=8)
        assert_attention_close(got[:, :, s], want, atol=ATOL[weights])
        empty = see == 0
        assert not got[:, :, s][empty].any() and np.all(np.isneginf(got_lse[:, :, s][empty]))
        assert np.all(np.isfinite(got_lse[:, :, s][~empty]))


def test_persistent_kernel_many_calls_on_one_workspace(monkeypatch):
    """The work-balanced kernel keeps counters and partial results in the workspace: a dozen
    calls of different shapes and lengths reuse one workspace back to back (no clearing in
    between); sampled queries of every call are compared with the oracle."""
    import paper_2406_11430_b200 as l2
    monkeypatch.setenv("L2KV_PREFIX_KERNEL", "persistent")
    rng = np.random.default_rng(4242)
    ws = None
    for call_no in range(12):
        G = int(rng.choice([2, 4, 8]))
        Hkv = int(rng.integers(1, 3))
        B, L = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        T = int(rng.choice([900, 3000, 6000]))
        n_q = int(rng.choice([2 * 128 // G, 3 * 128 // G + 1, 150]))      # two or more query tiles
        causal = bool(rng.integers(0, 2))
        w = synth.WORKLOADS[2].scaled(B=B, L=L, Hkv=Hkv, Hq=Hkv * G, T=T, seed=500 + call_no)
        K, V = synth.make_cache(w, DEV)
        q = make_queries(w, n_q, 600 + call_no)
        cur = rng.integers(0, T + 1, size=(B, L)).astype(np.int32)
        cur[0, 0] = T
        need = l2.prefix_attention_workspace(K, q, T).numel()
        if ws is None:
            ws = torch.zeros(need, dtype=torch.uint8, device=DEV)
        assert need == ws.numel()                        # that kernel's ask does not depend on the call
        out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
        lse = torch.full(q.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
        call(l2, "split", q, K, V, i32(cur), T, out, lse, workspace=ws, causal=causal)
        torch.cuda.synchronize()
        assert l2.read_device_status(ws) == 0
        got = out.cpu().numpy()
        assert not np.isnan(got).any()
        Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
        for s in sorted(set(rng.integers(0, n_q, size=3).tolist() + [n_q - 1])):
            see = (np.maximum(cur - n_q + s + 1, 0) if causal else cur).astype(np.int32)
            want = oracle.attention(synth.to_numpy(q[:, :, s].contiguous()), Kn, Vn, "bf16", see, nthreads=8)
            assert_attention_close(got[:, :, s], want, atol=ATOL["split"])


@pytest.mark.parametrize("kernel", KERNELS)
def test_prefix_attention_all_caches_empty(kernel, monkeypatch):
    """Nothing cached anywhere: zeros and lse = -inf for every query, from every kernel."""
    import paper_2406_11430_b200 as l2
    choose(monkeypatch, kernel)
    w = synth.WORKLOADS[2].scaled(B=2, L=3, Hkv=2, Hq=8, T=300)
    K, V = synth.make_cache(w, DEV)
    q = make_queries(w, 70, 21)
    cur = np.zeros((2, 3), dtype=np.int32)
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    lse = torch.full(q.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
    ws = l2.prefix_attention_workspace(K, q, 300)
    if ws.numel() == 256 and kernel == "persistent":
        pytest.skip("no room asked for")
    call(l2, "single", q, K, V, i32(cur), 300, out, lse, workspace=ws)
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    assert not out.cpu().numpy().any() and np.all(np.isneginf(lse.cpu().numpy()))
