"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by
element, on the same seeded bytes.

Bars: index maps, kept rows and stored keys bit-exact against the oracle run on the
library's documented fp32 key order, and against the oracle's fp64 keys everywhere
outside a 1e-6 relative norm band around each unit's threshold (swaps inside the band
are counted); attention within |err| <= 2e-3 + 1e-2 |ref|.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import (DEV, i32, gpu_compress, gpu_attention, assert_attention_close,
                      compare_with_band)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def l2():
    import paper_2406_11430_b200 as lib
    lib.lib()
    return lib


def make(w, t_cap=None):
    K, V = synth.make_cache(w, DEV, t_cap=t_cap)
    return K, V, synth.to_numpy(K), synth.to_numpy(V)


def check_compress(l2, w, K, V, Kn, Vn, lens, keep, unc=(), policy=0, t_cap_out=None, seed=0,
                   sumsq_in=None):
    dev, got = gpu_compress(l2, K, V, lens, keep, unc, policy, t_cap_out, seed=seed,
                            sumsq_in=sumsq_in)
    got["_dev"] = dev                                   # the device tensors, for callers that go on
    exact = oracle.compress(Kn, Vn, w.dtype, lens, keep, unc, key_mode=1, policy=policy,
                            t_cap_out=t_cap_out, nthreads=8, seed=seed)
    assert np.array_equal(got["kept_len"], exact["kept_len"])
    assert np.array_equal(got["idx"], exact["idx"])
    assert np.array_equal(got["K_c"], exact["K_c"])
    assert np.array_equal(got["V_c"], exact["V_c"])
    assert np.array_equal(got["sumsq"].astype(np.float64), exact["key"], equal_nan=True)
    # against the fp64 definition: identical outside the tie band
    ref = oracle.compress(Kn, Vn, w.dtype, lens, keep, unc, key_mode=0, policy=policy,
                          t_cap_out=t_cap_out, nthreads=8)
    key64 = oracle.key_sumsq(Kn, w.dtype)
    swaps = 0
    B, L, H = Kn.shape[:3]
    for b in range(B):
        for l in range(L):
            n = int(ref["kept_len"][b, l])
            if l in unc or n == 0 or policy != 0:
                continue
            for h in range(H):
                swaps += compare_with_band(got["idx"][b, l, h, :n], ref["idx"][b, l, h, :n],
                                           key64[b, l, h, :lens[b]], n)
    return got, swaps


# ------------------------------------------------------------------ key norms

@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("bf16", 64), ("f32", 64), ("f32", 128)])
def test_key_norms(l2, dtype, D):
    w = synth.WORKLOADS[0].scaled(dtype=dtype, D=D, B=2, L=2, Hkv=3, T=1500)
    K, V, Kn, Vn = make(w, t_cap=1536)
    lens = [1500, 333]
    sumsq = torch.full(K.shape[:4], -1.0, dtype=torch.float32, device=DEV)
    norm = torch.full(K.shape[:4], -1.0, dtype=torch.float32, device=DEV)
    l2.key_norms(K, i32(lens), 1500, sumsq, norm)
    torch.cuda.synchronize()
    s, nrm = sumsq.cpu().numpy(), norm.cpu().numpy()
    want32 = oracle.key_sumsq_f32(Kn, dtype)
    want64 = oracle.key_sumsq(Kn, dtype)
    for b in range(2):
        n = lens[b]
        assert np.array_equal(s[b, :, :, :n], want32[b, :, :, :n])            # same bits
        rel = np.abs(s[b, :, :, :n] - want64[b, :, :, :n]) / want64[b, :, :, :n]
        assert rel.max() <= 1e-6
        np.testing.assert_allclose(nrm[b, :, :, :n], np.sqrt(want64[b, :, :, :n]), rtol=1e-6)
        assert np.all(s[b, :, :, n:] == -1.0) and np.all(nrm[b, :, :, n:] == -1.0)  # untouched


# ---------------------------------------------------------- select + compact

def test_compress_tiny_config(l2):
    w = synth.WORKLOADS[0]
    K, V, Kn, Vn = make(w)
    keep = [oracle.keep_count(w.T, w.keep_ratio)]
    got, _ = check_compress(l2, w, K, V, Kn, Vn, [w.T], keep)
    assert np.all(got["idx"][0, 0, :, 0] == 0)           # the low-norm first token is kept


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("bf16", 64), ("f32", 128)])
def test_compress_ragged_multi_chunk(l2, dtype, D):
    w = synth.WORKLOADS[1].scaled(dtype=dtype, D=D, B=3, L=3, Hkv=2, Hq=2, T=2500)
    K, V, Kn, Vn = make(w, t_cap=2560)
    check_compress(l2, w, K, V, Kn, Vn, [2500, 777, 1], [1250, 100, 1], unc=(1,), t_cap_out=2500)


@pytest.mark.parametrize("case", range(10))
def test_compress_and_attention_random_shapes(l2, case):
    """Seeded random shapes, lengths, keep counts, layer lists, policies and element types: the whole
    path (compression, then decode attention over the result) against the oracle."""
    rng = np.random.default_rng(1000 + case)
    dtype = ("bf16", "f32")[int(rng.integers(0, 2))]
    D = (64, 128)[int(rng.integers(0, 2))]
    Hkv = int(rng.integers(1, 4))
    G = (1, 2, 4, 8)[int(rng.integers(0, 4))]
    B, L = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    T = int(rng.integers(1, 3000))
    w = synth.WORKLOADS[2].scaled(dtype=dtype, D=D, B=B, L=L, Hkv=Hkv, Hq=Hkv * G, T=T, seed=50 + case)
    t_cap = T + int(rng.integers(0, 70))
    K, V, Kn, Vn = make(w, t_cap=t_cap)
    lens = [int(rng.integers(0, T + 1)) for _ in range(B)]
    lens[0] = T
    keep = [int(rng.integers(0, n + 1)) for n in lens]
    unc = tuple(sorted(set(int(x) for x in rng.integers(0, L, size=int(rng.integers(0, 2))))))
    policy = int(rng.integers(0, 3))
    got, _ = check_compress(l2, w, K, V, Kn, Vn, lens, keep, unc=unc, policy=policy, seed=case)
    q = synth.make_query(w, case, DEV)
    dev = got["_dev"]
    out = gpu_attention(l2, q, dev["K_c"], dev["V_c"], dev["kept_len"])
    want = oracle.attention(synth.to_numpy(q), got["K_c"], got["V_c"], dtype, got["kept_len"], nthreads=8)
    assert_attention_close(out, want)


def test_compress_exact_ties(l2):
    # Rows of small integers: many keys are exactly equal, so the tie rule decides.
    w = synth.WORKLOADS[1].scaled(B=1, L=2, Hkv=2, Hq=2, T=1300)
    g = torch.Generator().manual_seed(5)
    K = torch.randint(-2, 3, (1, 2, 2, 1300, 128), generator=g).to(torch.bfloat16).to(DEV)
    V = torch.randn((1, 2, 2, 1300, 128), generator=g).to(torch.bfloat16).to(DEV)
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    for keep in (1, 2, 650, 1299):
        _, swaps = check_compress(l2, w, K, V, Kn, Vn, [1300], [keep])
        assert swaps == 0                                  # exact keys: fp32 and fp64 agree
    check_compress(l2, w, K, V, Kn, Vn, [1300], [300], policy=1)


def near_tie_pair(seed=0):
    """Two bf16 key rows A, B with fp64 sums ordered A < B (by ~1e-10 relative) and the
    library's documented fp32 sums ordered the other way.  B is A's elements in another order
    (only rounding differs) with one small element nudged up by one bf16 step."""
    def bf16(x):
        return (torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))[None]
    rng = np.random.default_rng(seed)
    for _ in range(2000):
        a = rng.standard_normal(128).astype(np.float32)
        a[5] = 2.0 ** -10                                   # the element that gets nudged
        b = a[rng.permutation(128)].copy()
        b[np.argmin(np.abs(b - 2.0 ** -10))] = 2.0 ** -10 * (1 + 2.0 ** -7)
        A, B = bf16(a), bf16(b)
        if (oracle.key_sumsq(A, "bf16")[0] < oracle.key_sumsq(B, "bf16")[0]
                and oracle.key_sumsq_f32(A, "bf16")[0] > oracle.key_sumsq_f32(B, "bf16")[0]):
            return A[0], B[0]
    raise AssertionError("no near-tie pair found")


def test_near_tie_is_decided_in_fp32_and_reported_as_a_swap_inside_the_band(l2):
    """A directed near-tie: the fp64 definition keeps row A, the fp32 keys keep row B.  The GPU
    must agree bit for bit with the oracle run on the fp32-ordered keys, and differ from the
    fp64 selection by exactly this one swap, which lies inside the 1e-6 norm band."""
    A, B = near_tie_pair()
    T, pa, pb = 96, 30, 61
    w = synth.WORKLOADS[2].scaled(B=1, L=1, Hkv=1, Hq=1, T=T)
    K, V, Kn, Vn = make(w)
    Kn = Kn.copy()
    # every other token: clearly smaller (first half) or clearly larger (second half) norms
    base = (torch.from_numpy(A.view(np.int16).copy()).view(torch.bfloat16).float()).numpy()
    for t in range(T):
        f = 0.25 + 0.5 * t / T if t < T // 2 else 1.5 + t / T
        row = torch.from_numpy((base * f).astype(np.float32)).to(torch.bfloat16)
        Kn[0, 0, 0, t] = row.view(torch.int16).numpy().view(np.uint16)
    Kn[0, 0, 0, pa], Kn[0, 0, 0, pb] = A, B
    K = torch.from_numpy(Kn.view(np.int16)).view(torch.bfloat16).to(DEV)
    keep = sum(1 for t in range(T // 2) if t != pa) + 1     # the smaller-norm tokens, then one of A / B
    got, swaps = check_compress(l2, w, K, V, Kn, Vn, [T], [keep])
    assert swaps == 1
    kept = set(got["idx"][0, 0, 0, :keep].tolist())
    assert pb in kept and pa not in kept                    # fp32 keys: B is the smaller
    ref = oracle.compress(Kn, Vn, "bf16", [T], [keep])
    kept64 = set(ref["idx"][0, 0, 0, :keep].tolist())
    assert pa in kept64 and pb not in kept64                # fp64 keys: A is the smaller


@pytest.mark.parametrize("T,keep", [(1, 1), (2, 1), (33, 17), (512, 512), (513, 1), (1024, 0)])
def test_compress_edge_sizes(l2, T, keep):
    w = synth.WORKLOADS[0].scaled(T=T)
    K, V, Kn, Vn = make(w)
    check_compress(l2, w, K, V, Kn, Vn, [T], [keep])


def test_compress_empty_sequence_and_highest_policy(l2):
    w = synth.WORKLOADS[0].scaled(B=2, T=600)
    K, V, Kn, Vn = make(w)
    check_compress(l2, w, K, V, Kn, Vn, [0, 600], [0, 300])
    check_compress(l2, w, K, V, Kn, Vn, [600, 600], [60, 599], policy=1)


def test_compress_strided_views(l2):
    # A per-layer call on a view of a larger cache: strides differ from the dense ones.
    w = synth.WORKLOADS[1].scaled(B=2, L=4, Hkv=2, Hq=2, T=700)
    K, V, Kn, Vn = make(w)
    Kv, Vv = K[:, 2:3], V[:, 2:3]
    _, got = gpu_compress(l2, Kv, Vv, [700, 650], [350, 300])
    want = oracle.compress(np.ascontiguousarray(Kn[:, 2:3]), np.ascontiguousarray(Vn[:, 2:3]),
                           "bf16", [700, 650], [350, 300], key_mode=1)
    for name in ("idx", "K_c", "V_c", "kept_len"):
        assert np.array_equal(got[name], want[name])


def test_planted_tokens_survive(l2):
    w = synth.WORKLOADS[3].scaled(L=3, T=16384)
    K, V, Kn, Vn = make(w)
    keep = oracle.keep_count(w.T, w.keep_ratio)
    got, _ = check_compress(l2, w, K, V, Kn, Vn, [w.T], [keep], unc=(0,))
    for l in (1, 2):
        pos = synth.planted_positions(w, 0, l).numpy()
        for h in range(w.Hkv):
            assert np.isin(pos[h], got["idx"][0, l, h, :keep]).all()


def test_compress_is_deterministic(l2):
    w = synth.WORKLOADS[1].scaled(L=2, Hkv=4, Hq=4, T=4096)
    K, V, _, _ = make(w)
    a = gpu_compress(l2, K, V, [4096], [2048])[1]
    b = gpu_compress(l2, K, V, [4096], [2048])[1]
    for name in a:
        assert np.array_equal(a[name], b[name], equal_nan=True)


def test_compress_random_policy(l2):
    w = synth.WORKLOADS[1].scaled(B=2, L=3, Hkv=2, Hq=2, T=2500)
    K, V, Kn, Vn = make(w, t_cap=2560)
    a, _ = check_compress(l2, w, K, V, Kn, Vn, [2500, 700], [1000, 699], unc=(1,), policy=2,
                          seed=12345, t_cap_out=2500)
    b, _ = check_compress(l2, w, K, V, Kn, Vn, [2500, 700], [1000, 699], unc=(1,), policy=2,
                          seed=(1 << 63) + 99, t_cap_out=2500)
    assert not np.array_equal(a["idx"], b["idx"])


@pytest.mark.parametrize("policy", [0, 1])
def test_compress_with_keys_from_write_time(l2, policy):
    # Keys computed once (as when rows are written to the cache) and handed back in: same
    # result as letting the call compute them, without its pass over K.
    w = synth.WORKLOADS[1].scaled(B=2, L=3, Hkv=2, Hq=2, T=2500)
    K, V, Kn, Vn = make(w, t_cap=2560)
    lens = [2500, 1200]
    keys = torch.full(K.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
    l2.key_norms(K, i32(lens), 2500, keys)
    check_compress(l2, w, K, V, Kn, Vn, lens, [1250, 7], unc=(1,), policy=policy, t_cap_out=2500,
                   sumsq_in=keys)


# ---------------------------------------------------------- decode attention

@pytest.mark.parametrize("dtype,D,Hkv,Hq", [
    ("f32", 64, 4, 4), ("bf16", 128, 2, 8), ("bf16", 128, 4, 4), ("bf16", 64, 2, 4),
    ("bf16", 128, 1, 8), ("f32", 128, 2, 4), ("bf16", 64, 1, 8), ("f32", 64, 1, 8)])
def test_attention_ragged(l2, dtype, D, Hkv, Hq):
    w = synth.WORKLOADS[2].scaled(dtype=dtype, D=D, Hkv=Hkv, Hq=Hq, B=2, L=3, T=2600)
    K, V, Kn, Vn = make(w)
    q = synth.make_query(w, 0, DEV)
    cur = np.array([[2600, 1, 1024], [0, 1025, 777]], dtype=np.int32)
    got = gpu_attention(l2, q, K, V, cur)
    want = oracle.attention(synth.to_numpy(q), Kn, Vn, dtype, cur, nthreads=8)
    assert_attention_close(got, want)
    assert not got[1, 0].any()                           # empty cache -> zeros
    rms = math.sqrt(np.mean(want ** 2))
    assert np.sqrt(np.mean((got - want) ** 2)) <= 2e-4 * max(rms, 1e-3) + 1e-6


def test_attention_copy_paths_agree(l2, monkeypatch):
    # bf16 / head_dim 128 streams K and V through TMA tensor maps by default and through
    # per-thread cp.async copies on request (or when a geometry cannot be encoded); the
    # arithmetic is the same, so the outputs must be bit-identical.
    w = synth.WORKLOADS[2].scaled(B=2, L=2, T=2300)
    K, V, Kn, Vn = make(w)
    q = synth.make_query(w, 0, DEV)
    cur = np.array([[2300, 1030], [129, 2047]], dtype=np.int32)
    monkeypatch.setenv("L2KV_DECODE_COPY", "tma")
    a = gpu_attention(l2, q, K, V, cur)
    monkeypatch.setenv("L2KV_DECODE_COPY", "cpasync")
    b = gpu_attention(l2, q, K, V, cur)
    assert np.array_equal(a, b)
    assert_attention_close(a, oracle.attention(synth.to_numpy(q), Kn, Vn, "bf16", cur, nthreads=8))
    # rows past the valid length must not leak in, whatever they hold (here: NaN and Inf)
    Kp, Vp = K.clone(), V.clone()
    Kp[0, 1, :, 1030:] = float("nan"); Vp[0, 1, :, 1030:] = float("inf")
    Kp[1, 0, :, 129:] = float("inf"); Vp[1, 0, :, 129:] = float("nan")
    for mode in ("tma", "cpasync"):
        monkeypatch.setenv("L2KV_DECODE_COPY", mode)
        assert np.array_equal(gpu_attention(l2, q, Kp, Vp, cur), a)


def test_attention_merge_inside_the_split_kernel_equals_the_merge_kernel(l2, monkeypatch):
    """The partial results of a unit's splits are merged by whichever split finishes last; the
    sums are formed in split order either way, so the result has the bits of the two-kernel form
    (split kernel, then merge kernel).  Ragged lengths: 0, 1, exactly one split, many splits."""
    w = synth.WORKLOADS[2].scaled(B=2, L=3, T=5000)
    K, V, _, _ = make(w)
    q = synth.make_query(w, 0, DEV)
    cur = [[5000, 0, 1024], [1, 1025, 3333]]
    a = gpu_attention(l2, q, K, V, cur)
    b = gpu_attention(l2, q, K, V, cur)                      # and it is deterministic
    monkeypatch.setenv("L2KV_DECODE_MERGE_KERNEL", "1")
    c = gpu_attention(l2, q, K, V, cur)
    assert np.array_equal(a, b) and np.array_equal(a, c)
    assert not a[0, 1].any()


def test_attention_special_cases(l2):
    w = synth.WORKLOADS[2].scaled(B=1, L=1, T=2048)
    K, V, Kn, Vn = make(w)
    q = synth.make_query(w, 0, DEV)
    # one cached token -> that token's value row, for every query head of the group
    got = gpu_attention(l2, q, K, V, [[1]])
    v0 = V[0, 0, :, 0].float().cpu().numpy()
    np.testing.assert_allclose(got[0, 0], np.repeat(v0, 4, axis=0), rtol=1e-6, atol=1e-7)
    # all keys equal -> mean of the values
    Ke = K[:, :, :, :1].expand_as(K).contiguous()
    got = gpu_attention(l2, q, Ke, V, [[2048]])
    mean = V[0, 0].double().mean(1).cpu().numpy()
    np.testing.assert_allclose(got[0, 0], np.repeat(mean, 4, axis=0), rtol=1e-4, atol=1e-5)
    # very large scores stay finite and select the arg-max row
    qbig = (q.float() * 256).to(torch.bfloat16)
    got = gpu_attention(l2, qbig, K, V, [[2048]])
    want = oracle.attention(synth.to_numpy(qbig), Kn, Vn, "bf16", [[2048]], nthreads=8)
    assert np.isfinite(got).all()
    assert_attention_close(got, want)
    # slot order does not matter beyond rounding
    perm = torch.randperm(2048, generator=torch.Generator().manual_seed(3)).to(DEV)
    a = gpu_attention(l2, q, K, V, [[2048]])
    b = gpu_attention(l2, q, K[:, :, :, perm].contiguous(), V[:, :, :, perm].contiguous(), [[2048]])
    np.testing.assert_allclose(a, b, rtol=1e-4, atol=1e-6)
    # explicit scale, and determinism
    c = gpu_attention(l2, q, K, V, [[2048]], scale=0.05)
    want = oracle.attention(synth.to_numpy(q), Kn, Vn, "bf16", [[2048]], scale=0.05, nthreads=8)
    assert_attention_close(c, want)
    assert np.array_equal(a, gpu_attention(l2, q, K, V, [[2048]]))


def test_keep_everything_then_attend_equals_uncompressed(l2):
    w = synth.WORKLOADS[2].scaled(B=1, L=2, T=1500)
    K, V, Kn, Vn = make(w)
    q = synth.make_query(w, 1, DEV)
    dev, got = gpu_compress(l2, K, V, [1500], [1500])
    assert np.array_equal(got["K_c"], Kn) and np.array_equal(got["V_c"], Vn)
    a = gpu_attention(l2, q, dev["K_c"], dev["V_c"], dev["kept_len"])
    b = gpu_attention(l2, q, K, V, [[1500, 1500]])
    assert np.array_equal(a, b)


def test_compress_then_attend_pipeline(l2):
    w = synth.WORKLOADS[2].scaled(B=2, L=4, T=3000)
    K, V, Kn, Vn = make(w)
    keep = oracle.keep_count(w.T, w.keep_ratio)
    dev, got = gpu_compress(l2, K, V, [3000, 2000], [keep, 1000], unc=(0, 1))
    ref = oracle.compress(Kn, Vn, "bf16", [3000, 2000], [keep, 1000], (0, 1), key_mode=1, nthreads=8)
    for s in range(2):
        q = synth.make_query(w, s, DEV)
        out = gpu_attention(l2, q, dev["K_c"], dev["V_c"], dev["kept_len"])
        want = oracle.attention(synth.to_numpy(q), ref["K_c"], ref["V_c"], "bf16", ref["kept_len"],
                                nthreads=8)
        assert_attention_close(out, want)


def test_compress_reads_v_from_pinned_host_memory(l2):
    """V left in pinned host memory: the compression reads the rows it keeps in place; same result."""
    w = synth.WORKLOADS[2].scaled(B=2, L=3, T=1500)
    K, V, Kn, Vn = make(w)
    lens, keep = [1500, 900], [700, 450]
    dev, host = gpu_compress(l2, K, V, lens, keep, unc=(0,))
    V_host = torch.empty(V.shape, dtype=V.dtype, pin_memory=True)
    V_host.copy_(V)
    torch.cuda.synchronize()
    dev2, host2 = gpu_compress(l2, K, V_host, lens, keep, unc=(0,))
    for name in ("K_c", "V_c", "idx", "kept_len"):
        assert np.array_equal(host[name], host2[name]), name


# -------------------------------------------------------------- append/evict

def _oracle_state(r, t_cap):
    B, L, H, t0, D = r["K_c"].shape
    st = dict(K_c=np.zeros((B, L, H, t_cap, D), r["K_c"].dtype),
              idx=np.full((B, L, H, t_cap), -1, np.int32),
              key=np.full((B, L, H, t_cap), np.nan), cur_len=r["kept_len"].copy())
    st["V_c"] = np.zeros_like(st["K_c"])
    for name in ("K_c", "V_c", "idx", "key"):
        st[name][:, :, :, :t0] = r[name]
    return st


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("f32", 64)])
def test_append_evict_stream(l2, dtype, D):
    steps, T0 = 48, 700
    w = synth.WORKLOADS[4].scaled(dtype=dtype, D=D, B=3, L=3, Hkv=2, Hq=8, T=T0, ragged_lo=0)
    K, V, Kn, Vn = make(w)
    lens, budget = [700, 300, 40], [350, 150, 60]        # the last sequence still grows
    keep = [350, 150, 40]
    t_cap = T0 + steps
    dev, _ = gpu_compress(l2, K, V, lens, keep, unc=(0,), t_cap_out=t_cap)
    st = _oracle_state(oracle.compress(Kn, Vn, dtype, lens, keep, (0,), key_mode=1, t_cap_out=T0),
                       t_cap)
    ws = l2.new_workspace(l2.Layout(dev["K_c"], q_heads=w.Hq), t_cap, DEV)
    bud = i32(budget)
    for s in range(steps):
        k, v = synth.make_new_kv(w, s, DEV)
        pos = [n + s for n in lens]
        l2.append_evict(dev["K_c"], dev["V_c"], dev["idx"], dev["sumsq"], dev["kept_len"], bud,
                        (0,), k, v, i32(pos), ws)
        assert oracle.append_evict(st, dtype, budget, (0,), synth.to_numpy(k), synth.to_numpy(v),
                                   pos, key_mode=1) == 0
        if s % 16 == 15 or s == steps - 1:
            torch.cuda.synchronize()
            cur = dev["kept_len"].cpu().numpy()
            assert np.array_equal(cur, st["cur_len"])
            for b in range(3):
                for l in range(3):
                    n = cur[b, l]
                    assert np.array_equal(dev["idx"][b, l, :, :n].cpu().numpy(), st["idx"][b, l, :, :n])
                    assert np.array_equal(synth.to_numpy(dev["K_c"][b, l, :, :n]), st["K_c"][b, l, :, :n])
                    assert np.array_equal(synth.to_numpy(dev["V_c"][b, l, :, :n]), st["V_c"][b, l, :, :n])
                    assert np.array_equal(dev["sumsq"][b, l, :, :n].cpu().numpy().astype(np.float64),
                                          st["key"][b, l, :, :n])
            q = synth.make_query(w, s, DEV)
            out = gpu_attention(l2, q, dev["K_c"], dev["V_c"], dev["kept_len"])
            want = oracle.attention(synth.to_numpy(q), st["K_c"], st["V_c"], dtype, st["cur_len"],
                                    nthreads=8)
            assert_attention_close(out, want)
    assert l2.read_device_status(ws) == 0


def test_append_evict_stream_against_fp64_keys(l2):
    """The same stream against the oracle with its fp64 keys: after every append the kept sets
    must agree outside the 1e-6 tie band around the threshold norm (the kernel decides in fp32)."""
    steps, T0 = 64, 600
    w = synth.WORKLOADS[4].scaled(B=2, L=3, Hkv=2, Hq=8, T=T0, ragged_lo=0)
    K, V, Kn, Vn = make(w)
    lens, budget = [600, 250], [300, 125]
    t_cap = T0 + steps
    dev, _ = gpu_compress(l2, K, V, lens, budget, unc=(0,), t_cap_out=t_cap)
    st = _oracle_state(oracle.compress(Kn, Vn, w.dtype, lens, budget, (0,), key_mode=0, t_cap_out=T0),
                       t_cap)
    ws = l2.new_workspace(l2.Layout(dev["K_c"], q_heads=w.Hq), t_cap, DEV)
    bud = i32(budget)
    rows = [[Kn[b, :, :, :lens[b]]] for b in range(w.B)]          # every key a unit has seen, by position
    swaps = 0
    for s in range(steps):
        k, v = synth.make_new_kv(w, s, DEV)
        kn, vn = synth.to_numpy(k), synth.to_numpy(v)
        pos = [n + s for n in lens]
        l2.append_evict(dev["K_c"], dev["V_c"], dev["idx"], dev["sumsq"], dev["kept_len"], bud,
                        (0,), k, v, i32(pos), ws)
        assert oracle.append_evict(st, w.dtype, budget, (0,), kn, vn, pos, key_mode=0) == 0
        for b in range(w.B):
            rows[b].append(kn[b][:, :, None, :])
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    cur = dev["kept_len"].cpu().numpy()
    assert np.array_equal(cur, st["cur_len"])
    for b in range(w.B):
        seen = np.concatenate(rows[b], axis=2)                    # [L, H, lens[b] + steps, D]
        key64 = oracle.key_sumsq(seen[None], w.dtype)[0]
        for l in range(1, w.L):                                   # layer 0 is uncompressed
            n = int(cur[b, l])
            assert n == budget[b]
            for h in range(w.Hkv):
                swaps += compare_with_band(dev["idx"][b, l, h, :n].cpu().numpy(), st["idx"][b, l, h, :n],
                                           key64[l, h], n)
    print(f"append/evict against fp64 keys: {swaps} swaps inside the tie band")


def test_append_evict_overflow_sets_status(l2):
    w = synth.WORKLOADS[4].scaled(B=1, L=2, Hkv=2, Hq=8, T=64, ragged_lo=0)
    K, V, Kn, Vn = make(w)
    dev, _ = gpu_compress(l2, K, V, [64], [32], unc=(0,))       # layer 0 is full: t_cap = 64
    ws = l2.new_workspace(l2.Layout(dev["K_c"]), 64, DEV)
    before = {k: v.clone() for k, v in dev.items()}
    k, v = synth.make_new_kv(w, 0, DEV)
    l2.append_evict(dev["K_c"], dev["V_c"], dev["idx"], dev["sumsq"], dev["kept_len"], i32([32]),
                    (0,), k, v, i32([64]), ws)
    assert l2.read_device_status(ws) == -7
    assert torch.equal(dev["K_c"][0, 0], before["K_c"][0, 0])    # nothing written for that layer
    assert dev["kept_len"].cpu().tolist() == [[64, 32]]
