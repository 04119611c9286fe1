"""Pins for the CPU oracle: what the paper and the mathematics fix, checked
against things other than the oracle itself (closed forms, brute force,
library routines, hand-worked values, invariants)."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import scipy.special

import oracle
import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_worked.json")


def bf16_round(x):
    """float32 array -> uint16 bfloat16 bit patterns (round to nearest even)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return u.astype(np.uint16)


def bf16_widen(h):
    return (h.astype(np.uint32) << 16).view(np.float32)


# ---------------------------------------------------------------- a1: norms

def test_norm_closed_forms():
    D = 64
    ones = np.ones((1, D), np.float32)
    assert oracle.key_sumsq(ones, "f32")[0] == D                      # ||1|| = sqrt(D)
    e = np.zeros((D, D), np.float32)
    c = np.arange(1, D + 1, dtype=np.float32) * 0.25
    e[np.arange(D), np.arange(D)] = -c                                # ||c e_i|| = |c|
    assert np.array_equal(oracle.key_sumsq(e, "f32"), (c.astype(np.float64)) ** 2)
    for h in (bf16_round(ones), ):
        assert oracle.key_sumsq(h, "bf16")[0] == D


def test_norm_matches_library_norm():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((37, 128)).astype(np.float32)
    ref = np.linalg.norm(x.astype(np.float64), axis=-1)
    np.testing.assert_allclose(np.sqrt(oracle.key_sumsq(x, "f32")), ref, rtol=1e-14)
    h = bf16_round(x)
    ref = np.linalg.norm(bf16_widen(h).astype(np.float64), axis=-1)
    np.testing.assert_allclose(np.sqrt(oracle.key_sumsq(h, "bf16")), ref, rtol=1e-14)


def test_norm_homogeneity_and_rotation():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((8, 64)).astype(np.float32)
    s = oracle.key_sumsq(x, "f32")
    assert np.array_equal(oracle.key_sumsq(x * np.float32(4.0), "f32"), s * 16.0)  # power of two
    # a rotary embedding rotates channel pairs; the norm does not change
    th = rng.uniform(0, 2 * math.pi, (8, 32))
    xr = np.empty_like(x, dtype=np.float64)
    xr[:, 0::2] = x[:, 0::2] * np.cos(th) - x[:, 1::2] * np.sin(th)
    xr[:, 1::2] = x[:, 0::2] * np.sin(th) + x[:, 1::2] * np.cos(th)
    np.testing.assert_allclose((xr ** 2).sum(-1), s, rtol=1e-13)


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("bf16", 64), ("f32", 64), ("f32", 128)])
def test_f32_ordered_key_within_rounding_of_exact(dtype, D):
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((500, D)) * np.exp(rng.standard_normal((500, 1)))).astype(np.float32)
    a = bf16_round(x) if dtype == "bf16" else x
    exact = oracle.key_sumsq(a, dtype)
    got = oracle.key_sumsq_f32(a, dtype).astype(np.float64)
    pieces = D // (8 if dtype == "bf16" else 4)
    n_round = (8 if dtype == "bf16" else 4) + int(math.log2(pieces))
    assert np.max(np.abs(got - exact) / exact) <= n_round * 2.0 ** -24
    # small integers: every partial sum is exact in fp32, whatever the order
    xi = rng.integers(-8, 9, (50, D)).astype(np.float32)
    ai = bf16_round(xi) if dtype == "bf16" else xi
    assert np.array_equal(oracle.key_sumsq_f32(ai, dtype).astype(np.float64), (xi.astype(np.float64) ** 2).sum(-1))


def test_f32_ordered_key_uses_the_documented_tree():
    # One big element per 16-byte piece and tiny ones elsewhere: the result
    # depends on where roundings happen.  Recomputed here with numpy float32.
    rng = np.random.default_rng(4)
    x = (rng.standard_normal((64, 128)) * 10.0 ** rng.integers(-3, 4, (64, 128))).astype(np.float32)
    h = bf16_round(x)
    xf = bf16_widen(h)
    p = np.zeros((64, 16), np.float32)
    for e in range(8):
        v = xf.reshape(64, 16, 8)[:, :, e]
        p = (v.astype(np.float64) * v.astype(np.float64) + p.astype(np.float64)).astype(np.float32)
    off = 8
    while off >= 1:
        p = (p + p[:, np.arange(16) ^ off]).astype(np.float32)
        off //= 2
    assert np.array_equal(oracle.key_sumsq_f32(h, "bf16"), p[:, 0])


# ------------------------------------------------------------ a2: selection

def test_selection_hand_worked():
    g = json.load(open(GOLDEN))["selection"]
    keys = np.array(g["keys"], dtype=np.float32)
    s = oracle.key_sumsq(keys, "f32")
    np.testing.assert_array_equal(np.sqrt(s), np.array(g["norms"], dtype=np.float64))
    for keep, want in g["kept"].items():
        assert oracle.select(s, int(keep)).tolist() == want


def test_selection_brute_force_subsets():
    # The kept set is the unique size-k subset whose largest (norm, position)
    # is below the smallest (norm, position) left outside.
    rng = np.random.default_rng(5)
    for T in (1, 2, 5, 9):
        s = rng.integers(0, 4, T).astype(np.float64)        # many exact ties
        for keep in range(1, T + 1):
            hits = []
            for sub in itertools.combinations(range(T), keep):
                rest = [t for t in range(T) if t not in sub]
                if not rest or max((s[t], t) for t in sub) < min((s[t], t) for t in rest):
                    hits.append(list(sub))
            assert len(hits) == 1
            assert oracle.select(s, keep).tolist() == hits[0]


def test_selection_vs_python_sort():
    rng = np.random.default_rng(6)
    for T in (3, 33, 64, 1000):
        s = np.round(rng.standard_normal(T) ** 2, 1)
        for keep in {1, 2, T // 2, T - 1, T} - {0}:
            want = sorted(sorted(range(T), key=lambda t: (s[t], t))[:keep])
            assert oracle.select(s, keep).tolist() == want
            hi = sorted(sorted(range(T), key=lambda t: (-s[t], t))[:keep])
            assert oracle.select(s, keep, policy=1).tolist() == hi


def test_keep_count():
    assert oracle.keep_count(4096, 0.5) == 2048
    assert oracle.keep_count(131072, 0.1) == 13108
    assert oracle.keep_count(1024, 1.0) == 1024
    assert oracle.keep_count(7, 0.0) == 1
    assert oracle.keep_count(7, 2.0) == 7
    assert oracle.keep_count(0, 0.5) == 0


# ------------------------------------------------- a1-a4: whole compression

def _tiny(dtype="f32", **kw):
    w = synth.WORKLOADS[0].scaled(dtype=dtype, **kw)
    K, V = synth.make_cache(w, "cpu")
    return w, synth.to_numpy(K), synth.to_numpy(V)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_compress_invariants(dtype):
    w, K, V = _tiny(dtype, L=3, T=512)
    keep = oracle.keep_count(w.T, w.keep_ratio)
    r = oracle.compress(K, V, dtype, [w.T], [keep], uncompressed=(1,))
    s = oracle.key_sumsq(K, dtype)
    assert r["kept_len"].tolist() == [[keep, w.T, keep]]
    for l in range(w.L):
        for h in range(w.Hkv):
            n = r["kept_len"][0, l]
            idx = r["idx"][0, l, h, :n]
            assert np.all(np.diff(idx) > 0)                                    # position order
            assert np.array_equal(r["K_c"][0, l, h, :n], K[0, l, h, idx])       # byte copies
            assert np.array_equal(r["V_c"][0, l, h, :n], V[0, l, h, idx])
            assert np.array_equal(r["key"][0, l, h, :n], s[0, l, h, idx])
            assert np.all(r["idx"][0, l, h, n:] == -1)                          # tail untouched
            assert not r["K_c"][0, l, h, n:].any()
            if l == 1:
                assert np.array_equal(idx, np.arange(w.T))                      # skipped layer
                continue
            assert n == keep
            dropped = np.setdiff1d(np.arange(w.T), idx)
            top = max((s[0, l, h, t], t) for t in idx)
            assert top < min((s[0, l, h, t], t) for t in dropped)
            assert 0 in idx                                                     # low-norm first token


def test_compress_keep_one_is_argmin_and_all_equal_keeps_first():
    w, K, V = _tiny("f32", T=256)
    r = oracle.compress(K, V, "f32", [w.T], [1])
    s = oracle.key_sumsq(K, "f32")
    assert np.array_equal(r["idx"][0, 0, :, 0], s[0, 0].argmin(-1))
    # rows that are permutations of the same small integers: exactly equal norms
    rng = np.random.default_rng(7)
    base = np.arange(w.D, dtype=np.float32) - 20
    Kp = np.stack([rng.permutation(base) for _ in range(w.Hkv * w.T)]).reshape(K.shape)
    r = oracle.compress(Kp, V, "f32", [w.T], [100])
    assert np.array_equal(r["idx"][0, 0, :, :100], np.tile(np.arange(100), (w.Hkv, 1)))


def test_planted_low_norm_tokens_survive_extreme_compression():
    w = synth.WORKLOADS[3].scaled(L=1, T=8192)
    K, V = synth.make_cache(w, "cpu")
    keep = oracle.keep_count(w.T, w.keep_ratio)
    r = oracle.compress(synth.to_numpy(K), synth.to_numpy(V), "bf16", [w.T], [keep])
    pos = synth.planted_positions(w, 0, 0).numpy()
    for h in range(w.Hkv):
        assert np.isin(pos[h], r["idx"][0, 0, h, :keep]).all()


def test_ragged_lengths_and_per_sequence_keep():
    w, K, V = _tiny("bf16", B=3, T=300)
    lens, keep = [300, 1, 77], [150, 1, 20]
    r = oracle.compress(K, V, "bf16", lens, keep, t_cap_out=160)
    s = oracle.key_sumsq(K, "bf16")
    for b in range(3):
        for h in range(w.Hkv):
            idx = r["idx"][b, 0, h, :keep[b]]
            want = sorted(sorted(range(lens[b]), key=lambda t: (s[b, 0, h, t], t))[:keep[b]])
            assert idx.tolist() == want
    with pytest.raises(ValueError):
        oracle.compress(K, V, "bf16", [301, 1, 1], [1, 1, 1])
    with pytest.raises(ValueError):
        oracle.compress(K, V, "bf16", [300, 1, 1], [2, 2, 1])


def test_per_head_keep_counts():
    """A keep count per (b, l, h): every unit is the sort-and-cut of its own keys; the
    uncompressed layer ignores the counts."""
    w, K, V = _tiny("bf16", B=2, L=3, T=200)
    lens = [200, 61]
    rng = np.random.default_rng(11)
    keep = np.stack([rng.integers(0, lens[b] + 1, size=(w.L, w.Hkv)) for b in range(2)])
    keep[0, 0, 0], keep[1, 2, 1] = 0, 61                                   # empty and whole
    r = oracle.compress(K, V, "bf16", lens, keep, uncompressed=(1,))
    s = oracle.key_sumsq(K, "bf16")
    assert r["kept_len"].shape == (2, w.L, w.Hkv)
    for b, l, h in itertools.product(range(2), range(w.L), range(w.Hkv)):
        n = lens[b] if l == 1 else keep[b, l, h]
        assert r["kept_len"][b, l, h] == n
        want = sorted(sorted(range(lens[b]), key=lambda t: (s[b, l, h, t], t))[:n])
        assert r["idx"][b, l, h, :n].tolist() == want
        assert np.all(r["idx"][b, l, h, n:] == -1)
        assert np.array_equal(r["V_c"][b, l, h, :n], V[b, l, h, want])
    # equal counts in every head are the per-sequence call
    same = oracle.compress(K, V, "bf16", lens, np.broadcast_to(np.array([90, 30])[:, None, None],
                                                               (2, w.L, w.Hkv)).copy())
    ref = oracle.compress(K, V, "bf16", lens, [90, 30])
    assert np.array_equal(same["idx"], ref["idx"]) and np.array_equal(same["K_c"], ref["K_c"])
    bad = keep.copy()
    bad[1, 0, 0] = 62
    with pytest.raises(ValueError):
        oracle.compress(K, V, "bf16", lens, bad)


# ------------------------------------------------------------ a5: attention

def _textbook_attention(q, K, V, G):
    """softmax(q K^T / sqrt(d)) V with library routines, fp64; K, V [H, n, D], q [Hq, D]."""
    out = np.empty(q.shape, np.float64)
    for j in range(q.shape[0]):
        z = K[j // G].astype(np.float64) @ q[j].astype(np.float64) / math.sqrt(q.shape[1])
        out[j] = scipy.special.softmax(z) @ V[j // G].astype(np.float64)
    return out


def test_attention_hand_worked():
    g = json.load(open(GOLDEN))["attention"]
    q = np.array(g["q"], np.float32).reshape(1, 1, 1, 4)
    K = np.zeros((1, 1, 1, 3, 4), np.float32)
    K[0, 0, 0, :, 0] = np.log([1.0, 2.0, 3.0]).astype(np.float32)
    V = np.array(g["values"], np.float32).reshape(1, 1, 1, 3, 4)
    out = oracle.attention(q, K, V, "f32", [3])
    np.testing.assert_allclose(out[0, 0, 0], g["out"], atol=2e-7)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_attention_matches_textbook_and_gqa_mapping(dtype):
    w = synth.WORKLOADS[0].scaled(dtype=dtype, L=2, Hkv=2, Hq=8, T=200)
    K, V = synth.make_cache(w, "cpu")
    q = synth.make_query(w, 0, "cpu")
    Kn, Vn, qn = synth.to_numpy(K), synth.to_numpy(V), synth.to_numpy(q)
    out = oracle.attention(qn, Kn, Vn, dtype, np.full((1, 2), 200))
    for l in range(2):
        want = _textbook_attention(q[0, l].float().numpy(), K[0, l].float().numpy(),
                                   V[0, l].float().numpy(), 4)
        np.testing.assert_allclose(out[0, l], want, rtol=1e-11, atol=1e-13)
    # cur_len limits the rows that are read
    out2 = oracle.attention(qn, Kn, Vn, dtype, [[50, 0]])
    want = _textbook_attention(q[0, 0].float().numpy(), K[0, 0, :, :50].float().numpy(),
                               V[0, 0, :, :50].float().numpy(), 4)
    np.testing.assert_allclose(out2[0, 0], want, rtol=1e-11, atol=1e-13)
    assert not out2[0, 1].any()                                            # empty cache -> zeros


def test_attention_with_a_length_per_kv_head():
    w = synth.WORKLOADS[0].scaled(dtype="bf16", L=2, Hkv=2, Hq=8, T=200)
    K, V = synth.make_cache(w, "cpu")
    q = synth.make_query(w, 0, "cpu")
    lens = np.array([[[200, 37], [0, 1]]])
    out = oracle.attention(synth.to_numpy(q), synth.to_numpy(K), synth.to_numpy(V), "bf16", lens)
    for l, h in itertools.product(range(2), range(2)):
        n = lens[0, l, h]
        got = out[0, l, 4 * h:4 * h + 4]
        if n == 0:
            assert not got.any()
            continue
        want = _textbook_attention(q[0, l, 4 * h:4 * h + 4].float().numpy(),
                                   K[0, l, h:h + 1, :n].float().numpy(),
                                   V[0, l, h:h + 1, :n].float().numpy(), 4)
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-13)


def test_keep_everything_reproduces_uncompressed_attention():
    w, K, V = _tiny("f32", T=128)
    q = synth.to_numpy(synth.make_query(w, 0, "cpu"))
    r = oracle.compress(K, V, "f32", [w.T], [w.T])
    assert np.array_equal(r["K_c"], K) and np.array_equal(r["V_c"], V)
    a = oracle.attention(q, r["K_c"], r["V_c"], "f32", r["kept_len"])
    b = oracle.attention(q, K, V, "f32", [[w.T]])
    assert np.array_equal(a, b)


def test_attention_special_cases():
    rng = np.random.default_rng(8)
    D, n = 64, 40
    q = rng.standard_normal((1, 1, 4, D)).astype(np.float32)
    K = rng.standard_normal((1, 1, 4, n, D)).astype(np.float32)
    V = rng.standard_normal((1, 1, 4, n, D)).astype(np.float32)
    # one cached token: the output is that token's value row
    out = oracle.attention(q, K, V, "f32", [1])
    np.testing.assert_allclose(out[0, 0], V[0, 0, :, 0], rtol=1e-15)
    # all keys equal: plain mean of the values
    Ke = np.broadcast_to(K[:, :, :, :1], K.shape).copy()
    out = oracle.attention(q, Ke, V, "f32", [n])
    np.testing.assert_allclose(out[0, 0], V[0, 0].astype(np.float64).mean(1), rtol=1e-12, atol=1e-14)
    # adding one vector to every key shifts all scores alike: softmax unchanged
    # (the shift is a multiple of 1/4 on quarter-integer data, so it is exact)
    Kq = np.round(K * 4) / 4
    base = oracle.attention(q, Kq, V, "f32", [n])
    shift = (np.round(rng.standard_normal(D) * 4) / 4).astype(np.float32)
    out = oracle.attention(q, Kq + shift, V, "f32", [n])
    np.testing.assert_allclose(out, base, rtol=1e-9, atol=1e-11)
    # very large scores stay finite and pick the arg-max row
    out = oracle.attention(q * 1e4, K, V, "f32", [n])
    z = np.einsum("hd,hnd->hn", q[0, 0].astype(np.float64), K[0, 0].astype(np.float64))
    assert np.isfinite(out).all()
    np.testing.assert_allclose(out[0, 0], V[0, 0][np.arange(4), z.argmax(1)], rtol=1e-9, atol=1e-12)
    # slot order does not matter
    perm = rng.permutation(n)
    out = oracle.attention(q, np.ascontiguousarray(K[:, :, :, perm]),
                           np.ascontiguousarray(V[:, :, :, perm]), "f32", [n])
    np.testing.assert_allclose(out, oracle.attention(q, K, V, "f32", [n]), rtol=1e-12, atol=1e-14)
    # explicit scale
    out = oracle.attention(q, K, V, "f32", [n], scale=0.0625)
    z = z * 0.0625
    np.testing.assert_allclose(out[0, 0], np.einsum("hn,hnd->hd", scipy.special.softmax(z, axis=1),
                                                    V[0, 0].astype(np.float64)), rtol=1e-11)


# --------------------------------------------------------- a6: append/evict

def _state_from(r, T_cap):
    B, L, H, t0, D = r["K_c"].shape
    st = dict(K_c=np.zeros((B, L, H, T_cap, D), r["K_c"].dtype), idx=np.full((B, L, H, T_cap), -1, np.int32),
              key=np.full((B, L, H, T_cap), np.nan), cur_len=r["kept_len"].copy())
    st["V_c"] = np.zeros_like(st["K_c"])
    for name in ("K_c", "V_c", "idx", "key"):
        st[name][:, :, :, :t0] = r[name]
    return st


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_streaming_eviction_equals_one_shot_selection(dtype):
    """After n appends the kept set is the `budget` lowest (norm, position) of
    everything seen -- append/evict pinned to the selection definition."""
    steps, T0 = 40, 64
    w = synth.WORKLOADS[0].scaled(dtype=dtype, B=2, L=3, T=T0)
    K, V = synth.make_cache(w, "cpu")
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    budget = [T0 // 2, T0 // 4]
    r = oracle.compress(Kn, Vn, dtype, [T0, T0], budget, uncompressed=(0,), t_cap_out=T0)
    st = _state_from(r, T0 + steps)
    allK, allV = [Kn], [Vn]
    for s in range(steps):
        k, v = synth.make_new_kv(w, s, "cpu")
        kn, vn = synth.to_numpy(k), synth.to_numpy(v)
        assert oracle.append_evict(st, dtype, budget, (0,), kn, vn, [T0 + s, T0 + s]) == 0
        allK.append(kn[:, :, :, None]); allV.append(vn[:, :, :, None])
    fullK, fullV = np.concatenate(allK, 3), np.concatenate(allV, 3)
    one = oracle.compress(fullK, fullV, dtype, [T0 + steps] * 2, budget, uncompressed=(0,))
    assert np.array_equal(st["cur_len"], one["kept_len"])
    for b in range(2):
        for l in range(3):
            n = st["cur_len"][b, l]
            assert n == (T0 + steps if l == 0 else budget[b])
            for h in range(w.Hkv):
                order = np.argsort(st["idx"][b, l, h, :n])
                assert np.array_equal(st["idx"][b, l, h, :n][order], one["idx"][b, l, h, :n])
                assert np.array_equal(st["K_c"][b, l, h, :n][order], one["K_c"][b, l, h, :n])
                assert np.array_equal(st["V_c"][b, l, h, :n][order], one["V_c"][b, l, h, :n])
                assert np.array_equal(st["key"][b, l, h, :n][order], one["key"][b, l, h, :n])


def test_streaming_eviction_with_a_budget_per_head():
    """Per-head budgets: every head ends with its own `budget` lowest (norm, position) of all
    the tokens it has seen (sort-and-cut per head); heads under budget keep growing."""
    steps, T0 = 30, 48
    w = synth.WORKLOADS[0].scaled(dtype="bf16", B=2, L=2, T=T0)
    K, V = synth.make_cache(w, "cpu")
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    rng = np.random.default_rng(2)
    keep = rng.integers(1, T0 + 1, size=(2, 2, w.Hkv)).astype(np.int32)
    budget = keep.copy()
    budget[0, 0, 0] = T0 + 10                                 # still filling: appends 10, then evicts
    budget[1, 1, 1] = T0 + steps + 5                          # never full: only appends
    keep[0, 0, 0] = keep[1, 1, 1] = T0
    r = oracle.compress(Kn, Vn, "bf16", [T0, T0], keep, t_cap_out=T0)
    st = _state_from(r, T0 + steps)
    assert st["cur_len"].shape == (2, 2, w.Hkv)
    allK = [Kn]
    for s in range(steps):
        k, v = synth.make_new_kv(w, s, "cpu")
        kn, vn = synth.to_numpy(k), synth.to_numpy(v)
        assert oracle.append_evict(st, "bf16", budget, (), kn, vn, [T0 + s, T0 + s]) == 0
        allK.append(kn[:, :, :, None])
    key = oracle.key_sumsq(np.concatenate(allK, 3), "bf16")
    T = T0 + steps
    for b, l, h in itertools.product(range(2), range(2), range(w.Hkv)):
        n = min(int(budget[b, l, h]), T)
        assert st["cur_len"][b, l, h] == n
        want = sorted(sorted(range(T), key=lambda t: (key[b, l, h, t], t))[:n])
        assert sorted(st["idx"][b, l, h, :n].tolist()) == want


def test_append_evict_cases():
    D = 64
    def row(c):
        r = np.zeros((1, 1, 1, D), np.float32); r[..., 0] = c; return r
    st = dict(K_c=np.zeros((1, 1, 1, 4, D), np.float32), V_c=np.zeros((1, 1, 1, 4, D), np.float32),
              idx=np.full((1, 1, 1, 4), -1, np.int32), key=np.full((1, 1, 1, 4), np.nan),
              cur_len=np.zeros((1, 1), np.int32))
    for t, c in enumerate([3.0, 5.0, 5.0]):                       # under budget: plain append
        oracle.append_evict(st, "f32", [3], (), row(c), row(10 + t), [t])
    assert st["cur_len"][0, 0] == 3 and st["idx"][0, 0, 0, :3].tolist() == [0, 1, 2]
    assert st["key"][0, 0, 0, :3].tolist() == [9.0, 25.0, 25.0]
    oracle.append_evict(st, "f32", [3], (), row(4.0), row(13), [3])  # tie at 25: the later one goes
    assert st["idx"][0, 0, 0, :3].tolist() == [0, 1, 3] and st["V_c"][0, 0, 0, 2, 0] == 13
    before = {k: v.copy() for k, v in st.items()}
    oracle.append_evict(st, "f32", [3], (), row(6.0), row(14), [4])  # newcomer is the largest: dropped
    assert all(np.array_equal(before[k], st[k], equal_nan=True) for k in st)
    oracle.append_evict(st, "f32", [3], (), row(5.0), row(15), [5])  # ties the stored 25 but is later: dropped
    assert st["idx"][0, 0, 0, :3].tolist() == [0, 1, 3]
    oracle.append_evict(st, "f32", [3], (0,), row(9.0), row(16), [6])  # uncompressed layer: grows
    assert st["cur_len"][0, 0] == 4 and st["idx"][0, 0, 0, 3] == 6
    assert oracle.append_evict(st, "f32", [3], (0,), row(1.0), row(17), [7]) == -2  # no room
    assert st["cur_len"][0, 0] == 4


# ------------------------------------------------- keep-random ablation policy

def test_random_key_is_splitmix64():
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "splitmix64.json")))
    gamma, mask = 0x9E3779B97F4A7C15, (1 << 64) - 1
    for k, out in enumerate(g["outputs"]):
        # the k-th output of the sequential generator is the output function at seed + k * gamma
        assert oracle.random_key((g["seed"] + k * gamma) & mask, 0, 0) == int(out) >> 32
    # the counter is seed + (unit * 2^32 + t)
    assert oracle.random_key(5, 3, 9) == oracle.random_key(5 + (3 << 32) + 9, 0, 0)
    assert oracle.random_key(5, 3, 9) != oracle.random_key(5, 3, 10)


def test_random_policy_keeps_the_lowest_random_keys():
    w, K, V = _tiny("f32", L=2, T=200)
    keep = 50
    r = oracle.compress(K, V, "f32", [w.T], [keep], uncompressed=(0,), policy=2, seed=77)
    s = oracle.key_sumsq(K, "f32")
    assert r["kept_len"].tolist() == [[w.T, keep]]
    counts = np.zeros(w.T)
    for h in range(w.Hkv):
        u = (0 * w.L + 1) * w.Hkv + h
        want = sorted(sorted(range(w.T), key=lambda t: (oracle.random_key(77, u, t), t))[:keep])
        idx = r["idx"][0, 1, h, :keep]
        assert idx.tolist() == want
        assert np.array_equal(r["K_c"][0, 1, h, :keep], K[0, 1, h, idx])
        assert np.array_equal(r["key"][0, 1, h, :keep], s[0, 1, h, idx])    # stored keys stay norms
        counts[idx] += 1
    again = oracle.compress(K, V, "f32", [w.T], [keep], uncompressed=(0,), policy=2, seed=77)
    other = oracle.compress(K, V, "f32", [w.T], [keep], uncompressed=(0,), policy=2, seed=78)
    assert np.array_equal(again["idx"], r["idx"]) and not np.array_equal(other["idx"], r["idx"])
    assert counts.max() <= w.Hkv and 0 < (counts > 0).mean() < 1             # heads differ
    # over many seeds every position is kept about keep / T of the time
    freq = np.zeros(w.T)
    for seed in range(200):
        freq[oracle.compress(K, V, "f32", [w.T], [keep], uncompressed=(0,), policy=2,
                             seed=seed)["idx"][0, 1, 0, :keep]] += 1
    assert abs(freq.mean() / 200 - keep / w.T) < 1e-12 and freq.min() > 20 and freq.max() < 85


# ----------------------------------------- attention loss / ALR (Eqs. 5-7)

def test_attention_loss_hand_worked():
    g = json.load(open(GOLDEN))["attention_loss"]
    ln = np.log([1.0, 2.0, 3.0])
    K = np.zeros((1, 1, 1, 3, 4), np.float64)
    K[0, 0, 0, :, 0] = ln
    K[0, 0, 0, :, 1] = np.sqrt(np.array([4.0, 1.0, 9.0]) - ln ** 2)    # norms 2, 1, 3
    q = np.array([2, 0, 0, 0], np.float32).reshape(1, 1, 1, 4)
    alr, loss, ref = oracle.attention_loss(q, K.astype(np.float32), "f32", [3], curves=True)
    np.testing.assert_allclose(loss[0, 0, 0], g["loss"], atol=1e-6)
    np.testing.assert_allclose(ref[0, 0, 0], g["loss_ref"], atol=1e-6)
    np.testing.assert_allclose(alr[0, 0, 0], g["alr"], atol=2e-6)


def test_attention_loss_invariants_and_brute_force():
    rng = np.random.default_rng(11)
    D, n = 64, 9
    q = rng.standard_normal((1, 1, 4, D)).astype(np.float32)
    K = (rng.standard_normal((1, 1, 2, n, D)) * rng.uniform(0.3, 2, (1, 1, 2, n, 1))).astype(np.float32)
    alr, loss, ref = oracle.attention_loss(q, K, "f32", [n], curves=True)
    s = oracle.key_sumsq(K, "f32")
    for j in range(4):
        h = j // 2
        z = K[0, 0, h].astype(np.float64) @ q[0, 0, j].astype(np.float64) / math.sqrt(D)
        a = scipy.special.softmax(z)
        drop = sorted(range(n), key=lambda t: (s[0, 0, h, t], t), reverse=True)
        for m in range(1, n + 1):
            np.testing.assert_allclose(loss[0, 0, j, m - 1], a[drop[:m]].sum(), rtol=1e-12)
            # the ideal compression loses the least attention any m-subset can lose
            best = min(sum(a[list(c)]) for c in itertools.combinations(range(n), m))
            np.testing.assert_allclose(ref[0, 0, j, m - 1], best, rtol=1e-12)
        assert np.all(loss[0, 0, j] >= ref[0, 0, j] - 1e-15)                    # Y^m >= 0
        np.testing.assert_allclose(loss[0, 0, j, -1], 1.0, rtol=1e-12)
        np.testing.assert_allclose(alr[0, 0, j], (loss[0, 0, j] - ref[0, 0, j]).sum(), rtol=1e-12)
        # rank identity: Y = sum_p a_p (rank in ideal order - rank in the method's drop order)
        rank_n = np.empty(n); rank_n[drop] = np.arange(1, n + 1)
        rank_a = np.empty(n); rank_a[np.argsort(a, kind="stable")] = np.arange(1, n + 1)
        np.testing.assert_allclose(alr[0, 0, j], (a * (rank_a - rank_n)).sum(), rtol=1e-10, atol=1e-12)
    # a cache whose norms fall exactly as the attention rises has no loss at all
    Kc = np.zeros((1, 1, 1, 5, D), np.float32)
    Kc[0, 0, 0, :, 0] = [0.5, 0.4, 0.3, 0.2, 0.1]        # scores rise with ... the first coordinate
    Kc[0, 0, 0, :, 1] = [0.0, 1.0, 2.0, 3.0, 4.0]        # norms rise the other way round
    qc = np.zeros((1, 1, 1, D), np.float32); qc[..., 0] = 8.0
    assert abs(oracle.attention_loss(qc, Kc, "f32", [5])[0, 0, 0]) < 1e-15
    assert oracle.attention_loss(qc, Kc, "f32", [0])[0, 0, 0] == 0.0
