"""Parity at the benchmark configurations' full sizes, in the launch configuration the
benchmark times: the library runs on the whole cache; the oracle recomputes a seeded
sample of (batch, layer, KV head) units one by one, and properties that hold at any
size are checked on everything (with torch ops on the GPU, not with the library)."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import DEV, i32, assert_attention_close, compare_with_band

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def l2():
    import paper_2406_11430_b200 as lib
    lib.lib()
    return lib


def _free():
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def compress_all(l2, w, K, V, lens, keep, t_cap_out):
    shape = (w.B, w.L, w.Hkv, t_cap_out, w.D)
    out = dict(K_c=torch.zeros(shape, dtype=K.dtype, device=DEV),
               V_c=torch.zeros(shape, dtype=K.dtype, device=DEV),
               idx=torch.full(shape[:4], -1, dtype=torch.int32, device=DEV),
               sumsq=torch.zeros(shape[:4], dtype=torch.float32, device=DEV),
               cur=torch.zeros((w.B, w.L), dtype=torch.int32, device=DEV))
    out["ws"] = l2.new_workspace(l2.Layout(out["K_c"], q_heads=w.Hq), t_cap_out, DEV)
    l2.select_compact(K, V, i32(lens), i32(keep), int(max(lens)), w.uncompressed, out["K_c"],
                      out["V_c"], out["idx"], out["sumsq"], out["cur"], out["ws"])
    torch.cuda.synchronize()
    return out


def check_properties(w, K, V, out, lens, keep):
    """Whole-cache checks that need no oracle: lengths, ordered index map, rows are the rows
    the index map names."""
    cur = out["cur"].cpu().numpy()
    for b in range(w.B):
        for l in range(w.L):
            n = lens[b] if l in w.uncompressed else keep[b]
            assert cur[b, l] == n
            idx = out["idx"][b, l, :, :n].long()
            assert bool((idx[:, 1:] > idx[:, :-1]).all()) and int(idx.max()) < lens[b]
            gi = idx.unsqueeze(-1).expand(-1, -1, w.D)
            assert torch.equal(out["K_c"][b, l, :, :n], torch.gather(K[b, l], 1, gi))
            assert torch.equal(out["V_c"][b, l, :, :n], torch.gather(V[b, l], 1, gi))


def check_sampled_units(w, K, V, out, lens, keep, units):
    """Oracle recomputation of sampled compressed units (b, l, h): index map, rows and keys
    bit-exact against the fp32-ordered keys, and equal to the fp64 selection outside the band."""
    swaps = 0
    for (b, l, h) in units:
        n_in, n = lens[b], keep[b]
        Kn = synth.to_numpy(K[b, l, h, :n_in])[None, None, None]
        Vn = synth.to_numpy(V[b, l, h, :n_in])[None, None, None]
        ex = oracle.compress(Kn, Vn, w.dtype, [n_in], [n], key_mode=1)
        assert np.array_equal(out["idx"][b, l, h, :n].cpu().numpy(), ex["idx"][0, 0, 0, :n])
        assert np.array_equal(synth.to_numpy(out["K_c"][b, l, h, :n]), ex["K_c"][0, 0, 0, :n])
        assert np.array_equal(synth.to_numpy(out["V_c"][b, l, h, :n]), ex["V_c"][0, 0, 0, :n])
        assert np.array_equal(out["sumsq"][b, l, h, :n].cpu().numpy().astype(np.float64),
                              ex["key"][0, 0, 0, :n])
        ref = oracle.compress(Kn, Vn, w.dtype, [n_in], [n], key_mode=0)
        swaps += compare_with_band(ex["idx"][0, 0, 0, :n], ref["idx"][0, 0, 0, :n],
                                   oracle.key_sumsq(Kn, w.dtype)[0, 0, 0], n)
    return swaps


def check_sampled_attention(l2, w, out, q, max_len, samples):
    """Runs decode attention on everything; the oracle recomputes sampled (b, l, kv head) groups."""
    res = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
    l2.decode_attention(q, out["K_c"], out["V_c"], out["cur"], max_len, res, out["ws"])
    torch.cuda.synchronize()
    assert bool(torch.isfinite(res).all())
    G = w.Hq // w.Hkv
    cur = out["cur"].cpu().numpy()
    worst = 0.0
    for (b, l, h) in samples:
        n = int(cur[b, l])
        Kn = synth.to_numpy(out["K_c"][b, l, h, :n])[None, None, None]
        Vn = synth.to_numpy(out["V_c"][b, l, h, :n])[None, None, None]
        qn = synth.to_numpy(q[b, l, h * G:(h + 1) * G])[None, None]
        want = oracle.attention(qn, Kn, Vn, w.dtype, [[n]], nthreads=8)
        worst = max(worst, assert_attention_close(res[b, l, h * G:(h + 1) * G].cpu().numpy()[None, None], want))
    return res, worst


def test_config1_llama2_7b_4k(l2):
    w = synth.WORKLOADS[1]
    K, V = synth.make_cache(w, DEV)
    lens, keep = [w.T], [oracle.keep_count(w.T, w.keep_ratio)]
    out = compress_all(l2, w, K, V, lens, keep, w.T)
    check_properties(w, K, V, out, lens, keep)
    units = [(0, 0, 0), (0, 5, 17), (0, 31, 31), (0, 16, 3)]
    check_sampled_units(w, K, V, out, lens, keep, units)
    assert bool((out["idx"][0, :, :, 0] == 0).all())        # the low-norm first token survives
    q = synth.make_query(w, 0, DEV)
    check_sampled_attention(l2, w, out, q, w.T, units)
    _free()


def test_config2_llama3_8b_32k(l2):
    w = synth.WORKLOADS[2]
    K, V = synth.make_cache(w, DEV)
    lens, keep = [w.T] * w.B, [oracle.keep_count(w.T, w.keep_ratio)] * w.B
    out = compress_all(l2, w, K, V, lens, keep, w.T)
    check_properties(w, K, V, out, lens, keep)
    units = [(0, 2, 0), (1, 17, 5), (3, 31, 7), (2, 9, 3)]
    swaps = check_sampled_units(w, K, V, out, lens, keep, units)
    print(f"config 2: {swaps} fp32/fp64 swaps inside the tie band over {len(units)} sampled units")
    del K, V
    _free()
    for step in (0, w.decode_steps - 1):                    # first and last decode step
        q = synth.make_query(w, step, DEV)
        check_sampled_attention(l2, w, out, q, w.T, units + [(0, 0, 1), (3, 1, 6)])
    _free()
    check_sampled_prefix_attention(l2, w, out, [(0, 2, 0, 0), (1, 17, 5, 127), (3, 31, 7, 64), (2, 9, 3, 31),
                                               (0, 0, 1, 100), (3, 1, 6, 5)])
    _free()


def check_sampled_prefix_attention(l2, w, out, samples, n_q=128, room=False):
    """Prefix attention in the launch the benchmark times (128 queries per (b, l) over the whole
    compressed cache), plain and causal, both forms of the weights; the oracle recomputes the
    sampled (b, l, kv head, query) rows with that row's own length.  room: with the workspace
    the library asks for (very long caches then go to the work-balanced kernel)."""
    g = torch.Generator().manual_seed(17)
    q = torch.randn((w.B, w.L, n_q, w.Hq, w.D), generator=g).to(torch.bfloat16).to(DEV)
    res = torch.empty(q.shape, dtype=torch.float32, device=DEV)
    ws = (l2.prefix_attention_workspace(out["K_c"], q, w.T) if room
          else torch.zeros(256, dtype=torch.uint8, device=DEV))
    assert (ws.numel() > 256) == room
    G = w.Hq // w.Hkv
    cur = out["cur"].cpu().numpy()
    for causal in (False, True):
        for weights, atol in (("split", 2e-3), ("single", 4e-3)):
            flags = (l2.PREFIX_CAUSAL if causal else 0) | (l2.PREFIX_SPLIT_WEIGHTS if weights == "split" else 0)
            res.fill_(float("nan"))
            l2.prefix_attention_flags(q, out["K_c"], out["V_c"], out["cur"], w.T, res, flags, workspace=ws)
            torch.cuda.synchronize()
            assert l2.read_device_status(ws) == 0
            assert bool(torch.isfinite(res).all())
            worst = 0.0
            for (b, l, h, s) in samples:
                n = int(cur[b, l]) - (n_q - s - 1 if causal else 0)
                Kn = synth.to_numpy(out["K_c"][b, l, h, :n])[None, None, None]
                Vn = synth.to_numpy(out["V_c"][b, l, h, :n])[None, None, None]
                qn = synth.to_numpy(q[b, l, s, h * G:(h + 1) * G])[None, None]
                want = oracle.attention(qn, Kn, Vn, w.dtype, [[n]], nthreads=8)
                got = res[b, l, s, h * G:(h + 1) * G].cpu().numpy()[None, None]
                worst = max(worst, assert_attention_close(got, want, atol=atol))
            print(f"prefix attention at full size, causal={causal}, {weights} weights: worst error {worst:.2e}")


def test_config3_extreme_128k(l2):
    w = synth.WORKLOADS[3]
    K, V = synth.make_cache(w, DEV)
    lens, keep = [w.T], [oracle.keep_count(w.T, w.keep_ratio)]
    assert keep[0] == 13108
    out = compress_all(l2, w, K, V, lens, keep, w.T)
    check_properties(w, K, V, out, lens, keep)
    units = [(0, 2, 0), (0, 30, 7), (0, 13, 4)]
    check_sampled_units(w, K, V, out, lens, keep, units)
    for l in range(2, w.L):                                  # every planted token is kept
        pos = synth.planted_positions(w, 0, l, DEV)
        kept = out["idx"][0, l, :, :keep[0]].long()
        for h in range(w.Hkv):
            assert bool(torch.isin(pos[h], kept[h]).all())
    del K, V
    _free()
    q = synth.make_query(w, 0, DEV)
    check_sampled_attention(l2, w, out, q, w.T, units + [(0, 1, 2)])
    _free()
    # 128 queries over the whole compressed cache (two layers of 131072 rows, thirty of 13108):
    # the work-balanced kernel, every item cut across several thread blocks
    check_sampled_prefix_attention(l2, w, out, [(0, 0, 0, 0), (0, 1, 7, 127), (0, 2, 0, 64), (0, 30, 7, 31),
                                               (0, 13, 4, 100)], room=True)
    _free()


def test_config4_serving_ragged_budget(l2):
    # The serving configuration at its stated size: 64 ragged sequences, all 32 layers, 256
    # steps of append + evict + decode attention.  The caches are packed (no padding): the
    # input holds len_b rows per (b, l); in the compressed cache an uncompressed layer has room
    # for len_b + 256 rows and a compressed one for its budget.  The oracle follows three
    # sequences end to end (dense per sequence); properties are checked on everything.
    w = synth.WORKLOADS[4]
    assert (w.B, w.L) == (64, 32)
    lens = synth.ragged_lengths(w).tolist()
    assert min(lens) >= 1024 and max(lens) <= 16384
    budget = [oracle.keep_count(n, 0.5) for n in lens]
    steps, unc = w.append_steps, w.uncompressed
    K, V, rin_host = synth.make_cache_packed(w, lens, DEV)
    rin = l2.Rows(*rin_host, DEV)
    caps = [[lens[b] + steps if l in unc else budget[b] for l in range(w.L)] for b in range(w.B)]
    rout_host = synth.packing(caps)
    ooff, _, total = rout_host
    ioff = rin_host[0]
    rows = l2.Rows(*rout_host, DEV)
    max_len = max(lens) + steps
    out = dict(K_c=torch.zeros((w.Hkv, total, w.D), dtype=K.dtype, device=DEV),
               idx=torch.full((w.Hkv, total), -1, dtype=torch.int32, device=DEV),
               sumsq=torch.zeros((w.Hkv, total), dtype=torch.float32, device=DEV),
               cur=torch.zeros((w.B, w.L), dtype=torch.int32, device=DEV))
    out["V_c"] = torch.zeros_like(out["K_c"])
    out["ws"] = l2.new_workspace(l2.Layout(out["K_c"], q_heads=w.Hq, rows=rows), max_len, DEV)
    l2.select_compact(K, V, i32(lens), i32(budget), max(lens), unc, out["K_c"], out["V_c"], out["idx"],
                      out["sumsq"], out["cur"], out["ws"], rows_in=rin, rows_out=rows)
    torch.cuda.synchronize()
    # whole-cache properties: lengths, ordered index map, rows are the rows the index map names
    cur = out["cur"].cpu().numpy()
    for b in range(w.B):
        for l in range(w.L):
            n = lens[b] if l in unc else budget[b]
            assert cur[b, l] == n
            o, i0 = int(ooff[b, l]), int(ioff[b, l])
            idx = out["idx"][:, o:o + n].long()
            assert bool((idx[:, 1:] > idx[:, :-1]).all()) and int(idx.max()) < lens[b]
            gi = idx.unsqueeze(-1).expand(-1, -1, w.D)
            assert torch.equal(out["K_c"][:, o:o + n], torch.gather(K[:, i0:i0 + lens[b]], 1, gi))
            assert torch.equal(out["V_c"][:, o:o + n], torch.gather(V[:, i0:i0 + lens[b]], 1, gi))

    follow = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 7})
    states = {}
    for b in follow:
        Kn = np.stack([synth.to_numpy(K[:, int(ioff[b, l]):int(ioff[b, l]) + lens[b]]) for l in range(w.L)])[None]
        Vn = np.stack([synth.to_numpy(V[:, int(ioff[b, l]):int(ioff[b, l]) + lens[b]]) for l in range(w.L)])[None]
        r = oracle.compress(Kn, Vn, w.dtype, [lens[b]], [budget[b]], unc, key_mode=1,
                            t_cap_out=lens[b], nthreads=8)
        t_cap = lens[b] + steps
        st = dict(K_c=np.zeros((1, w.L, w.Hkv, t_cap, w.D), np.uint16),
                  idx=np.full((1, w.L, w.Hkv, t_cap), -1, np.int32),
                  key=np.full((1, w.L, w.Hkv, t_cap), np.nan), cur_len=r["kept_len"].copy())
        st["V_c"] = np.zeros_like(st["K_c"])
        for name in ("K_c", "V_c", "idx", "key"):
            st[name][:, :, :, :lens[b]] = r[name]
        states[b] = st
    del K, V, Kn, Vn, r
    _free()

    def compare(b):
        st = states[b]
        cur_b = out["cur"][b].cpu().numpy()
        assert np.array_equal(cur_b, st["cur_len"][0])
        for l in range(w.L):
            n, o = int(cur_b[l]), int(ooff[b, l])
            assert np.array_equal(out["idx"][:, o:o + n].cpu().numpy(), st["idx"][0, l, :, :n])
            assert np.array_equal(synth.to_numpy(out["K_c"][:, o:o + n]), st["K_c"][0, l, :, :n])
            assert np.array_equal(synth.to_numpy(out["V_c"][:, o:o + n]), st["V_c"][0, l, :, :n])
            assert np.array_equal(out["sumsq"][:, o:o + n].cpu().numpy().astype(np.float64),
                                  st["key"][0, l, :, :n])

    for b in follow:
        compare(b)
    bud = i32(budget)
    worst = 0.0
    for s in range(steps):
        k, v = synth.make_new_kv(w, s, DEV)
        pos = [n + s for n in lens]
        l2.append_evict(out["K_c"], out["V_c"], out["idx"], out["sumsq"], out["cur"], bud, unc, k, v,
                        i32(pos), out["ws"], rows=rows)
        kn, vn = synth.to_numpy(k), synth.to_numpy(v)
        for b in follow:
            assert oracle.append_evict(states[b], w.dtype, [budget[b]], unc,
                                       np.ascontiguousarray(kn[b:b + 1]),
                                       np.ascontiguousarray(vn[b:b + 1]), [pos[b]], key_mode=1) == 0
        if s in (0, steps // 2, steps - 1):
            q = synth.make_query(w, s, DEV)
            res = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
            l2.decode_attention(q, out["K_c"], out["V_c"], out["cur"], max_len, res, out["ws"], rows=rows)
            torch.cuda.synchronize()
            assert bool(torch.isfinite(res).all())
            for b in follow:
                compare(b)
                st = states[b]
                want = oracle.attention(synth.to_numpy(q[b:b + 1]), st["K_c"], st["V_c"], w.dtype,
                                        st["cur_len"], nthreads=8)
                worst = max(worst, assert_attention_close(res[b:b + 1].cpu().numpy(), want))
    assert l2.read_device_status(out["ws"]) == 0
    print(f"config 4 (32 layers, packed): worst attention error {worst:.2e}")
    cur = out["cur"].cpu().numpy()
    for b in range(w.B):
        assert cur[b].tolist() == [lens[b] + steps] * 2 + [budget[b]] * (w.L - 2)
    _free()
