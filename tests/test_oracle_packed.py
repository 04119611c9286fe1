"""The oracle's packed (unpadded, ragged) forms pinned to its dense forms, which the other
pin tests tie to the paper: the same numbers must come out whichever way the rows are laid
out in memory.  The packing itself is checked by hand on a small example."""
import numpy as np
import pytest

import oracle
import synth


def test_packing_by_hand():
    off, cap, total = synth.packing([[3, 1], [0, 5]])
    assert off.tolist() == [[0, 3], [4, 4]] and cap.tolist() == [[3, 1], [0, 5]] and total == 9
    dense = np.arange(2 * 2 * 2 * 5).reshape(2, 2, 2, 5).astype(np.float32)
    p = synth.pack_rows(dense, (off, cap, total))
    # head 0: (0,0) rows 0..2, (0,1) row 0, (1,1) rows 0..4
    assert p[0].tolist() == [0, 1, 2, 10, 30, 31, 32, 33, 34]
    assert p[1].tolist() == [5, 6, 7, 15, 35, 36, 37, 38, 39]
    back = synth.unpack_rows(p, (off, cap, total), 2, 2, 5)
    assert back[0, 0, 1].tolist() == [5, 6, 7, 0, 0] and back[1, 0].tolist() == [[0] * 5] * 2


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("policy", [0, 1, 2])
def test_packed_compress_attention_append_equal_dense(dtype, policy):
    B, L, T0, steps, unc = 3, 3, 90, 12, (1,)
    w = synth.WORKLOADS[2].scaled(dtype=dtype, B=B, L=L, T=T0, Hkv=2, Hq=4, D=64)
    lens, keep = [90, 7, 41], [45, 7, 5]
    K, V = synth.make_cache(w, "cpu")
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    t_cap = T0 + steps
    dense = oracle.compress(Kn, Vn, dtype, lens, keep, unc, policy=policy, seed=9, t_cap_out=t_cap)

    # packed input: exactly lens[b] rows per (b, l); packed output: every (b, l) has just the
    # room it will ever need (layer 1 grows by `steps`, the others never exceed keep[b])
    rin = synth.packing([[n] * L for n in lens])
    rout = synth.packing([[lens[b] + steps if l in unc else keep[b] for l in range(L)] for b in range(B)])
    Kp, Vp = synth.pack_rows(Kn, rin), synth.pack_rows(Vn, rin)
    pk = oracle.compress_packed(Kp, Vp, dtype, rin, lens, keep, unc, rout, L, policy=policy, seed=9)
    assert np.array_equal(pk["kept_len"], dense["kept_len"])
    n_rows = dense["kept_len"]
    for name in ("K_c", "V_c", "idx", "key"):
        assert np.array_equal(synth.pack_rows(dense[name], rout, n_rows),
                              synth.pack_rows(synth.unpack_rows(pk[name], rout, B, L, t_cap), rout, n_rows))

    # the budget-maintained loop and attention, step by step
    sd = dict(K_c=dense["K_c"], V_c=dense["V_c"], idx=dense["idx"], key=dense["key"],
              cur_len=dense["kept_len"].copy())
    sp = dict(K_c=pk["K_c"], V_c=pk["V_c"], idx=pk["idx"], key=pk["key"], cur_len=pk["kept_len"].copy())
    for s in range(steps):
        k, v = synth.make_new_kv(w, s, "cpu")
        kn, vn = synth.to_numpy(k), synth.to_numpy(v)
        pos = [n + s for n in lens]
        assert oracle.append_evict(sd, dtype, keep, unc, kn, vn, pos) == 0
        assert oracle.append_evict_packed(sp, dtype, rout, keep, unc, kn, vn, pos) == 0
        assert np.array_equal(sd["cur_len"], sp["cur_len"])
        for name in ("K_c", "V_c", "idx", "key"):
            assert np.array_equal(synth.pack_rows(sd[name], rout, sd["cur_len"]),
                                  synth.pack_rows(synth.unpack_rows(sp[name], rout, B, L, t_cap),
                                                  rout, sd["cur_len"]))
        q = synth.to_numpy(synth.make_query(w, s, "cpu"))
        a_d = oracle.attention(q, sd["K_c"], sd["V_c"], dtype, sd["cur_len"])
        a_p = oracle.attention_packed(q, sp["K_c"], sp["V_c"], dtype, rout, sp["cur_len"])
        assert np.array_equal(a_d, a_p)
    # one more append: the growing layer has used up its rows -> overflow reported, nothing written
    k, v = synth.make_new_kv(w, steps, "cpu")
    before = {n: a.copy() for n, a in sp.items()}
    assert oracle.append_evict_packed(sp, dtype, rout, keep, unc, synth.to_numpy(k), synth.to_numpy(v),
                                      [n + steps for n in lens]) == -2
    assert np.array_equal(before["cur_len"][:, 1], sp["cur_len"][:, 1])
    o, c, _ = rout
    for b in range(B):                                      # rows of the full layer are untouched
        sl = slice(int(o[b, 1]), int(o[b, 1] + c[b, 1]))
        assert np.array_equal(before["K_c"][:, sl], sp["K_c"][:, sl])


def test_packed_compress_rejects_rows_that_do_not_fit():
    w = synth.WORKLOADS[2].scaled(B=1, L=2, T=16, Hkv=2, Hq=2, D=64)
    K, V = synth.make_cache(w, "cpu")
    rin = synth.packing([[16, 16]])
    Kp, Vp = synth.pack_rows(synth.to_numpy(K), rin), synth.pack_rows(synth.to_numpy(V), rin)
    with pytest.raises(ValueError):                         # layer 0 is copied whole: needs 16 rows
        oracle.compress_packed(Kp, Vp, "bf16", rin, [16], [8], (0,), synth.packing([[8, 8]]), 2)
    with pytest.raises(ValueError):                         # 17 valid rows in a range of 16
        oracle.compress_packed(Kp, Vp, "bf16", rin, [17], [8], (), synth.packing([[8, 8]]), 2)
    oracle.compress_packed(Kp, Vp, "bf16", rin, [16], [8], (0,), synth.packing([[16, 8]]), 2)
