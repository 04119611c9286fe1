"""GPU parity for packed (ragged, unpadded) caches: the rows of (b, l) are a range of one
shared row axis, each (b, l) with the room it needs and no more.  Every call is compared
with the oracle's packed forms on the same bytes: index maps, rows and keys bit-exact
(fp32-ordered keys), the fp64 selection equal outside the 1e-6 norm band, attention within
|err| <= 2e-3 + 1e-2 |ref|."""
import os

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


class Packed:
    """A compressed packed cache on the device with everything the calls need."""

    def __init__(self, l2, w, rows_host, max_len):
        off, cap, total = rows_host
        self.rows_host = rows_host
        self.rows = l2.Rows(off, cap, total, DEV)
        self.K_c = torch.zeros((w.Hkv, total, w.D), dtype=w.torch_dtype, device=DEV)
        self.V_c = torch.zeros_like(self.K_c)
        self.idx = torch.full((w.Hkv, total), -1, dtype=torch.int32, device=DEV)
        self.sumsq = torch.full((w.Hkv, total), float("nan"), dtype=torch.float32, device=DEV)
        self.cur = torch.zeros((w.B, w.L), dtype=torch.int32, device=DEV)
        self.max_len = min(max_len, self.rows.t_cap)         # what decode attention may be told
        self.ws = l2.new_workspace(l2.Layout(self.K_c, q_heads=w.Hq, rows=self.rows), max_len, DEV)

    def host(self):
        return dict(K_c=synth.to_numpy(self.K_c), V_c=synth.to_numpy(self.V_c),
                    idx=self.idx.cpu().numpy(), key=self.sumsq.cpu().numpy().astype(np.float64),
                    cur_len=self.cur.cpu().numpy())


def assert_states_equal(got, want, rows_host, B, L):
    """Valid rows of every (b, l) equal; nothing is compared past a unit's length."""
    off, cap, _ = rows_host
    assert np.array_equal(got["cur_len"], want["cur_len"])
    for b in range(B):
        for l in range(L):
            sl = slice(int(off[b, l]), int(off[b, l]) + int(want["cur_len"][b, l]))
            for name in ("idx", "K_c", "V_c", "key"):
                assert np.array_equal(got[name][:, sl], want[name][:, sl]), (name, b, l)


def run_packed_pipeline(l2, w, lens, keep, unc, steps, packed_input=True, policy=0):
    B, L = w.B, w.L
    if packed_input:
        K, V, rin_host = synth.make_cache_packed(w, lens, DEV)
        rin = l2.Rows(*rin_host, DEV)
        Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    else:
        K, V = synth.make_cache(w, DEV)
        rin, rin_host = None, synth.packing([[n] * L for n in lens])
        Kn = synth.pack_rows(synth.to_numpy(K), rin_host)
        Vn = synth.pack_rows(synth.to_numpy(V), rin_host)
    caps = [[lens[b] + steps if l in unc else keep[b] for l in range(L)] for b in range(B)]
    rout_host = synth.packing(caps)
    max_len = max(int(max(max(r) for r in caps)), int(max(lens)))   # the workspace serves both sides
    pc = Packed(l2, w, rout_host, max_len)
    l2.select_compact(K, V, i32(lens), i32(keep), int(max(lens)), unc, pc.K_c, pc.V_c, pc.idx,
                      pc.sumsq, pc.cur, pc.ws, policy=policy, seed=5, rows_in=rin, rows_out=pc.rows)
    torch.cuda.synchronize()
    want = oracle.compress_packed(Kn, Vn, w.dtype, rin_host, lens, keep, unc, rout_host, L, key_mode=1,
                                  policy=policy, seed=5, nthreads=8)
    st = dict(K_c=want["K_c"], V_c=want["V_c"], idx=want["idx"], key=want["key"],
              cur_len=want["kept_len"].copy())
    assert_states_equal(pc.host(), st, rout_host, B, L)
    if policy == 0:
        # against the fp64 definition: identical outside the tie band
        ref = oracle.compress_packed(Kn, Vn, w.dtype, rin_host, lens, keep, unc, rout_host, L, nthreads=8)
        ioff, ooff = rin_host[0], rout_host[0]
        got_idx = pc.idx.cpu().numpy()
        for b in range(B):
            for l in range(L):
                if l in unc or keep[b] == 0:
                    continue
                key64 = oracle.key_sumsq(np.ascontiguousarray(Kn[:, ioff[b, l]:ioff[b, l] + lens[b]]), w.dtype)
                for h in range(w.Hkv):
                    o = int(ooff[b, l])
                    compare_with_band(got_idx[h, o:o + keep[b]], ref["idx"][h, o:o + keep[b]], key64[h], keep[b])

    bud = i32(keep)
    for s in range(steps):
        k, v = synth.make_new_kv(w, s, DEV)
        pos = [n + s for n in lens]
        l2.append_evict(pc.K_c, pc.V_c, pc.idx, pc.sumsq, pc.cur, bud, unc, k, v, i32(pos), pc.ws,
                        rows=pc.rows)
        assert oracle.append_evict_packed(st, w.dtype, rout_host, keep, unc, synth.to_numpy(k),
                                          synth.to_numpy(v), pos, key_mode=1) == 0
        if s in (0, steps // 2, steps - 1):
            q = synth.make_query(w, s, DEV)
            out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
            l2.decode_attention(q, pc.K_c, pc.V_c, pc.cur, pc.max_len, out, pc.ws, rows=pc.rows)
            torch.cuda.synchronize()
            assert_states_equal(pc.host(), st, rout_host, B, L)
            ref = oracle.attention_packed(synth.to_numpy(q), st["K_c"], st["V_c"], w.dtype, rout_host,
                                          st["cur_len"], nthreads=8)
            assert_attention_close(out.cpu().numpy(), ref)
    assert l2.read_device_status(pc.ws) == 0
    return pc, st


@pytest.mark.parametrize("copy_mode", ["tma", "cpasync"])
def test_packed_bf16_gqa_pipeline(l2, copy_mode, monkeypatch):
    if copy_mode == "cpasync":
        monkeypatch.setenv("L2KV_DECODE_COPY", "cpasync")
    w = synth.WORKLOADS[2].scaled(B=3, L=3, T=2600)
    run_packed_pipeline(l2, w, lens=[2600, 515, 1029], keep=[1300, 258, 515], unc=(1,), steps=9)


def test_packed_output_from_a_dense_input(l2):
    w = synth.WORKLOADS[2].scaled(B=2, L=2, T=1400)
    run_packed_pipeline(l2, w, lens=[1400, 33], keep=[700, 1], unc=(0,), steps=3, packed_input=False)


@pytest.mark.parametrize("policy", [1, 2])
def test_packed_other_policies(l2, policy):
    w = synth.WORKLOADS[2].scaled(B=2, L=2, T=1100)
    run_packed_pipeline(l2, w, lens=[1100, 600], keep=[400, 599], unc=(), steps=2, policy=policy)


def test_packed_fp32_mha_pipeline(l2):
    w = synth.WORKLOADS[0].scaled(B=3, L=2, T=1500)
    run_packed_pipeline(l2, w, lens=[1500, 2, 700], keep=[750, 1, 350], unc=(0,), steps=5)


def test_packed_key_norms_and_keys_from_write_time(l2):
    w = synth.WORKLOADS[2].scaled(B=2, L=2, T=900)
    lens, keep = [900, 301], [450, 100]
    K, V, rin_host = synth.make_cache_packed(w, lens, DEV)
    rin = l2.Rows(*rin_host, DEV)
    sumsq = torch.full(K.shape[:2], -1.0, dtype=torch.float32, device=DEV)
    norm = torch.full(K.shape[:2], -1.0, dtype=torch.float32, device=DEV)
    l2.key_norms(K, i32(lens), 900, sumsq, norm, rows=rin)
    torch.cuda.synchronize()
    want = oracle.key_sumsq_f32(synth.to_numpy(K), w.dtype)
    assert np.array_equal(sumsq.cpu().numpy(), want)          # packed input has no unused rows
    assert np.array_equal(norm.cpu().numpy(), np.sqrt(want))
    # compression that takes those keys instead of reading K again gives the same cache
    rout_host = synth.packing([[k] * w.L for k in keep])
    a, b = Packed(l2, w, rout_host, 900), Packed(l2, w, rout_host, 900)
    for pc, keys in ((a, None), (b, sumsq)):
        l2.select_compact(K, V, i32(lens), i32(keep), 900, (), pc.K_c, pc.V_c, pc.idx, pc.sumsq, pc.cur,
                          pc.ws, sumsq_in=keys, rows_in=rin, rows_out=pc.rows)
    torch.cuda.synchronize()
    assert_states_equal(a.host(), b.host(), rout_host, w.B, w.L)


def test_packed_overflow_sets_status_and_leaves_neighbours_alone(l2):
    w = synth.WORKLOADS[2].scaled(B=2, L=2, T=64)
    lens, keep, unc = [64, 40], [32, 20], (0,)
    K, V, rin_host = synth.make_cache_packed(w, lens, DEV)
    rout_host = synth.packing([[lens[b] + 1 if l in unc else keep[b] for l in range(2)] for b in range(2)])
    pc = Packed(l2, w, rout_host, 65)
    l2.select_compact(K, V, i32(lens), i32(keep), 64, unc, pc.K_c, pc.V_c, pc.idx, pc.sumsq, pc.cur,
                      pc.ws, rows_in=l2.Rows(*rin_host, DEV), rows_out=pc.rows)
    for s in range(2):                                       # the second append has no row left
        k, v = synth.make_new_kv(w, s, DEV)
        if s == 1:
            torch.cuda.synchronize()
            before = pc.host()
        l2.append_evict(pc.K_c, pc.V_c, pc.idx, pc.sumsq, pc.cur, i32(keep), unc, k, v,
                        i32([n + s for n in lens]), pc.ws, rows=pc.rows)
    assert l2.read_device_status(pc.ws) == -7
    after = pc.host()
    assert after["cur_len"][:, 0].tolist() == [65, 41]       # layer 0 stayed full
    off, cap, _ = rout_host
    for b in range(2):                                       # nothing of the full layer was touched
        sl = slice(int(off[b, 0]), int(off[b, 0] + cap[b, 0]))
        assert np.array_equal(before["K_c"][:, sl], after["K_c"][:, sl])
        assert np.array_equal(before["idx"][:, sl], after["idx"][:, sl])


def test_packed_static_decode(l2):
    w = synth.WORKLOADS[2].scaled(B=2, L=2, T=1300)
    pc, st = run_packed_pipeline(l2, w, lens=[1300, 700], keep=[650, 350], unc=(0,), steps=1)
    q = synth.make_query(w, 7, DEV)
    want = torch.empty(q.shape, dtype=torch.float32, device=DEV)
    got = torch.empty_like(want)
    l2.decode_attention(q, pc.K_c, pc.V_c, pc.cur, pc.max_len, want, pc.ws, rows=pc.rows)
    l2.decode_attention_static(q, pc.K_c, pc.V_c, pc.cur, pc.max_len, got, rows=pc.rows)
    torch.cuda.synchronize()
    assert torch.equal(got, want)


@pytest.mark.parametrize("kernel", ["auto", "persistent"])
def test_packed_prefix_attention(l2, kernel, monkeypatch):
    """Several new queries per (b, l) over a packed compressed cache, plain and causal, both weight
    precisions, against the packed oracle query by query; lengths differ per (b, l).  With the
    library's own choice of kernel and with the work-balanced one."""
    if kernel == "auto":
        monkeypatch.delenv("L2KV_PREFIX_KERNEL", raising=False)
    else:
        monkeypatch.setenv("L2KV_PREFIX_KERNEL", kernel)
    B, L, Hkv, Hq, D, Sq = 3, 2, 2, 8, 128, 40
    w = synth.WORKLOADS[2].scaled(B=B, L=L, Hkv=Hkv, Hq=Hq, T=64)
    caps = [[700, 90], [300, 1], [64, 1500]]
    cur = np.array([[650, 90], [300, 0], [40, 1500]], dtype=np.int32)
    rows_host = synth.packing(caps)
    off, cap, total = rows_host
    rows = l2.Rows(off, cap, total, DEV)
    g = torch.Generator(device="cpu").manual_seed(7)
    K = torch.randn((Hkv, total, D), generator=g).to(torch.bfloat16).to(DEV)
    V = torch.randn((Hkv, total, D), generator=g).to(torch.bfloat16).to(DEV)
    q = torch.randn((B, L, Sq, Hq, D), generator=g).to(torch.bfloat16).to(DEV)
    Kn, Vn = synth.to_numpy(K), synth.to_numpy(V)
    max_len = int(cap.max())
    for causal in (False, True):
        for weights, atol in (("split", 2e-3), ("single", 4e-3)):
            flags = (l2.PREFIX_CAUSAL if causal else 0) | (l2.PREFIX_SPLIT_WEIGHTS if weights == "split" else 0)
            out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=DEV)
            lse = torch.full(q.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
            ws = l2.prefix_attention_workspace(K, q, max_len, rows=rows)
            l2.prefix_attention_flags(q, K, V, i32(cur), max_len, out, flags, lse_out=lse, workspace=ws, rows=rows)
            torch.cuda.synchronize()
            assert l2.read_device_status(ws) == 0
            got = out.cpu().numpy()
            for s in range(Sq):
                n_s = np.maximum(cur - Sq + s + 1, 0) if causal else cur
                want = oracle.attention_packed(synth.to_numpy(q[:, :, s].contiguous()), Kn, Vn, "bf16", rows_host,
                                               n_s, nthreads=4)
                assert_attention_close(got[:, :, s], want, atol=atol)
            assert np.all(np.isneginf(lse.cpu().numpy()[1, 1]))      # the empty cache
