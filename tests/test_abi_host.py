"""Host-side checks of the C library that need no GPU: every declared symbol is
exported, and argument validation returns the documented codes without launching."""
import ctypes
import os
import re

import pytest
import torch

import paper_2406_11430_b200 as l2
from paper_2406_11430_b200 import build as l2build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_builds_and_exports_every_declared_symbol():
    l2build.build()
    lib = ctypes.CDLL(l2.library_path())
    names = set()
    for hdr in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", hdr)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(l2kv_[a-z0-9_]+)\s*\(", text))
    assert {"l2kv_key_norms", "l2kv_select_compact", "l2kv_decode_attention",
            "l2kv_append_evict"} <= names
    for n in names:
        assert hasattr(lib, n), n


def test_keep_count_and_status_strings():
    assert l2.keep_count(4096, 0.5) == 2048
    assert l2.keep_count(131072, 0.1) == 13108
    assert l2.keep_count(10, 0.0) == 1 and l2.keep_count(10, 3.0) == 10 and l2.keep_count(0, 0.5) == 0
    assert l2.status_string(0) == "ok"
    for code in range(-7, 0):
        assert l2.status_string(code) not in ("ok", "unknown status")
    with pytest.raises(l2.L2KVError):
        l2.keep_count(-1, 0.5)


def _fake(shape, dtype=torch.bfloat16):
    return torch.empty(shape, dtype=dtype)          # host tensor: only used for failing checks


def test_validation_rejects_before_launch():
    K = _fake((1, 2, 4, 128, 128))
    lay = l2.Layout(K)
    assert l2.workspace_bytes(lay, 128) > 256
    with pytest.raises(l2.L2KVError) as e:          # head_dim outside {64, 128}
        l2.workspace_bytes(l2.Layout(_fake((1, 1, 1, 8, 32))), 8)
    assert e.value.status == -2
    ws = _fake((l2.workspace_bytes(lay, 128),), torch.uint8)
    lens = torch.zeros(1, dtype=torch.int32)
    out = _fake((1, 2, 4, 128), torch.float32)
    with pytest.raises(l2.L2KVError) as e:          # max_len beyond t_cap
        l2.key_norms(K, lens, 129, out)
    assert e.value.status == -5
    Ko = _fake((1, 2, 4, 64, 128))
    idx = torch.zeros((1, 2, 4, 64), dtype=torch.int32)
    kl = torch.zeros((1, 2), dtype=torch.int32)
    args = (K, K, lens, lens, 128)
    with pytest.raises(l2.L2KVError) as e:          # layer index out of range
        l2.select_compact(*args, (2,), Ko, Ko, idx, out, kl, ws)
    assert e.value.status == -5
    with pytest.raises(l2.L2KVError) as e:          # uncompressed layers do not fit the output
        l2.select_compact(*args, (0,), Ko, Ko, idx, out, kl, ws)
    assert e.value.status == -5
    with pytest.raises(l2.L2KVError) as e:          # workspace too small
        l2.select_compact(*args, (), Ko, Ko, idx, out, kl, ws[:512])
    assert e.value.status == -4
    with pytest.raises(l2.L2KVError) as e:          # bad policy
        l2.select_compact(*args, (), Ko, Ko, idx, out, kl, ws, policy=7)
    assert e.value.status == -1
    with pytest.raises(l2.L2KVError) as e:          # misaligned base pointer
        l2.select_compact(K.view(-1)[4:4 + 128 * 128].view(1, 1, 1, 128, 128), K, lens, lens, 128,
                          (), Ko[:, :1, :1], Ko[:, :1, :1], idx, out, kl, ws)
    assert e.value.status == -3
    q = _fake((1, 2, 12, 128))
    with pytest.raises(l2.L2KVError) as e:          # 12 query heads over 4 KV heads: G = 3
        l2.decode_attention(q, K, K, kl, 128, out, ws)
    assert e.value.status == -2
    with pytest.raises(l2.L2KVError) as e:          # null output
        l2.decode_attention(_fake((1, 2, 4, 128)), K, K, kl, 128, None, ws)
    assert e.value.status == -1


def test_validation_of_the_analysis_and_prefix_entry_points():
    K = _fake((1, 2, 4, 128, 128))
    kl = torch.zeros((1, 2), dtype=torch.int32)
    q = _fake((1, 2, 5, 8, 128))
    out = _fake((1, 2, 5, 8, 128), torch.float32)
    with pytest.raises(l2.L2KVError) as e:          # fp32 caches are not served by the tensor-core path
        l2.prefix_attention(q.float(), K.float(), K.float(), kl, 128, out)
    assert e.value.status == -2
    with pytest.raises(l2.L2KVError) as e:          # max_len beyond t_cap
        l2.prefix_attention(q, K, K, kl, 129, out)
    assert e.value.status == -5
    with pytest.raises(l2.L2KVError) as e:          # 12 query heads over 4 KV heads
        l2.prefix_attention(_fake((1, 2, 5, 12, 128)), K, K, kl, 128, out)
    assert e.value.status == -2
    with pytest.raises(l2.L2KVError) as e:          # status workspace too small
        l2.prefix_attention(q, K, K, kl, 128, out, workspace=_fake((16,), torch.uint8))
    assert e.value.status == -4
    sumsq = _fake((1, 2, 4, 128), torch.float32)
    alr = _fake((1, 2, 8), torch.float32)
    qd = _fake((1, 2, 8, 128))
    with pytest.raises(l2.L2KVError) as e:          # workspace too small for the sorts
        l2.attention_loss(qd, K, kl, 128, sumsq, alr, workspace=_fake((1024,), torch.uint8))
    assert e.value.status == -4
    with pytest.raises(l2.L2KVError) as e:          # keys are required
        l2.attention_loss(qd, K, kl, 128, None, alr, workspace=_fake((1 << 20,), torch.uint8))
    assert e.value.status == -1


def _prefix_ws_bytes(B, L, H, Hq, t_cap, max_len, n_q, dtype=torch.bfloat16, D=128):
    cache = torch.empty((B, L, H, t_cap, D), dtype=dtype, device="meta")
    lay = l2.Layout(cache, q_heads=Hq)
    out = ctypes.c_size_t(0)
    rc = l2.lib().l2kv_prefix_attention_workspace_bytes(lay.ref(), max_len, n_q, ctypes.byref(out))
    return rc, out.value


def test_prefix_attention_workspace_plan():
    """Host side of the split over the cache: room for partial results is asked for only when
    the unsplit grid would leave SMs idle or the cache is very long; sizes follow from the plan."""
    rows = lambda B, L, n_q, Hq: B * L * n_q * Hq
    persistent = 256 + 2 * 148 * 256 * 129 * 4
    # the benchmark call (all 32 layers, 2048 CTAs): no split
    assert _prefix_ws_bytes(4, 32, 8, 32, 32768, 32768, 128) == (0, 256)
    # one layer of it (64 CTAs unsplit, 256 sub-blocks each): the work-balanced kernel -- two
    # partial results of 256 rows (129 floats each) per CTA of its fixed grid of 148
    assert _prefix_ws_bytes(4, 1, 8, 32, 32768, 16384, 128) == (0, persistent)
    # a small grid with little work per CTA is cut into chunks: scratch = chunks * rows * (128 + 1) floats
    rc, b = _prefix_ws_bytes(4, 1, 8, 32, 4096, 4096, 128)
    per_chunk = rows(4, 1, 128, 32) * 129 * 4
    assert rc == 0 and b > 256 and (b - 256) % per_chunk == 0 and 2 <= (b - 256) // per_chunk <= 16
    # a very long cache goes to the work-balanced kernel whatever the grid
    assert _prefix_ws_bytes(1, 32, 8, 32, 131072, 131072, 128) == (0, persistent)
    assert _prefix_ws_bytes(2, 4, 8, 32, 70000, 70000, 64)[1] == persistent
    # short caches are never split below 1024 tokens; unsupported types ask for the status block only
    assert _prefix_ws_bytes(1, 1, 2, 8, 1000, 1000, 16) == (0, 256)
    assert _prefix_ws_bytes(1, 1, 4, 4, 1024, 1024, 16, dtype=torch.float32, D=64) == (0, 256)
    assert _prefix_ws_bytes(1, 1, 8, 32, 4096, 8192, 16)[0] == -5          # max_len beyond t_cap
