"""The workspace-free decode entry point, for callers that cannot allocate device memory
(see l2kv_decode_attention_static in include/l2kv.h): it must give what the ordinary entry
point gives, call after call, although all its calls share one built-in scratch array.

Collected last on purpose: if this addition breaks, a run that stops at the first failure
has already exercised everything else."""
import numpy as np
import pytest
import torch

import oracle
import synth
from gpu_util import DEV, i32, gpu_attention, assert_attention_close

pytestmark = pytest.mark.gpu


def _static(l2, q, K, V, cur, max_len):
    out = torch.full(q.shape, float("nan"), dtype=torch.float32, device=q.device)
    l2.decode_attention_static(q, K, V, cur, max_len, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    import paper_2406_11430_b200 as l2
    w = synth.WORKLOADS[2].scaled(B=2, L=3, T=2600)
    K, V = synth.make_cache(w, DEV)
    # two calls back to back, different queries and different lengths, so that the second
    # one meets whatever the first one left in the shared scratch
    for step, cur in enumerate([[[2600, 1, 1024], [0, 1025, 777]], [[300, 2600, 2], [2600, 0, 2047]]]):
        q = synth.make_query(w, step, DEV)
        cur_dev = i32(np.asarray(cur))
        want = gpu_attention(l2, q, K, V, cur_dev)
        got = _static(l2, q, K, V, cur_dev, w.T)
        assert_attention_close(got, want.astype(np.float64))
        np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-7)
        # and against the definition itself, not only the other entry point
        ref = oracle.attention(synth.to_numpy(q), synth.to_numpy(K), synth.to_numpy(V), w.dtype, cur, nthreads=8)
        assert_attention_close(got, ref)
    # fp32 caches go through the other kernel family; same contract
    w32 = synth.WORKLOADS[0].scaled(T=1500)
    K32, V32 = synth.make_cache(w32, DEV)
    q32 = synth.make_query(w32, 0, DEV)
    cur32 = i32([[1500]])
    np.testing.assert_allclose(_static(l2, q32, K32, V32, cur32, w32.T),
                               gpu_attention(l2, q32, K32, V32, cur32), rtol=1e-6, atol=1e-7)


def test_static_scratch_rejects_problems_beyond_its_size():
    import paper_2406_11430_b200 as l2
    # batch 4 x 32 layers x 32 query heads x 32 splits needs 68 MB of partials: more than the
    # built-in 16 MiB, so the call must refuse (status -4) before launching anything.
    rows = torch.zeros((32768, 128), dtype=torch.bfloat16, device=DEV)
    K = rows.as_strided((4, 32, 8, 32768, 128), (0, 0, 0, 128, 1))
    q = torch.zeros((4, 32, 32, 128), dtype=torch.bfloat16, device=DEV)
    out = torch.zeros((4, 32, 32, 128), dtype=torch.float32, device=DEV)
    cur = torch.zeros((4, 32), dtype=torch.int32, device=DEV)
    with pytest.raises(l2.L2KVError) as e:
        l2.decode_attention_static(q, K, K, cur, 32768, out)
    assert e.value.status == -4
    l2.decode_attention_static(q, K, K, cur, 7168, out)      # 7 splits: 14.9 MB, fits
    torch.cuda.synchronize()
    assert not out.any()                                     # empty caches -> zeros
