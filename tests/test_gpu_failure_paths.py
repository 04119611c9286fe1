"""Failure paths on the GPU, exercised without faulting anything: a bounded wait that runs out
(a barrier nothing completes; no copy in flight), the sticky abort mark and its reset, stale
completion counters, and the bounds-checked debug build of the library."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import synth
from gpu_util import DEV, i32, gpu_compress

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def l2():
    import paper_2406_11430_b200 as lib
    lib.lib()
    return lib


def test_a_wait_that_runs_out_is_reported_stops_later_calls_and_can_be_cleared(l2):
    w = synth.WORKLOADS[2].scaled(B=1, L=2, T=2100)
    K, V = synth.make_cache(w, DEV)
    q = synth.make_query(w, 0, DEV)
    cur = i32([[2100, 700]])
    lay = l2.Layout(K, q_heads=w.Hq)
    ws = l2.new_workspace(lay, w.T, DEV)
    good = torch.empty(q.shape, dtype=torch.float32, device=DEV)
    l2.decode_attention(q, K, V, cur, w.T, good, ws)
    assert l2.read_device_status(ws) == 0

    l2.selftest_wait_timeout(ws)                              # returns; the context stays usable
    assert l2.read_device_status(ws) == -8
    assert l2.status_string(-8) != "unknown status"
    # the mark is sticky: decode and prefix attention on this workspace now write nothing
    out = torch.full(q.shape, 7.0, dtype=torch.float32, device=DEV)
    l2.decode_attention(q, K, V, cur, w.T, out, ws)
    qp = torch.zeros((1, 2, 8, w.Hq, w.D), dtype=torch.bfloat16, device=DEV)
    op = torch.full(qp.shape, 7.0, dtype=torch.float32, device=DEV)
    l2.prefix_attention(qp, K, V, cur, w.T, op, workspace=ws)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all()) and bool((op == 7.0).all())
    assert l2.read_device_status(ws) == -8

    l2.workspace_reset(ws, lay)
    l2.decode_attention(q, K, V, cur, w.T, out, ws)
    torch.cuda.synchronize()
    assert l2.read_device_status(ws) == 0
    assert torch.equal(out, good)


def test_stale_completion_counters_are_cleared_by_a_reset(l2):
    """What a launch that died midway leaves behind: counters that do not rest at zero."""
    w = synth.WORKLOADS[2].scaled(B=2, L=2, T=2500)
    K, V = synth.make_cache(w, DEV)
    lens, keep = [2500, 1200], [1250, 600]
    _, want = gpu_compress(l2, K, V, lens, keep)
    lay = l2.Layout(K)
    ws = l2.new_workspace(lay, w.T, DEV)
    ws[256:256 + 4 * w.B * w.L * w.Hkv] = 1                   # every unit's counter is off
    l2.workspace_reset(ws, lay)
    K_c, V_c = torch.zeros_like(K), torch.zeros_like(K)
    idx = torch.full(K.shape[:4], -1, dtype=torch.int32, device=DEV)
    sumsq = torch.full(K.shape[:4], float("nan"), dtype=torch.float32, device=DEV)
    kl = torch.zeros((w.B, w.L), dtype=torch.int32, device=DEV)
    l2.select_compact(K, V, i32(lens), i32(keep), w.T, (), K_c, V_c, idx, sumsq, kl, ws)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), want["idx"])
    assert np.array_equal(synth.to_numpy(K_c), want["K_c"])


def test_static_scratch_has_a_status_block(l2):
    w = synth.WORKLOADS[2].scaled(B=1, L=1, T=1500)
    K, V = synth.make_cache(w, DEV)
    q = synth.make_query(w, 0, DEV)
    out = torch.empty(q.shape, dtype=torch.float32, device=DEV)
    l2.decode_attention_static(q, K, V, i32([[1500]]), w.T, out)
    assert l2.decode_attention_static_status() == 0
    assert l2.decode_attention_static_status(reset=True) == 0


def test_parity_cases_pass_on_the_bounds_checked_build():
    """The tiny-shape and ragged parity cases again, in a fresh process bound to the library
    built with -DL2KV_DEBUG: any index outside its range would be recorded and the access
    skipped, so the comparisons with the oracle (and the status checks inside those tests)
    would fail."""
    from paper_2406_11430_b200 import build as l2build
    lib = l2build.build_debug()
    env = dict(os.environ, L2KV_LIBRARY=lib)
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu",
                        os.path.join(ROOT, "tests", "test_gpu_parity.py"),
                        os.path.join(ROOT, "tests", "test_gpu_packed.py"),
                        os.path.join(ROOT, "tests", "test_gpu_per_head.py")],
                       env=env, cwd=ROOT, capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
