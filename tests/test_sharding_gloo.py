"""The N > 1 path on CPU: two gloo ranks each take their share of a batch, compress it and
attend over it on their own (with the oracle standing in for the GPU), and the pieces equal
the unsharded result -- the path needs no exchange of data between ranks.  Also covers the
barrier / max-over-ranks plumbing that the benchmark uses."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import oracle
    import synth
    from paper_2406_11430_b200 import sharding
    r, w_ = sharding.init("gloo")
    assert (r, w_) == (rank, world)
    w = synth.WORKLOADS[2].scaled(B=3, L=2, Hkv=2, Hq=8, T=300)
    K, V = synth.make_cache(w, "cpu")
    q = synth.make_query(w, 0, "cpu")
    lo, hi = sharding.shard_range(w.B, world, rank)
    lens, keep = [300, 123, 77], [150, 60, 77]
    Kn, Vn, qn = (synth.to_numpy(x[lo:hi].contiguous()) for x in (K, V, q))
    res = oracle.compress(Kn, Vn, "bf16", lens[lo:hi], keep[lo:hi], (0,))
    att = oracle.attention(qn, res["K_c"], res["V_c"], "bf16", res["kept_len"])
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), lo=lo, hi=hi, idx=res["idx"], att=att,
             kept=res["kept_len"])
    sharding.barrier()
    t = sharding.max_over_ranks(10.0 + rank)
    assert t == 10.0 + world - 1
    torch.distributed.destroy_process_group()


def test_two_ranks_shard_the_batch_without_exchange(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    import oracle
    import synth
    w = synth.WORKLOADS[2].scaled(B=3, L=2, Hkv=2, Hq=8, T=300)
    K, V = synth.make_cache(w, "cpu")
    q = synth.make_query(w, 0, "cpu")
    full = oracle.compress(synth.to_numpy(K), synth.to_numpy(V), "bf16", [300, 123, 77],
                           [150, 60, 77], (0,))
    att = oracle.attention(synth.to_numpy(q), full["K_c"], full["V_c"], "bf16", full["kept_len"])
    seen = 0
    for rank in range(world):
        z = np.load(os.path.join(tmp_path, f"rank{rank}.npz"))
        lo, hi = int(z["lo"]), int(z["hi"])
        assert np.array_equal(z["idx"], full["idx"][lo:hi])
        assert np.array_equal(z["kept"], full["kept_len"][lo:hi])
        assert np.array_equal(z["att"], att[lo:hi])
        seen += hi - lo
    assert seen == w.B


def test_shard_range_covers_everything_once():
    from paper_2406_11430_b200 import sharding
    for n in (0, 1, 7, 64):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_range(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
