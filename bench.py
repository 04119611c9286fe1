#!/usr/bin/env python
"""Benchmark of the l2kv hot path on B200.

One step = one pass of the whole path over one synthetic batch of the Llama-3-8B
32k-context workload: a compression pass over the full cache (key norms, selection,
compaction; the uncompressed layers are copied) followed by the workload's 64
single-query decode-attention steps over the compressed cache.  The metric is the
throughput of KV bytes the algorithm has to move (GB/s), reported with the fraction
of the HBM roofline, plus decode tokens/s.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl l2kv|reference]

With N > 1 (under torchrun) every rank runs the same per-GPU workload on its own
batch: the path shards over independent (batch, layer, head) units with no exchange,
so there is no collective on the data path (weak scaling).
"""
import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

GIB = 1 << 30
METRIC = "compress + decode GB/s of KV read and % of B200 HBM peak; decode tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + written) per algorithmic byte of the dominant kernel, from an ncu capture of
# the decode split kernel on a 4-layer case of the benchmark workload (the traffic is
# proportional to the tokens streamed).  Set to None whenever that kernel changes.
DECODE_TRAFFIC_RATIO = 1.0069


def workload(args):
    """The benchmark workload: configuration 2 (Llama-3-8B, 32k context) unless --workload
    picks another of the five.  The ragged serving workload runs on packed (unpadded) caches,
    so all of its 32 layers fit one GPU."""
    w = synth.WORKLOADS[args.workload]
    if args.layers:
        w = w.scaled(L=args.layers)
    if args.context:
        w = w.scaled(T=args.context)
    if args.decode_steps:
        w = w.scaled(decode_steps=args.decode_steps,
                     append_steps=args.decode_steps if w.append_steps else 0)
    return w


def algorithmic_bytes(w, lens=None):
    """Bytes the method must move, per step, from the shapes alone:
    (compression pass, all decode-attention steps together, all append/evict steps together)."""
    e, row = w.elem_bytes, w.D * w.elem_bytes
    lens = [w.T] * w.B if lens is None else [int(n) for n in lens]
    n_unc = len([l for l in w.uncompressed if l < w.L])
    n_cmp = w.L - n_unc
    compress = decode = append = 0
    for n in lens:
        keep = int(np.ceil(w.keep_ratio * n))
        # compressed unit: read K once for the norms, read kept K and V rows, write them, plus
        # the index map and stored keys; uncompressed unit: read and write K and V once
        compress += w.Hkv * (n_cmp * (n * row + 4 * keep * row + 8 * keep) + n_unc * (4 * n * row + 8 * n))
        for s in range(w.decode_steps):
            grown = n + (s + 1 if w.append_steps else 0)          # uncompressed layers only append
            decode += w.Hkv * (n_cmp * keep + n_unc * grown) * 2 * row
            if w.append_steps:
                append += w.Hkv * (n_cmp * keep * 8 + w.L * (4 * row + 8))
    decode += w.decode_steps * w.B * w.L * w.Hq * w.D * (e + 4)
    return compress, decode, append


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(index), "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        self.p.wait()
        self.f.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f:
            c = [x.strip() for x in line.split(",")]
            if len(c) < 8:
                continue
            try:
                sm.append(float(c[0])); smax.append(float(c[1]))
            except ValueError:
                continue
            for n, v in zip(names, c[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def dist_setup(n):
    """One process per GPU (torchrun sets RANK / LOCAL_RANK / WORLD_SIZE)."""
    from paper_2406_11430_b200 import sharding
    if n <= 1:
        return 0, 1, 0
    local = int(os.environ.get("LOCAL_RANK", os.environ.get("RANK", "0")))
    torch.cuda.set_device(local)
    rank, world = sharding.init("nccl", torch.device("cuda", local))
    return rank, world, local


def max_over_ranks(x, world, device):
    from paper_2406_11430_b200 import sharding
    return sharding.max_over_ranks(x, device) if world > 1 else x


def barrier(world):
    from paper_2406_11430_b200 import sharding
    sharding.barrier()


# ------------------------------------------------------------------------------ GPU arm

class Job:
    """Device-resident state of one rank: the full cache, the compressed cache, queries.
    Ragged workloads use packed caches (no padding): the input holds len_b rows per (b, l); in
    the compressed cache an uncompressed layer has room for len_b + steps rows and a compressed
    one for its keep count."""

    def __init__(self, w, device, rank):
        import paper_2406_11430_b200 as l2
        self.l2, self.w, self.dev = l2, w, device
        ws = w.scaled(seed=w.seed + 1000 * rank)          # each rank its own batch
        self.lens_host = synth.ragged_lengths(ws)
        self.keep_host = np.ceil(w.keep_ratio * self.lens_host.astype(np.float64)).astype(np.int32)
        self.unc = tuple(l for l in w.uncompressed if l < w.L)
        self.packed = bool(w.ragged_lo)
        self.t_cap = w.T + w.append_steps                 # uncompressed layers grow by one per step
        if self.packed:
            self.K, self.V, rin = synth.make_cache_packed(ws, self.lens_host, device)
            self.rin_host, self.rin = rin, l2.Rows(*rin, device)
            caps = [[int(self.lens_host[b]) + w.append_steps if l in self.unc else int(self.keep_host[b])
                     for l in range(w.L)] for b in range(w.B)]
            self.rows_host = synth.packing(caps)
            self.rows = l2.Rows(*self.rows_host, device)
            total = self.rows_host[2]
            self.K_c = torch.zeros((w.Hkv, total, w.D), dtype=w.torch_dtype, device=device)
            meta = (w.Hkv, total)
        else:
            self.K, self.V = synth.make_cache(ws, device)
            self.rin = self.rows = None
            shape = (w.B, w.L, w.Hkv, self.t_cap, w.D)
            self.K_c = torch.zeros(shape, dtype=w.torch_dtype, device=device)
            meta = shape[:4]
        self.V_c = torch.zeros_like(self.K_c)
        self.idx = torch.zeros(meta, dtype=torch.int32, device=device)
        self.sumsq = torch.zeros(meta, dtype=torch.float32, device=device)
        self.cur = torch.zeros((w.B, w.L), dtype=torch.int32, device=device)
        self.keep_n = int(self.keep_host.max())
        self.max_in = int(self.lens_host.max())           # longest sequence handed to compression
        self.max_dec = self.rows.t_cap if self.packed else self.t_cap   # longest cache decode may meet
        self.lens = torch.tensor(self.lens_host, dtype=torch.int32, device=device)
        self.keep = torch.tensor(self.keep_host, dtype=torch.int32, device=device)
        self.q = torch.stack([synth.make_query(ws, s, device) for s in range(w.decode_steps)])
        self.out = torch.zeros((w.decode_steps, w.B, w.L, w.Hq, w.D), dtype=torch.float32,
                               device=device)
        self.q_step = list(self.q.unbind(0))              # views made once, not per call
        self.out_step = list(self.out.unbind(0))
        self.ws = l2.new_workspace(l2.Layout(self.K_c, q_heads=w.Hq, rows=self.rows),
                                   max(self.max_dec, self.max_in), device)
        self.new_rows, self.new_pos = [], []
        for s in range(w.append_steps):                   # budget-maintained serving loop
            self.new_rows.append(synth.make_new_kv(ws, s, device))
            self.new_pos.append(self.lens + s)
        # norm pass (with the selection and the copies of uncompressed layers inside) + gather;
        # per decode step one launch (bf16, head_dim 128: the last split of a unit merges its
        # partial results) or two (other types: split + merge), and one append/evict launch when
        # the workload maintains a budget
        dec = 1 if (w.dtype == "bf16" and w.D == 128) else 2
        self.launches_per_step = 2 + (dec + (1 if w.append_steps else 0)) * w.decode_steps

    def kv_bytes(self):
        return 2 * self.K.numel() * self.w.elem_bytes

    def compress(self, b=None, V=None):
        """The whole batch, or (b given; dense caches) sequence b alone: every tensor of one
        sequence is dense.  V: the V cache to read instead of the device copy (same shape; a
        pinned host tensor is read in place)."""
        i = slice(None) if b is None or self.packed else slice(b, b + 1)
        V = self.V if V is None else V
        self.l2.select_compact(self.K[i], V[i], self.lens[i], self.keep[i], self.max_in, self.unc,
                               self.K_c[i], self.V_c[i], self.idx[i], self.sumsq[i], self.cur[i], self.ws,
                               rows_in=self.rin, rows_out=self.rows)

    def compress_variant(self, policy=0, sumsq_in=None):
        self.l2.select_compact(self.K, self.V, self.lens, self.keep, self.max_in, self.unc, self.K_c,
                               self.V_c, self.idx, self.sumsq, self.cur, self.ws, policy=policy,
                               seed=1, sumsq_in=sumsq_in, rows_in=self.rin, rows_out=self.rows)

    def decode(self, s, b=None):
        if b is None or self.packed:                      # the whole batch: no views to make
            if self.w.append_steps:
                k, v = self.new_rows[s]
                self.l2.append_evict(self.K_c, self.V_c, self.idx, self.sumsq, self.cur, self.keep, self.unc,
                                     k, v, self.new_pos[s], self.ws, rows=self.rows)
            self.l2.decode_attention(self.q_step[s], self.K_c, self.V_c, self.cur, self.max_dec,
                                     self.out_step[s], self.ws, rows=self.rows)
            return
        i = slice(b, b + 1)
        if self.w.append_steps:
            k, v = self.new_rows[s]
            self.l2.append_evict(self.K_c[i], self.V_c[i], self.idx[i], self.sumsq[i], self.cur[i],
                                 self.keep[i], self.unc, k[i], v[i], self.new_pos[s][i], self.ws,
                                 rows=self.rows)
        self.l2.decode_attention(self.q[s][i], self.K_c[i], self.V_c[i], self.cur[i], self.max_dec,
                                 self.out[s][i], self.ws, rows=self.rows)

    def step(self, ev=None):
        """One pass of the whole path.  ev: optional list collecting (start, mid, end) events."""
        if ev is not None:
            e0 = torch.cuda.Event(enable_timing=True); e0.record()
        self.compress()
        if ev is not None:
            e1 = torch.cuda.Event(enable_timing=True); e1.record()
        for s in range(self.w.decode_steps):
            self.decode(s)
        if ev is not None:
            e2 = torch.cuda.Event(enable_timing=True); e2.record()
            ev.append((e0, e1, e2))

    def unit_input_rows(self, b, l, h):
        """K rows of unit (b, l, h) of the input cache (device view) and its kept positions."""
        n_in, keep = int(self.lens_host[b]), int(self.keep_host[b])
        if self.packed:
            i0, o0 = int(self.rin_host[0][b, l]), int(self.rows_host[0][b, l])
            return self.K[h, i0:i0 + n_in], self.idx[h, o0:o0 + keep]
        return self.K[b, l, h, :n_in], self.idx[b, l, h, :keep]


def measure(job, w, steps, warmup, world, device, rank, local):
    """warmup untimed steps, then `steps` timed ones between barriers; device times, max over
    ranks; SM clocks sampled during the timed region (rank 0)."""
    for _ in range(warmup):
        job.step()
    barrier(world)
    sampler = ClockSampler(local) if rank == 0 else None
    ev = []
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        job.step(ev)
    t1.record()
    barrier(world)
    total_ms = max_over_ranks(t0.elapsed_time(t1), world, device)
    clocks = sampler.stop() if sampler else None
    c_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in ev)
    d_ms = statistics.mean(b.elapsed_time(c) for _, b, c in ev) / w.decode_steps
    return (total_ms, max_over_ranks(c_ms, world, device), max_over_ranks(d_ms, world, device), clocks)


def stage_report(w, job, c_ms, d_ms, world, peak, peak_kind):
    """The per-stage numbers of one workload: ms, algorithmic GB/s, fractions of both peaks."""
    cbytes, dbytes_all, abytes_all = algorithmic_bytes(w, job.lens_host)
    dbytes = (dbytes_all + abytes_all) / w.decode_steps   # per decode step (with its append, if any)
    dec_gbs = dbytes / (d_ms * 1e-3) / 1e9
    cmp_gbs = cbytes / (c_ms * 1e-3) / 1e9
    return {
        "compress": {"ms": round(c_ms, 3), "GBps": round(cmp_gbs, 1), "bytes": int(cbytes),
                     "frac_of_8TBps": round(cmp_gbs / NOMINAL_HBM_GBS, 4),
                     f"frac_of_{peak_kind}": round(cmp_gbs / peak, 4)},
        "decode": {"ms_per_decode_step": round(d_ms, 4), "GBps": round(dec_gbs, 1), "bytes": int(dbytes),
                   "frac_of_8TBps": round(dec_gbs / NOMINAL_HBM_GBS, 4),
                   f"frac_of_{peak_kind}": round(dec_gbs / peak, 4),
                   "tokens_per_s": round(world * w.B / (d_ms * 1e-3), 1)},
    }, cbytes + dbytes_all + abytes_all, dbytes, dec_gbs


def workload_config(w, job, world):
    return {"workload": w.name, "batch": w.B, "layers": w.L, "kv_heads": w.Hkv,
            "q_heads": w.Hq, "head_dim": w.D, "context": w.T, "storage": w.dtype,
            "ragged_lengths": bool(w.ragged_lo), "cache_layout": "packed" if job.packed else "dense",
            "append_evict_per_decode_step": bool(w.append_steps),
            "keep_ratio": w.keep_ratio, "keep_per_head": job.keep_n,
            "uncompressed_layers": list(job.unc), "decode_steps_per_step": w.decode_steps}


def run_gpu(args):
    rank, world, local = dist_setup(args.gpus)
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    w = workload(args)
    job = Job(w, device, rank)
    peak, peak_kind = measured_peak()
    warmup = max(args.warmup, 3)
    total_ms, c_ms, d_ms, clocks = measure(job, w, args.steps, warmup, world, device, rank, local)
    stages, step_bytes, dbytes, dec_gbs = stage_report(w, job, c_ms, d_ms, world, peak, peak_kind)
    cbytes = stages["compress"]["bytes"]

    variants = None
    if rank == 0 and not args.no_variants and not w.append_steps and not w.ragged_lo:
        variants = time_variants(job, w, cbytes)

    # end to end: inputs start in pinned host memory, results end there
    e2e = None
    if not args.no_e2e and not job.packed:
        e2e = run_e2e(job, w, step_bytes, world, device, args)

    line = None
    if rank == 0:
        ms_per_step = total_ms / args.steps
        value = world * step_bytes / (ms_per_step * 1e-3) / 1e9
        cfg = workload_config(w, job, world)
        cfg["l2"] = (f"inputs larger than L2 ({dbytes / GIB:.1f} GiB read per decode step, "
                     f"{job.kv_bytes() / GIB:.0f} GiB of K and V per compress)")
        cfg["parallelism"] = f"independent replicas x{world}, no collective"
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": warmup, "ms_per_step": round(ms_per_step, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": cfg,
            "compress": stages["compress"], "decode": stages["decode"],
            "roofline": {"bound": "hbm", "kernel": "decode_split_mma_kernel (the merge of the splits runs inside it)",
                         "achieved": round(dec_gbs, 1), "peak": peak, "peak_kind": peak_kind,
                         "unit": "GB/s", "frac": round(dec_gbs / peak, 4),
                         "traffic": args.traffic if args.traffic is not None else
                         (round(DECODE_TRAFFIC_RATIO * dbytes)
                          if DECODE_TRAFFIC_RATIO and args.workload == 2 and not w.append_steps else None)},
            "gpu_launches": job.launches_per_step * args.steps,
            "clocks": clocks,
        }
        if variants:
            line["variants"] = variants
        if e2e:
            line["e2e"] = e2e
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(w, target_s=args.cpu_seconds)
            line["tie_band"] = tie_band_report(job, w)

    # the other four configurations, a few steps each (same job, same measurement)
    if not args.no_other_configs and args.workload == 2 and not (args.layers or args.context):
        del job
        free_device_memory()
        others = {}
        for i, wo in enumerate(synth.WORKLOADS):
            if i == args.workload:
                continue
            jo = Job(wo, device, rank)
            n = 2 if wo.append_steps else (5 if wo.T >= 32768 else 200)   # short steps: enough of them for a clock sample
            _, c2, d2, clk = measure(jo, wo, n, 3, world, device, rank, local)
            if rank == 0:
                st, _, _, _ = stage_report(wo, jo, c2, d2, world, peak, peak_kind)
                if not wo.append_steps:
                    # the decode call alone, launched back to back (no event or other launch between
                    # calls): what a serving loop that replays its steps sees
                    jo.compress()
                    reps = max(20, min(400, int(60.0 / max(d2, 1e-3))))
                    for _ in range(3):
                        jo.decode(0)
                    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
                    t0.record()
                    for r in range(reps):
                        jo.decode(r % wo.decode_steps)
                    t1.record(); torch.cuda.synchronize()
                    ms = t0.elapsed_time(t1) / reps
                    st["decode"]["back_to_back"] = {"ms": round(ms, 4), "calls": reps,
                                                    "GBps": round(st["decode"]["bytes"] / ms / 1e6, 1),
                                                    "frac_of_8TBps": round(st["decode"]["bytes"] / ms / 1e6 / NOMINAL_HBM_GBS, 4)}
                entry = {"config": workload_config(wo, jo, world), "steps": n, "warmup": 3,
                         "compress": st["compress"], "decode": st["decode"], "clocks": clk,
                         "gpu_launches": jo.launches_per_step * n}
                if not args.no_cpu_baseline and world == 1:
                    entry["tie_band"] = tie_band_report(jo, wo)
                if wo.dtype == "bf16" and wo.D == 128:
                    entry["prefix_attention"] = time_prefix_over_compressed(jo, wo)
                others[wo.name] = entry
            del jo
            free_device_memory()
        if rank == 0:
            line["configs"] = others
    if rank == 0:
        print(json.dumps(line))


def time_prefix_over_compressed(job, w, n_q=128, reps=3):
    """A block of n_q new queries per sequence over the compressed caches as they stand (dense, or
    packed and ragged: a chunk of a chunked prefill in a serving batch): prefix attention on the
    tensor cores with the workspace the library asks for, so that it may cut the caches up."""
    q = torch.randn((w.B, w.L, n_q, w.Hq, w.D), dtype=torch.bfloat16, device=job.dev)
    out = torch.empty(q.shape, dtype=torch.float32, device=job.dev)
    max_len = int(job.cur.max().item())                  # the caller knows its longest cache
    ws = job.l2.prefix_attention_workspace(job.K_c, q, max_len, rows=job.rows)
    call = lambda: job.l2.prefix_attention_flags(q, job.K_c, job.V_c, job.cur, max_len, out, 0,
                                                 workspace=ws, rows=job.rows)
    call()
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(reps):
        call()
    t1.record(); torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / reps
    flops = 4.0 * n_q * w.Hq * w.D * float(job.cur.sum().item())
    status = job.l2.read_device_status(ws)
    return {"ms": round(ms, 3), "queries_per_sequence": n_q, "TFLOPs": round(flops / ms / 1e9, 1),
            "cached_rows": int(job.cur.sum().item()), "workspace_MiB": round(ws.numel() / 2**20, 1),
            "device_status": status}


def free_device_memory():
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def time_variants(job, w, cbytes, reps=5):
    """Other forms of the compression pass, outside the main timed region: keys kept from
    cache-write time (no pass over K), and the keep-random / keep-highest ablation policies."""
    keys = torch.zeros((w.B, w.L, w.Hkv, w.T), dtype=torch.float32, device=job.dev)
    job.l2.key_norms(job.K, job.lens, w.T, keys)
    n_unc = len(job.unc)
    norm_pass = w.B * (w.L - n_unc) * w.Hkv * w.T * w.D * w.elem_bytes
    out = {}
    for name, kw, nbytes in (("keys_given", dict(sumsq_in=keys), cbytes - norm_pass),
                             ("keep_random", dict(policy=2), cbytes - norm_pass),
                             ("keep_highest", dict(policy=1), cbytes)):
        for _ in range(2):
            job.compress_variant(**kw)
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(reps):
            job.compress_variant(**kw)
        t1.record(); torch.cuda.synchronize()
        ms = t0.elapsed_time(t1) / reps
        out[name] = {"ms": round(ms, 3), "bytes": nbytes, "GBps": round(nbytes / ms / 1e6, 1)}
    job.compress()                     # leave the cache as the method's own policy makes it
    torch.cuda.synchronize()
    out["append_evict"] = time_append_evict(job, w)
    if not w.append_steps:
        out["decode_cuda_graph"] = time_decode_graph(job, w)
    # attention-loss analysis (Eqs. 5-7) of the full cache: keys from above, first query
    lens_bl = torch.full((w.B, w.L), w.T, dtype=torch.int32, device=job.dev)
    alr = torch.zeros((w.B, w.L, w.Hq), dtype=torch.float32, device=job.dev)
    need = ctypes.c_size_t(0)
    job.l2.lib().l2kv_attention_loss_workspace_bytes(job.l2.Layout(job.K, q_heads=w.Hq).ref(), w.T,
                                                     ctypes.byref(need))
    ws_al = torch.empty(need.value, dtype=torch.uint8, device=job.dev)
    job.l2.attention_loss(job.q[0], job.K, lens_bl, w.T, keys, alr, workspace=ws_al)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    job.l2.attention_loss(job.q[0], job.K, lens_bl, w.T, keys, alr, workspace=ws_al)
    t1.record(); torch.cuda.synchronize()
    out["attention_loss"] = {"ms": round(t0.elapsed_time(t1), 2), "heads": w.B * w.L * w.Hq,
                             "tokens_per_head": w.T, "mean_alr": round(float(alr.mean().item()), 2)}
    del ws_al
    # prefix attention: 128 new queries per (b, l) over the compressed cache (tensor-bound)
    if w.dtype == "bf16" and w.D == 128:             # the tensor-core kernel's types
        n_q = 128
        job.compress()
        qp = torch.randn((w.B, w.L, n_q, w.Hq, w.D), device=job.dev).to(torch.bfloat16)
        op = torch.empty(qp.shape, dtype=torch.float32, device=job.dev)
        tf_peak = None
        try:
            tf_peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"])
        except Exception:
            pass

        def timed(q_, K_, V_, cur_, o_, reps=3, split=True):
            max_len_ = int(cur_.max().item())               # the caller knows its longest cache
            ws_ = (job.l2.prefix_attention_workspace(K_, q_, max_len_) if split  # room to split the cache
                   else torch.zeros(256, dtype=torch.uint8, device=job.dev))
            job.l2.prefix_attention(q_, K_, V_, cur_, max_len_, o_, workspace=ws_)
            t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
            t0.record()
            for _ in range(reps):
                job.l2.prefix_attention(q_, K_, V_, cur_, max_len_, o_, workspace=ws_)
            t1.record(); torch.cuda.synchronize()
            ms_ = t0.elapsed_time(t1) / reps
            flop_ = 4.0 * n_q * w.Hq * w.D * float(cur_.sum().item())
            return {"ms": round(ms_, 3), "TFLOPs": round(flop_ / ms_ / 1e9, 1),
                    "frac": round(flop_ / ms_ / 1e9 / tf_peak, 4) if tf_peak else None,
                    "split_scratch_MiB": round((ws_.numel() - 256) / 2**20, 1)}

        r = timed(qp, job.K_c, job.V_c, job.cur, op)
        out["prefix_attention"] = {"ms": r["ms"], "queries_per_sequence": n_q, "TFLOPs": r["TFLOPs"],
                                   "bound": "tensor", "peak_TFLOPs_measured_sustained": tf_peak,
                                   "frac": r["frac"], "split_scratch_MiB": r["split_scratch_MiB"]}
        # the same for one layer at a time, as a model calls it: few CTAs unless the cache is split
        l1 = min(2, w.L - 1)
        r1 = timed(qp[:, l1:l1 + 1].contiguous(), job.K_c[:, l1:l1 + 1], job.V_c[:, l1:l1 + 1],
                   job.cur[:, l1:l1 + 1].contiguous(), op[:, l1:l1 + 1].contiguous(), reps=10)
        out["prefix_attention"]["one_layer"] = r1
        out["prefix_attention"]["one_layer_unsplit"] = timed(
            qp[:, l1:l1 + 1].contiguous(), job.K_c[:, l1:l1 + 1], job.V_c[:, l1:l1 + 1],
            job.cur[:, l1:l1 + 1].contiguous(), op[:, l1:l1 + 1].contiguous(), reps=10, split=False)
        del qp, op
    job.compress()
    torch.cuda.synchronize()
    return out


def time_decode_graph(job, w, reps=5):
    """The step's decode calls captured once in a CUDA graph and replayed: what a serving loop
    does to take the launch overhead off short decode steps (the calls allocate nothing and are
    ordered on the caller's stream, so they capture as they are)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        job.decode(0)                                   # first call on this stream, outside capture
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for s in range(w.decode_steps):
            job.decode(s)

    def timed(fn):
        fn(); torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(reps):
            fn()
        t1.record(); torch.cuda.synchronize()
        return t0.elapsed_time(t1) / reps / w.decode_steps

    def eager():
        for s in range(w.decode_steps):
            job.decode(s)

    ms_graph, ms_eager = timed(graph.replay), timed(eager)
    return {"ms_per_decode_step": round(ms_graph, 5), "eager_ms_per_decode_step": round(ms_eager, 5),
            "decode_steps_in_graph": w.decode_steps}


def time_append_evict(job, w, reps=20):
    """One budget-maintenance step (a new K/V row per head, eviction of the highest norm) on
    the compressed cache of this workload, every sequence at its budget.  Not part of the
    workload's step (its cache is static); timed here so that the kernel has a number."""
    budget = torch.full((w.B,), job.keep_n, dtype=torch.int32, device=job.dev)
    pos = torch.full((w.B,), w.T, dtype=torch.int32, device=job.dev)
    rows = [synth.make_new_kv(w, s, job.dev) for s in range(4)]
    cur = job.cur.cpu()
    stored = int(cur.sum().item()) * w.Hkv                 # (key, position) pairs scanned
    nbytes = stored * 8 + w.B * w.L * w.Hkv * (4 * w.D * w.elem_bytes + 8)

    def one(i):
        k, v = rows[i % len(rows)]
        # no layer list: the full-length layers 0-1 are over budget too and evict like the rest
        job.l2.append_evict(job.K_c, job.V_c, job.idx, job.sumsq, job.cur, budget, (), k, v,
                            pos + i, job.ws)
    for i in range(3):
        one(i)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for i in range(reps):
        one(3 + i)
    t1.record(); torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / reps
    return {"ms": round(ms, 4), "bytes": nbytes, "GBps": round(nbytes / ms / 1e6, 1),
            "stored_entries": stored}


def host_memory_is_device_addressable(device_index):
    """True when kernels may read pinned host memory through its host pointer (unified addressing
    with mapped host memory), which the V-on-demand schedule relies on."""
    try:
        try:
            from cuda.bindings import runtime as cudart
        except ImportError:
            from cuda import cudart
        a = cudart.cudaDeviceAttr
        e1, ua = cudart.cudaDeviceGetAttribute(a.cudaDevAttrUnifiedAddressing, device_index)
        e2, mh = cudart.cudaDeviceGetAttribute(a.cudaDevAttrCanMapHostMemory, device_index)
        return int(e1) == 0 and int(e2) == 0 and bool(ua) and bool(mh)
    except Exception:
        return False


def run_e2e(job, w, step_bytes, world, device, args):
    """The same step with the cache arriving from pinned host memory and the attention outputs
    returning to it, all inside the timed region.  Two schedules are timed.  "copy everything":
    K and V are both uploaded.  "V rows on demand" (the reported one): only K is uploaded; the
    compression call is handed the V cache where it lies in pinned host memory (a device-
    accessible pointer), so the rows of V that the method drops never cross the link -- the
    gather reads the kept rows straight from the host."""
    Kh = torch.empty(job.K.shape, dtype=job.K.dtype, pin_memory=True)
    Vh = torch.empty_like(Kh, pin_memory=True)
    qh = torch.empty(job.q.shape, dtype=job.q.dtype, pin_memory=True)
    oh = torch.empty(job.out.shape, dtype=torch.float32, pin_memory=True)
    Kh.copy_(job.K); Vh.copy_(job.V); qh.copy_(job.q)
    job.step()
    torch.cuda.synchronize()
    want = job.out.clone()                              # what the device-resident step produces
    kv_bytes = Kh.numel() * Kh.element_size()
    q_bytes = qh.numel() * qh.element_size()
    d2h = oh.numel() * 4
    # rows of V that the compression reads: every row of an uncompressed layer, the kept rows elsewhere
    n_unc = len(job.unc)
    v_rows = sum((n_unc * int(n) + (w.L - n_unc) * int(k)) for n, k in zip(job.lens_host, job.keep_host))
    v_read = v_rows * w.Hkv * w.D * w.elem_bytes

    # Part by part -- a part is a group of consecutive layers of one sequence, whose tensors are
    # dense, so the same entry points take it as a batch of one with fewer layers: the upload of
    # the next part (copy stream) runs under the compression and the decode steps of this one
    # (the caller's stream).  The smaller the parts, the less of the step runs with the link idle
    # (the first upload, the last part's decode steps).
    comp = torch.cuda.current_stream()
    copy = torch.cuda.Stream()
    n_groups = max(1, min(w.L, args.e2e_layer_groups))
    bounds = [round(i * w.L / n_groups) for i in range(n_groups + 1)]
    parts = [(b, l0, l1) for b in range(w.B) for l0, l1 in zip(bounds[:-1], bounds[1:]) if l1 > l0]
    l2 = job.l2

    def run_part(b, l0, l1, V):
        i, ls = slice(b, b + 1), slice(l0, l1)
        unc = tuple(l - l0 for l in job.unc if l0 <= l < l1)
        l2.select_compact(job.K[i, ls], V[i, ls], job.lens[i], job.keep[i], job.max_in, unc,
                          job.K_c[i, ls], job.V_c[i, ls], job.idx[i, ls], job.sumsq[i, ls], job.cur[i, ls],
                          job.ws)
        for s in range(w.decode_steps):
            if w.append_steps:
                k, v = job.new_rows[s]
                l2.append_evict(job.K_c[i, ls], job.V_c[i, ls], job.idx[i, ls], job.sumsq[i, ls],
                                job.cur[i, ls], job.keep[i], unc, k[i, ls], v[i, ls], job.new_pos[s][i],
                                job.ws)
            l2.decode_attention(job.q_step[s][i, ls], job.K_c[i, ls], job.V_c[i, ls], job.cur[i, ls],
                                job.max_dec, job.out_step[s][i, ls], job.ws)

    def step(copy_v):
        copy.wait_stream(comp)                          # the last step is done with the buffers
        landed = []
        with torch.cuda.stream(copy):
            job.q.copy_(qh, non_blocking=True)
            for b, l0, l1 in parts:
                job.K[b, l0:l1].copy_(Kh[b, l0:l1], non_blocking=True)
                if copy_v:
                    job.V[b, l0:l1].copy_(Vh[b, l0:l1], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(copy)
                landed.append(ev)
        for ev, (b, l0, l1) in zip(landed, parts):
            comp.wait_event(ev)
            run_part(b, l0, l1, job.V if copy_v else Vh)
        oh.copy_(job.out, non_blocking=True)

    def timed(copy_v):
        job.out.zero_()
        step(copy_v)
        torch.cuda.synchronize()
        same = bool(torch.equal(oh.to(job.out.device), want))
        barrier(world)
        n = max(1, min(args.steps, args.e2e_steps))
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(n):
            step(copy_v)
        t1.record()
        barrier(world)
        return max_over_ranks(t0.elapsed_time(t1), world, device) / n, n, same

    ms_all, n, same_all = timed(True)
    if not host_memory_is_device_addressable(job.K.device.index or 0):
        # no mapped host memory on this system: only the copying schedule can run
        del Kh, Vh
        return {"value": round(world * step_bytes / (ms_all * 1e-3) / 1e9, 1), "unit": "GB/s",
                "ms_per_step": round(ms_all, 2), "steps": n, "h2d_bytes_per_step": 2 * kv_bytes + q_bytes,
                "d2h_bytes_per_step": d2h, "outputs_equal_device_resident_step": same_all,
                "parts_per_step": len(parts),
                "schedule": "per part (some layers of one sequence): the upload of the next part overlaps "
                            "compress + decode of this one"}
    ms_dem, _, same_dem = timed(False)
    del Kh, Vh
    rate = lambda ms: round(world * step_bytes / (ms * 1e-3) / 1e9, 1)
    return {"value": rate(ms_dem), "unit": "GB/s", "ms_per_step": round(ms_dem, 2), "steps": n,
            "h2d_bytes_per_step": kv_bytes + q_bytes + v_read, "d2h_bytes_per_step": d2h,
            "outputs_equal_device_resident_step": same_dem,
            "parts_per_step": len(parts),
            "schedule": "per part (some layers of one sequence): the upload of K of the next part overlaps "
                        "compress + decode of this one; V stays in pinned host memory and the compression "
                        "reads only the rows it keeps",
            "copy_everything": {"value": rate(ms_all), "ms_per_step": round(ms_all, 2),
                                "h2d_bytes_per_step": 2 * kv_bytes + q_bytes,
                                "outputs_equal_device_resident_step": same_all}}


# ------------------------------------------------------------------------- oracle arm

def oracle_sample_step(w, seed_shift=0, n_dec=2, n_comp=1, nthreads=None):
    """One bounded sample of the workload through the CPU oracle: sequence 0, one
    uncompressed layer and n_comp compressed layers, all KV heads, full context, a
    compression pass and n_dec decode steps.  Returns (seconds, bytes, threads, layers)."""
    import oracle
    nthreads = nthreads or oracle.hardware_threads()
    unc = [l for l in w.uncompressed if l < w.L][:1]
    comp = [l for l in range(w.L) if l not in w.uncompressed][:n_comp]
    layers = unc + comp
    ws = w.scaled(seed=w.seed + seed_shift)
    K = np.ascontiguousarray(np.stack(
        [synth.to_numpy(synth.make_kv_slab(ws, "K", 0, l, "cpu")) for l in layers])[None])
    V = np.ascontiguousarray(np.stack(
        [synth.to_numpy(synth.make_kv_slab(ws, "V", 0, l, "cpu")) for l in layers])[None])
    sub = w.scaled(B=1, L=len(layers), uncompressed=tuple(range(len(unc))))
    qs = [np.ascontiguousarray(synth.to_numpy(synth.make_query(ws, s, "cpu"))[:1, layers])
          for s in range(n_dec)]
    keep = oracle.keep_count(w.T, w.keep_ratio)
    t0 = time.perf_counter()
    r = oracle.compress(K, V, w.dtype, [w.T], [keep], sub.uncompressed, nthreads=nthreads)
    for q in qs:
        oracle.attention(q, r["K_c"], r["V_c"], w.dtype, r["kept_len"], nthreads=nthreads)
    dt = time.perf_counter() - t0
    cb, db, _ = algorithmic_bytes(sub.scaled(decode_steps=n_dec, append_steps=0, ragged_lo=0))
    return dt, cb + db, nthreads, layers


def cpu_baseline(w, target_s=15.0):
    """The oracle, as it stands, on the host cores: a sample sized to about target_s seconds."""
    probe, _, _, _ = oracle_sample_step(w, n_dec=w.decode_steps, n_comp=1)   # one layer pair, all steps
    # the uncompressed layer of the pair costs about two compressed ones (twice the rows)
    n_comp = int(max(1, min(w.L - len(w.uncompressed), round(3 * target_s / max(probe, 1e-3) - 2))))
    dt, nbytes, nthreads, layers = oracle_sample_step(w, n_dec=w.decode_steps, n_comp=n_comp)
    # the same oracle on one thread, on a smaller sample (one layer pair, a few decode steps)
    n1 = min(4, w.decode_steps)
    dt1, nbytes1, _, layers1 = oracle_sample_step(w, n_dec=n1, n_comp=1, nthreads=1)
    return {"value": round(nbytes / dt / 1e9, 4), "unit": "GB/s", "cores": nthreads,
            "kind": "oracle", "seconds": round(dt, 2),
            "sample": f"sequence 0, layers {layers} (first one uncompressed), all {w.Hkv} KV "
                      f"heads, full {w.T}-token context: one compression pass + "
                      f"{w.decode_steps} decode steps",
            "single_thread": {"value": round(nbytes1 / dt1 / 1e9, 4), "unit": "GB/s", "cores": 1,
                              "seconds": round(dt1, 2),
                              "sample": f"sequence 0, layers {layers1}, all {w.Hkv} KV heads, full "
                                        f"{w.T}-token context: one compression pass + {n1} decode steps"}}


def tie_band_report(job, w, n_units=6, band=1e-6):
    """Part of the CPU leg: the kept sets of a few compressed units against the oracle's fp64
    selection.  Tokens may differ only where the fp64 norm lies within `band` (relative) of the
    unit's threshold norm; such swaps are counted, anything else is reported as a mismatch."""
    import oracle
    job.compress()
    torch.cuda.synchronize()
    comp = [l for l in range(w.L) if l not in job.unc]
    if not comp:
        return {"units_checked": 0, "swaps_inside_band": 0, "mismatches_outside_band": 0, "band": band}
    swaps = bad = 0
    for i in range(n_units):
        b, l, h = i % w.B, comp[(i * 7) % len(comp)], (i * 3) % w.Hkv
        keep = int(job.keep_host[b])
        rows, kept = job.unit_input_rows(b, l, h)
        key = oracle.key_sumsq(np.ascontiguousarray(synth.to_numpy(rows)), w.dtype)
        want = set(oracle.select(key, keep).tolist())
        got = set(kept.cpu().tolist())
        norm = np.sqrt(key)
        thr = np.sort(norm)[keep - 1]
        for t in got ^ want:
            if abs(norm[t] - thr) <= band * thr:
                swaps += 1
            else:
                bad += 1
    return {"units_checked": n_units, "swaps_inside_band": swaps // 2,
            "mismatches_outside_band": bad, "band": band}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload(args)
    import oracle
    n_dec = 2
    for _ in range(min(args.warmup, 1)):
        oracle_sample_step(w, n_dec=n_dec)
    times, nbytes, nthreads, layers = [], 0, 0, []
    for s in range(args.steps):
        dt, nbytes, nthreads, layers = oracle_sample_step(w, seed_shift=s, n_dec=n_dec, n_comp=1)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = round(nbytes / (ms * 1e-3) / 1e9, 4)
    sample = (f"per step: sequence 0, layers {layers}, all {w.Hkv} KV heads, full {w.T}-token "
              f"context, one compression pass + {n_dec} decode steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": round(ms, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": nthreads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="l2kv", choices=["l2kv", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-layer-groups", type=int, default=4,
                    help="the end-to-end schedule cuts every sequence into this many groups of layers")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short runs of the other four configurations")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--workload", type=int, default=2, choices=range(len(synth.WORKLOADS)),
                    help="which of the five configurations (default 2: llama3-8b-32k)")
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: fewer layers")
    ap.add_argument("--context", type=int, default=0, help="profiling aid: shorter context")
    ap.add_argument("--decode-steps", type=int, default=0, help="profiling aid")
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per launch of the dominant kernel from an ncu capture")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
