#!/usr/bin/env python
"""Benchmark of the FedAttn attention hot path on B200.

One step = one pass of the whole hot path over one batch of synthetic input with the shapes of
the bf16 Llama-3-8B attention configuration (cfg2: N=4 participants x 2048 tokens, 32 query heads /
8 KV heads, head_dim 128):

    fedattn_local                      per-participant causal attention
    fedattn_aggregate_kv (CONCAT)      dense KV aggregation
    fedattn_sync                       queries over the 8192-token aggregated KV
    fedattn_aggregate_kv (TOPK_KNORM)  sparse aggregation, top 25% keys per participant and KV head
    fedattn_sync (sparse)              queries over the selected KV, global-position mask
    fedattn_decode (LOCAL)             one new token per participant over its own 2048-token cache
    fedattn_decode (SYNC)              the same tokens over the shared 8192-token cache

`value` is the algorithmic attention TFLOP/s of the whole step (exact unmasked (q,k) pairs x 4*d
flop per query head, divided by the step time, inputs resident in HBM).  `e2e` is the same metric
through the same calls with pinned HOST inputs and outputs (copies inside the timed region).
`roofline` covers the dominant kernel (the tcgen05 prefill kernel); `calls` gives every call's
own time and rate.  `--impl reference` times the fp64 CPU oracle on a bounded row sample.

With one GPU the default run (`--workload all`) also times the other seeded configurations at
their own sizes and folds them into the same line (`calls` entries prefixed with the configuration,
`rooflines` with one entry per bound):
    cfg1   fp32, 2 x 128 tokens, 4 heads, d=64: time of local, concat and sync; the oracle in full
    cfg3   32-block schedules over 8 heterogeneous segments, sync every H-th block, H in
           {1,2,4,8,32}, four non-uniform schedules, and a block in which half the participants
           exchange (explicit query positions)
    cfg4   sparse aggregation (16 x 1024, top 256 keys per KV head; per-head, token-level and a
           seeded random selection), sync over the selected KV, and the exchange block that keeps
           the own segment complete
    cfg5   decode, 8 caches x 4096 tokens, a step = 3 local + 1 sync call (H=4)
`--workload cfgN` prints one line for that configuration alone with its own metric (cfg2: the step
only, e.g. for a profiler capture).  With --gpus N > 1 every rank runs an independent replica of the
cfg2 step (the path has no exchange step on one device; participants are simulated per GPU) and the
value is the sum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import fedattn_inputs as fi  # noqa: E402

METRIC = "fedattn_prefill_tflops"
UNIT = "TFLOP/s"
N_SETS = 3            # rotating input sets: ~600 MB touched per cycle, larger than the 126 MB L2
SPARSE_RATIO_NUM, SPARSE_RATIO_DEN = 1, 4
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (None: the kernel has changed since its counters were taken)
PREFILL_DRAM_BYTES = 365_672_000        # prefill_sm100_kernel, the three cfg2 launches the roofline covers: local 133.5 MB,
                                        # sync 132.5 MB, sparse sync 99.7 MB (read + written)
DECODE_DRAM_BYTES = 140_620_000         # one cfg5 call: decode_stream_kernel 138.45 MB + decode_merge_kernel 2.17 MB
                                        # (the merge reads its partials from DRAM only under the profiler's cache flush)
TOPK_DRAM_BYTES = 42_223_000            # topk_fused_kernel, one cfg4 sparse aggregation (42.0 MB read + 0.2 MB written)
NOMINAL_TENSOR, NOMINAL_HBM = 2250.0, 8000.0     # B200 spec: dense bf16 TFLOP/s, HBM3e GB/s
MIN_REGION_S = 0.2                  # every microsecond-scale leg is timed over a region at least this long


def env_rank():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(tensor=float(d["bf16_tflops"]), tensor_sustained=float(d.get("bf16_tflops_sustained", 0.0)),
                    hbm=float(d["hbm_gbs"]), kind="measured")
    return dict(tensor=1590.0, tensor_sustained=1400.0, hbm=6650.0, kind="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# workload bookkeeping (algorithmic flops / bytes; no arithmetic of the method)
# ------------------------------------------------------------------------------------------------
def workload():
    return fi.cfg2()


def flops_local(w):
    return 4.0 * w.head_dim * w.n_q_heads * sum(n * (n + 1) // 2 for n in w.seqlens)


def flops_sync(w):
    L = w.total_tokens
    return 4.0 * w.head_dim * w.n_q_heads * (L * (L + 1) // 2)


def flops_decode(w):
    L = w.total_tokens
    return 4.0 * w.head_dim * w.n_q_heads * L, 4.0 * w.head_dim * w.n_q_heads * w.n_participants * L


# ------------------------------------------------------------------------------------------------
# multi-rank bookkeeping (replicas only: no data-path collective; the ranks only agree on the time)
# ------------------------------------------------------------------------------------------------
def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks of the default process group
    (device: where the reduction tensor lives, None for CPU / gloo); identity without a group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(x) for x in values]
    t = torch.tensor([float(x) for x in values], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def replica_throughput(work_per_rank, ms_per_step, world):
    """Whole-job units per second when `world` independent replicas each do work_per_rank per step
    and the slowest one needs ms_per_step."""
    return world * work_per_rank / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2511_02647_b200 as fa

    rank, local_rank, world = env_rank()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    w = workload()
    N, Hq, Hkv, d, L = w.n_participants, w.n_q_heads, w.n_kv_heads, w.head_dim, w.total_tokens
    seqlens = list(w.seqlens)
    cu = [0] + list(np.cumsum(seqlens))
    ksel = [n * SPARSE_RATIO_NUM // SPARSE_RATIO_DEN for n in seqlens]
    T = sum(ksel)
    shape = fa.Shape(N, Hq, Hkv, d, fa.BF16)
    ctx = fa.Context(shape, L, L, device=local_rank)
    dev = torch.device("cuda", local_rank)
    bf = torch.bfloat16

    n_sets = max(1, args.sets)
    # host inputs (pinned) -- also the e2e source
    host_sets = []
    for s in range(n_sets):
        q, k, v = w.qkv(block=s)
        qd = w.decode_q(s)
        host_sets.append([torch.from_numpy(x).to(bf).pin_memory() for x in (q, k, v, qd)])

    class Buf:
        pass

    def make_set(hs):
        b = Buf()
        b.q, b.k, b.v, b.qd = [x.to(dev, non_blocking=True) for x in hs]
        b.o_local = torch.empty_like(b.q); b.o_sync = torch.empty_like(b.q); b.o_sparse = torch.empty_like(b.q)
        b.k_agg = torch.empty_like(b.k); b.v_agg = torch.empty_like(b.v)
        b.kv_pos = torch.empty(L, dtype=torch.int32, device=dev)
        b.cu_kv = torch.empty(N + 1, dtype=torch.int32, device=dev)
        b.k_sp = torch.empty((Hkv, T, d), dtype=bf, device=dev); b.v_sp = torch.empty_like(b.k_sp)
        b.pos_sp = torch.empty((Hkv, T), dtype=torch.int32, device=dev)
        b.sel = torch.empty((Hkv, T), dtype=torch.int32, device=dev)
        b.cu_sp = torch.empty(N + 1, dtype=torch.int32, device=dev)
        b.o_dl = torch.empty_like(b.qd); b.o_ds = torch.empty_like(b.qd)
        b.len_local = torch.tensor(seqlens, dtype=torch.int32, device=dev)
        b.len_sync = torch.tensor([L], dtype=torch.int32, device=dev)
        return b

    sets = [make_set(hs) for hs in host_sets]
    torch.cuda.synchronize()
    set_mb = sum(t.numel() * t.element_size() for t in vars(sets[0]).values() if torch.is_tensor(t)) // 2 ** 20
    stream = torch.cuda.current_stream()
    call_names = ["local", "aggregate_concat", "sync", "aggregate_topk", "sync_sparse", "decode_local", "decode_sync"]

    def step(b, ev=None):
        def mark(i):
            if ev is not None:
                ev[i].record(stream)
        kp = [b.k[cu[n]:cu[n + 1]] for n in range(N)]
        vp = [b.v[cu[n]:cu[n + 1]] for n in range(N)]
        mark(0)
        fa.fedattn_local(ctx, shape, b.q, b.k, b.v, cu, b.o_local)
        mark(1)
        fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_CONCAT, kp, vp, seqlens, None, None, b.k_agg, b.v_agg, b.kv_pos,
                                b.cu_kv, None)
        mark(2)
        fa.fedattn_sync(ctx, shape, b.q, None, b.k_agg, b.v_agg, b.kv_pos, L, False, b.o_sync)
        mark(3)
        fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_TOPK_KNORM, kp, vp, seqlens, ksel, None, b.k_sp, b.v_sp, b.pos_sp,
                                b.cu_sp, b.sel)
        mark(4)
        fa.fedattn_sync(ctx, shape, b.q, None, b.k_sp, b.v_sp, b.pos_sp, T, True, b.o_sparse)
        mark(5)
        # decode: the prefill K/V act as the caches (local: participant n's own rows; sync: aggregated)
        fa.fedattn_decode(ctx, shape, fa.DECODE_LOCAL, b.qd, b.k, b.v, seqlens[0] * Hkv * d, b.len_local,
                          max(seqlens), b.o_dl)
        mark(6)
        fa.fedattn_decode(ctx, shape, fa.DECODE_SYNC, b.qd, b.k_agg, b.v_agg, 0, b.len_sync, L, b.o_ds)
        mark(7)

    assert len(set(seqlens)) == 1, "local decode uses a constant cache stride"

    # one untimed pass to obtain the sparse pair count from the positions the library produced
    step(sets[0])
    assert ctx.poll() == 0
    pos = sets[0].pos_sp.to(torch.int64)                                     # [Hkv, T], ascending per head
    rows = torch.arange(L, device=dev, dtype=torch.int64)
    pairs_sparse = sum(int(torch.searchsorted(pos[h].contiguous(), rows, right=True).sum().item()) for h in range(Hkv))
    f_local, f_sync = flops_local(w), flops_sync(w)
    f_sparse = 4.0 * d * (Hq // Hkv) * pairs_sparse
    f_dl, f_ds = flops_decode(w)
    step_flops = f_local + f_sync + f_sparse + f_dl + f_ds
    eb = 2
    kv_bytes = 2 * L * Hkv * d * eb
    call_flops = dict(local=f_local, sync=f_sync, sync_sparse=f_sparse, decode_local=f_dl, decode_sync=f_ds)
    call_bytes = dict(aggregate_concat=2 * kv_bytes,
                      aggregate_topk=kv_bytes // 2 + (kv_bytes // 2) * T // L + kv_bytes * T // L,
                      decode_local=kv_bytes + 2 * N * Hq * d * eb, decode_sync=kv_bytes + 2 * N * Hq * d * eb)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        step(sets[i % n_sets])
    barrier()

    # ---- timed region: K steps, per-call events on the launching stream ----
    K = args.steps
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(8)] for _ in range(K)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)
    launches0 = ctx.launch_count()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(K):
        step(sets[i % n_sets], evs[i])
    t_end.record(stream)
    barrier()
    total_ms = t_start.elapsed_time(t_end)
    launches = ctx.launch_count() - launches0
    status = ctx.poll()
    time.sleep(0.25)
    clocks = sampler.stop()
    if status != 0:
        raise RuntimeError("device status %d after the timed region" % status)
    call_ms = {nm: sum(evs[i][j].elapsed_time(evs[i][j + 1]) for i in range(K)) / K for j, nm in enumerate(call_names)}

    # ---- e2e: pinned host inputs -> device, the same step, results -> pinned host ----
    e2e_steps = max(3, min(K, 10))
    hout = [torch.empty((L, Hq, d), dtype=bf).pin_memory() for _ in range(3)] + \
           [torch.empty((N, Hq, d), dtype=bf).pin_memory() for _ in range(2)]
    h2d = sum(x.numel() * x.element_size() for x in host_sets[0])
    d2h = sum(x.numel() * x.element_size() for x in hout)

    def e2e_in(i):
        b, hs = sets[i % n_sets], host_sets[i % n_sets]
        b.q.copy_(hs[0], non_blocking=True); b.k.copy_(hs[1], non_blocking=True)
        b.v.copy_(hs[2], non_blocking=True); b.qd.copy_(hs[3], non_blocking=True)

    def e2e_out(i):
        b = sets[i % n_sets]
        for dst, src in zip(hout, (b.o_local, b.o_sync, b.o_sparse, b.o_dl, b.o_ds)):
            dst.copy_(src, non_blocking=True)

    barrier()
    e2e_ms = _pipelined(torch, stream, e2e_in, lambda i: step(sets[i % n_sets]), e2e_out, e2e_steps, n_sets)
    barrier()

    # ---- max over ranks; replicas: every rank did the same work, the job did `world` times as much ----
    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dev if world > 1 else None)
    ms_per_step = total_ms / K
    value = replica_throughput(step_flops, ms_per_step, world) / 1e12
    e2e_value = replica_throughput(step_flops, e2e_ms, world) / 1e12

    if rank == 0:
        pk = peaks()
        pre_ms = call_ms["local"] + call_ms["sync"] + call_ms["sync_sparse"]
        pre_flops = f_local + f_sync + f_sparse
        achieved = pre_flops / (pre_ms * 1e-3) / 1e12
        calls = {}
        for nm in call_names:
            c = {"ms": round(call_ms[nm], 5)}
            if nm in call_flops:
                c["tflops"] = round(call_flops[nm] / (call_ms[nm] * 1e-3) / 1e12, 3)
            if nm in call_bytes:
                c["gbs"] = round(call_bytes[nm] / (call_ms[nm] * 1e-3) / 1e9, 1)
                c["frac_hbm"] = round(c["gbs"] / pk["hbm"], 4)
            if nm in ("local", "sync", "sync_sparse"):
                c["frac_tensor"] = round(c["tflops"] / pk["tensor"], 4)
            calls[nm] = c
        out = {
            "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "participants": N, "tokens_per_participant": seqlens[0],
                       "q_heads": Hq, "kv_heads": Hkv, "head_dim": d, "sparse_keep": "1/4 per KV head",
                       "step": "local+concat+sync+topk+sparse_sync+decode_local+decode_sync",
                       "l2": "%d rotating input/output sets of %d MB each (> 126 MB L2), no flush" % (n_sets, set_mb),
                       "parallelism": "replicas" if world > 1 else "single"},
            "clocks": clocks,
            "e2e": {"value": round(e2e_value, 3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": round(e2e_ms, 4), "pipeline": "copy-in, kernels and copy-out of neighbouring steps overlap on three streams"},
            "gpu_launches": int(launches),
            "roofline": {"bound": "tensor", "kernel": "prefill_sm100_kernel (local + sync + sparse sync launches)",
                         "achieved": round(achieved, 2), "peak": pk["tensor"], "unit": "TFLOP/s",
                         "frac": round(achieved / pk["tensor"], 4), "peak_kind": "burst bf16, " + pk["kind"],
                         "frac_of_sustained": round(achieved / pk["tensor_sustained"], 4) if pk["tensor_sustained"] else None,
                         "frac_of_nominal_2250": round(achieved / NOMINAL_TENSOR, 4),
                         "traffic": PREFILL_DRAM_BYTES},
            "calls": calls,
            "step_tflop": round(step_flops / 1e12, 5),
        }
        out["rooflines"] = {"prefill": out["roofline"]}
        if world == 1 and args.workload == "all":
            # the other configurations at their own sizes, folded into this line
            del sets, host_sets, hout
            torch.cuda.empty_cache()
            legs_launches = {}
            for name in ("cfg5", "cfg4", "cfg3", "cfg1"):
                r = LEGS[name](args)
                for nm, c in r["calls"].items():
                    out["calls"]["%s.%s" % (name, nm)] = c
                out["rooflines"].update(r["rooflines"])
                legs_launches[name] = {"launches_per_step": int(r["launches"]), "step": r["config"]["step"],
                                       "ms_per_step": round(r["ms_step"], 5), "e2e": r["e2e"], "clocks": r["clocks"]}
                if "extra" in r:
                    out.setdefault("schedules_cfg3", r["extra"].get("schedules"))
                torch.cuda.empty_cache()
            out["other_workloads"] = legs_launches
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(w, target_seconds=10.0)
            if args.workload == "all":
                out["cpu_baseline"]["other_workloads"] = oracle_legs(["cfg1", "cfg4", "cfg5"])
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# the other configurations (one process, one GPU; same timing rules).  Every leg returns a dict:
#   calls      per-call figures              rooflines   {"decode"|"aggregate"|...: roofline object}
#   launches   kernels launched per `step`   ms_step, value, metric, unit, config, e2e   for a line of its own
# ------------------------------------------------------------------------------------------------
def _setup(local_rank=0):
    import torch
    import paper_2511_02647_b200 as fa
    torch.cuda.set_device(local_rank)
    return torch, fa, torch.device("cuda", local_rank)


def _timed(torch, stream, fn, iters, warmup, min_seconds=0.0):
    """Runs fn(i) warmup + iters times; returns ms per iteration (CUDA events on the launching stream).
    With min_seconds the iteration count is raised until the timed region lasts at least that long."""
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    while True:
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(iters):
            fn(i)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        if ms * 1e-3 >= min_seconds or iters >= 1 << 20:
            return ms / iters
        iters = int(iters * max(2.0, 1.25 * min_seconds / max(ms * 1e-3, 1e-6))) + 1


def _pipelined(torch, stream, h2d, compute, d2h, iters, n_sets, warmup=1):
    """End-to-end ms per step of a three-stage pipeline: step i's host->device copies run on a copy-in
    stream, its kernels on `stream` (one library context, so the calls stay in order), its
    device->host copies on a copy-out stream; the inputs of step i + n_sets reuse the device set of
    step i and wait for that step's results to have left.  Every step's copies are inside the timed
    region; they overlap the neighbouring steps' kernels."""
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    for i in range(warmup):
        h2d(i); compute(i); d2h(i)
    torch.cuda.synchronize()
    ev_in = [torch.cuda.Event() for _ in range(iters)]
    ev_cmp = [torch.cuda.Event() for _ in range(iters)]
    ev_out = [torch.cuda.Event() for _ in range(iters)]
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    s_in.wait_stream(stream); s_out.wait_stream(stream)
    for i in range(iters):
        with torch.cuda.stream(s_in):
            if i >= n_sets:
                s_in.wait_event(ev_out[i - n_sets])
            h2d(i)
            ev_in[i].record(s_in)
        stream.wait_event(ev_in[i])
        compute(i)
        ev_cmp[i].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[i])
            d2h(i)
            ev_out[i].record(s_out)
    stream.wait_stream(s_out)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _graph_timed(torch, fn, n_calls, iters=20):
    """ms per call of n_calls consecutive calls fn(i, stream) replayed as one CUDA graph: the device
    time of back-to-back launches without the host's marshalling between them.  None when the capture
    is refused."""
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            for i in range(n_calls):
                fn(i, side.cuda_stream)
            torch.cuda.synchronize()
            with torch.cuda.graph(g, stream=side):
                for i in range(n_calls):
                    fn(i, side.cuda_stream)
            torch.cuda.synchronize()
            for _ in range(3):
                g.replay()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(iters):
                g.replay()
            e1.record(side)
            torch.cuda.synchronize()
        torch.cuda.current_stream().wait_stream(side)
        return e0.elapsed_time(e1) / iters / n_calls
    except Exception:
        torch.cuda.synchronize()
        return None


def _hbm_call(pk, nbytes, ms, graph_ms=None):
    gbs = nbytes / (ms * 1e-3) / 1e9
    c = {"ms": round(ms, 5), "gbs": round(gbs, 1), "frac_hbm": round(gbs / pk["hbm"], 4),
         "frac_hbm_nominal": round(gbs / NOMINAL_HBM, 4), "bytes": int(nbytes)}
    if graph_ms:
        g = nbytes / (graph_ms * 1e-3) / 1e9
        c.update({"graph_ms": round(graph_ms, 5), "graph_gbs": round(g, 1), "graph_frac_hbm": round(g / pk["hbm"], 4)})
    return c


def _tensor_call(pk, flops, ms, launches=None):
    tf = flops / (ms * 1e-3) / 1e12
    c = {"ms": round(ms, 5), "tflops": round(tf, 2), "frac_tensor": round(tf / pk["tensor"], 4),
         "frac_tensor_sustained": round(tf / pk["tensor_sustained"], 4) if pk["tensor_sustained"] else None,
         "frac_tensor_nominal": round(tf / NOMINAL_TENSOR, 4)}
    if launches:
        c["launches"] = launches
    return c


def _hbm_roofline(pk, kernel, nbytes, ms, traffic, timing):
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": kernel, "achieved": round(gbs, 1), "peak": pk["hbm"], "unit": "GB/s",
            "frac": round(gbs / pk["hbm"], 4), "peak_kind": "copy, " + pk["kind"], "frac_of_nominal_8000": round(gbs / NOMINAL_HBM, 4),
            "timing": timing, "traffic": traffic}


EVENTS = "CUDA events on the launching stream around back-to-back calls, region >= %.1f s" % MIN_REGION_S


def leg_cfg5(args, quick=False):
    """Decode: N=8 caches x 4096 tokens; a step = 3 local calls + 1 sync call (sync every H=4)."""
    quick = quick or args.quick
    torch, fa, dev = _setup()
    w = fi.cfg5()
    N, Hq, Hkv, d, L = w.n_participants, w.n_q_heads, w.n_kv_heads, w.head_dim, w.total_tokens
    seqlens = list(w.seqlens)
    cu = [0] + list(np.cumsum(seqlens))
    shape = fa.Shape(N, Hq, Hkv, d, fa.BF16)
    ctx = fa.Context(shape, L, L)
    bf = torch.bfloat16
    n_sets = max(2, args.sets)
    stream = torch.cuda.current_stream()
    caches = []
    for s_ in range(n_sets):
        _, k, v = w.qkv(block=s_)
        tk, tv = (torch.from_numpy(x).to(bf).to(dev) for x in (k, v))
        kg, vg = torch.empty_like(tk), torch.empty_like(tv)
        kp = [tk[cu[n]:cu[n + 1]] for n in range(N)]; vp = [tv[cu[n]:cu[n + 1]] for n in range(N)]
        fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_CONCAT, kp, vp, seqlens, None, None, kg, vg, None, None, None)
        caches.append((tk, tv, kg, vg))
    n_q = 8
    hq = [torch.from_numpy(w.decode_q(i)).to(bf).pin_memory() for i in range(n_q)]
    qs = [x.to(dev) for x in hq]
    o = torch.empty_like(qs[0])
    ho = torch.empty((N, Hq, d), dtype=bf).pin_memory()
    len_local = torch.tensor(seqlens, dtype=torch.int32, device=dev)
    len_sync = torch.tensor([L], dtype=torch.int32, device=dev)
    stride = seqlens[0] * Hkv * d
    # every (cache set, query) combination marshalled once: the loop below costs one foreign call per decode call
    period = n_sets * n_q
    p_local = [fa.prepare_decode(ctx, shape, fa.DECODE_LOCAL, qs[i % n_q], caches[i % n_sets][0], caches[i % n_sets][1], stride,
                                 len_local, max(seqlens), o) for i in range(period)]
    p_sync = [fa.prepare_decode(ctx, shape, fa.DECODE_SYNC, qs[i % n_q], caches[i % n_sets][2], caches[i % n_sets][3], 0,
                                len_sync, L, o) for i in range(period)]

    def call(i, sync, stream=None):
        (p_sync if sync else p_local)[i % period](stream)

    def step(i):                                         # decode steps 4i+1 .. 4i+4: the 4th is a sync step
        for j in range(4):
            call(4 * i + j, fi.is_sync_block(j + 1, 4))

    W = max(args.warmup, 3)
    floor = 0.0 if quick else MIN_REGION_S
    sampler = ClockSampler(0); sampler.start(); time.sleep(0.25)
    n_it = 8 if quick else 400
    ms_local = _timed(torch, stream, lambda i: call(i, False), n_it, W, floor)
    ms_sync = _timed(torch, stream, lambda i: call(i, True), n_it, W, floor)
    l0 = ctx.launch_count()
    step(0)
    launches = ctx.launch_count() - l0
    ms_step = _timed(torch, stream, step, 4 if quick else 100, W, floor)
    time.sleep(0.25); clocks = sampler.stop()
    assert ctx.poll() == 0

    def e2e_step(i):                                     # 64 KB each way: copies stay on the launching stream
        qs[i % n_q].copy_(hq[i % n_q], non_blocking=True)
        step(i)
        ho.copy_(o, non_blocking=True)
    ms_e2e = _timed(torch, stream, e2e_step, 2 if quick else 50, 2)

    g_local = None if quick else _graph_timed(torch, lambda i, st: call(i, False, st), 2 * n_sets)
    g_sync = None if quick else _graph_timed(torch, lambda i, st: call(i, True, st), 2 * n_sets)
    kv_bytes = 2 * L * Hkv * d * 2 + 2 * N * Hq * d * 2        # per call: every K/V row once + q + o
    pk = peaks()
    calls = {"decode_local": _hbm_call(pk, kv_bytes, ms_local, g_local), "decode_sync": _hbm_call(pk, kv_bytes, ms_sync, g_sync),
             "decode_step_3local_1sync": _hbm_call(pk, 4 * kv_bytes, ms_step)}
    calls["decode_step_3local_1sync"]["launches"] = launches
    roof = _hbm_roofline(pk, "decode_stream_kernel + decode_merge_kernel (two launches per decode call; 3 local + 1 sync)",
                         4 * kv_bytes, ms_step, 4 * DECODE_DRAM_BYTES, EVENTS)
    return {"calls": calls, "rooflines": {"decode": roof}, "launches": launches, "ms_step": ms_step, "clocks": clocks,
            "metric": "fedattn_decode_gbs", "unit": "GB/s", "value": 4 * kv_bytes / (ms_step * 1e-3) / 1e9,
            "config": {"workload": w.name, "participants": N, "cache_tokens": seqlens[0], "q_heads": Hq, "kv_heads": Hkv, "head_dim": d,
                       "step": "3 x decode_local + 1 x decode_sync (sync every 4th decode step)",
                       "l2": "%d rotating cache sets of %d MB (K+V, > 126 MB L2 each)" % (n_sets, 2 * L * Hkv * d * 2 // 2 ** 20),
                       "parallelism": "single"},
            "e2e": {"value": round(4 * kv_bytes / (ms_e2e * 1e-3) / 1e9, 1), "unit": "GB/s", "h2d_bytes_per_step": hq[0].numel() * 2,
                    "d2h_bytes_per_step": ho.numel() * 2, "ms_per_step": round(ms_e2e, 4)}}


def leg_cfg4(args, quick=False):
    """Sparse aggregation (top 256 of 1024 keys per participant and KV head) + sync over the selected KV,
    and the exchange block that keeps the own segment complete (top-k and seeded random selection)."""
    quick = quick or args.quick
    torch, fa, dev = _setup()
    w = fi.cfg4()
    N, Hq, Hkv, d, L = w.n_participants, w.n_q_heads, w.n_kv_heads, w.head_dim, w.total_tokens
    seqlens = list(w.seqlens)
    cu = [0] + list(np.cumsum(seqlens))
    ksel = [w.k_sel] * N
    T = sum(ksel)
    shape = fa.Shape(N, Hq, Hkv, d, fa.BF16)
    ctx = fa.Context(shape, L, L)
    bf = torch.bfloat16
    n_sets = max(3, args.sets)
    stream = torch.cuda.current_stream()
    host, sets = [], []
    for s_ in range(n_sets):
        q, k, v = w.qkv(block=s_)
        hs = [torch.from_numpy(x).to(bf).pin_memory() for x in (q, k, v)]
        host.append(hs)
        tq, tk, tv = (x.to(dev) for x in hs)
        sets.append(dict(q=tq, k=tk, v=tv, kp=[tk[cu[n]:cu[n + 1]] for n in range(N)], vp=[tv[cu[n]:cu[n + 1]] for n in range(N)],
                         k_sp=torch.empty((Hkv, T, d), dtype=bf, device=dev), v_sp=torch.empty((Hkv, T, d), dtype=bf, device=dev),
                         pos=torch.empty((Hkv, T), dtype=torch.int32, device=dev), sel=torch.empty((Hkv, T), dtype=torch.int32, device=dev),
                         o=torch.empty_like(tq)))
    ho = torch.empty((L, Hq, d), dtype=bf).pin_memory()
    # a seeded random selection at the same ratio: the draw is an input (int32 [Hkv, T] local indices)
    sel_rand = torch.from_numpy(fi.random_selection(w.seed, seqlens, ksel, Hkv)).to(dev)
    for b in sets:                                       # token-level outputs, one set per input set like the rest
        b["k_tok"] = torch.empty((T, Hkv, d), dtype=bf, device=dev); b["v_tok"] = torch.empty_like(b["k_tok"])
        b["pos_tok"] = torch.empty((T,), dtype=torch.int32, device=dev); b["sel_tok"] = torch.empty_like(b["pos_tok"])
    o_b = torch.empty_like(sets[0]["q"])
    lse_a = torch.empty((L, Hq), dtype=torch.float32, device=dev); lse_b = torch.empty_like(lse_a)

    def prep(b):
        return dict(
            agg=fa.prepare_aggregate_kv(ctx, shape, fa.AGG_TOPK_KNORM, b["kp"], b["vp"], seqlens, ksel, None, b["k_sp"], b["v_sp"],
                                        b["pos"], None, b["sel"]),
            agg_tok=fa.prepare_aggregate_kv(ctx, shape, fa.AGG_TOPK_TOKEN, b["kp"], b["vp"], seqlens, ksel, None, b["k_tok"],
                                            b["v_tok"], b["pos_tok"], None, b["sel_tok"]),
            agg_rand=fa.prepare_aggregate_kv(ctx, shape, fa.AGG_INDEXED, b["kp"], b["vp"], seqlens, ksel, sel_rand, b["k_sp"],
                                             b["v_sp"], b["pos"], None, None),
            sync=fa.prepare_sync(ctx, shape, b["q"], None, b["k_sp"], b["v_sp"], b["pos"], T, True, b["o"]),
            local=fa.prepare_local(ctx, shape, b["q"], b["k"], b["v"], cu, b["o"], lse_a),
            remote=fa.prepare_sync_remote(ctx, shape, b["q"], cu, b["k_sp"], b["v_sp"], b["pos"], T, True, o_b, lse_b),
            merge=fa.prepare_merge(ctx, shape, L, b["o"], lse_a, o_b, lse_b, b["o"], None))
    P = [prep(b) for b in sets]

    def agg(i, stream=None): P[i % n_sets]["agg"](stream)
    def agg_tok(i, stream=None): P[i % n_sets]["agg_tok"](stream)
    def agg_rand(i): P[i % n_sets]["agg_rand"]()
    def sync(i): P[i % n_sets]["sync"]()

    def step(i):
        agg(i); sync(i)

    def exchange(i):                                     # positions/selection of set i are already in place
        pc = P[i % n_sets]
        pc["local"](); pc["remote"](); pc["merge"]()

    def exchange_random(i):                              # indexed aggregation of the random draw, then the block
        pc = P[i % n_sets]
        pc["agg_rand"](); pc["local"](); pc["remote"](); pc["merge"]()

    K, W = args.steps, max(args.warmup, 3)
    floor = 0.0 if quick else MIN_REGION_S
    for i in range(n_sets):
        step(i)
    assert ctx.poll() == 0
    pos = sets[0]["pos"].to(torch.int64)
    rows = torch.arange(L, device=dev, dtype=torch.int64)
    pairs = sum(int(torch.searchsorted(pos[h].contiguous(), rows, right=True).sum().item()) for h in range(Hkv))
    f_sync = 4.0 * d * (Hq // Hkv) * pairs
    f_exch = 4.0 * d * Hq * (sum(n * (n + 1) // 2 for n in seqlens) + sum(seqlens[n] * sum(ksel[:n]) for n in range(N)))
    sampler = ClockSampler(0); sampler.start(); time.sleep(0.25)
    n_it = 8 if quick else 200
    ms_agg = _timed(torch, stream, agg, n_it, W, floor)
    ms_tok = _timed(torch, stream, agg_tok, n_it, W, floor)
    ms_sync = _timed(torch, stream, sync, K, W)
    ms_exch = _timed(torch, stream, exchange, K, W)
    l0 = ctx.launch_count()
    step(0)
    launches = ctx.launch_count() - l0
    ms_step = _timed(torch, stream, step, K, W)
    g_agg = None if quick else _graph_timed(torch, agg, 2 * n_sets)
    g_tok = None if quick else _graph_timed(torch, agg_tok, 2 * n_sets)
    # the random draw last: it overwrites the sparse aggregate of every set
    ms_rand = _timed(torch, stream, agg_rand, n_it, W, floor)
    ms_exch_rand = _timed(torch, stream, exchange_random, K, W)
    time.sleep(0.25); clocks = sampler.stop()
    assert ctx.poll() == 0
    for i in range(n_sets):                              # back to the top-k aggregate for the end-to-end leg
        agg(i)

    def e2e_in(i):
        b, hs = sets[i % n_sets], host[i % n_sets]
        b["q"].copy_(hs[0], non_blocking=True); b["k"].copy_(hs[1], non_blocking=True); b["v"].copy_(hs[2], non_blocking=True)
    ms_e2e = _pipelined(torch, stream, e2e_in, step, lambda i: ho.copy_(sets[i % n_sets]["o"], non_blocking=True),
                        max(3, min(K, 10)), n_sets)
    assert ctx.poll() == 0
    kv_bytes = 2 * L * Hkv * d * 2
    agg_bytes = kv_bytes // 2 + (kv_bytes // 2) * T // L + kv_bytes * T // L     # K once + selected V + selected K,V written
    idx_bytes = 2 * kv_bytes * T // L + Hkv * T * 4                              # selected K,V read and written + the indices
    pk = peaks()
    calls = {"aggregate_topk": _hbm_call(pk, agg_bytes, ms_agg, g_agg), "aggregate_topk_token": _hbm_call(pk, agg_bytes, ms_tok, g_tok),
             "aggregate_indexed_random": _hbm_call(pk, idx_bytes, ms_rand),
             "sync_sparse": _tensor_call(pk, f_sync, ms_sync),
             "sync_exchange_own_complete_topk": _tensor_call(pk, f_exch, ms_exch, 3),
             "sync_exchange_own_complete_random": _tensor_call(pk, f_exch, ms_exch_rand, 4)}
    roof = _hbm_roofline(pk, "topk_fused_kernel (scores, selection and gather of one sparse aggregation)", agg_bytes, ms_agg,
                         TOPK_DRAM_BYTES, EVENTS)
    return {"calls": calls, "rooflines": {"aggregate": roof}, "launches": launches, "ms_step": ms_step, "clocks": clocks,
            "metric": "fedattn_aggregate_gbs", "unit": "GB/s", "value": agg_bytes / (ms_agg * 1e-3) / 1e9,
            "config": {"workload": w.name, "participants": N, "tokens_per_participant": seqlens[0], "q_heads": Hq, "kv_heads": Hkv,
                       "head_dim": d, "keep_per_kv_head": w.k_sel, "step": "aggregate_topk + sync over the selected KV",
                       "l2": "%d rotating input/output sets (> 126 MB L2 in total)" % n_sets, "parallelism": "single"},
            "e2e": {"value": round(agg_bytes / (ms_e2e * 1e-3) / 1e9, 1), "unit": "GB/s",
                    "h2d_bytes_per_step": sum(x.numel() * 2 for x in host[0]), "d2h_bytes_per_step": ho.numel() * 2,
                    "ms_per_step": round(ms_e2e, 4),
                    "pipeline": "copy-in, kernels and copy-out of neighbouring steps overlap on three streams"}}


def leg_cfg3(args, quick=False):
    """32-block schedules over 8 heterogeneous segments: block m is a sync block iff m mod H == 0."""
    torch, fa, dev = _setup()
    w = fi.cfg3()
    N, Hq, Hkv, d, L = w.n_participants, w.n_q_heads, w.n_kv_heads, w.head_dim, w.total_tokens
    seqlens = list(w.seqlens)
    cu = [0] + list(np.cumsum(seqlens))
    shape = fa.Shape(N, Hq, Hkv, d, fa.BF16)
    ctx = fa.Context(shape, L, L)
    bf = torch.bfloat16
    n_sets = max(3, args.sets)
    stream = torch.cuda.current_stream()
    host, sets = [], []
    for s_ in range(n_sets):
        q, k, v = w.qkv(block=s_)
        hs = [torch.from_numpy(x).to(bf).pin_memory() for x in (q, k, v)]
        host.append(hs)
        tq, tk, tv = (x.to(dev) for x in hs)
        sets.append(dict(q=tq, k=tk, v=tv, kp=[tk[cu[n]:cu[n + 1]] for n in range(N)], vp=[tv[cu[n]:cu[n + 1]] for n in range(N)],
                         kg=torch.empty_like(tk), vg=torch.empty_like(tv), o=torch.empty_like(tq)))
    ho = torch.empty((L, Hq, d), dtype=bf).pin_memory()
    M = w.n_blocks

    def block(m, H):
        # H: the uniform interval, or the explicit set of sync blocks of a non-uniform schedule
        b = sets[m % n_sets]
        if (m in H) if isinstance(H, frozenset) else fi.is_sync_block(m, H):
            fa.fedattn_aggregate_kv(ctx, shape, fa.AGG_CONCAT, b["kp"], b["vp"], seqlens, None, None, b["kg"], b["vg"], None, None, None)
            fa.fedattn_sync(ctx, shape, b["q"], None, b["kg"], b["vg"], None, L, False, b["o"])
        else:
            fa.fedattn_local(ctx, shape, b["q"], b["k"], b["v"], cu, b["o"])

    f_local = 4.0 * d * Hq * sum(n * (n + 1) // 2 for n in seqlens)
    f_sync = 4.0 * d * Hq * (L * (L + 1) // 2)
    K, W = (1 if quick else max(1, args.steps // 8)), 1
    sampler = ClockSampler(0); sampler.start(); time.sleep(0.25)
    per_h = {}
    for blk in range(1, 4):
        block(blk, 1); block(blk, M + 1)                     # warm-up of both paths
    l0 = ctx.launch_count()
    [block(m, 1) for m in range(1, M + 1)]
    launches = ctx.launch_count() - l0
    for H in (1, 2, 4, 8, 32):
        ms = _timed(torch, stream, lambda i, H=H: [block(m, H) for m in range(1, M + 1)], K, W)
        n_sync = sum(1 for m in range(1, M + 1) if fi.is_sync_block(m, H))
        fl = n_sync * f_sync + (M - n_sync) * f_local
        per_h[str(H)] = {"ms": round(ms, 4), "sync_blocks": n_sync, "ms_per_block": round(ms / M, 4),
                         "tflops": round(fl / (ms * 1e-3) / 1e12, 2)}
    # Non-uniform schedules with four exchanges each (Theorem 3: H_t local forwards in round t): exchanges
    # in the shallow or the deep half, intervals growing or shrinking with depth.  The paper does not
    # print its intervals; these are stand-ins of that form.
    named = {"shallow_half": fi.sync_blocks_of_rounds([4, 4, 4, 4]), "deep_half": [20, 24, 28, 32],
             "progressive": fi.sync_blocks_of_rounds([2, 4, 8, 18]), "regressive": fi.sync_blocks_of_rounds([18, 8, 4, 2])}
    for name, blocks in named.items():
        sset = frozenset(blocks)
        ms = _timed(torch, stream, lambda i, sset=sset: [block(m, sset) for m in range(1, M + 1)], K, W)
        fl = len(sset) * f_sync + (M - len(sset)) * f_local
        per_h[name] = {"ms": round(ms, 4), "sync_blocks": sorted(sset), "ms_per_block": round(ms / M, 4),
                       "tflops": round(fl / (ms * 1e-3) / 1e12, 2)}
    # A block in which only the first half of the participants exchange (adaptive aggregation): their rows
    # attend the members' aggregated KV through explicit query positions (tensor-core kernel with position
    # tables), the other participants run their local attention.
    half = N // 2
    Lm = cu[half]
    shape_m = fa.Shape(half, Hq, Hkv, d, fa.BF16)
    shape_r = fa.Shape(N - half, Hq, Hkv, d, fa.BF16)
    cu_r = [c - Lm for c in cu[half:]]
    q_pos = torch.arange(Lm, dtype=torch.int32, device=dev)
    kv_pos_m = torch.empty(Lm, dtype=torch.int32, device=dev)
    tc0 = ctx.tensor_core_launch_count()

    def subset_block(i):
        b = sets[i % n_sets]
        fa.fedattn_aggregate_kv(ctx, shape_m, fa.AGG_CONCAT, b["kp"][:half], b["vp"][:half], seqlens[:half], None, None,
                                b["kg"][:Lm], b["vg"][:Lm], kv_pos_m, None, None)
        fa.fedattn_sync(ctx, shape_m, b["q"][:Lm], q_pos, b["kg"][:Lm], b["vg"][:Lm], kv_pos_m, Lm, False, b["o"][:Lm])
        fa.fedattn_local(ctx, shape_r, b["q"][Lm:], b["k"][Lm:], b["v"][Lm:], cu_r, b["o"][Lm:])
    subset_block(0)
    subset_tc = ctx.tensor_core_launch_count() - tc0
    ms_subset = _timed(torch, stream, subset_block, max(3, 4 * K), 2)
    f_subset = 4.0 * d * Hq * (Lm * (Lm + 1) // 2 + sum(n * (n + 1) // 2 for n in seqlens[half:]))
    time.sleep(0.25); clocks = sampler.stop()
    assert ctx.poll() == 0

    def e2e_in(i):                                             # one sync block through host buffers
        b, hs = sets[i % n_sets], host[i % n_sets]
        b["q"].copy_(hs[0], non_blocking=True); b["k"].copy_(hs[1], non_blocking=True); b["v"].copy_(hs[2], non_blocking=True)
    # block(m, 1) works on set m mod n_sets
    ms_e2e = _pipelined(torch, stream, e2e_in, lambda i: block(i, 1), lambda i: ho.copy_(sets[i % n_sets]["o"], non_blocking=True),
                        6, n_sets)

    pk = peaks()
    value = per_h["1"]["tflops"]
    calls = {"schedule_H%s" % h: {"ms": v["ms"], "tflops": v["tflops"], "sync_blocks": v["sync_blocks"]} for h, v in per_h.items()}
    calls["subset_exchange_block"] = _tensor_call(pk, f_subset, ms_subset, 4)
    calls["subset_exchange_block"]["tensor_core_launches"] = subset_tc
    roof = {"bound": "tensor", "kernel": "prefill_sm100_kernel (32 sync blocks of the H=1 schedule)", "achieved": value,
            "peak": pk["tensor"], "unit": "TFLOP/s", "frac": round(value / pk["tensor"], 4), "peak_kind": "burst bf16, " + pk["kind"],
            "frac_of_sustained": round(value / pk["tensor_sustained"], 4) if pk["tensor_sustained"] else None,
            "frac_of_nominal_2250": round(value / NOMINAL_TENSOR, 4), "traffic": None}
    return {"calls": calls, "rooflines": {"prefill_cfg3": roof}, "launches": launches, "ms_step": per_h["1"]["ms"], "clocks": clocks,
            "metric": METRIC, "unit": UNIT, "value": value,
            "config": {"workload": w.name, "participants": N, "segment_lengths": seqlens, "q_heads": Hq, "kv_heads": Hkv, "head_dim": d,
                       "blocks": M, "step": "the H=1 schedule: 32 x (concat + sync); `schedules` lists every H",
                       "l2": "%d rotating seeded blocks of inputs stand in for the 32 fresh ones (> 126 MB L2 each)" % n_sets,
                       "parallelism": "single"},
            "e2e": {"value": round(f_sync / (ms_e2e * 1e-3) / 1e12, 2), "unit": UNIT,
                    "h2d_bytes_per_step": sum(x.numel() * 2 for x in host[0]), "d2h_bytes_per_step": ho.numel() * 2,
                    "ms_per_step": round(ms_e2e, 4),
                    "pipeline": "copy-in, kernels and copy-out of neighbouring steps overlap on three streams"},
            "extra": {"schedules": per_h, "local_block_tflop": round(f_local / 1e12, 4), "sync_block_tflop": round(f_sync / 1e12, 4)}}


def leg_cfg1(args, quick=False):
    """fp32, N=2 x 128 tokens, 4 heads, d=64: latency-bound; time per call of local, concat and sync."""
    torch, fa, dev = _setup()
    w = fi.cfg1()
    N, H, d, L = w.n_participants, w.n_q_heads, w.head_dim, w.total_tokens
    seqlens = list(w.seqlens)
    cu = [0] + list(np.cumsum(seqlens))
    shape = fa.Shape(N, H, H, d, fa.F32)
    ctx = fa.Context(shape, L, L)
    stream = torch.cuda.current_stream()
    q, k, v = w.qkv()
    hq, hk, hv = (torch.from_numpy(x).pin_memory() for x in (q, k, v))
    tq, tk, tv = (x.to(dev) for x in (hq, hk, hv))
    o = torch.empty_like(tq); kg = torch.empty_like(tk); vg = torch.empty_like(tv)
    ho = torch.empty_like(hq).pin_memory()
    kv_pos = torch.empty(L, dtype=torch.int32, device=dev)
    kp = [tk[cu[n]:cu[n + 1]] for n in range(N)]; vp = [tv[cu[n]:cu[n + 1]] for n in range(N)]
    p_local = fa.prepare_local(ctx, shape, tq, tk, tv, cu, o)
    p_cat = fa.prepare_aggregate_kv(ctx, shape, fa.AGG_CONCAT, kp, vp, seqlens, None, None, kg, vg, kv_pos, None, None)
    p_sync = fa.prepare_sync(ctx, shape, tq, None, kg, vg, kv_pos, L, False, o)
    floor = 0.0 if quick else MIN_REGION_S / 4
    ms_local = _timed(torch, stream, lambda i: p_local(), 200, 5, floor)
    ms_cat = _timed(torch, stream, lambda i: p_cat(), 200, 5, floor)
    ms_sync = _timed(torch, stream, lambda i: p_sync(), 200, 5, floor)

    def step(i):
        p_local(); p_cat(); p_sync()
    ms_step = _timed(torch, stream, step, 200, 5, floor)

    def e2e(i):
        tq.copy_(hq, non_blocking=True); tk.copy_(hk, non_blocking=True); tv.copy_(hv, non_blocking=True)
        step(i)
        ho.copy_(o, non_blocking=True)
    ms_e2e = _timed(torch, stream, e2e, 100, 3)
    assert ctx.poll() == 0
    f_local = 4.0 * d * H * sum(n * (n + 1) // 2 for n in seqlens)
    f_sync = 4.0 * d * H * (L * (L + 1) // 2)
    calls = {"local": {"us": round(ms_local * 1e3, 2), "gflops": round(f_local / (ms_local * 1e-3) / 1e9, 1)},
             "aggregate_concat": {"us": round(ms_cat * 1e3, 2)},
             "sync": {"us": round(ms_sync * 1e3, 2), "gflops": round(f_sync / (ms_sync * 1e-3) / 1e9, 1)},
             "step_local_concat_sync": {"us": round(ms_step * 1e3, 2)}}
    return {"calls": calls, "rooflines": {}, "launches": 3, "ms_step": ms_step, "clocks": None,
            "metric": "fedattn_cfg1_step_us", "unit": "us", "value": ms_step * 1e3, "higher_is_better": False,
            "config": {"workload": w.name, "participants": N, "tokens_per_participant": seqlens[0], "heads": H, "head_dim": d,
                       "step": "local + concat + sync (fp32, SIMT kernel; latency-bound, no roofline target)",
                       "l2": "inputs of 0.2 MB stay in L2: this configuration is a latency measurement", "parallelism": "single"},
            "e2e": {"value": round(ms_e2e * 1e3, 2), "unit": "us", "h2d_bytes_per_step": 3 * hq.numel() * 4,
                    "d2h_bytes_per_step": ho.numel() * 4, "ms_per_step": round(ms_e2e, 5)}}


LEGS = {"cfg1": leg_cfg1, "cfg3": leg_cfg3, "cfg4": leg_cfg4, "cfg5": leg_cfg5}


def run_leg(args, name):
    """One configuration alone, as a line of its own."""
    r = LEGS[name](args)
    dominant = next(iter(r["rooflines"].values()), None)
    out = {"metric": r["metric"], "value": round(r["value"], 3), "unit": r["unit"], "n_gpus": 1, "steps": args.steps,
           "warmup": max(args.warmup, 3), "ms_per_step": round(r["ms_step"], 5), "higher_is_better": r.get("higher_is_better", True),
           "scaling": "weak", "vs_baseline": None, "dtype": "f32" if name == "cfg1" else "bf16", "data": "synthetic",
           "config": r["config"], "clocks": r["clocks"], "e2e": r["e2e"], "gpu_launches": int(r["launches"]),
           "roofline": dominant, "rooflines": r["rooflines"], "calls": r["calls"]}
    out.update(r.get("extra", {}))
    if not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_legs([name])[name]
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample(w, q, k, v, n_rows, seed):
    """Runs the oracle's local and sync attention on n_rows seeded rows (all heads).
    Returns (seconds, algorithmic flops of the sample)."""
    import oracle
    rng = np.random.default_rng(seed)
    rows = np.sort(rng.choice(w.total_tokens, size=n_rows, replace=False)).astype(np.int64)
    off = np.concatenate([[0], np.cumsum(w.seqlens)])
    seg = np.searchsorted(off, rows, side="right") - 1
    pairs = int((rows - off[seg] + 1).sum() + (rows + 1).sum())
    t0 = time.perf_counter()
    oracle.local(q, k, v, w.seqlens, rows=rows)
    oracle.sync(q, k, v, rows=rows)
    dt = time.perf_counter() - t0
    return dt, 4.0 * w.head_dim * w.n_q_heads * pairs


def cpu_baseline(w, target_seconds):
    import oracle
    q, k, v = w.qkv(0)
    q, k, v = (x.astype(np.float64) for x in (q, k, v))
    dt, fl = oracle_sample(w, q, k, v, 16, 0)
    n = int(min(w.total_tokens, max(16, 16 * target_seconds / max(dt, 1e-3))))
    dt, fl = oracle_sample(w, q, k, v, n, 1)
    return {"value": round(fl / dt / 1e12, 6), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "fp64 oracle local+sync attention on %d seeded query rows x %d heads of %s (%.1f s)"
                      % (n, w.n_q_heads, w.name, dt)}


def oracle_legs(names):
    """The oracle as it stands, timed on the host cores at full size where that takes seconds:
    cfg1 local + sync; cfg4 the sparse aggregation (scores, selection, gather); cfg5 one local and
    one sync decode step.  A reported baseline, not a target."""
    import oracle
    out = {}
    for name in names:
        w = fi.ALL[name]()
        if name == "cfg1":
            q, k, v = (x.astype(np.float64) for x in w.qkv())
            t0 = time.perf_counter()
            oracle.local(q, k, v, w.seqlens)
            oracle.sync(q, k, v)
            dt = time.perf_counter() - t0
            out[name] = {"value": round(dt, 4), "unit": "s", "cores": oracle.threads(), "kind": "oracle",
                         "sample": "full size: fp64 local + sync attention of %s" % w.name}
        elif name == "cfg4":
            _, k, v = w.qkv()
            cuts = np.cumsum(w.seqlens)[:-1]
            kp = [x.astype(np.float64) for x in np.split(k, cuts)]; vp = [x.astype(np.float64) for x in np.split(v, cuts)]
            t0 = time.perf_counter()
            oracle.aggregate_topk(kp, vp, [w.k_sel] * w.n_participants)
            dt = time.perf_counter() - t0
            kv_bytes = 2 * w.total_tokens * w.n_kv_heads * w.head_dim * 2
            nbytes = kv_bytes // 2 + (kv_bytes // 2) // 4 + kv_bytes // 4
            out[name] = {"value": round(nbytes / dt / 1e9, 4), "unit": "GB/s", "seconds": round(dt, 3), "cores": 1, "kind": "oracle",
                         "sample": "full size: fp64 key-norm scores, selection and gather of %s (bf16-equivalent bytes)" % w.name}
        elif name == "cfg5":
            _, k, v = w.qkv()
            k, v = k.astype(np.float64), v.astype(np.float64)
            n, cap = w.n_participants, w.seqlens[0]
            q = w.decode_q(1).astype(np.float64)
            t0 = time.perf_counter()
            oracle.decode(q, k.reshape(n, cap, w.n_kv_heads, w.head_dim), v.reshape(n, cap, w.n_kv_heads, w.head_dim), [cap] * n, False)
            t1 = time.perf_counter()
            oracle.decode(q, k, v, [n * cap], True)
            t2 = time.perf_counter()
            kv_bytes = 2 * w.total_tokens * w.n_kv_heads * w.head_dim * 2
            out[name] = {"value": round(2 * kv_bytes / (t2 - t0) / 1e9, 4), "unit": "GB/s", "local_step_s": round(t1 - t0, 3),
                         "sync_step_s": round(t2 - t1, 3), "cores": oracle.threads(), "kind": "oracle",
                         "sample": "full size: one local and one sync decode step of %s in fp64 (bf16-equivalent bytes)" % w.name}
        else:
            q, k, v = (x.astype(np.float64) for x in w.qkv(0))
            dt, fl = oracle_sample(w, q, k, v, 64, 3)
            out[name] = {"value": round(fl / dt / 1e12, 6), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": "fp64 local + sync attention on 64 seeded query rows of %s (%.1f s)" % (w.name, dt)}
    return out


def run_reference(args):
    rank, _, world = env_rank()
    if rank != 0:
        return
    import oracle
    w = workload()
    q, k, v = w.qkv(0)
    q, k, v = (x.astype(np.float64) for x in (q, k, v))
    dt, _ = oracle_sample(w, q, k, v, 16, 0)
    budget = 120.0 / max(1, args.steps + max(args.warmup, 1))
    n = int(min(w.total_tokens, max(16, 16 * min(budget, 8.0) / max(dt, 1e-3))))
    for i in range(max(args.warmup, 1)):
        oracle_sample(w, q, k, v, n, 10 + i)
    tot_t, tot_f = 0.0, 0.0
    for i in range(args.steps):
        dt, fl = oracle_sample(w, q, k, v, n, 100 + i)
        tot_t += dt; tot_f += fl
    value = tot_f / tot_t / 1e12
    sample = "fp64 oracle local+sync attention on %d seeded query rows x %d heads of %s per step" % (
        n, w.n_q_heads, w.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 1), "ms_per_step": round(tot_t / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample": sample},
        "cpu_baseline": {"value": round(value, 6), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": round(value, 6), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="all", choices=["all", "cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--quick", action="store_true",
                    help="few iterations per leg and no graph replays (keeps a profiler capture short)")
    ap.add_argument("--sets", type=int, default=N_SETS,
                    help="rotating input sets (1 keeps device memory small for a profiler capture)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload in ("all", "cfg2"):
        run_ours(args)
    else:
        run_leg(args, args.workload)


if __name__ == "__main__":
    main()
