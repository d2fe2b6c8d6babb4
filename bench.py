#!/usr/bin/env python
"""Composed-prefill bench: one step = one layer's pass of the whole hot path (gather + RoPE shift,
fresh-row scatter, partial-prefill attention) over one synthetic batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is composed-prefill tokens/s per layer over all ranks with
inputs resident in HBM; `e2e` is the same metric through the host-buffer entry point (activations
copied from and to pinned host memory every step); `roofline` describes the dominant kernel;
`cpu_baseline` is the fp64 oracle timed on this machine's cores on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM traffic per launch of the two main kernels on config 4, from the ncu capture summarised under
# profiles/ (one request captured; a full launch is `requests` times that, traffic grows with the
# number of requests because requests share nothing).  Bytes per request per launch.
NCU_TRAFFIC_PER_REQUEST_C4 = {"attn": 253.5e6 + 14.7e6, "gather": 134.5e6 + 79.4e6}

METRIC = "composed_prefill_tokens_per_s_per_layer"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(w, tensors_host_bits, budget_s: float, seed: int = 0):
    """Times the oracle as it stands on a bounded sample of workload `w` and extrapolates to one
    whole layer: assembly (gather + rotation) by token count, attention by (query, key) pair count."""
    from oracle import tessera_oracle as orc
    kb, vb, qb, knb, vnb = tensors_host_bits
    rng = np.random.default_rng(seed)
    r = int(np.argmax(w.seq_len))
    t0 = time.perf_counter()
    a = orc.assemble(w, r, kb, vb, knb, vnb)
    t_asm = time.perf_counter() - t0
    asm_per_token = t_asm / max(int(w.seq_len[r]), 1)
    j0, j1 = int(w.recompute_off[r]), int(w.recompute_off[r + 1])
    H = w.shape.num_q_heads
    n_rows, pairs, t_att = 0, 0, 0.0
    chunk = 64
    while t_att < budget_s and j1 > j0:
        jj = rng.integers(j0, j1, size=chunk).astype(np.int32)
        hh = rng.integers(0, H, size=chunk).astype(np.int32)
        pp = w.recompute_pos[jj].astype(np.int32)
        t0 = time.perf_counter()
        orc.attention_rows(w, a.k, a.v_bits, qb, jj, hh, pp)
        t_att += time.perf_counter() - t0
        n_rows += chunk
        pairs += int(pp.astype(np.int64).sum() + chunk)
        chunk = min(chunk * 2, 4096)
    att_per_pair = t_att / max(pairs, 1)
    layer_s = asm_per_token * w.total_tokens + att_per_pair * w.qk_pairs * H
    return {"layer_seconds_extrapolated": layer_s, "assemble_s": t_asm, "attention_s": t_att,
            "rows": n_rows, "pairs": pairs, "cores": orc.num_threads(),
            "sample": "request %d assembled in full (%d tokens) + %d random (row, head) attention rows (%d q-k pairs); "
                      "extrapolated by token count and pair count" % (r, int(w.seq_len[r]), n_rows, pairs)}


def host_bits(t):
    from oracle import tessera_oracle as orc
    return tuple(orc.bits(x) for x in (t.k_pool, t.v_pool, t.q, t.k_new, t.v_new))


def rank_workload(config: int, rank: int, requests=None, policy=None):
    """Every rank owns an independent batch of the same configuration: requests never interact
    (no cross-request attention), so the path shards by request with no data-path collective."""
    from paper_2609_32999_b200 import workloads as wl
    return wl.config(config, seed=wl.BASE_SEED + config + 7919 * rank, requests_override=requests, policy=policy)


def aggregate(times_ms, tokens, world: int, device: str):
    """Max over ranks of every timing and sum over ranks of the tokens processed."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    n = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return t.tolist(), n.item()


def run_reference(args):
    """The reference arm: the oracle on the host cores, on the same workload and metric.  Each step is
    a bounded sample (a fixed share of one layer), extrapolated to a whole layer."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_32999_b200 import workloads as wl
    w = wl.config(args.config, requests_override=args.requests, policy=args.policy)
    t = wl.make_tensors(w, layer=0, device="cpu")
    bits = host_bits(t)
    per_step_budget = max(2.0, min(20.0, 90.0 / max(args.steps + args.warmup, 1)))
    for i in range(args.warmup):
        oracle_sample(w, bits, per_step_budget / 4, seed=100 + i)
    t0 = time.perf_counter()
    layer_s = []
    for i in range(args.steps):
        s = oracle_sample(w, bits, per_step_budget, seed=i)
        layer_s.append(s["layer_seconds_extrapolated"])
    wall = time.perf_counter() - t0
    ms = float(np.mean(layer_s)) * 1e3
    value = w.total_tokens / (ms / 1e3)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "config_index": args.config, "total_tokens": w.total_tokens,
                       "n_q": w.n_q, "note": "each step times a bounded sample of one layer and extrapolates"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": s["cores"], "kind": "oracle", "sample": s["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": wall}
    print(json.dumps(line))


def run_fp8_tier(args):
    """Side measurement, not the headline metric: the cached units of the workload sit in an e4m3 pool
    and are expanded into the requests' bf16 pages (rotation fused), and the reverse (retain).  L2 is
    flushed between timed launches; bytes are the algorithmic ones (1 + 2 per element either way)."""
    import copy
    import torch
    from paper_2609_32999_b200 import binding as tb
    from paper_2609_32999_b200 import workloads as wl
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    dev = "cuda:0"
    torch.cuda.set_device(0)
    w = rank_workload(args.config, 0, args.requests, None)
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    plan = tb.Plan(w2)
    t = wl.make_tensors(w, layer=0, device=dev, seed=wl.BASE_SEED)
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.BASE_SEED)
    shape8 = tuple(t.k_pool.shape)
    k8 = torch.randint(0, 0x78, shape8, dtype=torch.uint8, device=dev, generator=gen)      # finite codes, both signs below
    v8 = torch.randint(0, 0x78, shape8, dtype=torch.uint8, device=dev, generator=gen)
    k8 |= torch.randint(0, 2, shape8, dtype=torch.uint8, device=dev, generator=gen) << 7
    v8 |= torch.randint(0, 2, shape8, dtype=torch.uint8, device=dev, generator=gen) << 7
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def timed(fn):
        ms = []
        for i in range(args.warmup + args.steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            if i >= args.warmup:
                ms.append(a.elapsed_time(b))
        return sum(ms) / len(ms)

    launches0 = tb.launch_count()
    ms_expand = timed(lambda: plan.kv_compose_from_fp8(k8, v8, 1 / 32, 1 / 32, t.k_pool, t.v_pool))
    ms_retain = timed(lambda: plan.kv_retain_fp8(t.k_pool, t.v_pool, k8, v8, 1 / 32, 1 / 32))
    elems = w.cached_tokens * w.shape.num_kv_heads * w.shape.head_dim * 2            # K and V
    peak = measured_peaks()["hbm_gbs"]
    line = {"metric": "fp8_tier_GBps", "unit": "GB/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "dtype": "e4m3 <-> bf16", "data": "synthetic",
            "config": {"workload": w.name, "cached_tokens": int(w.cached_tokens), "l2": "flushed between launches"},
            "expand": {"ms": ms_expand, "GBps": elems * 3 / ms_expand / 1e6, "frac_of_measured_copy": elems * 3 / ms_expand / 1e6 / peak},
            "retain": {"ms": ms_retain, "GBps": elems * 3 / ms_retain / 1e6, "frac_of_measured_copy": elems * 3 / ms_retain / 1e6 / peak},
            "bytes_per_launch": elems * 3, "gpu_launches": tb.launch_count() - launches0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--requests", type=int, default=None, help="override the number of requests (profiling small cases)")
    ap.add_argument("--layers", type=int, default=4, help="distinct per-layer pools cycled through")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle attention sampling")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--policy", default=None, choices=["reuse", "lru", "lfu"],
                    help="residency of the units decided by a cache policy instead of 'all cached' (configs 2-4)")
    ap.add_argument("--graph", action="store_true",
                    help="replay each layer's launches from a captured CUDA graph (latency-bound small batches)")
    ap.add_argument("--tier", default=None, choices=["fp8"],
                    help="time the 8-bit storage tier's two kernels on the workload instead of the hot path (one GPU)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.tier == "fp8":
        return run_fp8_tier(args)

    import torch
    import torch.distributed as dist
    from paper_2609_32999_b200 import binding as tb
    from paper_2609_32999_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = "cuda:%d" % local
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    w = rank_workload(args.config, rank, args.requests, args.policy)
    t_plan = time.perf_counter()
    plan = tb.Plan(w)
    torch.cuda.synchronize()
    plan_create_ms = (time.perf_counter() - t_plan) * 1e3      # host placement + table upload, once per batch
    info = plan.info
    layers = [wl.make_tensors(w, layer=l, device=dev, seed=wl.BASE_SEED + rank) for l in range(args.layers)]
    sh = w.shape
    out = torch.empty(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(w.n_q, sh.num_q_heads, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def step(i, ev=None):
        t = layers[i % args.layers]
        if ev is not None:
            ev[0].record(stream)
        plan.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
        if ev is not None:
            ev[1].record(stream)
        plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse)
        if ev is not None:
            ev[2].record(stream)

    graphs = None
    if args.graph:
        # one graph per layer pool: compose + scatter + attention (+ combine) replayed as one launch
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(args.layers):
                step(i)                         # warm up outside capture (function attributes, descriptors)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graphs = []
        for i in range(args.layers):
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph):
                t = layers[i]
                plan.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
                plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse)
            graphs.append(gph)
        eager_step = step

        def step(i, ev=None):                   # noqa: F811  (graph replay has no inner events)
            if ev is not None:
                ev[0].record(stream)
            graphs[i % args.layers].replay()
            if ev is not None:
                ev[1].record(stream)
                ev[2].record(stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    launches0 = tb.launch_count()
    barrier()
    for i in range(args.steps):
        step(i, evs[i])
    end = torch.cuda.Event(enable_timing=True)
    end.record(stream)
    barrier()
    launches = tb.launch_count() - launches0
    total_ms = evs[0][0].elapsed_time(end)
    gather_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
    attn_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
    clocks = sampler.stop() if rank == 0 else None
    assert plan.status() == 0, "a kernel reported a bounded-wait timeout"

    # ---- end to end through the host-buffer entry point
    t0 = layers[0]
    qh, kh, vh = (x.cpu().pin_memory() for x in (t0.q, t0.k_new, t0.v_new))
    oh = torch.empty_like(qh).pin_memory()
    lh = torch.empty(w.n_q, sh.num_q_heads, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 16))
    for i in range(2):
        plan.composed_prefill_host(t0.k_pool, t0.v_pool, qh, kh, vh, oh, lh)
    barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(stream)
    for i in range(e2e_steps):
        t = layers[i % args.layers]
        plan.composed_prefill_host(t.k_pool, t.v_pool, qh, kh, vh, oh, lh)
    eb.record(stream)
    barrier()
    e2e_ms = ea.elapsed_time(eb) / e2e_steps

    (total_ms_max, e2e_ms_max), all_tokens = aggregate([total_ms, e2e_ms], w.total_tokens, world, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    ms_per_step = total_ms_max / args.steps
    value = all_tokens / (ms_per_step / 1e3)
    attn_tflops = info.attn_flops / (attn_ms / 1e3) / 1e12
    gather_gbs = info.gather_bytes / (gather_ms / 1e3) / 1e9
    tensor_peak = peaks["bf16_tflops_sustained"]     # the kernel is timed inside a long step
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "config_index": args.config, "requests_per_gpu": w.batch,
                   "total_tokens_per_gpu": w.total_tokens, "recompute_tokens_per_gpu": w.n_q,
                   "cached_tokens_per_gpu": w.cached_tokens, "H_q": sh.num_q_heads, "H_kv": sh.num_kv_heads,
                   "head_dim": sh.head_dim, "page_size": sh.page_size,
                   "l2": "inputs larger than L2: %d per-layer KV pools of %.2f GB cycled"
                         % (args.layers, 2 * t0.k_pool.numel() * 2 / 1e9),
                   "attn_kernel": "tcgen05",
                   "cuda_graph": bool(args.graph), "residency": args.policy or "all units cached"},
        "clocks": clocks,
        "gpu_launches": launches,
        "e2e": {"value": all_tokens / (e2e_ms_max / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": int(qh.numel() * 2 + kh.numel() * 2 + vh.numel() * 2),
                "d2h_bytes_per_step": int(oh.numel() * 2 + lh.numel() * 4), "ms_per_step": e2e_ms_max,
                "note": "q, k_new, v_new from pinned host memory, out and lse back to it, every step; "
                        "the KV pools are the resident cache"},
        "roofline": {"kernel": "partial_prefill_attn (fresh-row scatter + attention kernel)", "bound": "tensor",
                     "achieved": attn_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
                     "frac": attn_tflops / tensor_peak, "peak_source": peaks["source"] + " sustained bf16 GEMM",
                     "frac_of_burst": attn_tflops / peaks["bf16_tflops"], "frac_of_nominal_2250": attn_tflops / 2250.0,
                     "ms_per_launch": attn_ms, "flops_per_launch": int(info.attn_flops),
                     "traffic": NCU_TRAFFIC_PER_REQUEST_C4["attn"] * w.batch if args.config == 4 else None,
                     "traffic_note": "DRAM bytes per launch: ncu capture of one request x requests (profiles/)"},
        "roofline_gather": {"kernel": "kv_compose (gather + RoPE shift)", "bound": "hbm", "achieved": gather_gbs,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gather_gbs / peaks["hbm_gbs"],
                            "peak_source": peaks["source"] + " copy", "frac_of_nominal_8000": gather_gbs / 8000.0,
                            "ms_per_launch": gather_ms, "bytes_per_launch": int(info.gather_bytes),
                            "traffic": NCU_TRAFFIC_PER_REQUEST_C4["gather"] * w.batch if args.config == 4 else None},
        "recompute_tokens_per_s": w.n_q * world / (ms_per_step / 1e3),
        "plan_create_ms": plan_create_ms,
    }
    if not args.no_cpu_baseline:
        s = oracle_sample(w, host_bits(t0), args.cpu_budget)
        line["cpu_baseline"] = {"value": w.total_tokens / s["layer_seconds_extrapolated"], "unit": UNIT,
                                "cores": s["cores"], "kind": "oracle", "sample": s["sample"],
                                "layer_seconds_extrapolated": s["layer_seconds_extrapolated"]}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
