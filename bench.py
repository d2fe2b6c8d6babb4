#!/usr/bin/env python
"""Composed-prefill bench: one step = one layer's pass of the whole hot path (gather + RoPE shift,
fresh-row scatter, partial-prefill attention) over one synthetic batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1..5] [--impl ours|reference]

Prints ONE JSON line (rank 0).  The headline leg runs `--config` (default 4, the long-context RAG
batch): `value` is composed-prefill tokens/s per layer over all ranks with inputs resident in HBM;
`e2e` is the same metric through the host-buffer entry point (activations copied from and to pinned
host memory every step); `roofline` / `roofline_gather` describe the two kernels of the headline leg
against the measured burst peaks (the timed region is well under a second); `sustained` repeats the
headline workload back to back for seconds and is rated against the measured sustained GEMM rate;
`per_config` holds the same measurements for the other configurations, each with its own clock
samples and a parity flag from a sampled oracle check; `host_tier` and `fp8_tier` time the side
tiers; `cpu_baseline` is the fp64 oracle timed on this machine's cores on a bounded sample.
"""
from __future__ import annotations

import argparse
import copy
import hashlib
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

METRIC = "composed_prefill_tokens_per_s_per_layer"
UNIT = "tokens/s"
NOMINAL_TFLOPS, NOMINAL_GBS = 2250.0, 8000.0
L2_BYTES = 126e6
MAX_ABS, MEAN_ABS = 2e-2, 2e-3          # tolerance of bf16 attention outputs and re-rotated keys


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def kernel_traffic():
    """DRAM bytes per launch of the two main kernels as ncu measured them on ONE config-4 request
    (profiles/traffic.json, which also records the kernel sources the capture was taken on).  Returns
    (per-request bytes or None, stale flag): stale when a kernel source has changed since."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(p):
        return None, True
    d = json.load(open(p))
    stale = False
    for name, want in d.get("kernel_sources_sha256", {}).items():
        src = os.path.join(ROOT, "paper_2609_32999_b200", "csrc", name)
        have = hashlib.sha256(open(src, "rb").read()).hexdigest() if os.path.exists(src) else None
        stale |= have != want
    return d, stale


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""
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
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [x.strip() for x in line.split(",")]))

    def stop(self, t_begin=None, t_end=None):
        """Summary of the samples taken in [t_begin, t_end] (perf_counter times); when none fell inside
        (a region shorter than the sampling period) every sample of the leg is summarised and a note says so."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.thread.join(timeout=2)
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

        def summarise(rows):
            sm, mx, power, reasons = [], None, [], set()
            for _, r in rows:
                if len(r) < 7:
                    continue
                try:
                    sm.append(float(r[0])); mx = float(r[1]); power.append(float(r[2]))
                except ValueError:
                    continue
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_min_mhz": float(np.min(sm)) if sm else None,
                    "sm_max_mhz": mx, "power_w_max": float(np.max(power)) if power else None,
                    "reasons": sorted(reasons), "samples": len(sm)}

        inside = [x for x in self.rows if t_begin is None or t_begin <= x[0] <= t_end]
        out = summarise(inside)
        if not out["samples"] and t_begin is not None:
            out = summarise(self.rows)
            out["note"] = "no sample fell inside the timed region; all samples of the leg are summarised"
        return out


# --------------------------------------------------------------------------- oracle legs (CPU)

def host_bits(t):
    from oracle import tessera_oracle as orc
    return tuple(orc.bits(x) for x in (t.k_pool, t.v_pool, t.q, t.k_new, t.v_new))


def oracle_sample(w, tensors_host_bits, budget_s: float, seed: int = 0, request=None, max_rows=None):
    """Times the oracle as it stands on a bounded sample of workload `w` - one request assembled in
    full (gather + rotation), then random (row, head) attention rows of that request until the time
    budget or `max_rows` is reached - and extrapolates to one whole layer: assembly by token count,
    attention by (query, key) pair count.  The rows it computed are returned for a parity check."""
    from oracle import tessera_oracle as orc
    kb, vb, qb, knb, vnb = tensors_host_bits
    rng = np.random.default_rng(seed)
    r = int(np.argmax(w.seq_len)) if request is None else request
    t_all = time.perf_counter()
    t0 = time.perf_counter()
    a = orc.assemble(w, r, kb, vb, knb, vnb)
    t_asm = time.perf_counter() - t0
    asm_per_token = t_asm / max(int(w.seq_len[r]), 1)
    j0, j1 = int(w.recompute_off[r]), int(w.recompute_off[r + 1])
    H = w.shape.num_q_heads
    n_rows, pairs, t_att = 0, 0, 0.0
    chunk = 64
    rows_j, rows_h, rows_o, rows_l = [], [], [], []
    while t_att < budget_s and j1 > j0 and (max_rows is None or n_rows < max_rows):
        jj = rng.integers(j0, j1, size=chunk).astype(np.int32)
        hh = rng.integers(0, H, size=chunk).astype(np.int32)
        pp = w.recompute_pos[jj].astype(np.int32)
        t0 = time.perf_counter()
        o, l = orc.attention_rows(w, a.k, a.v_bits, qb, jj, hh, pp)
        t_att += time.perf_counter() - t0
        rows_j.append(jj); rows_h.append(hh); rows_o.append(o); rows_l.append(l)
        n_rows += chunk
        pairs += int(pp.astype(np.int64).sum() + chunk)
        chunk = min(chunk * 2, 4096)
    att_per_pair = t_att / max(pairs, 1)
    layer_s = asm_per_token * w.total_tokens + att_per_pair * w.qk_pairs * H
    cat = lambda xs, d: np.concatenate(xs) if xs else np.zeros(d)
    return {"layer_seconds_extrapolated": layer_s, "assemble_s": t_asm, "attention_s": t_att,
            "sample_seconds": time.perf_counter() - t_all,
            "rows": n_rows, "pairs": pairs, "cores": orc.num_threads(), "request": r, "assembled": a,
            "row_q": cat(rows_j, 0).astype(np.int64), "row_h": cat(rows_h, 0).astype(np.int64),
            "row_o": cat(rows_o, (0, w.shape.head_dim)), "row_lse": cat(rows_l, 0),
            "sample": "request %d assembled in full (%d tokens) + %d random (row, head) attention rows (%d q-k pairs); "
                      "extrapolated by token count and pair count" % (r, int(w.seq_len[r]), n_rows, pairs)}


def parity_of_sample(w, s, plan_tables, k_after_bits, v_after_bits, out, lse):
    """Compares what the GPU left behind with the oracle rows of `oracle_sample` (same bytes in): block
    table and per-position sources bit for bit, the sampled request's V and un-shifted / fresh K rows
    bit for bit, its rotated K rows and the sampled attention rows within the stated tolerance."""
    from oracle import tessera_oracle as orc
    page_off, pages, src_slot = plan_tables
    st, o_off, o_pages, o_src, _ = orc.placement(w)
    res = {"placement_exact": bool(st == 0 and np.array_equal(page_off, o_off) and np.array_equal(pages, o_pages)
                                   and np.array_equal(src_slot, o_src))}
    r, a = s["request"], s["assembled"]
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    T, B = int(w.seq_len[r]), sh.page_size
    p = np.arange(T)
    slots = pages[page_off[r] + p // B].astype(np.int64) * B + p % B
    gv, gk = v_after_bits.reshape(-1, row)[slots], k_after_bits.reshape(-1, row)[slots]
    ex = a.k_exact != 0
    res["v_rows_exact"] = bool(np.array_equal(gv, a.v_bits.reshape(T, row)))
    res["k_copy_rows_exact"] = bool(np.array_equal(gk[ex], a.k_bits.reshape(T, row)[ex]))
    if (~ex).any():
        d = np.abs(orc.bf16_bits_to_f64(gk[~ex]) - a.k.reshape(T, row)[~ex])
        res["k_rotated_max_abs"], res["k_rotated_mean_abs"] = float(d.max()), float(d.mean())
    else:
        res["k_rotated_max_abs"] = res["k_rotated_mean_abs"] = 0.0
    if len(s["row_q"]):
        got = out[s["row_q"], s["row_h"]].float().cpu().numpy().astype(np.float64)
        e = np.abs(got - s["row_o"])
        res["attn_max_abs"], res["attn_mean_abs"] = float(e.max()), float(e.mean())
        res["lse_max_abs"] = float(np.abs(lse[s["row_q"], s["row_h"]].cpu().numpy().astype(np.float64) - s["row_lse"]).max())
    else:
        res["attn_max_abs"] = res["attn_mean_abs"] = res["lse_max_abs"] = 0.0
    res["rows_checked"] = int(len(s["row_q"]))
    res["ok"] = bool(res["placement_exact"] and res["v_rows_exact"] and res["k_copy_rows_exact"]
                     and res["k_rotated_max_abs"] <= MAX_ABS and res["k_rotated_mean_abs"] <= MEAN_ABS
                     and res["attn_max_abs"] <= MAX_ABS and res["attn_mean_abs"] <= MEAN_ABS
                     and res["lse_max_abs"] <= 2e-2 and np.isfinite(res["attn_max_abs"]))
    return res


# --------------------------------------------------------------------------- workloads

def rank_workload(config: int, rank: int, requests=None, policy=None):
    """Every rank owns an independent batch of the same configuration: requests never interact
    (no cross-request attention), so the path shards by request with no data-path collective."""
    from paper_2609_32999_b200 import workloads as wl
    return wl.config(config, seed=wl.BASE_SEED + config + 7919 * rank, requests_override=requests, policy=policy)


def config_dict(w, config_index, layers, pool_gb, flushed, policy, graph=False):
    sh = w.shape
    l2 = ("L2 flushed (256 MB written) between timed steps" if flushed else
          "inputs larger than L2: %d per-layer KV pools of %.2f GB cycled" % (layers, pool_gb))
    return {"workload": w.name, "config_index": config_index, "requests_per_gpu": w.batch,
            "total_tokens_per_gpu": w.total_tokens, "recompute_tokens_per_gpu": w.n_q,
            "cached_tokens_per_gpu": w.cached_tokens, "H_q": sh.num_q_heads, "H_kv": sh.num_kv_heads,
            "head_dim": sh.head_dim, "page_size": sh.page_size, "l2": l2, "attn_kernel": "tcgen05",
            "cuda_graph": bool(graph), "residency": policy or "all units cached"}


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


def fractions(attn_tflops, gather_gbs, peaks):
    return {"attn_frac_of_burst": attn_tflops / peaks["bf16_tflops"],
            "attn_frac_of_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
            "attn_frac_of_nominal_2250": attn_tflops / NOMINAL_TFLOPS,
            "gather_frac_of_measured_copy": gather_gbs / peaks["hbm_gbs"],
            "gather_frac_of_nominal_8000": gather_gbs / NOMINAL_GBS}


class Leg:
    """One workload on one GPU: plan, per-layer pools, the step function and its timing."""

    def __init__(self, w, dev, n_layers, seed, want_out=True):
        import torch
        from paper_2609_32999_b200 import binding as tb
        from paper_2609_32999_b200 import workloads as wl
        self.w, self.dev, self.tb = w, dev, tb
        t0 = time.perf_counter()
        self.plan = tb.Plan(w)
        torch.cuda.synchronize()
        self.plan_create_ms = (time.perf_counter() - t0) * 1e3      # host placement + table upload, once per batch
        self.layers = [wl.make_tensors(w, layer=l, device=dev, seed=seed) for l in range(n_layers)]
        sh = w.shape
        self.out = torch.empty(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty(w.n_q, sh.num_q_heads, dtype=torch.float32, device=dev)
        self.stream = torch.cuda.current_stream()
        self.pool_bytes = 2 * self.layers[0].k_pool.numel() * 2
        # small pools stay in L2 from one step to the next: flush between steps instead of cycling
        self.flush = None
        if self.pool_bytes * n_layers < 2 * L2_BYTES:
            self.flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def step(self, i, ev=None):
        t = self.layers[i % len(self.layers)]
        if ev is not None:
            ev[0].record(self.stream)
        self.plan.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
        if ev is not None:
            ev[1].record(self.stream)
        self.plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, self.out, self.lse)
        if ev is not None:
            ev[2].record(self.stream)

    def timed(self, steps, warmup, barrier, sampler_index=None, step_fn=None):
        """W warm-up steps, then K timed steps.  Returns per-step ms of the whole step, of the gather and
        of scatter + attention (CUDA events on the launching stream), launches made and clock summary."""
        import torch
        step_fn = step_fn or self.step
        for i in range(warmup):
            if self.flush is not None:
                self.flush.zero_()
            step_fn(i)
        barrier()
        sampler = ClockSampler(sampler_index).start() if sampler_index is not None else None
        if sampler:
            time.sleep(0.15)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
        launches0 = self.tb.launch_count()
        barrier()
        t_begin = time.perf_counter()
        for i in range(steps):
            if self.flush is not None:
                self.flush.zero_()
            step_fn(i, evs[i])
        end = torch.cuda.Event(enable_timing=True)
        end.record(self.stream)
        barrier()
        t_end = time.perf_counter()
        launches = self.tb.launch_count() - launches0
        if self.flush is None:
            total_ms = evs[0][0].elapsed_time(end)                  # back to back: first event to last
        else:
            total_ms = float(sum(e[0].elapsed_time(e[2]) for e in evs))   # the flushes in between are not counted
        gather_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))
        attn_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in evs]))
        clocks = sampler.stop(t_begin, t_end) if sampler else None
        return {"total_ms": total_ms, "ms_per_step": total_ms / steps, "gather_ms": gather_ms, "attn_ms": attn_ms,
                "launches": launches, "clocks": clocks, "wall_s": t_end - t_begin}

    def rates(self, r):
        info = self.plan.info
        return (info.attn_flops / (r["attn_ms"] / 1e3) / 1e12 if info.attn_flops else 0.0,
                info.gather_bytes / (r["gather_ms"] / 1e3) / 1e9 if info.gather_bytes else 0.0)

    def parity(self, budget_s, max_rows, layer=0):
        """Runs layer `layer` once more on fresh tensors, keeps the pools as the GPU left them and checks
        them and sampled attention rows against the oracle run on the very same input bytes."""
        import torch
        from oracle import tessera_oracle as orc
        from paper_2609_32999_b200 import workloads as wl
        t = wl.make_tensors(self.w, layer=layer, device=self.dev, seed=977)
        bits_in = host_bits(t)
        bits_in = tuple(b.copy() for b in bits_in)
        self.plan.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
        self.plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, self.out, self.lse)
        torch.cuda.synchronize()
        s = oracle_sample(self.w, bits_in, budget_s, seed=5, max_rows=max_rows)
        res = parity_of_sample(self.w, s, self.plan.block_table(), orc.bits(t.k_pool), orc.bits(t.v_pool), self.out, self.lse)
        res["kernel_status"] = int(self.plan.status())
        res["ok"] = bool(res["ok"] and res["kernel_status"] == 0)
        return res, s

    def extend_write_record(self, steps, warmup, peaks):
        """Write side of the extend pass, two ways, on this leg's workload: un-rotated fresh projections
        -> (a) tessera_rope_fresh then the attention call's own scatter, (b) the fused tessera_extend_write
        and attention without scatter.  Times the rotation / fused write kernels alone (L2 flushed) and the
        whole layer both ways."""
        import torch
        t = self.layers[0]
        sh, n_q = self.w.shape, self.w.n_q
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=self.dev)
        stream = self.stream

        def timed(fn, do_flush):
            ms = []
            for i in range(warmup + steps):
                if do_flush:
                    flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                if i >= warmup:
                    ms.append(a.elapsed_time(b))
            return sum(ms) / len(ms)

        p = self.plan
        # (the scatter of the unfused way is part of the attention call and has no entry point of its own:
        # its cost shows in the whole-layer times)
        m_rot = timed(lambda: p.rope_fresh(t.q, t.k_new), True)
        m_fused = timed(lambda: p.extend_write(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new), True)

        def layer_unfused():
            p.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
            p.rope_fresh(t.q, t.k_new)
            p.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, self.out, self.lse)

        def layer_fused():
            p.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
            p.extend_write(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new)
            p.partial_prefill_attn(t.k_pool, t.v_pool, t.q, None, None, self.out, self.lse)

        m_layer_unfused = timed(layer_unfused, self.flush is not None)
        m_layer_fused = timed(layer_fused, self.flush is not None)
        kv_row = sh.num_kv_heads * sh.head_dim * 2
        q_row = sh.num_q_heads * sh.head_dim * 2
        fused_bytes = n_q * (2 * q_row + 4 * kv_row)                 # q read + written, K and V read + written once
        unfused_bytes = n_q * (2 * q_row + 2 * kv_row + 4 * kv_row)  # + the rotated K written in place and read again
        return {"workload": self.w.name, "recompute_rows": n_q, "steps": steps,
                "rope_fresh_ms": m_rot, "unfused_bytes": int(unfused_bytes),
                "extend_write_ms": m_fused, "extend_write_bytes": int(fused_bytes),
                "extend_write_GBps": fused_bytes / m_fused / 1e6,
                "extend_write_frac_of_measured_copy": fused_bytes / m_fused / 1e6 / peaks["hbm_gbs"],
                "layer_ms_unfused": m_layer_unfused, "layer_ms_fused": m_layer_fused}

    def k8_attention_record(self, steps, warmup, peaks):
        """Attention over 8-bit key pages (tessera_partial_prefill_attn_k8: queries quantised by the call, fresh
        rows scattered as codes) against the 16-bit call on the same composed layer; flops are the same
        algorithmic count (the 8-bit S = Q K^T runs at twice the tensor rate, P.V stays 16-bit)."""
        import torch
        t = self.layers[0]
        p = self.plan
        p.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
        ks = qs = 1.0 / 32
        k8 = (t.k_pool.float() * (1.0 / ks)).clamp_(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=self.dev)
        stream = self.stream

        def timed(fn):
            ms = []
            for i in range(warmup + steps):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                if i >= warmup:
                    ms.append(a.elapsed_time(b))
            return sum(ms) / len(ms)

        f16 = lambda: p.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, self.out, self.lse)
        f8 = lambda: p.partial_prefill_attn_k8(k8, ks, t.v_pool, t.q, qs, t.k_new, t.v_new, self.out, self.lse)
        # the two calls alternate, so that both see the same clock and power state; medians are reported
        a16, a8 = [], []
        for i in range(warmup + 2 * steps):
            for fn, acc in ((f16, a16), (f8, a8)):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn()
                b.record(stream)
                torch.cuda.synchronize()
                if i >= warmup:
                    acc.append(a.elapsed_time(b))
        m16, m8 = float(np.median(a16)), float(np.median(a8))

        def block(fn, n=20):                 # back to back, no flush: the power-capped regime
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(stream)
            for _ in range(n):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n

        b16, b8 = block(f16), block(f8)
        # whole layer both ways: compose + attention (the 8-bit-key compose reads a separate source pool)
        w2 = copy.copy(self.w)
        w2.num_source_pages = self.w.num_pool_pages
        p2 = self.tb.Plan(w2)
        src_k, src_v = t.k_pool.clone(), t.v_pool.clone()

        def layer16():
            p.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
            p.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, self.out, self.lse)

        def layer8():
            p2.kv_compose_k8(src_k, src_v, k8, t.v_pool, ks)
            p2.partial_prefill_attn_k8(k8, ks, t.v_pool, t.q, qs, t.k_new, t.v_new, self.out, self.lse)

        l16, l8 = timed(layer16), timed(layer8)
        m_c8 = timed(lambda: p2.kv_compose_k8(src_k, src_v, k8, t.v_pool, ks))
        assert p2.status() == 0
        p2.destroy()
        flops = p.info.attn_flops
        cached_elems = self.w.cached_tokens * self.w.shape.num_kv_heads * self.w.shape.head_dim
        return {"workload": self.w.name, "steps": steps, "l2": "flushed between calls",
                "bf16_ms": m16, "bf16_tflops": flops / m16 / 1e9, "k8_ms": m8, "k8_tflops_algorithmic": flops / m8 / 1e9,
                "speedup": m16 / m8, "k8_ms_min": float(min(a8)), "bf16_ms_min": float(min(a16)),
                "back_to_back_ms": {"bf16": b16, "k8": b8}, "compose_k8_ms": m_c8, "compose_k8_GBps": cached_elems * 7 / m_c8 / 1e6,
                "layer_ms_bf16": l16, "layer_ms_k8": l8,
                "timing": "bf16 and k8 calls alternate (L2 flushed before each); medians",
                "note": "k8 time includes quantising q (one pass over q) and the 8-bit fresh-row scatter; compose_k8 moves "
                        "7 bytes per cached element pair (K 2 in, 1 out; V 2 in, 2 out)"}

    def close(self):
        self.plan.destroy()
        self.layers = None
        self.out = self.lse = self.flush = None


# --------------------------------------------------------------------------- side tiers

def fp8_tier_record(w, dev, steps, warmup, peaks):
    """The cached units of the workload sit in an e4m3 pool and are expanded into the requests' bf16
    pages (rotation fused), and the reverse (retain).  L2 is flushed between timed launches; bytes are
    the algorithmic ones (1 + 2 per element either way)."""
    import torch
    from paper_2609_32999_b200 import binding as tb
    from paper_2609_32999_b200 import workloads as wl
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
        for i in range(warmup + steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            if i >= warmup:
                ms.append(a.elapsed_time(b))
        return sum(ms) / len(ms)

    launches0 = tb.launch_count()
    ms_expand = timed(lambda: plan.kv_compose_from_fp8(k8, v8, 1 / 32, 1 / 32, t.k_pool, t.v_pool))
    ms_retain = timed(lambda: plan.kv_retain_fp8(t.k_pool, t.v_pool, k8, v8, 1 / 32, 1 / 32))
    elems = w.cached_tokens * w.shape.num_kv_heads * w.shape.head_dim * 2            # K and V
    peak = peaks["hbm_gbs"]
    rec = {"workload": w.name, "cached_tokens": int(w.cached_tokens), "l2": "flushed between launches",
           "dtype": "e4m3 <-> bf16", "steps": steps, "bytes_per_launch": elems * 3,
           "expand": {"ms": ms_expand, "GBps": elems * 3 / ms_expand / 1e6, "frac_of_measured_copy": elems * 3 / ms_expand / 1e6 / peak},
           "retain": {"ms": ms_retain, "GBps": elems * 3 / ms_retain / 1e6, "frac_of_measured_copy": elems * 3 / ms_retain / 1e6 / peak},
           "gpu_launches": tb.launch_count() - launches0}
    plan.destroy()
    return rec


def host_tier_record(w, dev, steps, warmup):
    """Local-hit tier: the cached units live in a pinned host-memory pool.  One layer = compose from that
    pool + fresh-row scatter + attention.  `zero_copy_then_attention`: the gather kernel reads the host
    pool over the link (tessera_kv_compose_from), attention follows.  `overlapped`: a small reader launch
    pulls chunk c + 1 while scatter + attention of chunk c run (tessera_composed_prefill_host_tier), for
    bf16 and for e4m3 units.  Bytes over the link = K and V rows of every cached token."""
    import torch
    from paper_2609_32999_b200 import binding as tb
    from paper_2609_32999_b200 import workloads as wl
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    plan = tb.Plan(w2)
    t = wl.make_tensors(w, layer=0, device=dev, seed=wl.BASE_SEED)
    host_k, host_v = t.k_pool.cpu().pin_memory(), t.v_pool.cpu().pin_memory()
    sh = w.shape
    out = torch.empty(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(w.n_q, sh.num_q_heads, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    row_bytes = sh.num_kv_heads * sh.head_dim * 2 * 2
    rec = {"workload": w.name, "cached_tokens": int(w.cached_tokens), "steps": steps}
    launches0 = tb.launch_count()

    def timed(fn):
        ms = []
        for i in range(warmup + steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            torch.cuda.synchronize()
            if i >= warmup:
                ms.append(a.elapsed_time(b))
        return sum(ms) / len(ms)

    m_gather = timed(lambda: plan.kv_compose_from(host_k, host_v, t.k_pool, t.v_pool))
    m_attn = timed(lambda: plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse))

    def zero_copy_layer():
        plan.kv_compose_from(host_k, host_v, t.k_pool, t.v_pool)
        plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse)

    m_zero = timed(zero_copy_layer)
    link_bytes = w.cached_tokens * row_bytes
    rec["zero_copy_then_attention"] = {"ms_per_layer": m_zero, "gather_ms": m_gather, "attention_ms": m_attn,
                                       "link_bytes_per_layer": int(link_bytes), "link_GBps_during_gather": link_bytes / m_gather / 1e6}
    m_over = timed(lambda: plan.composed_prefill_host_tier(host_k, host_v, t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse))
    rec["overlapped"] = {"ms_per_layer": m_over, "link_GBps": link_bytes / m_over / 1e6,
                         "saved_ms_vs_sequential": m_zero - m_over,
                         # share of the attention time that ran under the transfer
                         "attention_hidden_frac": max(0.0, min(1.0, (m_zero - m_over) / m_attn))}
    # e4m3 units: half the bytes over the link
    gen = torch.Generator(device="cpu")
    gen.manual_seed(wl.BASE_SEED)
    shape8 = tuple(t.k_pool.shape)
    draw8 = lambda: (torch.randint(0, 0x78, shape8, dtype=torch.uint8, generator=gen)
                     | (torch.randint(0, 2, shape8, dtype=torch.uint8, generator=gen) << 7)).pin_memory()
    k8, v8 = draw8(), draw8()

    def zero_copy_layer8():
        plan.kv_compose_from_fp8(k8, v8, 1 / 32, 1 / 32, t.k_pool, t.v_pool)
        plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse)

    m_zero8 = timed(zero_copy_layer8)
    m8 = timed(lambda: plan.composed_prefill_host_tier(k8, v8, t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse,
                                                       src_format=1, k_scale=1 / 32, v_scale=1 / 32))
    rec["e4m3_units"] = {"sequential_ms_per_layer": m_zero8, "overlapped_ms_per_layer": m8,
                         "link_bytes_per_layer": int(link_bytes // 2), "link_GBps": link_bytes / 2 / m8 / 1e6}
    rec["gpu_launches"] = tb.launch_count() - launches0
    assert plan.status() == 0
    plan.destroy()
    return rec


def run_fp8_tier(args):
    """Side measurement on its own (`--tier fp8`): prints the fp8_tier record as one JSON line."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(0)
    w = rank_workload(args.config, 0, args.requests, None)
    rec = fp8_tier_record(w, "cuda:0", args.steps, args.warmup, measured_peaks())
    rec.update({"metric": "fp8_tier_GBps", "unit": "GB/s", "n_gpus": 1, "warmup": args.warmup, "data": "synthetic"})
    print(json.dumps(rec))


# --------------------------------------------------------------------------- reference arm

def run_reference(args):
    """The reference arm: the oracle on the host cores, on the same workload and metric.  Each step
    times a bounded sample of one layer (one request assembled in full plus random attention rows);
    `ms_per_step` is that sampled step as timed, `layer_ms_extrapolated` the whole layer it stands for,
    and `value` = tokens of the layer / extrapolated layer time."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_32999_b200 import workloads as wl
    w = rank_workload(args.config, 0, args.requests, args.policy)
    t = wl.make_tensors(w, layer=0, device="cpu")
    bits = host_bits(t)
    per_step_budget = max(1.0, min(20.0, 80.0 / max(args.steps + args.warmup, 1)))
    for i in range(args.warmup):
        oracle_sample(w, bits, per_step_budget / 4, seed=100 + i)
    t0 = time.perf_counter()
    layer_s, step_s = [], []
    for i in range(args.steps):
        s = oracle_sample(w, bits, per_step_budget, seed=i)
        layer_s.append(s["layer_seconds_extrapolated"])
        step_s.append(s["sample_seconds"])
    wall = time.perf_counter() - t0
    layer_ms = float(np.mean(layer_s)) * 1e3
    value = w.total_tokens / (layer_ms / 1e3)
    pool_gb = 2 * t.k_pool.numel() * 2 / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(step_s)) * 1e3,
            "layer_ms_extrapolated": layer_ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w, args.config, args.layers, pool_gb, pool_gb * 1e9 * args.layers < 2 * L2_BYTES, args.policy),
            "note": "each step times a bounded sample of one layer on the host cores (ms_per_step) and extrapolates "
                    "to the whole layer by token and pair count (layer_ms_extrapolated, value)",
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": s["cores"], "kind": "oracle", "sample": s["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": wall}
    print(json.dumps(line))


# --------------------------------------------------------------------------- main arm

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
    ap.add_argument("--only-headline", action="store_true",
                    help="skip the sustained leg, the other configurations and the side tiers (profiling runs)")
    ap.add_argument("--sustained-steps", type=int, default=1000, help="back-to-back layers of the seconds-long leg")
    ap.add_argument("--other-steps", type=int, default=16, help="timed steps of each of the other configurations")
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

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = measured_peaks()
    w = rank_workload(args.config, rank, args.requests, args.policy)
    leg = Leg(w, dev, args.layers, wl.BASE_SEED + rank)
    info = leg.plan.info
    sh = w.shape
    stream = leg.stream

    step_fn = None
    if args.graph:
        # one graph per layer pool: compose + scatter + attention (+ combine) replayed as one launch
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(args.layers):
                leg.step(i)                     # warm up outside capture (function attributes, descriptors)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graphs = []
        for i in range(args.layers):
            gph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gph):
                leg.step(i)
            graphs.append(gph)

        def step_fn(i, ev=None):                # graph replay has no inner events
            if ev is not None:
                ev[0].record(stream)
            graphs[i % args.layers].replay()
            if ev is not None:
                ev[1].record(stream)
                ev[2].record(stream)

    head = leg.timed(args.steps, args.warmup, barrier, sampler_index=local if rank == 0 else None, step_fn=step_fn)
    assert leg.plan.status() == 0, "a kernel reported a bounded-wait timeout"
    launches = head["launches"]

    # ---- end to end through the host-buffer entry point
    t0 = leg.layers[0]
    qh, kh, vh = (x.cpu().pin_memory() for x in (t0.q, t0.k_new, t0.v_new))
    oh = torch.empty_like(qh).pin_memory()
    lh = torch.empty(w.n_q, sh.num_q_heads, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 16))
    for i in range(3):
        leg.plan.composed_prefill_host(t0.k_pool, t0.v_pool, qh, kh, vh, oh, lh)
    barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(stream)
    for i in range(e2e_steps):
        t = leg.layers[i % args.layers]
        leg.plan.composed_prefill_host(t.k_pool, t.v_pool, qh, kh, vh, oh, lh)
    eb.record(stream)
    barrier()
    e2e_ms = ea.elapsed_time(eb) / e2e_steps

    (total_ms_max, e2e_ms_max), all_tokens = aggregate([head["total_ms"], e2e_ms], w.total_tokens, world, dev)

    # ---- seconds-long leg: the same workload back to back until the power cap has settled
    sustained = None
    if not args.only_headline and not args.graph and args.sustained_steps > 0:
        s_run = leg.timed(args.sustained_steps, 3, barrier, sampler_index=local if rank == 0 else None)
        s_att, s_gat = leg.rates(s_run)
        (s_total_max,), _ = aggregate([s_run["total_ms"]], w.total_tokens, world, dev)
        sustained = {"steps": args.sustained_steps, "seconds": s_total_max / 1e3, "ms_per_step": s_total_max / args.sustained_steps,
                     "value": all_tokens / (s_total_max / args.sustained_steps / 1e3), "attn_ms": s_run["attn_ms"],
                     "attn_tflops": s_att, "gather_ms": s_run["gather_ms"], "gather_GBps": s_gat,
                     "frac": s_att / peaks["bf16_tflops_sustained"], "peak": peaks["bf16_tflops_sustained"],
                     "peak_source": peaks["source"] + " sustained bf16 GEMM (seconds-long timed region)",
                     "frac_of_burst": s_att / peaks["bf16_tflops"], "frac_of_nominal_2250": s_att / NOMINAL_TFLOPS,
                     "clocks": s_run["clocks"]}
        if s_run["clocks"] and s_run["clocks"].get("sm_mhz"):
            mhz = s_run["clocks"]["sm_mhz"]
            sustained["attn_ms_x_sm_mhz"] = s_run["attn_ms"] * mhz
            sustained["headline_attn_ms_x_sm_mhz"] = (head["attn_ms"] * head["clocks"]["sm_mhz"]
                                                      if head["clocks"] and head["clocks"].get("sm_mhz") else None)
        assert leg.plan.status() == 0, "a kernel reported a bounded-wait timeout"

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms_max / args.steps
    value = all_tokens / (ms_per_step / 1e3)
    attn_tflops, gather_gbs = leg.rates(head)
    traffic, stale = kernel_traffic()
    scale = w.batch if (traffic and args.config == 4) else None

    def traffic_of(kernel):
        if not scale:
            return None
        k = traffic["config4_one_request"][kernel]
        return (k["dram_bytes_read"] + k["dram_bytes_write"]) * scale

    long_region = total_ms_max > 1000.0
    tensor_peak = peaks["bf16_tflops_sustained"] if long_region else peaks["bf16_tflops"]
    pool_gb = leg.pool_bytes / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_dict(w, args.config, args.layers, pool_gb, leg.flush is not None, args.policy, args.graph),
        "clocks": head["clocks"],
        "gpu_launches": launches,
        "e2e": {"value": all_tokens / (e2e_ms_max / 1e3), "unit": UNIT,
                "h2d_bytes_per_step": int(qh.numel() * 2 + kh.numel() * 2 + vh.numel() * 2),
                "d2h_bytes_per_step": int(oh.numel() * 2 + lh.numel() * 4), "ms_per_step": e2e_ms_max,
                "note": "q, k_new, v_new from pinned host memory, out and lse back to it, every step; "
                        "the KV pools are the resident cache"},
        "roofline": {"kernel": "partial_prefill_attn (fresh-row scatter + attention kernel)", "bound": "tensor",
                     "achieved": attn_tflops, "peak": tensor_peak, "unit": "TFLOP/s",
                     "frac": attn_tflops / tensor_peak,
                     "peak_source": peaks["source"] + (" sustained bf16 GEMM (timed region over a second)" if long_region
                                                      else " burst bf16 GEMM (timed region %.0f ms)" % total_ms_max),
                     "frac_of_burst": attn_tflops / peaks["bf16_tflops"],
                     "frac_of_sustained": attn_tflops / peaks["bf16_tflops_sustained"],
                     "frac_of_nominal_2250": attn_tflops / NOMINAL_TFLOPS,
                     "ms_per_launch": head["attn_ms"], "flops_per_launch": int(info.attn_flops),
                     "traffic": traffic_of("attn"), "traffic_stale": bool(stale),
                     "traffic_note": "DRAM bytes per launch: ncu capture of one request (profiles/traffic.json) x requests; "
                                     "algorithmic minimum (assembled K,V once + Q + O) %.1f MB"
                                     % ((w.total_tokens * sh.num_kv_heads * sh.head_dim * 2 * 2
                                         + 2 * w.n_q * sh.num_q_heads * sh.head_dim * 2) / 1e6)},
        "roofline_gather": {"kernel": "kv_compose (gather + RoPE shift)", "bound": "hbm", "achieved": gather_gbs,
                            "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gather_gbs / peaks["hbm_gbs"],
                            "peak_source": peaks["source"] + " copy", "frac_of_nominal_8000": gather_gbs / NOMINAL_GBS,
                            "ms_per_launch": head["gather_ms"], "bytes_per_launch": int(info.gather_bytes),
                            "traffic": traffic_of("gather"), "traffic_stale": bool(stale),
                            "dram_level_GBps": (traffic_of("gather") / (head["gather_ms"] / 1e3) / 1e9) if scale else None},
        "recompute_tokens_per_s": w.n_q * world / (ms_per_step / 1e3),
        "plan_create_ms": leg.plan_create_ms,
        "masked_mma_fraction": leg.plan.masked_mma_fraction,
    }
    if sustained:
        line["sustained"] = sustained
    k8_record = None
    if not args.only_headline and world == 1 and sh.head_dim == 128:
        k8_record = leg.k8_attention_record(8, 3, peaks)
    if not args.no_cpu_baseline:
        par, s = leg.parity(args.cpu_budget, None)
        line["cpu_baseline"] = {"value": w.total_tokens / s["layer_seconds_extrapolated"], "unit": UNIT,
                                "cores": s["cores"], "kind": "oracle", "sample": s["sample"],
                                "layer_seconds_extrapolated": s["layer_seconds_extrapolated"]}
        line["parity"] = par
    leg.close()
    del leg
    torch.cuda.empty_cache()

    if not args.only_headline and world == 1:
        # ---- the other configurations: same step, fewer timed iterations, own clock samples
        per_config = []
        for c in (1, 2, 3, 4, 5):
            if c == args.config:
                att, gat = attn_tflops, gather_gbs
                rec = {"config_index": c, "workload": w.name, "steps": args.steps, "ms_per_step": ms_per_step,
                       "value": value, "attn_ms": head["attn_ms"], "attn_tflops": att, "gather_ms": head["gather_ms"],
                       "gather_GBps": gat, **fractions(att, gat, peaks), "clocks": head["clocks"],
                       "timed_region_ms": total_ms_max, "l2": line["config"]["l2"],
                       "masked_mma_fraction": line["masked_mma_fraction"],
                       "parity_ok": line.get("parity", {}).get("ok"), "parity": line.get("parity")}
                per_config.append(rec)
                continue
            wc = rank_workload(c, rank, None, None)
            n_layers = 2 if c == 5 else 4
            lg = Leg(wc, dev, n_layers, wl.BASE_SEED + rank)
            r = lg.timed(args.other_steps, 3, barrier, sampler_index=local)
            att, gat = lg.rates(r)
            rec = {"config_index": c, "workload": wc.name, "steps": args.other_steps, "ms_per_step": r["ms_per_step"],
                   "value": wc.total_tokens / (r["ms_per_step"] / 1e3), "attn_ms": r["attn_ms"], "attn_tflops": att,
                   "gather_ms": r["gather_ms"], "gather_GBps": gat, **fractions(att, gat, peaks), "clocks": r["clocks"],
                   "timed_region_ms": r["total_ms"], "total_tokens": wc.total_tokens, "recompute_tokens": wc.n_q,
                   "l2": config_dict(wc, c, n_layers, lg.pool_bytes / 1e9, lg.flush is not None, None)["l2"],
                   "masked_mma_fraction": lg.plan.masked_mma_fraction, "gpu_launches": r["launches"]}
            if not args.no_cpu_baseline:
                par, s = lg.parity(3.0, 2048)
                rec["parity_ok"], rec["parity"] = par["ok"], par
                rec["cpu_oracle_tokens_per_s"] = wc.total_tokens / s["layer_seconds_extrapolated"]
            if c in (3, 5):
                rec["extend_write"] = lg.extend_write_record(5, 2, peaks)
            per_config.append(rec)
            lg.close()
            del lg
            torch.cuda.empty_cache()
        line["per_config"] = per_config
        w4 = w if args.config == 4 else rank_workload(4, rank, None, None)
        line["host_tier"] = [host_tier_record(w4, dev, 3, 2), host_tier_record(rank_workload(3, rank, None, None), dev, 5, 2)]
        torch.cuda.empty_cache()
        line["fp8_tier"] = fp8_tier_record(w4, dev, 8, 3, peaks)
        if k8_record:
            line["fp8_key_attention"] = k8_record
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
