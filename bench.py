#!/usr/bin/env python
"""Benchmark of the branch-isolated attention step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload serving-mix] [--layers 28]
    python bench.py --impl reference ...        # the fp64 CPU oracle on the host cores

A *step* is one pass of the whole hot path -- RoPE + paged write of the new tokens (a3, done by
the attention pass itself through aspd_branch_step; --separate-append uses aspd_kv_append) ->
split-K branch attention -> log-sum-exp combine -- over every attention layer of a
Qwen2.5-7B-shaped stack (28 layers, each with its own K/V pools, one shared plan), for one
decoding step of the synthetic batch.  The pools of all layers together are far larger than
L2, so every layer streams its KV from HBM.

metric  : branch-decode attention tokens/s = query tokens x layers / time, with the achieved
          HBM GB/s (algorithmic bytes / time) beside it.
value   : inputs resident in HBM before the timed region.
e2e     : same metric through aspd_step_host with q / k_new / v_new / positions in pinned HOST
          memory and the output read back to the host, per layer, copies inside the timed region
          (the KV pools are the state of the decoder and stay on the device).
roofline: for the dominant kernel (the split-K attention pass), algorithmic bytes of one launch /
          its mean duration, timed alone with CUDA events over all layers, against the measured
          HBM copy bandwidth.
cpu_baseline: the oracle as it stands on this machine's host cores (a reported baseline only).

Multi-GPU: the path has no exchange step; requests are independent, so each rank runs its own
batch of requests (weak scaling) and the ranks only meet at the timing barrier.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "branch_decode_attn_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes moved per algorithmic byte by the split-K attention kernel, from an ncu capture of the
# 8-request case of the serving mix (62.36 MB of dram read + write for 61.44 MB algorithmic; the
# kernel streams every page once, so traffic scales with the cached tokens).
TRAFFIC_PER_ALGORITHMIC_BYTE = 1.015


def measured_tensor_peak():
    """Dense bf16 TFLOP/s of a library GEMM inside a long step (the sustained figure)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["bf16_tflops_sustained"]), "measured (sustained)"
        except Exception:
            pass
    return 1400.0, "fallback (sustained)"


def attention_flops(desc, Hq: int, d: int) -> float:
    """2 contractions x 2 flops x d per (query row, visible key) of a parallel-mode step."""
    pairs = 0
    for r in range(len(desc["prefix_len"])):
        b0, nb = int(desc["branch_begin"][r]), int(desc["n_branches"][r])
        ql, kl = desc["br_q_len"][b0:b0 + nb].astype(np.int64), desc["br_kv_len"][b0:b0 + nb].astype(np.int64)
        shared = int(desc["prefix_len"][r]) + int(kl[ql < 0].sum())
        for q, k in zip(ql, kl):
            if q > 0:
                pairs += q * (shared + k - q) + q * (q + 1) // 2
    return 4.0 * d * Hq * float(pairs)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def build_workload(name: str, rank: int, requests: int = 0):
    from paper_2508_08895_b200 import workloads as W
    if name == "serving-mix" and requests > 0:      # a smaller batch of the same mix (profiling captures)
        return W.config_serving_mix(seed=W.SEED_BASE + 4 + 16 * rank, n_req=requests)
    if name == "masked-prefill":
        return W.config_masked_prefill(seed=W.SEED_BASE + 5 + 16 * rank, n_req=requests or 32)
    if name == "serving-mix-serial":
        return W.config_serving_mix_serial(seed=W.SEED_BASE + 4 + 16 * rank, n_req=requests or 32)
    fn = W.CONFIGS[name]
    base = {"tiny-f32": 0, "qwen7b-layer": 1, "branch-open": 2, "long-rag": 3, "serving-mix": 4}[name]
    if name == "branch-open":
        return fn(seed=W.SEED_BASE + base + 16 * rank, serial_steps=0)
    return fn(seed=W.SEED_BASE + base + 16 * rank)


# ------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            try:
                sm.append(float(row[0])); mx.append(float(row[1]))
                for n, v in zip(names, row[2:6]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------ reference arm
def oracle_sample(wl, budget_s: float):
    """Time the oracle's attention on the measured step (all requests), repeated until about
    budget_s seconds of CPU work; returns (tokens/s per layer, threads, description)."""
    import oracle
    from oracle.run import OracleRun
    run = OracleRun(wl)
    for ph in wl.phases[:-1]:
        run.step(ph, attend=False)
    ph = wl.phases[-1]
    pos, slot, req = oracle.new_tokens(ph.desc, ph.mode)
    reps, total = 0, 0.0
    while total < budget_s and reps < 50:
        t0 = time.perf_counter()
        oracle.kv_append(ph.desc, ph.k_new, ph.v_new, pos, req, slot, run.k_pool, run.v_pool, wl.theta)
        oracle.attn(ph.desc, ph.mode, ph.q, run.k_pool, run.v_pool, wl.theta, wl.sm_scale)
        total += time.perf_counter() - t0
        reps += 1
    n_new = len(pos)
    return n_new * reps / total, oracle.threads(), total / reps, reps, n_new


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    wl = build_workload(args.workload, 0, args.requests)
    steps = max(1, args.steps)
    # each "step" of this arm is one layer-step of the oracle on the full batch; warm-up once
    value, cores, sec, reps, n_new = oracle_sample(wl, budget_s=min(30.0, 2.0 * (steps + args.warmup)))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "layers": 1, "query_tokens": n_new,
                   "note": "fp64 CPU oracle, one attention layer-step of the full batch per repetition"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{reps} repetitions of one layer-step ({n_new} query tokens), {sec:.3f} s each"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def reduce_over_ranks(times_ms, units, device, world):
    """Whole-job figures from per-rank ones: every time becomes its maximum over the ranks, the
    units (query tokens a rank processed) their sum.  A no-op for one rank."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x) for x in times_ms], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(u.item())


# ------------------------------------------------------------------------------ our arm
def fill_caches(wl, shape, caches):
    """Fill every layer's pools through the library's own append (same values, distinct memory)."""
    import torch
    from paper_2508_08895_b200 import binding as B, engine as E
    for ph in wl.phases[:-1]:
        plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode)
        pos, _, _ = B.positions(ph.desc, ph.mode)
        pos_d = torch.from_numpy(pos.copy()).cuda()
        k_d, v_d = E.to_device(ph.k_new, wl.dtype), E.to_device(ph.v_new, wl.dtype)
        for c in caches:
            B.kv_append(plan, k_d, v_d, pos_d, c.k, c.v)
        torch.cuda.synchronize()
        plan.destroy()
        del k_d, v_d


def graph_of(fn, use_graph=True):
    """fn captured into a CUDA graph (after two plain runs); returns the callable to replay."""
    import torch
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    if not use_graph:
        return fn
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g.replay


def time_replays(run, reps, warmup=3):
    """Milliseconds of `reps` back-to-back calls of `run`, CUDA events on the current stream."""
    import torch
    for _ in range(warmup):
        run()
    stream = torch.cuda.current_stream()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    for _ in range(reps):
        run()
    b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b)


def attention_kernel_call(plan, mode, q_d, k_d, v_d, fused):
    """The call that launches ONLY the attention kernel the step really runs: for plans whose kernel
    writes the output itself (single-launch plans, plans that deal whole streams) the step or
    attention call, which is that one launch; otherwise the fused pass that also writes the new rows
    (aspd_step_partials) or the plain split-K pass (aspd_attn_partials)."""
    from paper_2508_08895_b200 import binding as B, workloads as W
    info = plan.info
    if info.single_launch and fused and info.fused_append:       # the step is this one launch
        fstep = B.branch_step if mode == W.MODE_BRANCH else B.serial_step
        return lambda c, o: fstep(plan, q_d, k_d, v_d, c.k, c.v, o)
    if info.direct_output or info.single_launch:
        attn = B.branch_attn if mode == W.MODE_BRANCH else B.serial_attn
        return lambda c, o: attn(plan, q_d, c.k, c.v, o)
    if fused and info.fused_append:
        return lambda c, o: B.step_partials(plan, q_d, k_d, v_d, c.k, c.v)
    return lambda c, o: B.attn_partials(plan, q_d, c.k, c.v)


def launches_per_layer(info, fused):
    """Kernel launches of one layer's step: the append kernel unless the attention pass writes the
    new rows itself, the attention pass, the combine unless the attention pass writes the output."""
    return (0 if (fused and info.fused_append) else 1) + 1 + (0 if (info.direct_output or info.single_launch) else 1)


def measure_step_workload(wl, layers, steps, warmup, plan_kw=None, fused=True, use_graph=True, sample_clocks=True, device_index=0):
    """One workload through the step the benchmark times: L layers with distinct pools (at least
    four times L2 together), one plan, CUDA-graph replay.  Returns the figures of the per-config
    block: the step per layer, the attention kernel back to back (consecutive launches overlap
    through programmatic dependent launch: throughput per launch) and isolated (median of single
    launches between synchronisations on cold pools: an upper bound of its duration, launch
    latency included), each also multiplied by the median SM clock sampled while it ran."""
    import torch
    from paper_2508_08895_b200 import binding as B, engine as E, workloads as W
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    ph = wl.phases[-1]
    probe = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, host_only=True)
    L = max(layers, int(np.ceil(4 * 126e6 / max(1, probe.info.algorithmic_bytes))))
    probe.destroy()
    caches = [E.LayerCache(shape, wl.n_pool_pages) for _ in range(L)]
    fill_caches(wl, shape, caches)
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, **(plan_kw or {}))
    info = plan.info
    pos, _, _ = B.positions(ph.desc, ph.mode)
    pos_d = torch.from_numpy(pos.copy()).cuda()
    q_d, k_d, v_d = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
    outs = [torch.empty_like(q_d) for _ in range(L)]
    attn = B.branch_attn if ph.mode == W.MODE_BRANCH else B.serial_attn
    fstep = B.branch_step if ph.mode == W.MODE_BRANCH else B.serial_step

    def step():
        for c, o in zip(caches, outs):
            if fused:
                fstep(plan, q_d, k_d, v_d, c.k, c.v, o)
            else:
                B.kv_append(plan, k_d, v_d, pos_d, c.k, c.v)
                attn(plan, q_d, c.k, c.v, o)
    kcall = attention_kernel_call(plan, ph.mode, q_d, k_d, v_d, fused)

    def kernels():
        for c, o in zip(caches, outs):
            kcall(c, o)
    sampler = ClockSampler(device_index)
    if sample_clocks:
        sampler.start()
    run_step = graph_of(step, use_graph)
    step_ms = time_replays(run_step, steps, warmup) / steps
    run_k = graph_of(kernels, use_graph)
    k_reps = max(3, min(steps, 50))
    kernel_ms = time_replays(run_k, k_reps, 1) / (k_reps * L)
    clocks = sampler.stop() if sample_clocks else None
    # one launch at a time, every launch on pools the L2 has long forgotten (or never held)
    stream = torch.cuda.current_stream()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    iso = []
    for i in range(50):
        torch.cuda.synchronize()
        a.record(stream)
        kcall(caches[i % L], outs[i % L])
        b.record(stream)
        torch.cuda.synchronize()
        iso.append(a.elapsed_time(b) * 1e3)
    if plan.status() != 0:
        raise SystemExit("bench.py: device status %d" % plan.status())
    same = all(torch.equal(outs[0], o) for o in outs[1:])
    res = {"layers": L, "query_tokens": int(plan.n_new), "kv_tokens_per_layer": int(info.kv_tokens_read),
           "alg_bytes": int(info.algorithmic_bytes), "step_ms": step_ms, "step_us_per_layer": step_ms / L * 1e3,
           "kernel_us": kernel_ms * 1e3, "kernel_us_isolated": float(np.median(iso)), "clocks": clocks,
           "launches_per_layer": launches_per_layer(info, fused), "layers_agree": bool(same),
           "n_ctas": int(info.n_ctas), "work_items": int(info.n_items), "kernel": {1: "generic", 2: "mma"}[info.kernel],
           "fused_append": bool(info.fused_append), "direct_output": bool(info.direct_output)}
    return res, dict(plan=plan, shape=shape, caches=caches, outs=outs, q_d=q_d, k_d=k_d, v_d=v_d, pos=pos, pos_d=pos_d, ph=ph,
                     run_step=run_step)


def per_config_entry(res, peak, flops=None, tensor_peak=None):
    """The per-config record of the benchmark line from measure_step_workload's figures."""
    mhz = (res["clocks"] or {}).get("sm_mhz")
    alg = float(res["alg_bytes"])
    e = {"layers": res["layers"], "query_tokens": res["query_tokens"], "kv_tokens_per_layer": res["kv_tokens_per_layer"],
         "alg_bytes": res["alg_bytes"], "launches_per_layer": res["launches_per_layer"],
         "step_us_per_layer": res["step_us_per_layer"], "kernel_us": res["kernel_us"], "kernel_us_isolated": res["kernel_us_isolated"],
         "tokens_per_s": res["query_tokens"] / (res["step_us_per_layer"] * 1e-6)}
    if flops is None:
        e.update({"bound": "hbm", "frac": alg / (res["kernel_us"] * 1e-6) / 1e9 / peak,
                  "frac_isolated": alg / (res["kernel_us_isolated"] * 1e-6) / 1e9 / peak,
                  "step_frac": alg / (res["step_us_per_layer"] * 1e-6) / 1e9 / peak})
    else:
        e.update({"bound": "tensor", "flops": flops, "frac": flops / (res["kernel_us"] * 1e-6) / 1e12 / tensor_peak,
                  "frac_isolated": flops / (res["kernel_us_isolated"] * 1e-6) / 1e12 / tensor_peak,
                  "step_frac": flops / (res["step_us_per_layer"] * 1e-6) / 1e12 / tensor_peak})
    if mhz:
        e.update({"sm_mhz": mhz, "step_us_x_ghz": res["step_us_per_layer"] * mhz * 1e-3, "kernel_us_x_ghz": res["kernel_us"] * mhz * 1e-3,
                  "reasons": res["clocks"]["reasons"]})
    return e


def run_rerotate(args):
    """--op rerotate: the Same-Re renumbering of a finished segment, the keys of every branch token
    of the workload re-rotated in all layers' pools (one launch for all layers; --rerotate-per-layer
    and --rerotate-by-token: one call per layer).  One GPU; prints its own JSON line."""
    print(json.dumps(measure_rerotate(args)))
    return 0


def measure_rerotate(args):
    import torch
    from paper_2508_08895_b200 import binding as B, engine as E
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    wl = build_workload(args.workload, 0, args.requests)
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    d = wl.phases[-1].desc
    # sequential renumbering of the finished segment: branch b of a request moves, as a whole, by the
    # number of tokens in the branches before it
    pages, rows, delta, ranges = [], [], [], []
    for r in range(len(d["prefix_len"])):
        moved = 0
        for b in range(int(d["branch_begin"][r]), int(d["branch_begin"][r]) + int(d["n_branches"][r])):
            k = np.arange(int(d["br_kv_len"][b]))
            s_ = int(d["br_kv_off"][b]) + k
            pages.append(d["page_ids"][int(d["page_begin"][r]) + s_ // wl.page_size]); rows.append(s_ % wl.page_size)
            delta.append(moved + 0 * k)
            ranges.append((int(d["page_begin"][r]), int(d["br_kv_off"][b]), len(k), moved))
            moved += len(k)
    pages, rows, delta = (torch.from_numpy(np.concatenate(x).astype(np.int32)).cuda() for x in (pages, rows, delta))
    ranges = np.array(ranges, dtype=np.int32)
    table_d = torch.from_numpy(np.ascontiguousarray(d["page_ids"], dtype=np.int32)).cuda()
    by_token = bool(getattr(args, "rerotate_by_token", False))
    n = int(pages.numel())
    es = 2 if wl.dtype == "bf16" else 4
    alg = n * (2 * wl.Hkv * wl.d * es + (12 if by_token else 0))
    L = max(args.layers, int(np.ceil(4 * 126e6 / alg)))
    caches = [E.LayerCache(shape, wl.n_pool_pages) for _ in range(L)]
    fill_caches(wl, shape, caches)

    per_layer = by_token or bool(getattr(args, "rerotate_per_layer", False))
    launches = 1 if by_token else (len(ranges) + 511) // 512
    launches *= L if per_layer else (L + 63) // 64

    def step():
        if not per_layer:                  # every layer's pool in one launch (64 pools per launch)
            return B.k_rerotate_ranges_layers(shape, [c.k for c in caches], table_d, ranges)
        for c in caches:
            if by_token:
                B.k_rerotate(shape, c.k, pages, rows, delta)
            else:
                B.k_rerotate_ranges(shape, c.k, table_d, ranges)
    for _ in range(2):
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for _ in range(max(args.warmup, 3)):
        graph.replay()
    sampler = ClockSampler(0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(args.steps):
        graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    peak, peak_kind = measured_peaks()
    achieved = alg * L * args.steps / (ms * 1e-3) / 1e9
    return ({
        "op": "rerotate", "metric": "rerotated_key_tokens_per_second", "value": n * L * args.steps / (ms * 1e-3),
        "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
        "higher_is_better": True, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "layers": L, "tokens_per_layer": n, "heads": wl.Hkv, "head_dim": wl.d,
                   "call": "aspd_k_rerotate" if by_token else "aspd_k_rerotate_ranges" if per_layer else "aspd_k_rerotate_ranges_layers",
                   "launches_per_step": launches, "l2": "%.1f GB of distinct keys per step" % (alg * L / 1e9)},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "peak_kind": "of " + peak_kind, "kernel": "rerotate_kernel" if by_token else "rerotate_ranges_kernel",
                     "kernel_us": ms / args.steps / L * 1e3, "algorithmic_bytes_per_launch": alg * L // launches,
                     "algorithmic_bytes_per_layer": alg},
        "gpu_launches": launches * args.steps, "clocks": clocks})


def run_serial_chain(args):
    """--op serial-chain: a segment of 6 branches opens (12-token headers) over a 1024-token
    prefix, merges, and 64 serial tokens are decoded one after the other (aspd_serial_step, one
    plan per step, every step through all layers); the whole chain is one CUDA graph.  Tiny data
    per call (2.3 MB): a latency measurement.  One GPU; prints its own JSON line."""
    print(json.dumps(measure_serial_chain(args)))
    return 0


def measure_serial_chain(args):
    import torch
    from paper_2508_08895_b200 import binding as B, engine as E, workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    n_serial = 64
    wl = W.config_branch_open(serial_steps=n_serial)
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    L = args.layers
    caches = [E.LayerCache(shape, wl.n_pool_pages) for _ in range(L)]
    serial = [ph for ph in wl.phases if ph.mode == W.MODE_SERIAL]
    assert len(serial) == n_serial and all(ph.mode != W.MODE_SERIAL for ph in wl.phases[:-n_serial])
    for ph in wl.phases[:-n_serial]:                  # prefix and the opening step: cache fill
        plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode)
        pos, _, _ = B.positions(ph.desc, ph.mode)
        pos_d = torch.from_numpy(pos.copy()).cuda()
        k_d, v_d = E.to_device(ph.k_new, wl.dtype), E.to_device(ph.v_new, wl.dtype)
        for c in caches:
            B.kv_append(plan, k_d, v_d, pos_d, c.k, c.v)
        torch.cuda.synchronize()
        plan.destroy()
    combine = {"auto": B.COMBINE_AUTO, "kernel": B.COMBINE_KERNEL, "fused": B.COMBINE_FUSED}[getattr(args, "combine", "auto")]
    plans = [B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, stable_cache=True, combine=combine) for ph in serial]
    qkv = [tuple(E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new)) for ph in serial]
    outs = [torch.empty_like(q) for q, _, _ in qkv]
    alg = float(sum(pl.info.algorithmic_bytes for pl in plans))

    def chain():
        for s_, pl in enumerate(plans):
            q, k, v = qkv[s_]
            for c in caches:
                B.serial_step(pl, q, k, v, c.k, c.v, outs[s_])
    chain()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        chain()
    reps = max(1, min(args.steps, 50))
    for _ in range(max(args.warmup, 3)):
        graph.replay()
    sampler = ClockSampler(0)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(reps):
        graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    if any(pl.status() != 0 for pl in plans):
        raise SystemExit("bench.py: device status")
    peak, peak_kind = measured_peaks()
    gbs = alg * L * reps / (ms * 1e-3) / 1e9
    launches = sum(launches_per_layer(pl.info, True) for pl in plans) * L * reps
    line = ({
        "op": "serial-chain", "metric": "serial_decode_steps_per_second", "value": n_serial * reps / (ms * 1e-3), "unit": "steps/s",
        "n_gpus": 1, "steps": reps, "warmup": max(args.warmup, 3), "ms_per_step": ms / reps, "higher_is_better": True,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "branch-open, then 64 serial steps over the merged cache (1097 + s keys at step s)", "layers": L,
                   "serial_steps": n_serial, "heads": f"{wl.Hq}/{wl.Hkv}", "head_dim": wl.d, "cuda_graph": True,
                   "calls": "aspd_serial_step per (step, layer), one plan per step"},
        "layer_step_us": ms / reps / (n_serial * L) * 1e3,
        "hbm_gbs": gbs, "hbm_frac_of_measured": gbs / peak, "peak_kind": "of " + peak_kind,
        "algorithmic_bytes_per_chain_per_layer": alg, "gpu_launches": launches, "clocks": clocks})
    for pl in plans:
        pl.destroy()
    return line


def run_decode_loop(args):
    """--op decode-loop: 64 consecutive parallel decoding steps of the serving mix as an engine would
    run them: every step the branches are one token longer, so every step gets its own plan
    (created on the host, uploaded, destroyed after its 28 layer calls were enqueued; no graph,
    no synchronisation inside the loop).  Measures what is left of the kernel rate once planning
    and host launches are part of the loop.  One GPU; prints its own JSON line."""
    import torch
    from paper_2508_08895_b200 import binding as B, engine as E, workloads as W
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    n_steps = 64
    prefix, prior = W.serving_mix_lengths(W.SEED_BASE + 4, args.requests or 32)
    # regions sized for the last step; step t reads prior + t + 1 tokens of every branch
    wl = W.build_segment_workload("serving-mix-loop", W.SEED_BASE + 4, 28, 4, 128, "bf16", 1.0e6, prefix,
                                  [[x + n_steps - 1 for x in p] for p in prior], [[1] * len(p) for p in prior])
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    L = args.layers
    caches = [E.LayerCache(shape, wl.n_pool_pages) for _ in range(L)]
    fill_caches(wl, shape, caches)
    ph = wl.phases[-1]
    q_d, k_d, v_d = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
    outs = [torch.empty_like(q_d) for _ in range(L)]
    n_new = int(q_d.shape[0])
    descs = []
    for t in range(n_steps):
        d = {k: v.copy() for k, v in ph.desc.items()}
        d["br_kv_len"] = (ph.desc["br_kv_len"] - (n_steps - 1 - t)).astype(np.int32)
        descs.append(d)

    # The C ABI called as a native engine would: descriptors packed ahead of the loop (an engine
    # keeps them up to date incrementally), pointers resolved once, one foreign call per library call.
    import ctypes
    lib = B.lib()
    packed = [B.pack_descriptors(d) for d in descs]
    tune = B.Tuning(B.KERNEL_AUTO, 0, 0, 0, 1, 0)
    stream = torch.cuda.current_stream().cuda_stream
    qp, kp, vp = q_d.data_ptr(), k_d.data_ptr(), v_d.data_ptr()
    layer_ptrs = [(c.k.data_ptr(), c.v.data_ptr(), o.data_ptr()) for c, o in zip(caches, outs)]
    shape_p, tune_p = ctypes.addressof(shape), ctypes.addressof(tune)
    handle = ctypes.c_void_p()
    handle_p = ctypes.addressof(handle)

    def loop():
        plan_s = 0.0
        for req, br, pages in packed:
            t0 = time.perf_counter()
            rc = lib.aspd_plan_create(shape_p, req.ctypes.data, br.ctypes.data, pages.ctypes.data, len(req), wl.n_pool_pages,
                                      ph.mode, None, tune_p, stream, handle_p)
            plan_s += time.perf_counter() - t0
            if rc:
                raise SystemExit("bench.py: aspd_plan_create returned %d" % rc)
            for kc, vc, oc in layer_ptrs:
                rc |= lib.aspd_branch_step(handle, qp, kp, vp, kc, vc, oc, stream)
            rc |= lib.aspd_plan_destroy(handle)
            if rc:
                raise SystemExit("bench.py: a step call returned %d" % rc)
        return plan_s
    if args.loop_graph:
        # One step captured once; every step re-plans IN PLACE (aspd_plan_update keeps the tables'
        # addresses) and replays the graph: no kernel launch from the host inside the loop.
        side = torch.cuda.Stream()
        torch.cuda.set_stream(side)
        stream = side.cuda_stream
        tune_u = B.Tuning(B.KERNEL_AUTO, 0, 0, 0, 1, 0, 1)
        req0, br0, pages0 = packed[0]
        if lib.aspd_plan_create(shape_p, req0.ctypes.data, br0.ctypes.data, pages0.ctypes.data, len(req0), wl.n_pool_pages, ph.mode,
                                None, ctypes.addressof(tune_u), stream, handle_p):
            raise SystemExit("bench.py: aspd_plan_create failed")

        def one_step():
            rc = 0
            for kc, vc, oc in layer_ptrs:
                rc |= lib.aspd_branch_step(handle, qp, kp, vp, kc, vc, oc, stream)
            if rc:
                raise SystemExit("bench.py: a step call returned %d" % rc)
        one_step()
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            stream = torch.cuda.current_stream().cuda_stream
            one_step()
        stream = side.cuda_stream

        def loop():                                  # noqa: F811  (replaces the host-launched loop above)
            plan_s = 0.0
            for req, br, pages in packed:
                t0 = time.perf_counter()
                rc = lib.aspd_plan_update(handle, req.ctypes.data, br.ctypes.data, pages.ctypes.data, len(req), None, stream)
                plan_s += time.perf_counter() - t0
                if rc:
                    raise SystemExit("bench.py: aspd_plan_update returned %d" % rc)
                graph.replay()
            return plan_s
    loop()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    reps = max(1, min(args.steps, 10))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    ev0.record()
    plan_s = sum(loop() for _ in range(reps))
    host_s = time.perf_counter() - t0
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop()
    total_steps = n_steps * reps
    probe = B.Plan(shape, descs[n_steps // 2], wl.n_pool_pages, ph.mode, host_only=True)
    alg = float(probe.info.algorithmic_bytes)
    probe.destroy()
    peak, peak_kind = measured_peaks()
    gbs = alg * L * total_steps / (ms * 1e-3) / 1e9
    print(json.dumps({
        "op": "decode-loop", "metric": METRIC, "value": n_new * L * total_steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1,
        "steps": total_steps, "warmup": n_steps, "ms_per_step": ms / total_steps, "higher_is_better": True, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": "serving-mix, 64 consecutive decoding steps, a new plan every step", "layers": L,
                   "query_tokens_per_step": n_new, "cuda_graph": bool(args.loop_graph),
                   "calls_per_step": ("aspd_plan_update, replay of the captured step (%d x aspd_branch_step)" % L) if args.loop_graph
                   else "aspd_plan_create, %d x aspd_branch_step, aspd_plan_destroy" % L},
        "host_ms_per_step": host_s / total_steps * 1e3, "plan_create_call_ms_per_step": plan_s / total_steps * 1e3,
        "plan_create_note": "time inside aspd_plan_create; when the host is ahead of the GPU it includes the wait for a parked block "
                            "whose table upload the GPU has not reached yet (the loop's backpressure)",
        "hbm_gbs": gbs, "hbm_frac_of_measured": gbs / peak, "peak_kind": "of " + peak_kind,
        "gpu_launches": L * total_steps + total_steps, "clocks": clocks}))
    return 0


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    from paper_2508_08895_b200 import binding as B, engine as E, workloads as W

    wl = build_workload(args.workload, rank, args.requests)
    kernel = {"auto": B.KERNEL_AUTO, "generic": B.KERNEL_GENERIC, "mma": B.KERNEL_MMA}[args.kernel]
    fused = not args.separate_append
    # decode loop: a layer's pools are written only by that layer's own step, so the plan may carry
    # the stable-cache promise (the kernel starts fetching before the previous layer's combine ends)
    plan_kw = dict(kernel=kernel, chunk_tokens=args.chunk, n_ctas=args.ctas, stable_cache=not args.no_stable_cache,
                   combine={"auto": B.COMBINE_AUTO, "kernel": B.COMBINE_KERNEL, "fused": B.COMBINE_FUSED}[args.combine],
                   wide_rows=args.wide_rows, mma_m=args.mma_m)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- set-up: L layers with distinct pools, one plan, the whole step captured into a CUDA graph
    # (2 launches per layer), so that the host's launch rate does not bound a step whose kernels
    # last tens of microseconds
    shape = B.make_shape(wl.Hq, wl.Hkv, wl.d, wl.page_size, wl.dtype, wl.theta, wl.sm_scale)
    ph = wl.phases[-1]
    probe = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, host_only=True)
    L = max(args.layers, int(np.ceil(4 * 126e6 / max(1, probe.info.algorithmic_bytes))))
    probe.destroy()
    caches = [E.LayerCache(shape, wl.n_pool_pages) for _ in range(L)]
    fill_caches(wl, shape, caches)
    plan = B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, **plan_kw)
    info = plan.info
    pos, _, _ = B.positions(ph.desc, ph.mode)
    n_new = plan.n_new
    pos_d = torch.from_numpy(pos.copy()).cuda()
    q_d, k_d, v_d = (E.to_device(x, wl.dtype) for x in (ph.q, ph.k_new, ph.v_new))
    outs = [torch.empty_like(q_d) for _ in range(L)]
    attn = B.branch_attn if ph.mode == W.MODE_BRANCH else B.serial_attn
    fstep = B.branch_step if ph.mode == W.MODE_BRANCH else B.serial_step
    step_name, attn_name = ("aspd_branch_step", "aspd_branch_attn") if ph.mode == W.MODE_BRANCH else ("aspd_serial_step", "aspd_serial_attn")

    def layer_call(l):
        if fused:      # the attention pass writes the step's new K/V rows itself: 2 launches per layer
            fstep(plan, q_d, k_d, v_d, caches[l].k, caches[l].v, outs[l])
        else:          # aspd_kv_append, then aspd_branch_attn: 3 launches per layer
            B.kv_append(plan, k_d, v_d, pos_d, caches[l].k, caches[l].v)
            attn(plan, q_d, caches[l].k, caches[l].v, outs[l])

    def step():
        for l in range(L):
            layer_call(l)

    run_step = graph_of(step, not args.no_graph)
    for _ in range(max(args.warmup, 3)):
        run_step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        run_step()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    if plan.status() != 0:
        raise SystemExit("bench.py: device status %d" % plan.status())

    # latency of a single layer call launched from the host (no graph), cold pools: median of 50
    lat = []
    la, lb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(50):
        torch.cuda.synchronize()
        la.record(stream)
        layer_call(i % L)
        lb.record(stream)
        torch.cuda.synchronize()
        lat.append(la.elapsed_time(lb) * 1e3)

    # the dominant kernel alone -- the attention kernel the step really runs (with the fused append
    # where the plan fuses it) -- over all layers, back to back (also a graph), then one launch at a
    # time between synchronisations on cold pools
    kcall = attention_kernel_call(plan, ph.mode, q_d, k_d, v_d, fused)

    def kernels():
        for l in range(L):
            kcall(caches[l], outs[l])
    run_k = graph_of(kernels, not args.no_graph)
    k_reps = max(3, min(args.steps, 50))
    kernel_ms = time_replays(run_k, k_reps, 1) / (k_reps * L)
    clocks = sampler.stop() if rank == 0 else None
    iso = []
    for i in range(50):
        torch.cuda.synchronize()
        la.record(stream)
        kcall(caches[i % L], outs[i % L])
        lb.record(stream)
        torch.cuda.synchronize()
        iso.append(la.elapsed_time(lb) * 1e3)
    kernel_iso_us = float(np.median(iso))
    run_step()            # the kernel-only launches left records without a combine: redo the outputs
    torch.cuda.synchronize()

    # ---- end to end through host buffers: q | k_new | v_new packed in one pinned buffer per step
    # (one host-to-device copy per layer), positions compared on the host, output read back
    es = 2 if wl.dtype == "bf16" else 4
    packed = torch.cat([t.reshape(-1).view(torch.uint8).cpu() for t in (q_d, k_d, v_d)]).pin_memory()
    nq, nk = q_d.numel() * es, k_d.numel() * es
    q_h, k_h, v_h = packed[:nq], packed[nq:nq + nk], packed[nq + nk:]
    pos_h = torch.from_numpy(pos.copy()).pin_memory()
    out_h = [torch.empty(nq, dtype=torch.uint8).pin_memory() for _ in range(L)]
    # The layers rotate over a few plans (each owns its staging memory), each on a stream of its
    # own, so that the host copies of one layer overlap the kernels of others; one
    # synchronisation per step, after which every layer's output is in host memory.
    n_e = max(1, args.e2e_streams)
    e_kw = dict(plan_kw, stable_cache=False)
    e_plans = [B.Plan(shape, ph.desc, wl.n_pool_pages, ph.mode, **e_kw) for _ in range(n_e)]
    e_streams = [torch.cuda.Stream() for _ in range(n_e)]

    def step_e2e():
        for l in range(L):
            B.step_host_async(e_plans[l % n_e], q_h, k_h, v_h, pos_h, caches[l].k, caches[l].v, out_h[l], stream=e_streams[l % n_e])
        for st in e_streams:
            st.synchronize()

    for _ in range(2):
        step_e2e()
    barrier()
    e_steps = max(1, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e_steps):
        step_e2e()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    e2e_same = all(torch.equal(out_h[l].view(torch.int16), outs[l].reshape(-1).view(torch.int16).cpu()) for l in range(L))

    # max over ranks, on the device-side times
    (ms, e2e_ms, kernel_ms), total_new = reduce_over_ranks([ms, e2e_ms, kernel_ms], n_new, "cuda", world)

    # parity of layer 0 against the oracle is the tests' business; here only a sanity check that
    # the layers agree with each other (same inputs, distinct pools)
    same = all(torch.equal(outs[0], o) for o in outs[1:])
    for pl in e_plans:
        pl.destroy()

    if rank == 0:
        peak, peak_kind = measured_peaks()
        alg = float(info.algorithmic_bytes)
        value = total_new * L * args.steps / (ms * 1e-3)
        achieved = alg / (kernel_ms * 1e-3) / 1e9
        mhz = (clocks or {}).get("sm_mhz")
        tensor = None
        if args.workload == "masked-prefill":      # many query rows per key: the contraction bounds it, not HBM
            tpeak, tkind = measured_tensor_peak()
            fl = attention_flops(ph.desc, wl.Hq, wl.d)
            tensor = {"bound": "tensor", "achieved": fl / (kernel_ms * 1e-3) / 1e12, "peak": tpeak, "unit": "TFLOP/s",
                      "frac": fl / (kernel_ms * 1e-3) / 1e12 / tpeak, "traffic": None, "peak_kind": "of " + tkind,
                      "kernel": "attention pass", "kernel_us": kernel_ms * 1e3, "kernel_us_isolated": kernel_iso_us, "flops_per_launch": fl}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "layers": L, "query_tokens_per_rank": n_new,
                       "kv_tokens_per_layer": int(info.kv_tokens_read), "heads": f"{wl.Hq}/{wl.Hkv}", "head_dim": wl.d,
                       "page_size": wl.page_size, "kernel": {1: "generic", 2: "mma"}[info.kernel],
                       "chunk_tokens": info.chunk_tokens, "work_items": info.n_items, "n_ctas": info.n_ctas,
                       "l2": "footprint %.1f GB of distinct K/V pools per step, far above L2" % (alg * L / 1e9),
                       "layers_agree": bool(same), "cuda_graph": not args.no_graph, "stable_cache": not args.no_stable_cache,
                       "launches_per_layer": launches_per_layer(info, fused), "combine": "inside the attention kernel" if info.single_launch
                       else "none needed" if info.direct_output else "combine kernel",
                       "calls_per_layer": (step_name + (" (new rows written by the attention pass)" if info.fused_append else " (append kernel, attention pass)")
                                           + ("" if info.single_launch or info.direct_output else " -> combine kernel")) if fused
                       else "aspd_kv_append -> " + attn_name},
            "hbm_gbs": alg * L * args.steps / (ms * 1e-3) / 1e9,
            "hbm_frac_of_measured": alg * L * args.steps / (ms * 1e-3) / 1e9 / peak,
            "hbm_frac_of_8000_nominal": alg * L * args.steps / (ms * 1e-3) / 1e9 / 8000.0,
            "step_us_per_layer": ms / args.steps / L * 1e3,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": alg * TRAFFIC_PER_ALGORITHMIC_BYTE if info.kernel == 2 else None,
                         "traffic_note": "ncu capture of a smaller case of the same mix, scaled by cached tokens",
                         "peak_kind": "of " + peak_kind,
                         "kernel": "attention pass of the step (split-K, new rows written inside)" if (fused and info.fused_append)
                         else "attention pass",
                         "kernel_us": kernel_ms * 1e3, "kernel_us_note": "launches back to back in a graph (consecutive launches overlap): time per launch",
                         "kernel_us_isolated": kernel_iso_us, "frac_isolated": alg / (kernel_iso_us * 1e-6) / 1e9 / peak,
                         "kernel_us_isolated_note": "median of 50 single launches between synchronisations on cold pools, launch latency included",
                         "algorithmic_bytes_per_launch": alg},
            "e2e": {"value": total_new * L * e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(L * (n_new * es * wl.d * (wl.Hq + 2 * wl.Hkv))),
                    "d2h_bytes_per_step": int(L * n_new * es * wl.d * wl.Hq), "ms_per_step": e2e_ms / e_steps,
                    "matches_device_path": bool(e2e_same),
                    "calls": "aspd_step_host_async per layer (one packed host-to-device copy, the fused step, one copy back), "
                             "layers rotating over %d plans on %d streams, one synchronisation per step" % (n_e, n_e)},
            "single_call_us": {"median": float(np.median(lat)), "best": float(np.min(lat)), "calls": len(lat),
                               "what": "one layer's step call launched from the host, CUDA events around it"},
            "gpu_launches": launches_per_layer(info, fused) * L * args.steps,
            "clocks": clocks,
        }
        if mhz:
            line["step_us_x_ghz"] = line["step_us_per_layer"] * mhz * 1e-3
            line["roofline"]["kernel_us_x_ghz"] = kernel_ms * 1e3 * mhz * 1e-3
        if tensor is not None:
            line["roofline_hbm"], line["roofline"] = line["roofline"], tensor
    plan.destroy()
    del caches, outs, plan
    torch.cuda.empty_cache()
    if rank == 0:
        if world == 1 and not args.no_per_config and args.workload == "serving-mix" and args.requests == 0:
            line["per_config"] = per_config_block(args, peak)
        if world == 1 and not args.no_cpu_baseline:
            v, cores, sec, reps_o, n_o = oracle_sample(wl, budget_s=args.cpu_budget)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{reps_o} repetitions of one layer-step of the same batch "
                                              f"({n_o} query tokens), {sec:.3f} s each"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def per_config_block(args, peak):
    """The other configurations on the same box, right after the headline: each parity config that
    runs on the tensor-core path, the serial step of the mix, the serial chain, masked prefill
    (against the tensor roofline) and the key re-rotation."""
    import copy
    import torch
    from paper_2508_08895_b200 import workloads as W
    steps = max(3, min(args.steps, 30))
    out = {}
    for name in ("qwen7b-layer", "branch-open", "long-rag", "serving-mix-serial", "masked-prefill"):
        wl = build_workload(name, 0, 0)
        layers = 4 if name == "masked-prefill" else 28
        res, keep = measure_step_workload(wl, layers, steps if name != "masked-prefill" else 5, 3, plan_kw=dict(stable_cache=True))
        if name == "masked-prefill":
            tpeak, tkind = measured_tensor_peak()
            out[name] = per_config_entry(res, peak, flops=attention_flops(keep["ph"].desc, wl.Hq, wl.d), tensor_peak=tpeak)
            out[name]["peak_kind"] = "of " + tkind
        else:
            out[name] = per_config_entry(res, peak)
        keep["plan"].destroy()
        del keep, res
        torch.cuda.empty_cache()
    sub = copy.copy(args)
    sub.steps, sub.layers = min(args.steps, 20), 28
    sc = measure_serial_chain(sub)
    out["serial-chain"] = {"layer_step_us": sc["layer_step_us"], "steps_per_s": sc["value"], "hbm_gbs": sc["hbm_gbs"],
                           "step_frac": sc["hbm_frac_of_measured"], "bound": "hbm", "layers": sc["config"]["layers"],
                           "sm_mhz": (sc["clocks"] or {}).get("sm_mhz"), "what": sc["config"]["workload"]}
    torch.cuda.empty_cache()
    sub.workload, sub.requests = "serving-mix", 0
    rr = measure_rerotate(sub)
    out["rerotate"] = {"kernel_us": rr["roofline"]["kernel_us"], "alg_bytes": rr["roofline"]["algorithmic_bytes_per_layer"],
                       "call": rr["config"]["call"], "launches": rr["config"]["launches_per_step"],
                       "frac": rr["roofline"]["frac"], "bound": "hbm", "tokens_per_layer": rr["config"]["tokens_per_layer"],
                       "layers": rr["config"]["layers"], "sm_mhz": (rr["clocks"] or {}).get("sm_mhz")}
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="serving-mix", choices=["qwen7b-layer", "branch-open", "long-rag", "serving-mix", "masked-prefill", "serving-mix-serial"])
    ap.add_argument("--op", default="step", choices=["step", "rerotate", "serial-chain", "decode-loop"],
                    help="step: the attention step (the benchmark); rerotate: the Same-Re key re-rotation kernel alone; "
                         "serial-chain: 64 serial steps after a merged segment, one graph; "
                         "decode-loop: 64 decoding steps with a new plan each, launched from the host")
    ap.add_argument("--layers", type=int, default=28)
    ap.add_argument("--kernel", default="auto", choices=["auto", "generic", "mma"])
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--ctas", type=int, default=0)
    ap.add_argument("--wide-rows", type=int, default=0, choices=[0, 128, 256],
                    help="plans that deal whole streams: query rows per row block (one or two tiles; 0 = automatic)")
    ap.add_argument("--mma-m", type=int, default=0, choices=[0, 64, 96, 128], help="stream-K plans: M of the tensor-core kernel's MMAs (0 = automatic)")
    ap.add_argument("--combine", default="auto", choices=["auto", "kernel", "fused"],
                    help="where the split-K records are merged: a combine launch, or inside the attention kernel (one launch per layer)")
    ap.add_argument("--requests", type=int, default=0, help="serving-mix only: number of requests (default 32)")
    ap.add_argument("--cpu-budget", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the per-configuration block of the default run")
    ap.add_argument("--separate-append", action="store_true",
                    help="call aspd_kv_append and aspd_branch_attn separately instead of aspd_branch_step")
    ap.add_argument("--no-stable-cache", action="store_true", help="create the plan without the stable-cache promise")
    ap.add_argument("--e2e-streams", type=int, default=4, help="plans/streams the layers rotate over in the end-to-end leg")
    ap.add_argument("--loop-graph", action="store_true",
                    help="decode-loop: capture the step once and re-plan in place every step (aspd_plan_update) instead of "
                         "making a new plan and launching from the host")
    ap.add_argument("--rerotate-by-token", action="store_true", help="rerotate: per-token index arrays (aspd_k_rerotate) instead of ranges")
    ap.add_argument("--rerotate-per-layer", action="store_true",
                    help="rerotate: one aspd_k_rerotate_ranges call per layer instead of all layers in one launch")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying a CUDA graph")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.op != "step" and int(os.environ.get("RANK", "0")) != 0:
        return 0          # the side measurements are single-GPU: rank 0 alone runs and prints them
    if args.op == "rerotate":
        return run_rerotate(args)
    if args.op == "serial-chain":
        return run_serial_chain(args)
    if args.op == "decode-loop":
        return run_decode_loop(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
