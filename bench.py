#!/usr/bin/env python
"""Benchmark of the partitioned decode-attention step (one layer, one decode step per "step").

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl cuda|reference]

Prints ONE JSON line.  `value` is decode-attention KV GB/s (bytes of cached K and V rows divided by
time) of spd_decode_step (fused) with every input resident in HBM; `e2e` is the same metric through
spd_decode_step_host, whose per-step inputs (q, page tables, lengths) start in one pinned host buffer and
whose output is read back inside the timed region.  The KV pools are the resident cache in both.

The headline workload is the largest single-GPU configuration (c5_many_user); the GQA configuration
(c3_llama3_8b_gqa) is measured the same way beside it (`co_headline`), the other two more briefly
(`other_configs`).  A timed region is `--steps` back-to-back steps between two CUDA events; it is repeated
until at least a second of GPU time has gone by, and the MEDIAN repeat is reported (the best one beside it),
so that the figure is the sustained, power-capped one.

With N > 1 (torchrun) every rank runs an independent replica on its own GPU (the path has no exchange
step) and `value` sums the replicas over the slowest rank's time.

`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2409_19134_b200 import workloads as wl  # noqa: E402

METRIC = "decode-attention KV GB/s"
NOMINAL_HBM_GBS = 8000.0
CO_HEADLINE = {"c5_many_user": "c3_llama3_8b_gqa", "c3_llama3_8b_gqa": "c5_many_user"}
BRIEF_CONFIGS = ["c2_llama2_7b", "c4_long_prompt", "c3_llama3_8b_gqa", "c5_many_user"]
MIN_GPU_SECONDS = 1.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                 "sw_thermal_slowdown": 0x20, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def max_over_ranks(x: float, device) -> float:
    """Slowest rank's time (every rank gets it).  Single process: x itself."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(bytes_per_replica: int, ms_slowest: float, world: int) -> float:
    """GB/s of `world` independent replicas that all finish within the slowest rank's time."""
    return world * bytes_per_replica / ms_slowest / 1e6


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ------------------------------------------------------------------------------------------------ oracle legs
def _slice_heads(w, n_users, n_kvh):
    """First n_users users and first n_kvh KV heads (with their query heads): pure slicing."""
    from oracle import spd_oracle as orc
    g = w.num_q_heads // w.num_kv_heads

    def part(p):
        lo = int(p.page_indptr[n_users])
        kv = orc.kv_from_torch(wl.PagedKV(p.k_pool[:, :n_kvh].contiguous(), p.v_pool[:, :n_kvh].contiguous(),
                                          p.page_indptr[:n_users + 1].contiguous(), p.page_indices[:lo].contiguous(),
                                          p.seq_lens[:n_users].contiguous()))
        return kv
    q = orc.q_from_torch(w.q[:n_users, :n_kvh * g].contiguous())
    toks = int(w.priv.seq_lens[:n_users].sum()) + int(w.pub.seq_lens[:n_users].sum())
    nbytes = toks * 2 * n_kvh * w.head_dim * w.elem_size
    return q, part(w.priv), part(w.pub), nbytes


def oracle_sample(w_cpu, budget_s):
    """Pick (users, kv heads) so that one oracle pass takes about budget_s; returns a timed closure."""
    from oracle import spd_oracle as orc
    q, a, b, nb = _slice_heads(w_cpu, 1, 1)
    t0 = time.perf_counter()
    orc.full(q, a, b, w_cpu.sm_scale)
    t1 = max(time.perf_counter() - t0, 1e-4)        # one user, one KV head (few threads busy)
    cores = orc.num_threads()
    g = w_cpu.num_q_heads // w_cpu.num_kv_heads
    unit = t1 * min(cores, g) / cores               # wall time of one (user, KV head) with all cores busy
    units = max(1.0, budget_s / unit)
    n_kvh = int(min(w_cpu.num_kv_heads, max(1, units)))
    n_users = int(min(w_cpu.batch, max(1, units // n_kvh)))
    q, a, b, nb = _slice_heads(w_cpu, n_users, n_kvh)

    def run():
        t = time.perf_counter()
        orc.full(q, a, b, w_cpu.sm_scale)
        return time.perf_counter() - t
    return run, nb, n_users, n_kvh, cores


def cpu_baseline(w_cpu, full_batch, budget_s=12.0):
    run, nb, n_users, n_kvh, cores = oracle_sample(w_cpu, budget_s)
    ts = [run()]
    while sum(ts) < 10.0 and len(ts) < 40:    # a short pass is repeated: about ten seconds of CPU work in all
        ts.append(run())
    dt = float(np.mean(ts))
    return {"value": nb / dt / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": f"first {n_users} of {full_batch} users x first {n_kvh} of {w_cpu.num_kv_heads} KV heads, "
                      f"mean of {len(ts)} passes of {dt:.2f} s", "user_tokens_per_s": n_users * n_kvh / w_cpu.num_kv_heads / dt}


def sample_workload_cpu(cfg_name, max_users=48, users=None):
    """The first users of a config, generated on the CPU: same seeded length draw as the full workload (so these
    are its first users' lengths), values from the CPU generator.  Keeps the oracle legs from building 5 GB pools."""
    cfg = wl.CONFIGS[cfg_name]
    lin, lout = wl.make_lengths(cfg)
    full = cfg["batch"] if users is None else min(users, cfg["batch"])
    n = min(full, max_users)
    w = wl.make_workload(dict(cfg, name=cfg_name, batch=n), lengths=(lin[:n], lout[:n]), device="cpu")
    w.full_kv_bytes = int(lin[:full].sum() + lout[:full].sum()) * 2 * cfg["hkv"] * cfg["d"] * w.elem_size
    return w, full


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    cfg = args.config
    w, full_batch = sample_workload_cpu(cfg, users=args.users)
    steps, warmup = args.steps or 5, args.warmup if args.warmup is not None else 1
    budget = min(15.0, 150.0 / (steps + warmup))
    run, nb, n_users, n_kvh, cores = oracle_sample(w, budget)
    for _ in range(warmup):
        run()
    ts = [run() for _ in range(steps)]
    dt = float(np.mean(ts))
    val = nb / dt / 1e9
    sample = (f"each step: first {n_users} of {full_batch} users x first {n_kvh} of {w.num_kv_heads} KV heads "
              f"({nb / 1e6:.1f} MB of KV)")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": steps,
            "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, w, full_batch, world, args, kv_bytes_per_step=w.full_kv_bytes, sample=sample),
            "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(cfg, w, users, world, args, **extra):
    """The `config` object of the JSON line: the same keys for both arms."""
    c = {"workload": cfg, "users": users, "q_heads": w.num_q_heads, "kv_heads": w.num_kv_heads,
         "head_dim": w.head_dim, "page_size": w.page_size,
         "parallelism": "replicas only" if world > 1 else "single GPU", "call": "spd_decode_step(fused=1)",
         "bf16_math": args.bf16_math}
    c.update(extra)
    return c


# ------------------------------------------------------------------------------------------------ CUDA arm
def time_config(spd, w, steps, warmup, fused=True, plan=None, min_seconds=MIN_GPU_SECONDS, max_repeats=400):
    """Device time of `steps` back-to-back decode steps between two CUDA events on the launching stream, repeated
    until `min_seconds` of GPU time have gone by.  Returns the median repeat (ms per step), all repeats, and the
    objects the other measurements reuse.  plan: None = the plain call; 'reuse' = one storing call, then every
    timed call loads the stored plan."""
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device=w.q.device)
    mode = None
    if plan == "reuse":
        spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=fused, plan=spd.SPD_PLAN_STORE)
        mode = spd.SPD_PLAN_REUSE

    def step():
        spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=fused, plan=mode)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    n0 = spd.spd_kernel_launch_count()
    per_step, total = [], 0.0
    while total < min_seconds * 1e3 and len(per_step) < max_repeats:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            step()
        e1.record()
        e1.synchronize()
        ms = e0.elapsed_time(e1)
        per_step.append(ms / steps)
        total += ms
    launches = spd.spd_kernel_launch_count() - n0
    code, bad = spd.spd_query_device_status(ws)
    if code != spd.SPD_OK or not bool(torch.isfinite(out).all()):
        raise RuntimeError(f"decode step failed: status {code}, first bad user {bad}")
    timing = {"repeats": len(per_step), "steps_per_repeat": steps, "median_ms_per_step": float(np.median(per_step)),
              "best_ms_per_step": float(np.min(per_step)), "worst_ms_per_step": float(np.max(per_step)),
              "gpu_seconds": total / 1e3}
    return timing["median_ms_per_step"], launches, shape, ws, out, timing


def kernel_split(spd, w, shape, ws, out, steps):
    """Average device time of the attention kernel alone, events recorded inside the library."""
    steps = max(1, min(steps, 2000))
    spd.spd_profile_begin(steps)
    for _ in range(steps):
        spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=True)
    r = spd.spd_profile_end()
    return {"attn_ms": r["kernel_ms"] / max(r["calls"], 1)}


def time_e2e(spd, w, shape, ws, steps, warmup, out_dtype=torch.float32):
    """Per step: q, page tables and lengths go in from one pinned host blob, the output comes back."""
    dev = w.q.device
    lay = spd.spd_step_blob_layout(shape, int(w.priv.page_indices.numel()), int(w.pub.page_indices.numel()), out_dtype)
    host = torch.zeros(lay.total_bytes, dtype=torch.uint8).pin_memory()
    spd.fill_step_blob(lay, host, w.q, w.priv, w.pub)
    devb = torch.empty(lay.total_bytes, dtype=torch.uint8, device=dev)
    pools = [(w.priv.k_pool, w.priv.v_pool), (w.pub.k_pool, w.pub.v_pool)]

    step = spd.HostStep(shape, lay, host, devb, pools[0], pools[1], out_dtype, ws)

    def call():
        code, bad = step()
        if code != spd.SPD_OK:
            raise RuntimeError(f"host-buffer step failed: status {code}, user {bad}")
    for _ in range(warmup):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    d2h = lay.total_bytes - lay.status
    n_out = w.batch * w.num_q_heads * w.head_dim
    es = 4 if out_dtype == torch.float32 else 2
    outh = host[lay.out:lay.out + es * n_out].view(out_dtype).reshape(w.batch, w.num_q_heads, w.head_dim).float().clone()
    return e0.elapsed_time(e1) / steps, lay.in_bytes, d2h, outh


def time_schedules(spd, w, shape, steps=200):
    """The same step scheduled four ways, microseconds per step by CUDA events: the two halves chained on one
    stream, the halves on two streams followed by the stand-alone merge, the fused step, and the fused
    step replayed from a CUDA graph (20 steps per graph); then each half alone, and the spread of single steps."""
    dev = w.q.device
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device=dev)
    ws_a, ws_b = spd.alloc_workspace(shape), spd.alloc_workspace(shape)
    pa, pb = spd.alloc_partial(shape), spd.alloc_partial(shape)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()

    def chained():
        spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws_a, fused=False, stream=sa)

    def fused():
        spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws_a, fused=True, stream=sa)

    def two_streams():
        sb.wait_stream(sa)                                   # the previous merge has read pb
        spd.spd_partial_attn(shape, w.q, w.priv, pa, ws_a, stream=sa)
        spd.spd_partial_attn(shape, w.q, w.pub, pb, ws_b, stream=sb)
        sa.wait_stream(sb)
        spd.spd_merge_partials(shape, [pa, pb], out, stream=sa)

    def timed(fn, n):
        for _ in range(10):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(sa)
        for _ in range(n):
            fn()
        e1.record(sa)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n * 1e3

    res = {"chained_us": timed(chained, steps), "two_streams_us": timed(two_streams, steps), "fused_us": timed(fused, steps)}
    # the two halves of the protocol on their own: the per-user call (private partial) and the service call
    # (public partial + merge of a given private partial)
    res["partial_attn_us"] = timed(lambda: spd.spd_partial_attn(shape, w.q, w.priv, pa, ws_a, stream=sa), steps)
    res["service_attn_merge_us"] = timed(lambda: spd.spd_service_attn_merge(shape, w.q, w.pub, pa, out, ws_a, stream=sa), steps)
    # spread of single fused steps: an event between every two calls
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    evs[0].record(sa)
    for i in range(steps):
        fused()
        evs[i + 1].record(sa)
    torch.cuda.synchronize()
    per = np.array([evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]) * 1e3
    res["fused_step_us"] = {"median": float(np.median(per)), "best": float(per.min()), "p95": float(np.percentile(per, 95))}
    per_graph = 20
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(sa):
        with torch.cuda.graph(graph, stream=sa):
            for _ in range(per_graph):
                spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws_a, fused=True, stream=sa)
        res["fused_graph_us"] = timed(graph.replay, max(1, steps // per_graph)) / per_graph
    for ws in (ws_a, ws_b):
        code, bad = spd.spd_query_device_status(ws, stream=sa)
        if code != spd.SPD_OK:
            raise RuntimeError(f"schedule study failed: status {code}, user {bad}")
    return res


PREFILL_CASE = dict(users=8, prompt_lo=2048, prompt_hi=8192, hq=32, hkv=8, d=128, seed=7)   # Llama-3-8B-shaped prompts


def prefill_inputs(spd, dev, case=PREFILL_CASE):
    """Seeded ragged prompts and an empty private cache with room for them (values drawn on `dev`)."""
    rng = np.random.default_rng(case["seed"])
    lens = rng.integers(case["prompt_lo"], case["prompt_hi"] + 1, size=case["users"])
    B, hq, hkv, D = case["users"], case["hq"], case["hkv"], case["d"]
    ip = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(ip[-1])
    gen = torch.Generator(device=dev)
    gen.manual_seed(case["seed"])
    q = torch.randn((T, hq, D), generator=gen, device=dev).to(torch.bfloat16)
    k = torch.randn((T, hkv, D), generator=gen, device=dev).to(torch.bfloat16)
    v = torch.randn((T, hkv, D), generator=gen, device=dev).to(torch.bfloat16)
    need = (lens + 15) // 16
    pidx = np.concatenate([[0], np.cumsum(need)]).astype(np.int32)
    pages = int(pidx[-1])
    perm = torch.from_numpy(rng.permutation(pages).astype(np.int32)).to(dev)
    part = wl.PagedKV(torch.zeros((pages, hkv, 16, D), dtype=torch.bfloat16, device=dev),
                      torch.zeros((pages, hkv, 16, D), dtype=torch.bfloat16, device=dev),
                      torch.from_numpy(pidx).to(dev), perm, torch.zeros(B, dtype=torch.int32, device=dev))
    shape = spd.make_shape(B, hq, hkv, D, torch.bfloat16, 1.0 / np.sqrt(D))
    return lens, ip, q, k, v, part, shape


def time_prefill(spd, dev, steps=5, case=PREFILL_CASE):
    """spd_prefill_attn on seeded ragged prompts: causal attention (tensor-bound) plus the K/V hand-over.
    Flops counted: 4 * D * Hq * sum over users of L (L + 1) / 2 (the causal half only)."""
    lens, ip, q, k, v, part, shape = prefill_inputs(spd, dev, case)
    B, hq, hkv, D = case["users"], case["hq"], case["hkv"], case["d"]
    T = int(ip[-1])
    ws = spd.alloc_workspace(shape, dev)
    out = torch.empty((T, hq, D), dtype=torch.bfloat16, device=dev)
    tip = torch.from_numpy(ip).to(dev)
    for _ in range(2):
        spd.spd_prefill_attn(shape, q, k, v, tip, part, out, ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        spd.spd_prefill_attn(shape, q, k, v, tip, part, out, ws)
    e1.record()
    torch.cuda.synchronize()
    code, bad = spd.spd_query_device_status(ws)
    if code != spd.SPD_OK or not bool(torch.isfinite(out.float()).all()):
        raise RuntimeError(f"prefill failed: status {code}, user {bad}")
    ms = e0.elapsed_time(e1) / steps
    flops = 4.0 * D * hq * float(sum(int(n) * (int(n) + 1) // 2 for n in lens))
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak, src = float(json.load(f)["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, burst)"
    except Exception:
        peak, src = 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"
    tf = flops / ms / 1e9
    return {"workload": f"{B} prompts, lengths U[{case['prompt_lo']},{case['prompt_hi']}] ({T} tokens), {hq}/{hkv} heads, D {D}, bf16",
            "ms": ms, "tokens_per_s": T / ms * 1e3,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                         "traffic": None, "kernel": "prefill_pair_kernel", "peak_source": src}}


def time_append(spd, w, shape, ws, calls=8):
    """spd_append_kv on the public cache: `calls` tokens per user appended back to back (the lengths are
    first moved back by `calls`, and restored afterwards, so that every row fits the pages already listed)."""
    if int(w.pub.seq_lens.min()) < 1:
        return None
    dev = w.q.device
    keep = w.pub.seq_lens.clone()
    gen = torch.Generator(device=dev)
    gen.manual_seed(99)
    k_new = torch.randn((w.batch, w.num_kv_heads, w.head_dim), generator=gen, device=dev).to(w.dtype)
    v_new = torch.randn((w.batch, w.num_kv_heads, w.head_dim), generator=gen, device=dev).to(w.dtype)
    ms = []
    for rep in range(4):
        w.pub.seq_lens.copy_(torch.clamp(keep - calls, min=0))
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(calls):
            spd.spd_append_kv(shape, k_new, v_new, w.pub, ws)
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1) / calls)
    code, bad = spd.spd_query_device_status(ws)
    w.pub.seq_lens.copy_(keep)     # the rows written sit where tokens already were or in unused slots: restore
    if code != spd.SPD_OK:
        raise RuntimeError(f"append failed: status {code}, user {bad}")
    nbytes = 2 * w.batch * w.num_kv_heads * w.head_dim * w.elem_size
    return {"us_per_call": min(ms) * 1e3, "bytes_written_per_call": nbytes, "note": "latency-bound: one small kernel"}


def time_token_step(spd, w, shape, ws, n_layers=8, replays=4):
    """spd_token_step: the append and the fused decode step, one launch per layer, for each of `n_layers` layers
    (every layer with its own copy of the caches), run eagerly and replayed from one CUDA graph; microseconds per token step.  Every
    run appends a token per user and layer, so the lengths are first moved back by the number of runs."""
    if int(w.pub.seq_lens.min()) < 1:
        return None
    dev = w.q.device
    runs = 2 * (replays + 2)
    gen = torch.Generator(device=dev)
    gen.manual_seed(101)
    layers = []
    for i in range(n_layers):
        priv = wl.PagedKV(w.priv.k_pool.clone(), w.priv.v_pool.clone(), w.priv.page_indptr, w.priv.page_indices, w.priv.seq_lens)
        pub = wl.PagedKV(w.pub.k_pool.clone(), w.pub.v_pool.clone(), w.pub.page_indptr, w.pub.page_indices,
                         torch.clamp(w.pub.seq_lens - runs, min=0))
        k_new = torch.randn((w.batch, w.num_kv_heads, w.head_dim), generator=gen, device=dev).to(w.dtype)
        v_new = torch.randn((w.batch, w.num_kv_heads, w.head_dim), generator=gen, device=dev).to(w.dtype)
        out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device=dev)
        layers.append((w.q, k_new, v_new, priv, pub, out))
    if any(int((p[4].seq_lens + runs > (p[4].page_indptr[1:] - p[4].page_indptr[:-1]) * 16).sum()) for p in layers[:1]):
        return None                                    # some user's listed pages cannot take that many tokens
    sa = torch.cuda.Stream()

    def timed(fn, n):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(sa)
        for _ in range(n):
            fn()
        e1.record(sa)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n * 1e3

    with torch.cuda.stream(sa):
        eager = timed(lambda: spd.spd_token_step(shape, layers, ws, stream=sa, same_lengths=True), replays)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=sa):
            spd.spd_token_step(shape, layers, ws, stream=sa, same_lengths=True)
        replay = timed(graph.replay, replays)
    code, bad = spd.spd_query_device_status(ws, stream=sa)
    if code != spd.SPD_OK:
        raise RuntimeError(f"token step failed: status {code}, user {bad}")
    kv = sum(int(p[3].seq_lens.sum()) + int(p[4].seq_lens.sum()) for p in layers) * 2 * w.num_kv_heads * w.head_dim * w.elem_size
    return {"layers": n_layers, "eager_us": eager, "graph_us": replay, "kernels_per_step": n_layers,
            "kv_gbs_graph": kv / replay / 1e3, "plan": "derived by layer 0, loaded by the other layers"}


PAPER_SCALE = dict(batch=8, hq=32, hkv=8, d=128, dtype="bf16", lin=("const", 512), lout=("uniform", 1, 128), seed=11)


def time_paper_scale(spd, dev, steps=300):
    """The scale of the paper's own runs (a handful of users, prompts of 64 to 512 tokens, a Llama-3-8B-shaped
    layer): latency of one fused decode step, of the per-user call alone (one user per call, as the paper's
    per-user processes issue it) and of the prefill of the same prompts.  Latency-bound: microseconds, no roofline."""
    w = wl.make_workload(dict(PAPER_SCALE, name="paper_scale"), device=dev)
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape, dev)
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device=dev)

    def timed(fn, n):
        for _ in range(10):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n * 1e3

    res = {"workload": "8 users, 512-token prompts, 1-128 generated tokens, 32/8 heads, D 128, bf16",
           "decode_step_us": timed(lambda: spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=True), steps)}
    spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=True, plan=spd.SPD_PLAN_STORE)
    res["decode_step_plan_cached_us"] = timed(
        lambda: spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=True, plan=spd.SPD_PLAN_REUSE), steps)
    one = wl.make_workload(dict(PAPER_SCALE, name="one_user", batch=1), device=dev)
    shape1 = spd.make_shape(1, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws1, part1 = spd.alloc_workspace(shape1, dev), spd.alloc_partial(shape1)
    res["per_user_partial_us"] = timed(lambda: spd.spd_partial_attn(shape1, one.q, one.priv, part1, ws1), steps)
    spd.spd_partial_attn(shape1, one.q, one.priv, part1, ws1, plan=spd.SPD_PLAN_STORE)
    res["per_user_partial_plan_cached_us"] = timed(
        lambda: spd.spd_partial_attn(shape1, one.q, one.priv, part1, ws1, plan=spd.SPD_PLAN_REUSE), steps)
    ts = time_token_step(spd, w, shape, ws, n_layers=8, replays=4)
    if ts is not None:
        res["token_step_8_layers"] = dict(ts, per_layer_graph_us=ts["graph_us"] / ts["layers"])
    case = dict(users=8, prompt_lo=512, prompt_hi=512, hq=32, hkv=8, d=128, seed=11)
    res["prefill_us"] = time_prefill(spd, dev, steps=20, case=case)["ms"] * 1e3
    for x in (ws, ws1):
        code, bad = spd.spd_query_device_status(x)
        if code != spd.SPD_OK:
            raise RuntimeError(f"paper-scale run failed: status {code}, user {bad}")
    return res


def make_gpu_workload(cfg, dev, users=None):
    """The named workload on `dev`; with `users`, its first users only (for profiler captures that must stay small)."""
    if users is None or users >= wl.CONFIGS[cfg]["batch"]:
        return wl.make_workload(cfg, device=dev)
    lin, lout = wl.make_lengths(wl.CONFIGS[cfg])
    return wl.make_workload(dict(wl.CONFIGS[cfg], name=cfg, batch=users), lengths=(lin[:users], lout[:users]), device=dev)


def roofline_block(kvb, attn_ms, cfg, users):
    peak, peak_src = measured_peak()
    achieved = kvb / attn_ms / 1e6
    traffic = TRAFFIC_BYTES.get(cfg) if users is None else None
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic, "kernel": "attn_kernel", "peak_source": peak_src, "kernel_ms": attn_ms,
            "algorithmic_bytes": kvb, "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
            "timing": "separate pass, CUDA events around each kernel on the launch stream"}


def measure_config(spd, cfg, dev, steps, warmup, local_rank, users=None, seconds=MIN_GPU_SECONDS, extras=True):
    """One configuration measured on its own: the fused step (median repeat of a >= `seconds` region, clocks
    sampled meanwhile), the attention kernel alone against the roofline, and -- with extras -- the step through
    host buffers, the chained step, the step on a stored plan and the step with the measured rates ignored."""
    w = make_gpu_workload(cfg, dev, users)
    kvb = w.kv_bytes()
    with ClockSampler(local_rank) as clocks:
        ms, launches, shape, ws, out, timing = time_config(spd, w, steps, warmup, min_seconds=seconds)
    res = {"workload": cfg, "users": w.batch, "kv_bytes_per_step": kvb, "ms_per_step": ms, "gbs": kvb / ms / 1e6,
           "best_gbs": kvb / timing["best_ms_per_step"] / 1e6, "timing": timing, "clocks": clocks.summary(),
           "user_tokens_per_s": w.batch / ms * 1e3, "pct_of_nominal_hbm_8000": 100.0 * kvb / ms / 1e6 / NOMINAL_HBM_GBS,
           "pct_of_measured_hbm": 100.0 * kvb / ms / 1e6 / measured_peak()[0], "gpu_launches": launches}
    split = kernel_split(spd, w, shape, ws, out, min(2000, max(steps, int(seconds * 1e3 / ms))))
    res["roofline"] = roofline_block(kvb, split["attn_ms"], cfg, users)
    res["sm_moves"] = dict(zip(("launches_compared", "ctas_on_another_sm"), spd.spd_debug_sm_moves(ws)))
    if extras:
        e2e_ms, h2d, d2h, outh = time_e2e(spd, w, shape, ws, min(500, max(steps, int(0.3 * seconds * 1e3 / ms))), warmup)
        if not torch.allclose(outh, out.cpu(), atol=2e-3, rtol=0):   # share sizes adapt, so rounding order may differ
            raise RuntimeError("host-buffer path and device path disagree")
        res["e2e"] = {"value": kvb / e2e_ms / 1e6, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "ms_per_step": e2e_ms, "call": "spd_decode_step_host", "out_dtype": "f32"}
        # the same with the output read back in bf16 (what a bf16 model consumes): half the device-to-host bytes
        b_ms, b_h2d, b_d2h, outb = time_e2e(spd, w, shape, ws, min(300, max(steps, int(0.2 * seconds * 1e3 / ms))), warmup, torch.bfloat16)
        if not torch.allclose(outb, out.cpu(), atol=2e-3 + 2.0 ** -8 * float(out.abs().max()), rtol=0):
            raise RuntimeError("host-buffer path with bf16 output and device path disagree")
        res["e2e_bf16_out"] = {"value": kvb / b_ms / 1e6, "unit": "GB/s", "h2d_bytes_per_step": b_h2d, "d2h_bytes_per_step": b_d2h,
                               "ms_per_step": b_ms}
        brief = 0.25 * seconds
        m, *_ = time_config(spd, w, steps, warmup, fused=False, min_seconds=brief)
        res["chained"] = {"ms_per_step": m, "gbs": kvb / m / 1e6}
        m, *_ = time_config(spd, w, steps, warmup, plan="reuse", min_seconds=brief)
        res["plan_cached"] = {"ms_per_step": m, "gbs": kvb / m / 1e6, "note": "every timed call loads the plan stored by one call before the region; the headline derives it inside every call (plan included)"}
        spd.spd_set_split(0, True)
        try:
            m, *_ = time_config(spd, w, steps, warmup, min_seconds=brief)
        finally:
            spd.spd_set_split(0, False)
        res["uniform_shares"] = {"ms_per_step": m, "gbs": kvb / m / 1e6, "note": "measured streaming rates ignored: what the rate-weighted shares are worth"}
    return res, w


def run_cuda(args):
    from paper_2409_19134_b200 import binding as spd
    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    steps = args.steps or 100
    warmup = args.warmup if args.warmup is not None else 20
    if warmup < 3:
        warmup = 3
    cfg = args.config
    spd.lib()
    spd.spd_set_bf16_math(1 if args.bf16_math == "fma" else 0)
    if args.prefill_only:
        if rank == 0:
            print(json.dumps({"prefill": time_prefill(spd, dev, steps=args.steps or 5)}), flush=True)
        return

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    head, w = measure_config(spd, cfg, dev, steps, warmup, local_rank, users=args.users, extras=not args.kernel_only)
    barrier()
    kvb = head["kv_bytes_per_step"]
    ms_max = max_over_ranks(head["ms_per_step"], dev)     # every rank: its own replica of the same seeded workload
    value = replica_throughput(kvb, ms_max, world)
    e2e = head.get("e2e")
    if e2e is not None:
        e2e_ms = max_over_ranks(e2e["ms_per_step"], dev)
        e2e = dict(e2e, value=replica_throughput(kvb, e2e_ms, world), ms_per_step=e2e_ms)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak = measured_peak()[0]
    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_max, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if w.dtype == torch.bfloat16 else "f32", "data": "synthetic",
        "config": workload_config(cfg, w, w.batch, world, args, kv_bytes_per_step=kvb,
                                  l2=("inputs larger than L2 (KV bytes per step >> 126 MB); no flush" if kvb > 4 * 126e6 else
                                      "inputs FIT in L2 and are not flushed: a latency figure, not comparable with the HBM roofline"),
                                  timed_region=f"{steps} back-to-back steps between two CUDA events, repeated {head['timing']['repeats']} "
                                               f"times ({head['timing']['gpu_seconds']:.2f} s of GPU time); value = median repeat"),
        "timing": head["timing"], "best_repeat_gbs": head["best_gbs"] * world,
        "user_tokens_per_s": world * w.batch / ms_max * 1e3,
        "pct_of_nominal_hbm_8000": 100.0 * value / world / NOMINAL_HBM_GBS,
        "pct_of_measured_hbm": 100.0 * value / world / peak,
        "e2e": e2e, "gpu_launches": head["gpu_launches"], "roofline": head["roofline"], "clocks": head["clocks"],
        "sm_moves": head["sm_moves"],
    }
    for k in ("e2e_bf16_out", "chained", "plan_cached", "uniform_shares"):
        if k in head:
            line[k] = head[k]
    if world == 1 and not args.no_extras and not args.kernel_only and args.users is None:
        del w
        torch.cuda.empty_cache()
        co = CO_HEADLINE.get(cfg)
        if co:
            line["co_headline"], w = measure_config(spd, co, dev, steps, warmup, local_rank)
            del w
            torch.cuda.empty_cache()
        others = {}
        for name in BRIEF_CONFIGS:
            if name in (cfg, co):
                continue
            others[name], w = measure_config(spd, name, dev, steps, warmup, local_rank, seconds=0.4)
            del w
            torch.cuda.empty_cache()
        line["other_configs"] = others
        # the studies around the path run on the Llama-2-7B-shaped layer (the smallest bf16 configuration)
        w = wl.make_workload("c2_llama2_7b", device=dev)
        shape2 = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
        ws2 = spd.alloc_workspace(shape2)
        line["prefill"] = time_prefill(spd, dev)
        line["schedules"] = dict(time_schedules(spd, w, shape2), workload="c2_llama2_7b")
        line["append_kv"] = time_append(spd, w, shape2, ws2)
        line["paper_scale"] = time_paper_scale(spd, dev)
        line["token_step"] = time_token_step(spd, w, shape2, ws2)
        del w
        torch.cuda.empty_cache()
        w_cpu, full_batch = sample_workload_cpu(cfg)
        line["cpu_baseline"] = cpu_baseline(w_cpu, full_batch)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one attn_kernel launch, from the ncu
# captures summarised under profiles/; configs without a capture of the current kernel report None.  The largest
# configuration holds too much memory for a capture: its figure is that of its first 256 users (2 615 303 936 bytes
# for 2 590 486 528 algorithmic) scaled to all 512 by the KV bytes, traffic being proportional to the tokens streamed.
TRAFFIC_BYTES = {"c2_llama2_7b": 1340836608, "c3_llama3_8b_gqa": 3021949696, "c4_long_prompt": 2587209728, "c5_many_user": 5084278250}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", default="c5_many_user", choices=list(wl.CONFIGS))
    ap.add_argument("--users", type=int, default=None,
                    help="only the first N users of the config (for profiler captures that must hold little memory)")
    ap.add_argument("--kernel-only", action="store_true",
                    help="only the fused step and the kernel-alone pass of the chosen config (for profiler captures)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the other configs and the CPU baseline")
    ap.add_argument("--prefill-only", action="store_true", help="run only the prefill measurement (for profiling)")
    ap.add_argument("--bf16-math", default="mma", choices=["mma", "fma"],
                    help="arithmetic of the bf16 kernels: tensor cores (default) or the FMA-pipe comparison arm")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
