#!/usr/bin/env python
"""Benchmark of the Superposed Decoding decode step on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b_k3] [--impl ours|reference]

A "step" is one decode timestep: superposed embedding -> decoder over the shared KV cache -> LM
head + KeepTopK -> k*k n-gram expansion -> selection and gamma.  The timed region is ONE
spd_generate_async(K) launch after a prefill and W warm-up steps, timed with CUDA events on the
launching stream; inputs (13 GB of weights) exceed L2, so nothing is flushed between steps.
With N > 1 (torchrun) every rank serves its own prefix on its own GPU: replicas, no collective
on the data path.  Prints one JSON line on rank 0.
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
import torch

import spd_inputs as si

# dram bytes (read + write) / algorithmic bytes measured by ncu on a 4-layer case of the decode kernel; traffic
# grows in proportion to the layers streamed.  The ratio stands only for the kernel sources it was taken with:
# `traffic` is null once any of them has changed.
TRAFFIC = {"ratio": 1.002, "sources_sha256": "3c1fcbd45d7e9f758b2c92916b647c16bcd76af04cf8b5c4ef89a0e2a56536e4"}
KERNEL_SOURCES = ("spd_kernel.cu", "spd_params.h", "spd_ptx.cuh", "spd_score.cuh", "spd_tail.cuh", "spd_nucleus.cuh", "spd_hash.h")


def kernel_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2405_18400_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def traffic_ratio():
    try:
        return TRAFFIC["ratio"] if TRAFFIC["ratio"] and kernel_sources_sha256() == TRAFFIC["sources_sha256"] else None
    except OSError:
        return None

METRIC = "k-draft tokens/s"
UNIT = "tokens/s"


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def measured_peak_bf16():
    """Dense bf16 peak of a kernel timed alone (the driver's cuBLAS burst figure), TFLOP/s."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


def step_bytes(wl, k, T):
    """Algorithmic bytes one decode step must move: every weight once, norm gains, k embedding rows,
    the KV cache of T positions, one 32-byte sector per table probe."""
    s = wl.shape
    kvb = 2 if wl.kv_dtype == "bf16" else 4
    return (s.step_weight_bytes + 2 * (2 * s.n_layers + 1) * s.d_model + k * s.d_model * 2
            + s.n_layers * 2 * T * s.d_model * kvb + (k + k * k) * len(wl.orders) * 32)


def config_of(wl, k, world, reps):
    """The workload's description, the same in both arms."""
    return {"workload": "%s: %s-shape decoder, prefix %d, k=%d, bs1, n-gram n=%d..%d, %d entries/order" % (
        wl.name, wl.shape.name, wl.prefix_len, k, min(wl.orders), max(wl.orders), wl.retain),
        "l2": "inputs_exceed_l2", "kv_dtype": wl.kv_dtype, "parallelism": "replicas x%d" % world, "reps": reps}


def max_over_ranks(x: float, dev, world: int) -> float:
    """The slowest rank's value (every rank gets it); a plain pass-through for one rank."""
    if world <= 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, k: int, steps: int, ms: float) -> float:
    """Whole-job k-draft tokens per second: every rank advances k drafts by `steps` tokens in `ms`."""
    return world * k * steps / (ms * 1e-3)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 9:
                continue
            try:
                sm.append(float(p[1])); mx.append(float(p[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), p[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def make_inputs(wl, device, rank):
    t0 = time.time()
    weights = si.make_weights(wl.shape, seed=0, device=device)
    log("[bench] weights %.1fs" % (time.time() - t0))
    t0 = time.time()
    tables = si.make_ngram_tables(wl.shape.vocab, wl.zipf_s, wl.stream_len, wl.orders, wl.retain, seed=1, device=device)
    log("[bench] n-gram tables %.1fs (%s entries)" % (time.time() - t0, [int(t["counts"].shape[0]) for t in tables]))
    prefix = si.make_prefix(wl.prefix_kind, wl.prefix_len, wl.shape.vocab, wl.zipf_s, seed=2, tensor_id=rank)
    return weights, tables, prefix


def run_batched(args, wl, P, dev, rank, world, packed, dtabs, k, K, W):
    """B requests stepped together: one pass over the weights per timestep (the paper's remark that batching is
    complementary).  Every request has its own prefix, cache and draft state."""
    B = args.batch
    max_pos = max(192, wl.prefix_len + W + K + 2)
    ctxs, prefixes = [], []
    for r in range(B):
        ctxs.append(P.SpdContext(wl.shape, packed, dtabs, k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, max_pos, wl.kv_dtype))
        prefixes.append(si.make_prefix(wl.prefix_kind, wl.prefix_len, wl.shape.vocab, wl.zipf_s, seed=2, tensor_id=rank * 1000 + r))
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = dev.index
    sampler = ClockSampler(gpu_id)
    ms_list, launches = [], 0
    sampler.start()
    time.sleep(0.3)
    for rep in range(max(1, args.reps)):
        for c, pf in zip(ctxs, prefixes):
            c.spd_prefill(pf)
        P.spd_batch_generate(ctxs, W)
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()
        l0 = ctxs[0].spd_launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        P.spd_batch_generate(ctxs, K)
        e1.record()
        torch.cuda.synchronize()
        launches = ctxs[0].spd_launch_count() - l0
        ms_list.append(e0.elapsed_time(e1))
    time.sleep(0.2)
    clocks = sampler.stop()
    ms = max_over_ranks(float(np.median(ms_list)), dev, world)
    s = wl.shape
    T_mid = wl.prefix_len + W + (K + 1) // 2
    kvb = 2 if wl.kv_dtype == "bf16" else 4
    per_request = k * s.d_model * 2 + s.n_layers * 2 * T_mid * s.d_model * kvb + (k + k * k) * len(wl.orders) * 32
    bytes_step = s.step_weight_bytes + 2 * (2 * s.n_layers + 1) * s.d_model + B * per_request
    peak, peak_kind = measured_peak_gbs()
    achieved = bytes_step * K / (ms * 1e-3) / 1e9
    # end to end: host ids in, ids / parents / gamma of every request out, per timestep
    e2e = None
    if not args.no_e2e:
        gen = wl.gen_tokens
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for c, pf in zip(ctxs, prefixes):
            c.spd_prefill(pf)
        for _ in range(gen - 1):
            P.spd_batch_step(ctxs)
        dt = max_over_ranks(time.perf_counter() - t0, dev, world)
        e2e = {"value": world * B * k * gen / dt, "unit": UNIT, "h2d_bytes_per_step": 4.0 * wl.prefix_len * B / gen,
               "d2h_bytes_per_step": 12.0 * k * B, "ms_per_request_batch": dt * 1e3,
               "what": "%d x spd_prefill(host ids), then %d spd_batch_step calls returning every request's ids, parents and gamma "
                       "to the host" % (B, gen - 1)}
    cfg = config_of(wl, k, world, max(1, args.reps))
    cfg["workload"] = cfg["workload"].replace("bs1", "bs%d (batched timesteps, one pass over the weights per step)" % B)
    out = {"metric": METRIC, "value": job_throughput(world, k * B, K, ms), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
           "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": cfg,
           "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "traffic": None,
                        "peak_kind": peak_kind, "bytes_per_step": bytes_step, "kernel": "spd_batch_gemm_kernel",
                        "note": "weights once per timestep + per request its KV cache, embedding rows and table probes; the time is "
                                "the whole timestep's (the products are about 70 % of it)"},
           "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "batch": B}
    for c in ctxs:
        c.close()
    if rank == 0:
        print(json.dumps(out), flush=True)


def run_ours(args, wl):
    import paper_2405_18400_b200 as P

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    P.load_library()
    k, K, W = args.k or wl.k, args.steps, args.warmup
    weights, tables, prefix = make_inputs(wl, dev, rank)
    host_weights = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        t0 = time.time()
        host_weights = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
        log("[bench] weights to host %.1fs" % (time.time() - t0))
    t0 = time.time()
    packed = P.pack_weights(weights, dev, consume=True, images=not args.no_images)
    del weights
    dtabs = P.build_ngram_tables(tables, dev)
    torch.cuda.empty_cache()
    log("[bench] pack + table build %.1fs" % (time.time() - t0))
    if args.batch > 1:
        run_batched(args, wl, P, dev, rank, world, packed, dtabs, k, K, W)
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return
    max_pos = max(wl.max_pos, wl.prefix_len + W + K + 2)
    ctx = P.SpdContext(wl.shape, packed, dtabs, k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, max_pos, wl.kv_dtype)
    if args.stage_bytes or args.stages:
        ctx.spd_set_ring(args.stage_bytes, args.stages)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident throughput: one launch of K steps
    ctx.spd_prefill(prefix)
    ctx.spd_generate_async(W)
    ctx.spd_sync()
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = local
    sampler = ClockSampler(gpu_id)
    reps = max(1, args.reps)
    ms_list = []
    sampler.start()
    time.sleep(0.3)
    launches0 = ctx.spd_launch_count()
    for rep in range(reps):
        if rep:
            ctx.spd_prefill(prefix)
            ctx.spd_generate_async(W)
            ctx.spd_sync()
            launches0 = ctx.spd_launch_count()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.spd_generate_async(K)
        e1.record()
        ctx.spd_sync()
        barrier()
        ms_list.append(e0.elapsed_time(e1))
    launches = ctx.spd_launch_count() - launches0
    time.sleep(0.2)
    clocks = sampler.stop()
    ms = max_over_ranks(float(np.median(ms_list)), dev, world)
    T_mid = wl.prefix_len + W + (K + 1) // 2
    bytes_step = step_bytes(wl, k, T_mid)
    peak, peak_kind = measured_peak_gbs()
    achieved = bytes_step * K / (ms * 1e-3) / 1e9
    value = job_throughput(world, k, K, ms)

    # ---- end to end through the C ABI with host buffers: prefill(host ids) + per-step calls returning to the host
    gen = wl.gen_tokens
    e2e_t, first_t = [], []
    for _ in range(0 if args.no_e2e else 2):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ctx.spd_prefill(prefix)
        first_t.append(time.perf_counter() - t0)
        for _ in range(gen - 1):
            ctx.spd_step()
        e2e_t.append(time.perf_counter() - t0)
    e2e_s = min(e2e_t) if e2e_t else None
    if e2e_s:
        e2e_s = max_over_ranks(e2e_s, dev, world)
    e2e = {"value": world * k * gen / e2e_s if e2e_s else None, "unit": UNIT, "h2d_bytes_per_step": 4.0 * wl.prefix_len / gen,
           "d2h_bytes_per_step": 12.0 * k, "what": "spd_prefill(host ids) + %d spd_step calls returning ids, parents and gamma "
           "to the host, per request of %d tokens per draft; prefill = one launch of the batched kernel per 16 prefix tokens, the last one ending with the LM head and the first timestep; "
           "prefixes over 32 tokens send all but their last 1..16 tokens through the tcgen05 long-prefix path" % (gen - 1, gen),
           "ms_per_request": e2e_s * 1e3 if e2e_s else None,
           "ms_to_first_drafts": min(first_t) * 1e3 if first_t else None}

    # ---- long prefixes: the prefill alone, device-timed, against the tensor roofline of its tcgen05 products
    prefill_rec = None
    if wl.prefix_len > 64 and not args.no_e2e:
        ts = []
        for _ in range(3):
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.spd_prefill(prefix)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        pf_ms = max_over_ranks(float(np.median(ts)), dev, world)
        n_tc = wl.prefix_len - ((wl.prefix_len - 1) % 16 + 1)
        sh = wl.shape
        layer_params = sh.n_layers * (4 * sh.d_model * sh.d_model + 3 * sh.d_model * sh.d_ffn)
        tflop = n_tc * layer_params * 2 / 1e12           # the method's own arithmetic: tokens x weights x 2
        tpeak, tkind = measured_peak_bf16()
        prefill_rec = {"ms": pf_ms, "tokens": wl.prefix_len, "tokens_through_tcgen05_products": n_tc, "bound": "tensor",
                       "achieved": tflop / (pf_ms * 1e-3), "peak": tpeak, "unit": "TFLOP/s", "frac": tflop / (pf_ms * 1e-3) / tpeak,
                       "peak_kind": tkind, "issued_tflops": 3 * tflop / (pf_ms * 1e-3), "issued_frac": 3 * tflop / (pf_ms * 1e-3) / tpeak,
                       "note": "whole spd_prefill call (products, attention, row-wise kernels, the last tokens' launch of the 16-token "
                               "kernel with LM head and first timestep); achieved / frac count the method's arithmetic (tokens x layer "
                               "weights x 2); issued_* count what the tensor cores execute, three bf16 terms per float32 activation"}

    # ---- the same number of drafts from k separate single-draft passes through the same kernels
    kpass = None
    if rank == 0 and not args.no_kpass and k > 1:
        c1 = P.SpdContext(wl.shape, packed, dtabs, 1, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, max_pos, wl.kv_dtype)
        c1.spd_prefill(prefix)
        c1.spd_generate_async(W)
        c1.spd_sync()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        c1.spd_generate_async(K)
        e1.record()
        c1.spd_sync()
        one = e0.elapsed_time(e1)
        kpass = {"ms_per_step_single_draft": one / K, "ms_per_step_k_passes": k * one / K, "ms_per_step_spd": ms / K,
                 "saving": k * one / ms, "note": "k sequential batch-1 passes (k=1 contexts, own KV cache) vs one superposed pass"}
        if e2e_s:
            # the paper's latency comparison (Section 4.3): k nucleus-sampled generations against one SPD request
            u = np.linspace(0.05, 0.95, gen - 1).astype(np.float32)
            ns_t = []
            for _ in range(2):
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                c1.spd_prefill(prefix)
                c1.spd_sample(u, 0.9, 1.0)
                ns_t.append(time.perf_counter() - t0)
            kpass.update({"nucleus_ms_per_request": min(ns_t) * 1e3, "nucleus_k_requests_ms": k * min(ns_t) * 1e3,
                          "spd_ms_per_request": e2e_s * 1e3, "request_saving": k * min(ns_t) / e2e_s,
                          "nucleus_note": "prefill + %d nucleus-sampled passes (top-p 0.9, T 1) through spd_sample, host to "
                                          "host; the draw of the last token (no pass) is not run; a sampled pass costs about 8 %% more than a "
                                          "decode step of one draft (the draw runs on one block while the others wait)" % (gen - 1)})
        c1.close()

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": config_of(wl, k, world, reps),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic_ratio() * bytes_step * K if traffic_ratio() else None, "peak_kind": peak_kind,
                     "bytes_per_step": bytes_step, "kernel": "spd_decode_img_kernel" if "lm_head_img" in packed else "spd_decode_kernel"},
        "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
    }
    if kpass:
        out["k_pass"] = kpass
    if prefill_rec:
        out["prefill"] = prefill_rec
    ctx.close()

    if rank == 0 and host_weights is not None:
        out["cpu_baseline"] = cpu_baseline(wl, k, host_weights, tables, prefix, args.cpu_steps)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def cpu_baseline(wl, k, host_weights, tables, prefix, n_steps):
    """The oracle as it stands on the host cores: n_steps decode steps after an untimed prefill."""
    from oracle import spd_oracle as so

    cfg = so.make_config(wl.shape, k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, wl.prefix_len + n_steps + 2,
                         wl.kv_dtype)
    orc = so.Oracle(cfg, host_weights, tables)
    t0 = time.time()
    orc.prefill(prefix)
    log("[bench] oracle prefill %.1fs" % (time.time() - t0))
    t0 = time.perf_counter()
    for _ in range(n_steps):
        orc.step()
    dt = time.perf_counter() - t0
    orc.close()
    return {"value": k * n_steps / dt, "unit": UNIT, "cores": so.max_threads(), "kind": "oracle",
            "ms_per_step": dt / n_steps * 1e3,
            "sample": "%d decode steps of the same workload after an untimed %d-token prefill" % (n_steps, wl.prefix_len)}


def run_reference(args, wl):
    """The CPU oracle timed on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import spd_oracle as so

    k, K, W = args.k or wl.k, args.steps, args.warmup
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    weights, tables, prefix = make_inputs(wl, dev, 0)
    host = {n: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for n, v in weights.items()}
    del weights
    cfg = so.make_config(wl.shape, k, wl.orders, wl.lambdas(), wl.alpha, wl.tau, wl.delta, wl.prefix_len + W + K + 2, wl.kv_dtype)
    orc = so.Oracle(cfg, host, tables)
    orc.prefill(prefix)
    t1 = time.perf_counter()
    for _ in range(W):
        orc.step()
    per = (time.perf_counter() - t1) / max(1, W)
    K_run = K if W == 0 else max(1, min(K, int(150.0 / max(per, 1e-9))))
    t0 = time.perf_counter()
    for _ in range(K_run):
        orc.step()
    dt = time.perf_counter() - t0
    value = k * K_run / dt
    cores = so.max_threads()
    sample = "%d decode steps (of %d asked) after an untimed %d-token prefill and %d warm-up steps" % (K_run, K, wl.prefix_len, W)
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1, "steps": K_run, "warmup": W,
           "ms_per_step": dt / K_run * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
           "data": "synthetic",
           "config": config_of(wl, k, 1, args.reps),
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=9)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="7b_k3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--k", type=int, default=0, help="override the number of drafts")
    ap.add_argument("--reps", type=int, default=5, help="timed launches (median reported)")
    ap.add_argument("--cpu-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kpass", action="store_true")
    ap.add_argument("--stage-bytes", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0, help="profiling only: keep this many layers of the shape")
    ap.add_argument("--retain", type=int, default=0, help="profiling only: n-grams kept per order")
    ap.add_argument("--stream-len", type=int, default=0, help="profiling only: tokens of the n-gram corpus")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-images", action="store_true",
                    help="comparison only: no fragment-order weight images, decode timesteps on the float32 multiply loop")
    ap.add_argument("--batch", type=int, default=1, help="requests stepped together (batched timesteps); 1 = the single-request kernel")
    args = ap.parse_args()
    if args.warmup < 1:
        args.warmup = 1
    wl = si.get_workload(args.workload)
    if args.layers or args.retain or args.stream_len:
        import dataclasses
        sh = wl.shape
        if args.layers:
            sh = dataclasses.replace(sh, n_layers=args.layers, name="%s[%d layers]" % (sh.name, args.layers))
        wl = dataclasses.replace(wl, shape=sh, retain=args.retain or wl.retain, stream_len=args.stream_len or wl.stream_len,
                                 name=wl.name + "-reduced")
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
        run_ours(args, wl)


if __name__ == "__main__":
    main()
