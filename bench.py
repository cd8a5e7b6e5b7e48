#!/usr/bin/env python
"""Benchmark of the path-attention hot path.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One step = one pass of the decode hot path over one batch of the synthetic workload:
gf_build_path_tables (K1) followed by gf_path_attention_decode (K2 + K4) for every layer of the
configuration.  The headline workload is configuration 4, the largest that fits one GPU (32 layers,
2048 decode requests over a 4096-node wGraph: table build plus all 32 layers' attention).  Without
--config the same JSON line also carries, under "configs", one sub-record each for configuration 1
(Llama-3-8B-shaped single layer, 256 requests), configuration 3 (1024 requests on one 8192-token
root) and configuration 2 (extend: 64 requests x 512 new tokens, tensor roofline), timed the same
way.  --config C times configuration C alone.  With N > 1 (torchrun) every rank runs an independent
replica on its own GPU: the path does not shard, no collective is on the data path.

Prints ONE JSON line.  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "path_attention_decode_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
NCU_TRAFFIC_PRUNE = 138.8e6  # bytes per k_transition_counts launch of bench.py --pruning (134.2 MB read + 4.6 MB written)
NCU_TRAFFIC_RECON = 278.6e6  # bytes per k_kv_reconstruct launch of bench.py --residual (181.6 MB read + 97.0 MB written)
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per decode launch from an ncu capture, keyed by
# configuration, each with the digest of the decode kernels' sources it was taken with: a capture says
# nothing about a kernel that has changed since, so the bench reports null when the digest differs.
# Config 4's figure comes from the capture with two layers held (each layer is a full-size launch).  Per layer:
# config 1: k_decode 740.3 MB read + 34.4 written; config 3: k_decode 1522.3 + 95.0, k_path_tc 50.0 + 5.3;
# config 4: k_decode 5266.4 + 129.0, k_path_tc 52.5 + 4.6.
NCU_TRAFFIC_DECODE = {1: (774.7e6, "e7be67436ca80d84"), 3: (1672.6e6, "e7be67436ca80d84"), 4: (5452.5e6, "e7be67436ca80d84")}
# The same for one k_path_tc<extend> launch of config 2 (560.5 MB read + 240.8 MB written).
NCU_TRAFFIC_EXTEND = {2: (801.3e6, "e7be67436ca80d84")}
DECODE_SOURCES = ("decode.cu", "attn_core.cuh", "extend_tc.cu", "tc_device.cuh", "gf_device.cuh")


def decode_sources_digest() -> str:
    h = hashlib.sha256()
    for name in DECODE_SOURCES:
        with open(os.path.join(ROOT, "paper_2605_22566_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return d, "measured"
        except Exception:
            pass
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (reads only) while a timed region runs."""

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
                 "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80)}
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self, histogram: bool = False):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2.0)
        med = float(np.median(self.samples)) if self.samples else None
        out = {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
               "samples": len(self.samples)}
        if histogram and self.samples:
            vals, cnt = np.unique(np.asarray(self.samples), return_counts=True)
            out["sm_mhz_histogram"] = {str(int(v)): int(c) for v, c in zip(vals, cnt)}
        return out


def max_over_ranks(value_ms: float, dist, device) -> float:
    """The step time of the job is the slowest rank's: MAX all-reduce (no-op for one process)."""
    if dist is None:
        return float(value_ms)
    import torch
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(units_per_rank_step: float, steps: int, world: int, total_ms: float) -> float:
    """Whole-job throughput of N independent replicas: units all ranks processed / slowest rank's time."""
    return units_per_rank_step * steps * world / (total_ms * 1e-3)


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------
def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


_KV_CACHE = {}


def oracle_decode_sample(w, n_req: int, layer: int = 0):
    """Times the oracle, as it stands, on n_req requests of the workload (one layer): the first n_req,
    or, where the workload has far more requests than that, n_req spread evenly over the batch.
    Returns (seconds, requests).  Input generation happens before the clock starts."""
    from oracle import attention as OA
    from paper_2605_22566_b200 import workloads as W
    cache = _KV_CACHE.setdefault((w.config_id, w.seed, layer), {})

    def node_kv(v):
        if v not in cache:
            k, vv = w.node_kv_bits(layer, v)
            cache[v] = (W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(vv))
        return cache[v]
    n_req = min(n_req, w.num_requests)
    reqs = list(range(n_req))
    paths = [[v for v in w.path(r).tolist() if w.node_len[v] > 0] for r in reqs]
    for p in paths:
        for v in p:
            node_kv(v)
    q = W.bf16_bits_to_f64(w.q_bits(layer, 0, len(reqs)))
    t0 = time.perf_counter()
    OA.decode(paths, node_kv, q, w.num_kv_heads)
    return time.perf_counter() - t0, len(reqs)


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the headline workload's shape.  The metric is
    decode tokens per second of a whole step (all layers of the configuration), so the oracle's rate on
    one layer is divided by the number of layers."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_22566_b200 import workloads as W
    cfg = 4 if args.config is None else args.config
    w = W.make_config(cfg)
    if w.mode != "decode":
        t, n, fl = oracle_extend_sample(w, args.oracle_rows)
        value = fl / t / 1e12
        line = {"impl": "reference", "metric": "path_attention_extend_tflops", "value": value, "unit": "TFLOP/s",
                "n_gpus": args.gpus, "steps": 1, "warmup": 0, "ms_per_step": 1e3 * t, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": workload_config(w, args),
                "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle",
                                 "sample": f"{n} seeded query rows x {w.num_q_heads} heads, 1 layer, {t:.1f} s"},
                "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return
    layers = w.num_layers if args.layers is None else args.layers
    # size the per-step sample from a short probe so that K steps take about two minutes
    t_probe, r_probe = oracle_decode_sample(w, 2)
    per_req = t_probe / r_probe
    n_req = max(1, min(w.num_requests, args.oracle_requests or w.num_requests, int(120.0 / max(args.steps, 1) / per_req)))
    for _ in range(min(args.warmup, 2)):
        oracle_decode_sample(w, n_req)
    total_t, total_r = 0.0, 0
    for _ in range(args.steps):
        t, r = oracle_decode_sample(w, n_req)
        total_t += t
        total_r += r
    value = total_r / total_t / layers
    sample = (f"first {n_req} of {w.num_requests} requests, 1 of {layers} layers per step "
              f"(rate divided by {layers}: a step of the metric covers every layer); per request the oracle "
              "concatenates the path's K/V and applies fp64 softmax attention")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": workload_config(w, args),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(w, args, layers=None):
    """The `config` object: identical for the GPU arm and the reference arm of one workload."""
    if layers is None:
        layers = w.num_layers if getattr(args, "layers", None) is None else args.layers
    kv_mb = w.resident_tokens() * w.kv_bytes_per_token() / 1e6
    step = ("gf_build_path_tables (extend) + gf_path_attention_extend per layer" if w.mode == "extend" else
            "gf_build_path_tables + gf_path_attention_decode per layer")
    return {"workload": f"config {w.config_id}: {w.name}", "requests": w.num_requests,
            "layers_timed": layers, "kv_layer_copies": min(layers, args.phys_layers), "q_heads": w.num_q_heads,
            "kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "wgraph_nodes": w.num_shared_nodes, "step": step,
            "l2": f"KV inputs ({kv_mb:.0f} MB per layer) exceed the 126 MB L2; a 512 MB buffer is also rewritten between timed steps",
            "parallelism": "replicas" if args.gpus > 1 else "single-gpu", "seed": w.seed}


# ------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------
class Env:
    """Process-wide state of the GPU arm: rank, device, process group."""

    def __init__(self):
        import torch
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.dist = None
        torch.cuda.set_device(self.local_rank)
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{self.local_rank}"))
            self.dist = dist
        self.dev = f"cuda:{self.local_rank}"
        self.flush = torch.empty(512 << 20, dtype=torch.uint8, device=self.dev)

    def barrier(self):
        import torch
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def decode_record(env, args, w, steps, warmup, sustained_s=0.0, cpu_baseline=True):
    """Times the decode step of one workload; returns the record (rank 0) or None (other ranks)."""
    import torch
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention

    dev, dist, rank, world = env.dev, env.dist, env.rank, env.world
    layers = w.num_layers if args.layers is None else min(args.layers, w.num_layers)
    # Physical layer copies of the KV pool: configuration 4's 32 layers do not fit one GPU, so layer l
    # reads copy l % phys (each copy is far larger than L2, so the bytes streamed are unchanged).
    phys = min(layers, args.phys_layers)
    policy = tuple(args.policy) if args.policy else None
    pa = PathAttention(w, device=dev, layers=phys, policy=policy)
    pa.write_nodes("device")
    q_dev = [pa.make_q(l) for l in range(layers)]
    out_dev = torch.empty_like(q_dev[0])
    flush = env.flush
    stream = torch.cuda.current_stream()

    def step():
        pa.build(deferred=True)  # nothing on the path waits for the host
        for l in range(layers):
            pa.decode(l % phys, q_dev[l], out=out_dev)

    warmup = max(warmup, 3)
    for _ in range(warmup):
        step()
    info = pa.build()
    assert pa.status() == 0

    # ---- timed region: K steps, device-timed, L2 flushed between steps -------------------
    B.gf_profile_enable(pa.g, True)
    B.gf_profile_read(pa.g)
    sampler = ClockSampler(visible_gpu_index(env.local_rank)) if rank == 0 else None
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    launches0 = B.gf_launch_count(pa.g)
    env.barrier()
    if sampler:
        sampler.start()
    wall0 = time.perf_counter()
    for a, b in evs:
        flush.fill_(1)
        a.record(stream)
        step()
        b.record(stream)
    env.barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.finish() if sampler else None
    launches = B.gf_launch_count(pa.g) - launches0
    prof = B.gf_profile_read(pa.g)
    assert pa.status() == 0
    step_ms = np.array([a.elapsed_time(b) for a, b in evs])
    total_ms = max_over_ranks(float(step_ms.sum()), dist, dev)

    # ---- sustained leg: the same step back to back for at least sustained_s seconds, clocks binned ----
    sustained = None
    if sustained_s > 0:
        n_sus = max(steps, int(np.ceil(sustained_s * 1e3 / max(float(step_ms.mean()), 1e-3))))
        sampler = ClockSampler(visible_gpu_index(env.local_rank)) if rank == 0 else None
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        env.barrier()
        if sampler:
            sampler.start()
        ea.record(stream)
        for _ in range(n_sus):
            step()
        eb.record(stream)
        env.barrier()
        sus_clocks = sampler.finish(histogram=True) if sampler else None
        sus_prof = B.gf_profile_read(pa.g)
        sus_ms = max_over_ranks(ea.elapsed_time(eb), dist, dev)
        assert pa.status() == 0
        sustained = {"steps": n_sus, "seconds": sus_ms * 1e-3, "ms_per_step": sus_ms / n_sus,
                     "value": replica_throughput(w.num_requests, n_sus, world, sus_ms), "unit": UNIT,
                     "decode_K2_ms_per_layer": sus_prof.decode_ms / max(n_sus * layers, 1),
                     "l2": "no flush between steps: every layer's KV exceeds the L2", "clocks": sus_clocks}
    B.gf_profile_enable(pa.g, False)

    # ---- end to end through the C ABI with host buffers ---------------------------------
    h_ptr = torch.from_numpy(w.path_ptr.astype(np.int32)).pin_memory()
    h_node = torch.from_numpy(w.path_node.astype(np.int32)).pin_memory()
    h_q = [q.cpu().pin_memory() for q in q_dev]
    h_out = torch.empty(q_dev[0].shape, dtype=torch.bfloat16).pin_memory()
    d_q = [torch.empty_like(q_dev[0]) for _ in range(2)]
    e2e_steps = max(3, min(steps, 50))
    # the queries of layer l + 1 travel on a second stream while the tables are built / layer l is computed,
    # and the output of layer l - 1 goes back on a third (two output buffers), so that only the first upload
    # and the last download of a step are not hidden behind a layer's kernels
    copy_stream = torch.cuda.Stream(device=dev)
    back_stream = torch.cuda.Stream(device=dev)
    q_ready = [torch.cuda.Event() for _ in range(2)]
    q_free = [torch.cuda.Event() for _ in range(2)]
    out_bufs = [out_dev, torch.empty_like(out_dev)]
    out_ready = [torch.cuda.Event() for _ in range(2)]
    out_free = [torch.cuda.Event() for _ in range(2)]

    def send_q(l):
        b = l & 1
        with torch.cuda.stream(copy_stream):
            if l >= 2:
                copy_stream.wait_event(q_free[b])  # the layer that last read this buffer is done
            d_q[b].copy_(h_q[l], non_blocking=True)
            q_ready[b].record(copy_stream)

    issued = [0]
    # A one-layer step shorter than the host's own work per step (a dozen calls through ctypes) gains nothing from
    # side streams: their event calls only add to what the host has to issue.
    one_stream = layers == 1 and total_ms / steps < 0.35

    def e2e_step():
        if one_stream:
            pa.path_ptr.copy_(h_ptr, non_blocking=True)
            pa.path_node.copy_(h_node, non_blocking=True)
            pa.build(deferred=True)
            d_q[0].copy_(h_q[0], non_blocking=True)
            pa.decode(0, d_q[0], out=out_dev)
            h_out.copy_(out_dev, non_blocking=True)
            stream.synchronize()
            return
        if layers == 1:
            # one layer per step: steps are issued back to back, the next step's queries go up and the previous
            # step's outputs come down on the two side streams while this step's kernels run
            i = issued[0]
            b = i & 1
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(q_free[b])
                d_q[b].copy_(h_q[0], non_blocking=True)
                q_ready[b].record(copy_stream)
            pa.path_ptr.copy_(h_ptr, non_blocking=True)
            pa.path_node.copy_(h_node, non_blocking=True)
            pa.build(deferred=True)
            stream.wait_event(q_ready[b])
            if i >= 2:
                stream.wait_event(out_free[b])
            pa.decode(0, d_q[b], out=out_bufs[b])
            q_free[b].record(stream)
            out_ready[b].record(stream)
            with torch.cuda.stream(back_stream):
                back_stream.wait_event(out_ready[b])
                h_out.copy_(out_bufs[b], non_blocking=True)
                out_free[b].record(back_stream)
            issued[0] = i + 1
            return
        send_q(0)
        pa.path_ptr.copy_(h_ptr, non_blocking=True)
        pa.path_node.copy_(h_node, non_blocking=True)
        pa.build(deferred=True)
        for l in range(layers):
            b = l & 1
            if l + 1 < layers:
                send_q(l + 1)
            stream.wait_event(q_ready[b])
            if l >= 2:
                stream.wait_event(out_free[b])  # the download that last read this buffer is done
            pa.decode(l % phys, d_q[b], out=out_bufs[b])
            q_free[b].record(stream)
            out_ready[b].record(stream)
            with torch.cuda.stream(back_stream):
                back_stream.wait_event(out_ready[b])
                h_out.copy_(out_bufs[b], non_blocking=True)
                out_free[b].record(back_stream)
        stream.synchronize()
        copy_stream.synchronize()
        back_stream.synchronize()

    def drain():
        stream.synchronize()
        copy_stream.synchronize()
        back_stream.synchronize()

    for _ in range(3):
        e2e_step()
    drain()
    env.barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    if layers == 1 and not one_stream:
        stream.wait_event(out_free[(issued[0] - 1) & 1])  # the last download ends inside the timed region
    eb.record(stream)
    drain()
    env.barrier()
    e2e_ms = max_over_ranks(ea.elapsed_time(eb), dist, dev)
    h2d = (h_ptr.numel() + h_node.numel()) * 4 + sum(x.numel() * 2 for x in h_q)
    d2h = h_out.numel() * 2 * layers
    assert pa.status() == 0
    pa.close()
    del pa, q_dev, d_q, out_dev, out_bufs
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    peaks, peak_kind = measured_peaks()
    R = w.num_requests
    value = replica_throughput(R, steps, world, total_ms)
    # algorithmic bytes of one decode launch: every resident K/V token once, Q in, out written
    btok = w.kv_bytes_per_token()
    alg_bytes = btok * info.resident_tokens + 2 * R * w.num_q_heads * w.head_dim * 2
    dec_ms = prof.decode_ms / max(steps * layers, 1)  # per layer: the decode kernels of one gf_path_attention_decode
    mrg_ms = prof.merge_ms / max(prof.merge_launches, 1)
    tab_ms = prof.tables_ms / max(steps, 1)
    step_ms_mean = total_ms / steps
    achieved = alg_bytes / (dec_ms * 1e-3) / 1e9
    peak = float(peaks["hbm_gbs"])
    traffic = args.traffic
    if traffic is None and policy is None:
        known = NCU_TRAFFIC_DECODE.get(w.config_id)
        if known is not None and known[1] == decode_sources_digest():
            traffic = known[0]

    def frac3(ms):  # algorithmic bytes of all timed layers over a time: GB/s and the two fractions
        gbs = alg_bytes * layers / (ms * 1e-3) / 1e9
        return {"gbs": gbs, "frac_of_measured": gbs / peak, "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}
    rec = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": step_ms_mean, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, args, layers), "clocks": clocks,
        "e2e": {"value": R * e2e_steps * world / (e2e_ms * 1e-3), "unit": UNIT,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": e2e_steps,
                "overlap": ("one stream, a host synchronisation per step" if one_stream else
                            "steps back to back; uploads and downloads on their own streams, two buffers each" if layers == 1 else
                            "per layer: next queries up and previous outputs down on their own streams, two buffers each")},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "K2: the decode kernels of one layer (k_decode, plus k_path_tc<decode> when chunks are widely shared)",
                     "bound": "hbm", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_source": f"{peak_kind} copy bandwidth",
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "traffic": traffic,
                     "algorithmic_bytes_per_launch": int(alg_bytes), "kernel_ms": dec_ms},
        # decode read three ways: K2 alone (the roofline object), K2 + K4 (decode as a whole), the whole step
        "decode_fracs": {"K2": frac3(dec_ms * layers), "K2_plus_K4": frac3((dec_ms + mrg_ms) * layers),
                         "whole_step": frac3(step_ms_mean)},
        "breakdown_us_per_step": {"tables_K1": 1e3 * tab_ms, "decode_K2": 1e3 * dec_ms * layers,
                                  "merge_K4": 1e3 * mrg_ms * layers, "step_total": 1e3 * step_ms_mean},
        "kv": {"resident_tokens": int(info.resident_tokens), "materialised_tokens": int(info.materialised_tokens),
               "resident_bytes_per_layer": int(info.resident_tokens * btok),
               "materialised_bytes_per_layer": int(info.materialised_tokens * btok),
               "ratio": info.materialised_tokens / max(info.resident_tokens, 1),
               "segments": info.num_segments, "items": info.num_items, "partial_slots": info.num_slots},
        "wall_s_timed_region": wall,
    }
    if sustained is not None:
        sustained["decode_K2_frac_of_measured"] = alg_bytes / (sustained["decode_K2_ms_per_layer"] * 1e-3) / 1e9 / peak
        rec["sustained"] = sustained
    if world == 1 and cpu_baseline and not args.no_cpu_baseline:
        n_req = args.oracle_requests
        if n_req is None:  # a sample of about ten seconds, sized from a short probe
            t_probe, r_probe = oracle_decode_sample(w, 4)
            n_req = int(max(4, min(R, 10.0 / (t_probe / r_probe))))
        t, r = oracle_decode_sample(w, n_req)
        rec["cpu_baseline"] = {"value": r / t / layers, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                               "sample": f"first {r} of {R} requests, 1 of {layers} layers, {t:.1f} s"
                                         + (f" (rate divided by {layers}: a step covers every layer)" if layers > 1 else "")}
    else:
        rec["cpu_baseline"] = None
    return rec


def extend_flops(w) -> float:
    """Causal-visible flops of one layer: 4*D*Hq * sum_r (T_r*P_r + T_r*(T_r+1)/2)."""
    T = w.q_rows_per_request().astype(np.float64)
    P = w.request_len().astype(np.float64) - T
    return float(4.0 * w.head_dim * w.num_q_heads * (T * P + T * (T + 1) / 2).sum())


def oracle_extend_sample(w, n_rows: int, layer: int = 0):
    """Times the oracle, as it stands, on n_rows seeded query rows (all heads) of the workload."""
    from oracle import attention as OA
    from paper_2605_22566_b200 import workloads as W
    cache = _KV_CACHE.setdefault((w.config_id, w.seed, layer), {})

    def node_kv(v):
        if v not in cache:
            k, vv = w.node_kv_bits(layer, v)
            cache[v] = (W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(vv))
        return cache[v]
    qp = w.q_row_ptr()
    total = int(qp[-1])
    rows = sorted(np.random.default_rng(3).choice(total, size=min(n_rows, total), replace=False).tolist())
    paths = [[v for v in w.path(r).tolist() if w.node_len[v] > 0] for r in range(w.num_requests)]
    reqs = sorted({int(np.searchsorted(qp, x, side="right") - 1) for x in rows})
    for r in reqs:
        for v in paths[r]:
            node_kv(v)
    # rows of other requests are never touched by the oracle; give it zeros there
    q = np.zeros((total, w.num_q_heads, w.head_dim), dtype=np.float64)
    for x in rows:
        q[x] = W.bf16_bits_to_f64(w.q_bits(layer, x, 1))[0]
    req_len = w.request_len()
    flops = 0.0
    for x in rows:
        r = int(np.searchsorted(qp, x, side="right") - 1)
        i = x - int(qp[r])
        T = int(qp[r + 1] - qp[r])
        flops += 4.0 * w.head_dim * w.num_q_heads * (int(req_len[r]) - T + i + 1)
    t0 = time.perf_counter()
    OA.extend(paths, node_kv, q, w.num_kv_heads, rows=rows)
    return time.perf_counter() - t0, len(rows), flops


def extend_record(env, args, w, steps, warmup, cpu_baseline=True):
    """Extend / prefill step: gf_build_path_tables (extend mode) + gf_path_attention_extend per layer."""
    import torch
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention

    dev, dist, rank, world = env.dev, env.dist, env.rank, env.world
    layers = w.num_layers if args.layers is None else min(args.layers, w.num_layers)
    pa = PathAttention(w, device=dev, layers=layers)
    pa.write_nodes("device")
    q_dev = [pa.make_q(l) for l in range(layers)]
    out_dev = torch.empty_like(q_dev[0])
    flush = env.flush
    stream = torch.cuda.current_stream()

    def step():
        pa.build()
        for l in range(layers):
            pa.extend(l, q_dev[l], out=out_dev)

    warmup = max(warmup, 3)
    for _ in range(warmup):
        step()
    info = pa.build()
    assert pa.status() == 0
    B.gf_profile_enable(pa.g, True)
    B.gf_profile_read(pa.g)
    sampler = ClockSampler(visible_gpu_index(env.local_rank)) if rank == 0 else None
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    launches0 = B.gf_launch_count(pa.g)
    env.barrier()
    if sampler:
        sampler.start()
    wall0 = time.perf_counter()
    for a, b in evs:
        flush.fill_(1)
        a.record(stream)
        step()
        b.record(stream)
    env.barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.finish(histogram=True) if sampler else None
    launches = B.gf_launch_count(pa.g) - launches0
    prof = B.gf_profile_read(pa.g)
    B.gf_profile_enable(pa.g, False)
    assert pa.status() == 0
    total_ms = max_over_ranks(float(sum(a.elapsed_time(b) for a, b in evs)), dist, dev)

    # The on-the-fly branch end to end (Sec. 5.2): the new segments' K/V arrive in the caller layout
    # every step.  Timed twice: a gf_node_kv_write per request ahead of gf_path_attention_extend, and
    # gf_path_attention_extend_append, which writes them inside the attention launch.
    qp = w.q_row_ptr()
    new_nodes = pa.new_nodes()
    k_new = torch.empty((int(qp[-1]), w.num_kv_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    v_new = torch.empty_like(k_new)
    for r, v in enumerate(new_nodes):
        B.check(B.gf_node_kv_read(pa.g, v, 0, k_new[int(qp[r]):].data_ptr(), v_new[int(qp[r]):].data_ptr(), pa.stream),
                "gf_node_kv_read")

    def step_separate():
        pa.build()
        for l in range(layers):
            for r, v in enumerate(new_nodes):
                B.check(B.gf_node_kv_write(pa.g, v, l, k_new[int(qp[r]):].data_ptr(), v_new[int(qp[r]):].data_ptr(),
                                           int(qp[r + 1] - qp[r]), pa.stream), "gf_node_kv_write")
            pa.extend(l, q_dev[l], out=out_dev)

    def step_fused():
        pa.build()
        for l in range(layers):
            pa.extend_append(l, q_dev[l], k_new, v_new, out=out_dev)

    append_ms = {}
    for name, fn in (("separate_write", step_separate), ("fused", step_fused)):
        for _ in range(2):
            fn()
        n_app = max(3, min(steps, 10))
        aev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_app)]
        env.barrier()
        for a, b in aev:
            flush.fill_(1)
            a.record(stream)
            fn()
            b.record(stream)
        env.barrier()
        append_ms[name] = max_over_ranks(float(sum(a.elapsed_time(b) for a, b in aev)), dist, dev) / n_app
    assert pa.status() == 0

    # end to end: paths and queries from pinned host memory, outputs back to the host
    h_ptr = torch.from_numpy(w.path_ptr.astype(np.int32)).pin_memory()
    h_node = torch.from_numpy(w.path_node.astype(np.int32)).pin_memory()
    h_q = [q.cpu().pin_memory() for q in q_dev]
    h_out = torch.empty(q_dev[0].shape, dtype=torch.bfloat16).pin_memory()
    e2e_steps = max(3, min(steps, 20))
    # Steps are issued back to back, as a server with a queue of batches would: the queries of step i + 1 are
    # uploaded (second stream, two buffers) while step i computes, and step i's outputs go back on a third
    # stream (two buffers).  Every step's upload and download lie inside the timed region; only the first
    # upload and the last download are not hidden.
    d_q = [torch.empty_like(q_dev[0]) for _ in range(2)]
    out_bufs = [out_dev, torch.empty_like(out_dev)]
    copy_stream = torch.cuda.Stream(device=dev)
    back_stream = torch.cuda.Stream(device=dev)
    q_ready = [torch.cuda.Event() for _ in range(2)]
    q_free = [torch.cuda.Event() for _ in range(2)]
    out_ready = [torch.cuda.Event() for _ in range(2)]
    out_free = [torch.cuda.Event() for _ in range(2)]
    issued = [0]

    def e2e_step():
        for l in range(layers):
            i = issued[0]
            b = i & 1
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(q_free[b])
                d_q[b].copy_(h_q[l], non_blocking=True)
                q_ready[b].record(copy_stream)
            if l == 0:
                pa.path_ptr.copy_(h_ptr, non_blocking=True)
                pa.path_node.copy_(h_node, non_blocking=True)
                pa.build()
            stream.wait_event(q_ready[b])
            if i >= 2:
                stream.wait_event(out_free[b])
            pa.extend(l, d_q[b], out=out_bufs[b])
            q_free[b].record(stream)
            out_ready[b].record(stream)
            with torch.cuda.stream(back_stream):
                back_stream.wait_event(out_ready[b])
                h_out.copy_(out_bufs[b], non_blocking=True)
                out_free[b].record(back_stream)
            issued[0] = i + 1

    def drain():
        stream.synchronize()
        copy_stream.synchronize()
        back_stream.synchronize()

    for _ in range(2):
        e2e_step()
    drain()
    env.barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    stream.wait_event(out_free[(issued[0] - 1) & 1])  # the last download ends inside the timed region
    eb.record(stream)
    drain()
    env.barrier()
    e2e_ms = max_over_ranks(ea.elapsed_time(eb), dist, dev)
    h2d = int((h_ptr.numel() + h_node.numel()) * 4 + sum(x.numel() * 2 for x in h_q))
    d2h = int(h_out.numel() * 2 * layers)
    pa.close()
    del pa, q_dev, d_q, out_dev, out_bufs
    torch.cuda.empty_cache()
    if rank != 0:
        return None
    peaks, peak_kind = measured_peaks()
    flops = extend_flops(w) * layers
    extend_traffic = args.traffic
    if extend_traffic is None:
        known = NCU_TRAFFIC_EXTEND.get(w.config_id)
        if known is not None and known[1] == decode_sources_digest():
            extend_traffic = known[0]
    # per gf_path_attention_extend call: the extend kernel and the exact variant queued behind it, which
    # leaves at once on inputs of ordinary range
    ext_ms = prof.extend_ms / max(steps * layers, 1)
    achieved = extend_flops(w) / (ext_ms * 1e-3) / 1e12
    # a launch of several ms runs under the power cap: the sustained GEMM figure is the denominator
    peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    rows = int(info.num_q_rows)
    value = flops * steps * world / (total_ms * 1e-3) / 1e12
    btok = w.kv_bytes_per_token()
    rec = {
        "metric": "path_attention_extend_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": total_ms / steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {**workload_config(w, args, layers), "new_tokens": rows,
                   "flops": "causal-visible: 4*D*Hq*sum(T*P + T*(T+1)/2)"},
        "clocks": clocks,
        "e2e": {"value": flops * e2e_steps * world / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                "overlap": "steps back to back; uploads and downloads on their own streams, two buffers each"},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "K3: k_path_tc<extend>", "bound": "tensor", "achieved": achieved, "peak": peak,
                     "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_source": f"{peak_kind} cuBLAS bf16, sustained",
                     "frac_of_measured_burst": achieved / float(peaks["bf16_tflops"]),
                     "frac_of_nominal_2250": achieved / 2250.0, "traffic": extend_traffic,
                     "algorithmic_flops_per_launch": extend_flops(w), "kernel_ms": ext_ms},
        "breakdown_us_per_step": {"tables_K1": 1e3 * prof.tables_ms / max(steps, 1),
                                  "extend_K3": 1e3 * ext_ms * layers, "step_total": 1e3 * total_ms / steps},
        "new_tokens_per_s": rows * steps * world / (total_ms * 1e-3),
        "append_step_ms": {**append_ms, "what": "the step when the new segments' K/V arrive with it: a node write per "
                                               "request ahead of the extend, against the extend that appends them itself"},
        "kv": {"resident_tokens": int(info.resident_tokens), "materialised_tokens": int(info.materialised_tokens),
               "resident_bytes_per_layer": int(info.resident_tokens * btok),
               "materialised_bytes_per_layer": int(info.materialised_tokens * btok),
               "ratio": info.materialised_tokens / max(info.resident_tokens, 1)},
        "wall_s_timed_region": wall,
    }
    if world == 1 and cpu_baseline and not args.no_cpu_baseline:
        t, n, fl = oracle_extend_sample(w, args.oracle_rows)
        rec["cpu_baseline"] = {"value": fl / t / 1e12, "unit": "TFLOP/s", "cores": blas_threads(), "kind": "oracle",
                               "sample": f"{n} seeded query rows x {w.num_q_heads} heads of {rows} rows, 1 layer, {t:.1f} s"}
    else:
        rec["cpu_baseline"] = None
    return rec


SUB_RECORD_KEYS = ("metric", "value", "unit", "steps", "ms_per_step", "config", "clocks", "e2e", "gpu_launches",
                   "roofline", "decode_fracs", "breakdown_us_per_step", "kv", "new_tokens_per_s", "append_step_ms")


def run_gpu(args):
    """The GPU arm.  --config C: that configuration alone.  Default: configuration 4 as the headline and
    configurations 1, 3 (decode) and 2 (extend) as sub-records of the same line."""
    from paper_2605_22566_b200 import workloads as W
    env = Env()
    if args.config is not None:
        w = W.make_config(args.config)
        fn = decode_record if w.mode == "decode" else extend_record
        kw = dict(sustained_s=args.sustained) if w.mode == "decode" else {}
        rec = fn(env, args, w, args.steps, args.warmup, **kw)
    else:
        rec = decode_record(env, args, W.make_config(4), args.steps, args.warmup, sustained_s=args.sustained)
        subs = {}
        for cfg in (1, 3, 2):
            w = W.make_config(cfg)
            fn = decode_record if w.mode == "decode" else extend_record
            sub_steps = max(args.steps, 50) if w.mode == "decode" else max(3, min(args.steps, 20))
            sub = fn(env, args, w, sub_steps, args.warmup, cpu_baseline=False)
            if sub is not None:
                subs[f"config{cfg}"] = {k: sub[k] for k in SUB_RECORD_KEYS if k in sub}
        if rec is not None:
            rec["configs"] = subs
    if rec is not None:
        print(json.dumps(rec))
    env.close()


def run_gpu_residual(args):
    """Differential KV (Sec. 5.1, Eq. 7): gf_node_kv_reconstruct of every variant node from its base and a
    sparse residual.  A step reconstructs all variants once; the metric is algorithmic bytes per second."""
    import torch
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200 import workloads as W
    from paper_2605_22566_b200.runtime import PathAttention

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    dev = f"cuda:{local_rank}"
    torch.cuda.set_device(local_rank)
    w = W.residual_workload()
    nb, T = w.num_shared_nodes, int(w.node_len[0])
    rows = T * w.num_kv_heads
    pa = PathAttention(w, device=dev, layers=1, extra_tiles=nb * ((T + 63) // 64))
    pa.write_nodes("device")
    dens = {"k": 0.25, "v": 0.30}  # shares of entries above the threshold that Sec. 5.1 reports
    host = {"k": W.residual_stream(w.seed, W.KIND_DK, 0, 0, 1, rows, w.head_dim, dens["k"]),
            "v": W.residual_stream(w.seed, W.KIND_DV, 0, 0, 1, rows, w.head_dim, dens["v"])}
    pinned = {n: tuple(torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a.view(np.int32)).pin_memory() for a in r)
              for n, r in host.items()}
    devr = {n: tuple(t.to(dev) for t in r) for n, r in pinned.items()}
    ptrs = {n: (r[0].data_ptr(), r[1].data_ptr(), r[2].data_ptr(), int(host[n][2][-1])) for n, r in devr.items()}
    stream = torch.cuda.current_stream()

    def step():
        for b in range(nb):  # the same residual for every base: what is timed does not depend on its values
            B.check(B.gf_node_kv_reconstruct(pa.g, nb + b, 0, b, ptrs["k"], ptrs["v"], pa.stream), "gf_node_kv_reconstruct")

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    assert pa.status() == 0
    sampler = ClockSampler(visible_gpu_index(local_rank)) if rank == 0 else None
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = B.gf_launch_count(pa.g)
    barrier()
    if sampler:
        sampler.start()
    wall0 = time.perf_counter()
    for a, b in evs:  # a step moves 1.2 GB: far more than the 126 MB L2
        a.record(stream)
        step()
        b.record(stream)
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.finish() if sampler else None
    launches = B.gf_launch_count(pa.g) - launches0
    assert pa.status() == 0
    total_ms = max_over_ranks(float(sum(a.elapsed_time(b) for a, b in evs)), dist, dev)

    # end to end: the residual arrives from pinned host memory every step, a checksum row goes back
    e2e_steps = max(3, min(args.steps, 10))
    h_back = torch.empty((w.num_kv_heads, w.head_dim), dtype=torch.bfloat16).pin_memory()
    k_out = torch.empty((T, w.num_kv_heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    v_out = torch.empty_like(k_out)

    def e2e_step():
        for n in ("k", "v"):
            for d_t, h_t in zip(devr[n], pinned[n]):
                d_t.copy_(h_t, non_blocking=True)
        step()
        B.check(B.gf_node_kv_read(pa.g, nb, 0, k_out.data_ptr(), v_out.data_ptr(), pa.stream), "gf_node_kv_read")
        h_back.copy_(k_out[T - 1], non_blocking=True)
        stream.synchronize()

    for _ in range(2):
        e2e_step()
    barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    eb.record(stream)
    barrier()
    e2e_ms = ea.elapsed_time(eb)
    if rank != 0:
        return
    peaks, peak_kind = measured_peaks()
    dense = rows * w.head_dim * 2 * 2                      # K and V of one node, bf16
    res_bytes = sum(int(r[2][-1]) * 2 + r[0].size * 4 + r[2].size * 4 for r in host.values())
    per_launch = 2 * dense + res_bytes                     # base read + state written + residual read
    ms = total_ms / args.steps / nb
    achieved = per_launch / (ms * 1e-3) / 1e9
    peak = float(peaks["hbm_gbs"])
    line = {
        "metric": "kv_reconstruct_gbs", "value": per_launch * nb * args.steps * world / (total_ms * 1e-3) / 1e9,
        "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"differential KV: {nb} variant nodes of {T} tokens reconstructed from their bases",
                   "kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "residual_density": dens,
                   "step": "gf_node_kv_reconstruct per variant node, one layer",
                   "l2": "a step moves 1.2 GB, every launch 316 MB: far more than the 126 MB L2", "parallelism":
                   "single-gpu" if world == 1 else f"{world} independent replicas"},
        "clocks": clocks,
        "e2e": {"value": per_launch * nb * e2e_steps * world / (e2e_ms * 1e-3) / 1e9, "unit": "GB/s",
                "h2d_bytes_per_step": int(res_bytes), "d2h_bytes_per_step": int(h_back.numel() * 2), "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "k_kv_reconstruct", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": f"{peak_kind} copy bandwidth",
                     "traffic": NCU_TRAFFIC_RECON if args.traffic is None else args.traffic,
                     "algorithmic_bytes_per_launch": int(per_launch), "kernel_ms": ms},
        "tokens_reconstructed_per_s": T * nb * args.steps * world / (total_ms * 1e-3),
        "wall_s_timed_region": wall,
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import residual as OR
        n_rows = 65536
        kb = W.fill_bits(W.stream_key(w.seed, W.KIND_K, 0, 0), 0, n_rows * w.head_dim).reshape(n_rows, w.head_dim)
        bm, vals, rp = host["k"]
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < 10.0:
            OR.reconstruct(kb, bm[:n_rows], vals[:int(rp[n_rows])], rp[:n_rows + 1])
            reps += 1
        t = time.perf_counter() - t0
        nnz = int(rp[n_rows])
        cpu_bytes = reps * (2 * n_rows * w.head_dim * 2 + nnz * 2 + n_rows * (w.head_dim // 8) + (n_rows + 1) * 4)
        line["cpu_baseline"] = {"value": cpu_bytes / t / 1e9, "unit": "GB/s", "cores": blas_threads(), "kind": "oracle",
                                "sample": f"K tensor, first {n_rows} rows of one node, {reps} repetitions, {t:.1f} s"}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    pa.close()
    if dist is not None:
        dist.destroy_process_group()


def run_gpu_residual_stream(args):
    """Differential KV inside the segment stream (Sec. 5.1, Eq. 7): p prefix-conditioned variants of one
    operation node, each shared by four requests, decoded (a) from materialised states
    (gf_node_kv_reconstruct: p dense extents) and (b) from the base node's tiles plus the sparse residuals
    (gf_node_kv_attach_residual: nothing materialised).  A step is table build + decode of one layer."""
    import dataclasses
    import torch
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200 import workloads as W
    from paper_2605_22566_b200.runtime import PathAttention
    env = Env()
    dev, rank, world, dist = env.dev, env.rank, env.world, env.dist
    T, P, share = 16384, 8, 4
    base = W.residual_workload(n_base=1, n_tokens=T)
    R = P * share
    w = dataclasses.replace(base, num_nodes=1 + P, node_len=np.full(1 + P, T, np.int32),
                            path_ptr=np.arange(R + 1, dtype=np.int32),
                            path_node=np.repeat(np.arange(1, 1 + P, dtype=np.int32), share))
    rows = T * w.num_kv_heads
    dens = {"k": 0.25, "v": 0.30}
    host = {"k": W.residual_stream(w.seed, W.KIND_DK, 0, 0, 1, rows, w.head_dim, dens["k"]),
            "v": W.residual_stream(w.seed, W.KIND_DV, 0, 0, 1, rows, w.head_dim, dens["v"])}
    res_bytes = sum(int(r[2][-1]) * 2 + r[0].size * 4 + r[2].size * 4 for r in host.values())
    dense = rows * w.head_dim * 2 * 2
    results = {}
    stream = torch.cuda.current_stream()
    for how in ("materialised", "in_stream"):
        pa = PathAttention(w, device=dev, layers=1, max_residual_nodes=P, extra_tiles=(T + 63) // 64)
        # one residual copy per variant (the same values; every variant reads its own memory)
        keep, ptrs = [], []
        for v in range(P):
            t = {n: tuple(torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a.view(np.int32)).to(dev)
                          for a in r) for n, r in host.items()}
            keep.append(t)
            ptrs.append({n: (t[n][0].data_ptr(), t[n][1].data_ptr(), t[n][2].data_ptr(), int(host[n][2][-1])) for n in t})
        pa.write_nodes("device", only=[0])  # the base node; the variants come from it
        fn = B.gf_node_kv_reconstruct if how == "materialised" else B.gf_node_kv_attach_residual
        for v in range(P):
            B.check(fn(pa.g, 1 + v, 0, 0, ptrs[v]["k"], ptrs[v]["v"], pa.stream), how)
        q = pa.make_q(0)
        out = torch.empty_like(q)

        def step():
            pa.build(deferred=True)
            pa.decode(0, q, out=out)
        for _ in range(max(args.warmup, 3)):
            step()
        assert pa.status() == 0
        B.gf_profile_enable(pa.g, True)
        B.gf_profile_read(pa.g)
        sampler = ClockSampler(visible_gpu_index(env.local_rank)) if rank == 0 else None
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        launches0 = B.gf_launch_count(pa.g)
        env.barrier()
        if sampler:
            sampler.start()
        for a, b in evs:
            env.flush.fill_(1)
            a.record(stream)
            step()
            b.record(stream)
        env.barrier()
        clocks = sampler.finish() if sampler else None
        prof = B.gf_profile_read(pa.g)
        B.gf_profile_enable(pa.g, False)
        assert pa.status() == 0
        total_ms = max_over_ranks(float(sum(a.elapsed_time(b) for a, b in evs)), dist, dev)
        pool = B.gf_pool_info(pa.g)
        results[how] = {"ms_per_step": total_ms / args.steps, "decode_K2_ms": prof.decode_ms / max(args.steps, 1),
                        "pool_bytes_in_use_per_layer": int(pool.tiles_in_use) * B.gf_pool_bytes_per_tile(w.head_dim) * w.num_kv_heads,
                        "clocks": clocks, "gpu_launches": int(B.gf_launch_count(pa.g) - launches0),
                        "out_bits": out.view(torch.int16).cpu().numpy().copy()}
        pa.close()
        del pa, keep
        torch.cuda.empty_cache()
    env.close()
    if rank != 0:
        return
    same = bool(np.array_equal(results["materialised"].pop("out_bits"), results["in_stream"].pop("out_bits")))
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    alg = {"materialised": P * dense, "in_stream": dense + P * res_bytes}   # bytes that have to come from HBM
    ins = results["in_stream"]
    achieved = alg["in_stream"] / (ins["decode_K2_ms"] * 1e-3) / 1e9
    line = {"metric": "residual_stream_decode_tokens_per_s", "value": R * world / (ins["ms_per_step"] * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ins["ms_per_step"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"differential KV in the stream: {P} variants of one {T}-token node, {share} requests each",
                       "kv_heads": w.num_kv_heads, "head_dim": w.head_dim, "residual_density": dens,
                       "step": "gf_build_path_tables + gf_path_attention_decode, one layer",
                       "l2": "residuals (355 MB) and, materialised, the variants (537 MB) exceed the 126 MB L2; a 512 MB buffer is rewritten between steps"},
            "clocks": ins["clocks"], "gpu_launches": ins["gpu_launches"],
            "e2e": None,
            "roofline": {"kernel": "K2: k_decode with the residual applied in shared memory", "bound": "hbm",
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": f"{peak_kind} copy bandwidth", "traffic": args.traffic,
                         "algorithmic_bytes_per_launch": int(alg["in_stream"]), "kernel_ms": ins["decode_K2_ms"]},
            "materialised": results["materialised"], "in_stream": {k: v for k, v in ins.items()},
            "bytes_from_hbm_per_layer": {"materialised": int(alg["materialised"]), "in_stream": int(alg["in_stream"]),
                                         "dense_state": int(dense), "one_residual": int(res_bytes)},
            "outputs_identical": same, "cpu_baseline": None}
    print(json.dumps(line))


def run_gpu_scoring(args):
    """Workflow generation scoring (Sec. 4.2): gf_edge_scores for a batch of tasks over config 3's wGraph
    (1024 operations) with the paper's model sizes (384 -> 256 -> 256 encoder, 768 -> 128 -> 128 -> 1
    scorer), seeded weights.  A step scores every edge for every task of the batch."""
    import torch
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200 import workloads as W
    from paper_2605_22566_b200.runtime import PathAttention
    env = Env()
    dev, rank, world, dist = env.dev, env.rank, env.world, env.dist
    w = W.make_config(3)
    nt, (d_in, dh, dm) = 256, (384, 256, 128)
    N, E = w.num_shared_nodes, len(w.edge_src)
    inp = W.scoring_inputs(w.seed, N, nt, d_in, dh, dm)
    pa = PathAttention(w, device=dev, layers=1)
    t = {k: torch.from_numpy(np.ascontiguousarray(v)).to(dev) for k, v in inp.items() if k != "b3"}
    h_task = torch.from_numpy(inp["x_task"]).pin_memory()
    sc = B.Scorer(d_in, dh, dm, t["w_gcn1"].data_ptr(), t["w_gcn2"].data_ptr(), t["w1"].data_ptr(), t["b1"].data_ptr(),
                  t["w2"].data_ptr(), t["b2"].data_ptr(), t["w3"].data_ptr(), float(inp["b3"]))
    per_pass = 64
    nbytes = B.gf_edge_scores_scratch_bytes(pa.g, sc, nt, per_pass)
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    scores = torch.empty((nt, E), dtype=torch.float32, device=dev)
    h_scores = torch.empty((nt, E), dtype=torch.float32).pin_memory()
    stream = torch.cuda.current_stream()

    def step():
        B.check(B.gf_edge_scores(pa.g, sc, t["x_op"].data_ptr(), nt, t["x_task"].data_ptr(), scores.data_ptr(),
                                 scratch.data_ptr(), nbytes, pa.stream), "gf_edge_scores")
    for _ in range(max(args.warmup, 3)):
        step()
    sampler = ClockSampler(visible_gpu_index(env.local_rank)) if rank == 0 else None
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = B.gf_launch_count(pa.g)
    env.barrier()
    if sampler:
        sampler.start()
    for a, b in evs:
        env.flush.fill_(1)
        a.record(stream)
        step()
        b.record(stream)
    env.barrier()
    clocks = sampler.finish() if sampler else None
    launches = B.gf_launch_count(pa.g) - launches0
    total_ms = max_over_ranks(float(sum(a.elapsed_time(b) for a, b in evs)), dist, dev)
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        t["x_task"].copy_(h_task, non_blocking=True)
        step()
        h_scores.copy_(scores, non_blocking=True)
        stream.synchronize()
    for _ in range(2):
        e2e_step()
    env.barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    eb.record(stream)
    env.barrier()
    e2e_ms = max_over_ranks(ea.elapsed_time(eb), dist, dev)
    pa.close()
    env.close()
    if rank != 0:
        return
    # multiply-adds the model needs per task (the aggregation's adds left out), two flops each
    flops = 2.0 * ((N + 1) * dh * dh + (N + 1) * dh * 3 * dm + E * dm * dm + E * dm) * nt + 2.0 * (N + nt) * d_in * dh
    ms = total_ms / args.steps
    mhz = (clocks or {}).get("sm_max_mhz") or 1965
    peak = 148 * 128 * 2 * mhz * 1e6 / 1e12   # fp32: 128 fused multiply-adds per SM and clock
    achieved = flops / (ms * 1e-3) / 1e12
    line = {"metric": "edge_scores_per_s", "value": nt * E * args.steps * world / (total_ms * 1e-3), "unit": "scores/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"workflow generation scoring: {nt} tasks over config 3's wGraph ({N} operations, {E} edges)",
                       "model": {"d_in": d_in, "d_hidden": dh, "d_mlp": dm}, "tasks_per_pass": per_pass,
                       "step": "gf_edge_scores", "l2": "a 512 MB buffer is rewritten between steps"},
            "clocks": clocks,
            "e2e": {"value": nt * E * e2e_steps * world / (e2e_ms * 1e-3), "unit": "scores/s",
                    "h2d_bytes_per_step": int(h_task.numel() * 4), "d2h_bytes_per_step": int(h_scores.numel() * 4),
                    "steps": e2e_steps},
            "gpu_launches": int(launches),
            "roofline": {"kernel": "k_linear / k_aggregate / k_edge_mlp (the whole step)", "bound": "alu", "achieved": achieved,
                         "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_source": "148 SMs x 128 fp32 FMA per clock x 2 x the maximum SM clock", "traffic": None,
                         "algorithmic_flops_per_step": flops, "kernel_ms": ms}}
    if world == 1 and not args.no_cpu_baseline:
        from oracle import scoring as OS
        nb = 2
        t0 = time.perf_counter()
        OS.edge_scores(inp["x_op"], inp["x_task"][:nb], w.edge_src, w.edge_dst, inp["w_gcn1"], inp["w_gcn2"], inp["w1"],
                       inp["b1"], inp["w2"], inp["b2"], inp["w3"], float(inp["b3"]))
        tt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": nb * E / tt, "unit": "scores/s", "cores": blas_threads(), "kind": "oracle",
                                "sample": f"{nb} of {nt} tasks, {tt:.1f} s"}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))


def run_gpu_pruning(args):
    """Effective path pruning (Sec. 5.2): gf_transition_counts over a trace of executed workflows, then
    gf_select_transitions.  The trace is config 3's batch of paths repeated until it exceeds the L2."""
    import torch
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200 import workloads as W
    from paper_2605_22566_b200.runtime import PathAttention

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    dev = f"cuda:{local_rank}"
    torch.cuda.set_device(local_rank)
    w = W.make_config(3)
    reps = 4096
    lens = np.diff(w.path_ptr)
    h_node = torch.from_numpy(np.tile(w.path_node.astype(np.int32), reps)).pin_memory()
    h_ptr = torch.from_numpy(np.concatenate([[0], np.cumsum(np.tile(lens, reps))]).astype(np.int32)).pin_memory()
    R, P, E = h_ptr.numel() - 1, h_node.numel(), len(w.edge_src)
    # hops between two operation nodes (the last node of most paths is a private suffix: not a transition)
    inner = np.ones(len(w.path_node), dtype=bool)
    inner[w.path_ptr[1:] - 1] = False
    a, b = w.path_node[:-1], w.path_node[1:]
    hops = int(reps * np.count_nonzero(inner[:-1] & (a < w.num_shared_nodes) & (b < w.num_shared_nodes)))
    pa = PathAttention(w, device=dev, layers=1)
    d_node, d_ptr = h_node.to(dev), h_ptr.to(dev)
    counts = torch.zeros(max(E, 1), dtype=torch.int32, device=dev)
    misses = torch.zeros(1, dtype=torch.int64, device=dev)
    keep = torch.zeros(max(E, 1), dtype=torch.uint8, device=dev)
    totals = torch.zeros(3, dtype=torch.int64, device=dev)
    h_totals = torch.zeros(3, dtype=torch.int64).pin_memory()
    min_count = reps  # keep the transitions taken at least once per repetition of the batch
    stream = torch.cuda.current_stream()

    def step():
        B.check(B.gf_transition_counts(pa.g, R, P, d_ptr.data_ptr(), d_node.data_ptr(), counts.data_ptr(),
                                       misses.data_ptr(), pa.stream), "gf_transition_counts")
        B.check(B.gf_select_transitions(pa.g, counts.data_ptr(), min_count, keep.data_ptr(), totals.data_ptr(),
                                        pa.stream), "gf_select_transitions")

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    sampler = ClockSampler(visible_gpu_index(local_rank)) if rank == 0 else None
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches0 = B.gf_launch_count(pa.g)
    barrier()
    if sampler:
        sampler.start()
    wall0 = time.perf_counter()
    for a, b in evs:  # the trace (134 MB) exceeds the 126 MB L2
        a.record(stream)
        step()
        b.record(stream)
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.finish() if sampler else None
    launches = B.gf_launch_count(pa.g) - launches0
    total_ms = max_over_ranks(float(sum(a.elapsed_time(b) for a, b in evs)), dist, dev)
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        d_ptr.copy_(h_ptr, non_blocking=True)
        d_node.copy_(h_node, non_blocking=True)
        step()
        h_totals.copy_(totals, non_blocking=True)
        stream.synchronize()

    for _ in range(2):
        e2e_step()
    barrier()
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record(stream)
    for _ in range(e2e_steps):
        e2e_step()
    eb.record(stream)
    barrier()
    e2e_ms = ea.elapsed_time(eb)
    if rank != 0:
        return
    assert int(misses.item()) == 0 and int(h_totals[2]) == hops
    peaks, peak_kind = measured_peaks()
    per_launch = 4 * (P + R + 1)  # the trace is read once
    ms = total_ms / args.steps
    achieved = per_launch / (ms * 1e-3) / 1e9
    peak = float(peaks["hbm_gbs"])
    line = {
        "metric": "transition_hops_per_s", "value": hops * args.steps * world / (total_ms * 1e-3), "unit": "hops/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": f"path pruning statistics: config 3's {w.num_requests} paths x {reps} = {R} executed workflows, "
                               f"{hops} hops, {E} wGraph edges", "min_count": min_count,
                   "step": "gf_transition_counts + gf_select_transitions",
                   "l2": f"the trace is {4 * (P + R + 1) / 1e6:.0f} MB, more than the 126 MB L2", "parallelism":
                   "single-gpu" if world == 1 else f"{world} independent replicas"},
        "clocks": clocks,
        "e2e": {"value": hops * e2e_steps * world / (e2e_ms * 1e-3), "unit": "hops/s",
                "h2d_bytes_per_step": int(4 * (P + R + 1)), "d2h_bytes_per_step": 24, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "k_transition_counts", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_source": f"{peak_kind} copy bandwidth",
                     "traffic": NCU_TRAFFIC_PRUNE if args.traffic is None else args.traffic,
                     "algorithmic_bytes_per_launch": int(per_launch), "kernel_ms": ms,
                     "note": "kernel_ms is the whole step (two memsets, the count kernel, the selection kernel)"},
        "kept": {"edges": int(h_totals[0]), "traversals_covered": int(h_totals[1]), "traversals": int(h_totals[2])},
        "wall_s_timed_region": wall,
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import pruning as OP
        t0 = time.perf_counter()
        n = 0
        while time.perf_counter() - t0 < 10.0:
            OP.transition_counts(w.num_shared_nodes, w.edge_src, w.edge_dst, w.path_ptr, w.path_node)
            n += 1
        t = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n * (hops // reps) / t, "unit": "hops/s", "cores": 1,
                                "kind": "oracle", "sample": f"config 3's {w.num_requests} paths, {n} repetitions, {t:.1f} s"}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    pa.close()
    if dist is not None:
        dist.destroy_process_group()


def relaunch_under_torchrun(args) -> bool:
    """`--gpus N` with N > 1 outside torchrun: start N ranks of this command on this node."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ:
        return False
    import subprocess
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None,
                    help="time this configuration alone (default: configuration 4 with sub-records for 1, 3 and 2)")
    ap.add_argument("--layers", type=int, default=None, help="materialise and time only this many layers")
    ap.add_argument("--phys-layers", type=int, default=16,
                    help="physical KV layer copies kept in HBM (timed layer l reads copy l %% this)")
    ap.add_argument("--policy", type=int, nargs=4, default=None,
                    metavar=("CHUNK", "GROUP_TILE", "GROUP_UNIT", "MAX_MULT"))
    ap.add_argument("--sustained", type=float, default=2.0,
                    help="seconds of back-to-back decode steps for the sustained leg (0: skip)")
    ap.add_argument("--oracle-requests", type=int, default=None,
                    help="requests the oracle is timed on (default: about ten seconds' worth)")
    ap.add_argument("--oracle-rows", type=int, default=48, help="query rows the oracle times in extend mode")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--traffic", type=float, default=None,
                    help="DRAM bytes per launch of the roofline kernel, from an ncu capture of this command "
                         "(dram__bytes_read.sum + dram__bytes_write.sum); default: the recorded capture if the "
                         "kernel sources are unchanged since, else null")
    ap.add_argument("--residual", action="store_true",
                    help="time the differential-KV reconstruction (gf_node_kv_reconstruct) instead of a decode / extend step")
    ap.add_argument("--residual-stream", action="store_true",
                    help="decode over prefix-conditioned variants kept as base + residual (gf_node_kv_attach_residual) "
                         "against the same variants materialised")
    ap.add_argument("--scoring", action="store_true",
                    help="time the workflow generation scoring (gf_edge_scores: graph convolutional encoder + perceptron)")
    ap.add_argument("--pruning", action="store_true",
                    help="time the path-pruning statistics (gf_transition_counts + gf_select_transitions)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    relaunch_under_torchrun(args)
    if args.scoring:
        run_gpu_scoring(args)
    elif args.residual_stream:
        run_gpu_residual_stream(args)
    elif args.residual:
        run_gpu_residual(args)
    elif args.pruning:
        run_gpu_pruning(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
