#!/usr/bin/env python
"""Benchmark of the MLPMoE forward path on B200.

    python bench.py --gpus N --steps K --warmup W            (N > 1: launched once per rank by torchrun)
    python bench.py --impl reference --steps K --warmup W     (the CPU oracle, timed on the host cores)

Workload: the 24-layer MLP-only stack with Qwen2.5-0.5B shapes (d_model 896, d_inter 4864,
bf16, B = 16 equal slices, 4 of 16 branches per layer dropped by Compensated Pruning with a
seeded keep set, RMSNorm before and residual add after each layer) over 4096 tokens ~ N(0, 1).
One step = one pass of the whole stack over one batch; every rank runs its own batch (token
split, no collective on the data path), so scaling is weak.

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_21089_b200 import synth  # noqa: E402

METRIC = "mlpmoe_mlp_tokens_per_s"
UNIT = "tokens/s"
WORKLOAD = ("configs[1]: 24-layer MLP-only stack, Qwen2.5-0.5B shapes (d_model=896, d_inter=4864), bf16, "
            "B=16 equal slices, Compensated Pruning 12 of 16 branches kept per layer (seeded), "
            "RMSNorm + residual, 4096 tokens")


def workload(layers=None, name="qwen_stack", tokens=None, branches=None, ratio=0.0, prune_k=None):
    """The default (and only driver-run) workload is the 24-layer Qwen-shaped stack; the others are
    the remaining configurations, for measurement of the decode and Llama-shaped prefill paths."""
    if name == "qwen_stack":
        c = synth.CONFIGS[2]
        return dict(name=name, cfg=2, d=c["d_model"], I=c["d_inter"], B=c["B"], n=tokens or c["n"], L=layers or c["layers"],
                    n_drop=c["n_drop"], stack=True, label=WORKLOAD)
    c = synth.CONFIGS[4]
    d, I = c["d_model"], c["d_inter"]
    if name == "llama_decode":
        n = tokens or 64
        return dict(name=name, cfg=4, d=d, I=I, B=64, n=n, L=layers or 32, prune_k=prune_k, stack=True,
                    label=f"configs[3]: 32-layer Llama-3-8B-shaped MLP stack, bf16, B=64 equal slices, decode, {n} tokens, "
                          + (f"first-K pruning K={prune_k}" if prune_k else "no pruning"))
    if name == "llama_layer_fade":
        n = tokens or 8192
        return dict(name=name, cfg=3, d=d, I=I, B=32, n=n, L=1, stack=False, fade=True,
                    label=f"configs[2]: single Llama-3-8B-shaped layer, bf16, B=32, Fractal Fade s_b=0.9b/B, alpha~U(0.8,1.2), {n} tokens")
    if name == "llama_prefill":
        n, B = tokens or 2048, branches or 16
        return dict(name=name, cfg=5, d=d, I=I, B=B, n=n, L=layers or 32, ratio=ratio, stack=True,
                    label=f"configs[4]: 32-layer Llama-3-8B-shaped MLP stack, bf16, B={B} unequal slices, {n} tokens, "
                          f"Compensated Pruning ratio {ratio}")
    raise ValueError(name)


def layer_inputs(layer: int, w):
    """Seeded inputs of one layer: (weights as bf16 bit patterns, partition, alpha or None, keep mask or None)."""
    cfg, B = w["cfg"], w["B"]
    wcfg = 4 if cfg == 5 else cfg          # the prefill sweep runs on the decode configuration's weights
    bits = synth.layer_weights(wcfg, layer, w["d"], w["I"], 0.02, bf16=True)
    alpha, keep = None, None
    if cfg == 2:
        d_b = synth.equal_partition(w["I"], B)
        keep = synth.keep_set((synth.BASE_SEED, cfg, layer, synth.T_KEEP), B, w["n_drop"])
    elif cfg == 3:
        d_b = synth.equal_partition(w["I"], B)
        alpha = [float(a) for a in synth.uniform_f64((synth.BASE_SEED, 3, layer, synth.T_ALPHA), B, 0.8, 1.2).astype(np.float32)]
    elif cfg == 4:
        d_b = synth.equal_partition(w["I"], B)
        if w.get("prune_k"):
            keep = [b < w["prune_k"] for b in range(B)]
    else:
        d_b = synth.random_partition((synth.BASE_SEED, 5, B, synth.T_PARTITION), w["I"], B, 64)
        n_drop = synth.n_drop_for_ratio(B, w["ratio"])
        if n_drop:
            keep = synth.keep_set((synth.BASE_SEED, 5, B, layer, synth.T_KEEP), B, n_drop)
    return bits, d_b, alpha, keep


# DRAM traffic of one launch of the persistent prefill-stack kernel on the default workload, from the
# committed ncu summary of that kernel (dram__bytes_read.sum + dram__bytes_write.sum), valid only
# while the kernel's sources are the ones that were profiled.
GATEUP_TRAFFIC_BYTES = 889.68e6 + 969.74e6
GATEUP_SOURCES = ("tc_stack.cu", "tc_common.cuh", "ptx.cuh")
GATEUP_SOURCES_SHA = "da40b6ea7d527727"


def gateup_traffic():
    import hashlib
    h = hashlib.sha256()
    for f in GATEUP_SOURCES:
        with open(os.path.join(ROOT, "paper_2511_21089_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return GATEUP_TRAFFIC_BYTES if h.hexdigest()[:16] == GATEUP_SOURCES_SHA else None


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"], hbm_gbs=p["hbm_gbs"],
                    source="measured")
    return dict(tflops_burst=1590.0, tflops_sustained=1400.0, hbm_gbs=6650.0, source="fallback")


# ------------------------------------------------------------------ oracle leg --
def oracle_layers(w):
    import oracle
    layers = []
    for l in range(w["L"]):
        bits, d_b, alpha, keep = layer_inputs(l, w)
        host = [synth.bf16_bits_to_f32(b) for b in bits]
        layers.append((host[0], host[1], host[2], d_b, oracle.prune_alpha([1.0] * w["B"], keep)))
    return layers


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i["num_threads"] for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(w, rows: int, steps: int, warmup: int, layers=None):
    """The oracle as it stands, on the first `rows` token rows of the batch (tokens are
    independent, so a row sample runs exactly the per-token work of the full batch)."""
    import oracle
    if layers is None:
        layers = oracle_layers(w)
    x = synth.tokens(w["cfg"], w["n"], w["d"])[:rows]
    for _ in range(warmup):
        oracle.stack_forward(x, layers, bf16_activations=True)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.stack_forward(x, layers, bf16_activations=True)
    dt = (time.perf_counter() - t0) / steps
    return rows / dt, dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload(args.layers)
    rows = 256
    tps, dt = time_oracle(w, rows, args.steps, args.warmup)
    cores = blas_threads()
    sample = f"first {rows} of {w['n']} token rows through all {w['L']} layers per step, numpy float64"
    out = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


# ------------------------------------------------------------- multi-rank glue --
def rank_batch(cfg: int, n: int, d: int, rank: int) -> np.ndarray:
    """Token split: every rank draws its own n-token batch (rows are independent, so the path
    shards by tokens with no collective on the data path)."""
    return synth.tokens(cfg, n, d, stream=rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a few per-rank timings over all ranks (the job is as slow as its
    slowest rank); a no-op outside torch.distributed."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(world: int, n: int, steps: int, ms_total_max: float) -> float:
    """Whole-job tokens/s: all ranks' tokens over the slowest rank's time."""
    return world * n * steps / (ms_total_max * 1e-3)


# ------------------------------------------------------------------- CUDA leg --
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.path = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".csv", delete=False).name
        self.f = open(self.path, "w")
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.p.kill()
        self.f.close()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                c = [v.strip() for v in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); smax.append(float(c[2])); power.append(float(c[3]))
                except ValueError:
                    continue
                for name, v in zip(names, c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": float(max(power))}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2511_21089_b200 import build
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    from paper_2511_21089_b200 import binding as lib

    w = workload(args.layers, args.workload, args.tokens, args.branches, args.ratio, args.prune_k)
    n, d, L = w["n"], w["d"], w["L"]
    stream = torch.cuda.current_stream()
    st = stream.cuda_stream
    layers, active = [], []
    for l in range(L):
        bits, d_b, alpha, keep = layer_inputs(l, w)
        dev = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).cuda() for b in bits]
        h = lib.mlpmoe_create(d, w["I"], d_b, dev[0], dev[1], dev[2], alpha, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, n, st)
        if w.get("fade"):
            lib.mlpmoe_fade(h, None, st)
        if keep is not None:
            lib.mlpmoe_prune(h, keep, True, st)
        if layers:
            lib.mlpmoe_share_workspace(h, layers[0])
        layers.append(h)
        active.append(lib.mlpmoe_get_active_neurons(h))
        del dev
    torch.cuda.synchronize()

    x_f32 = rank_batch(w["cfg"], n, d, rank)
    y_host = torch.empty((n, d), dtype=torch.float32).pin_memory()
    if w["stack"]:
        x0_host = torch.from_numpy(x_f32).pin_memory()
        x0 = x0_host.cuda()
        xw = torch.empty_like(x0)

        def step():
            xw.copy_(x0, non_blocking=True)      # fresh residual stream; inputs already resident in HBM
            lib.mlpmoe_stack_forward(layers, xw, n, 1e-6, st)

        def step_host():
            lib.mlpmoe_stack_forward_host(layers, x0_host, y_host, n, 1e-6, st)
        in_bytes = n * d * 4
    else:
        xb = synth.f32_to_bf16_bits(x_f32)
        x0_host = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()
        x0 = x0_host.cuda()
        xw = torch.empty((n, d), dtype=torch.float32, device="cuda")

        def step():
            lib.mlpmoe_forward(layers[0], x0, xw, n, st)

        def step_host():
            lib.mlpmoe_forward_host(layers[0], x0_host, y_host, n, st)
        in_bytes = n * d * 2

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    launches0 = sum(lib.mlpmoe_get_launch_count(h) for h in layers)
    for h in layers:
        lib.mlpmoe_set_timing(h, bool(args.kernel_events))     # allocates the event pools (set-up)
        lib.mlpmoe_get_timing(h)
        lib.mlpmoe_set_timing(h, False)
    gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    sampler = ClockSampler(gpu_id)
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        # per-kernel events on every 8th step only: each record costs about a microsecond of stream time
        timed = bool(args.kernel_events) and i % 8 == 0
        if timed:
            for h in layers:
                lib.mlpmoe_set_timing(h, True)
        step()
        if timed:
            for h in layers:
                lib.mlpmoe_set_timing(h, False)
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    launches = sum(lib.mlpmoe_get_launch_count(h) for h in layers) - launches0
    kms, kcnt = np.zeros(3), np.zeros(3, dtype=np.int64)
    for h in layers:
        ms, cnt = lib.mlpmoe_get_timing(h)
        kms += np.array(ms); kcnt += np.array(cnt)
        lib.mlpmoe_set_timing(h, False)
    status = max(lib.mlpmoe_get_status(h) for h in layers)
    if status != lib.MLPMOE_OK:
        raise RuntimeError("a kernel reported " + lib.mlpmoe_status_string(status))

    # end to end through the host-buffer entry point: H2D of x and D2H of y inside the timed region
    for _ in range(2):
        step_host()
    barrier()
    e2e_steps = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_host()                                  # synchronises the stream itself
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    if not np.isfinite(y_host.numpy()).all():
        raise RuntimeError("non-finite output")

    ms_total, e2e_ms = max_over_ranks([ms_total, e2e_ms], device="cuda")
    ms_step = ms_total / args.steps
    value = job_throughput(world, n, args.steps, ms_total)

    if rank == 0:
        pk = peaks()
        flops_gu = [4.0 * n * d * a for a in active]              # algorithmic FLOPs of each gate|up launch
        flops_dn = [2.0 * n * d * a for a in active]
        wbytes_gu = [2.0 * d * a * 2 for a in active]             # weight bytes each gate|up launch must stream
        wbytes_dn = [1.0 * d * a * 2 for a in active]
        default = w["name"] == "qwen_stack" and L == synth.CONFIGS[2]["layers"] and n == synth.CONFIGS[2]["n"]
        weights_gb = (sum(wbytes_gu) + sum(wbytes_dn)) / 1e9
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": w["label"] if default or w["name"] != "qwen_stack" else w["label"] + f" [REDUCED to {L} layers, {n} tokens]",
                       "l2": f"inputs larger than L2: each step streams {weights_gb:.2f} GB of distinct weights",
                       "surviving_neurons_per_layer": int(np.mean(active)), "tokens_per_rank": n},
            "clocks": clocks,
            "e2e": {"value": world * n / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
                    "d2h_bytes_per_step": n * d * 4, "ms_per_step": e2e_ms},
            "gpu_launches": int(launches),
            "tflops": (sum(flops_gu) + sum(flops_dn)) / (ms_step * 1e-3) / 1e12,
            "weight_gbs": weights_gb / (ms_step * 1e-3),
        }
        if kcnt[0] > 0:
            # per-kernel events exist on every 8th step only: shares are taken of those steps' time
            timed_steps = len(range(0, args.steps, 8))
            ms_timed = ms_total * timed_steps / args.steps
            gu_ms = kms[0] / kcnt[0]
            dn_ms = kms[1] / max(kcnt[1], 1)
            fused = n > 128            # one kernel runs both GEMMs of a layer call
            # ... and, for a stack of short layers, every layer and its RMSNorm (one launch per step)
            whole_stack = fused and w["stack"] and int(kcnt[0]) == timed_steps
            if n > 64:
                if whole_stack:
                    flops = float(np.sum(flops_gu)) + float(np.sum(flops_dn))
                else:
                    flops = float(np.mean(flops_gu)) + (float(np.mean(flops_dn)) if fused else 0.0)
                achieved = flops / (gu_ms * 1e-3) / 1e12
                out["roofline"] = {"bound": "tensor",
                                   "kernel": "persistent stack kernel: per layer RMSNorm, gate|up GEMM + SiLU*up epilogue, down GEMM + "
                                             "residual add (tcgen05, CTA pairs, all layers in one launch)" if whole_stack else
                                   "fused layer kernel: gate|up GEMM + SiLU*up epilogue, then down GEMM (tcgen05, CTA pairs)"
                                   if fused else "gate|up GEMM + SiLU*up epilogue (tcgen05)",
                                   "achieved": achieved, "peak": pk["tflops_sustained"], "unit": "TFLOP/s",
                                   "frac": achieved / pk["tflops_sustained"], "traffic": gateup_traffic() if default else None,
                                   "peak_source": pk["source"] + " (sustained bf16 matmul)", "avg_launch_us": gu_ms * 1e3}
            elif not w["stack"]:
                # decode, one layer call: two kernels, each streams its part of the weights once
                achieved = float(np.mean(wbytes_gu)) / (gu_ms * 1e-3) / 1e9
                out["roofline"] = {"bound": "hbm", "kernel": "decode gate|up kernel (TMA weight ring + tcgen05)",
                                   "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"],
                                   "traffic": None, "peak_source": pk["source"] + " (copy bandwidth)", "avg_launch_us": gu_ms * 1e3}
            else:
                # decode: one persistent kernel runs the whole stack and streams every layer's weights once
                achieved = (sum(wbytes_gu) + sum(wbytes_dn)) / (gu_ms * 1e-3) / 1e9
                out["roofline"] = {"bound": "hbm", "kernel": "persistent decode-stack kernel (TMA weight ring + tcgen05, all layers)",
                                   "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"],
                                   "traffic": None, "peak_source": pk["source"] + " (copy bandwidth)", "avg_launch_us": gu_ms * 1e3}
            if n <= 64 and w["stack"]:
                out["kernels"] = {"decode_stack": {"avg_us": gu_ms * 1e3, "launches": int(kcnt[0]), "share": float(kms[0] / ms_timed),
                                                   "weight_gbs": achieved}}
            elif whole_stack:
                out["kernels"] = {"prefill_stack": {"avg_us": gu_ms * 1e3, "launches": int(kcnt[0]), "share": float(kms[0] / ms_timed),
                                                    "tflops": achieved}}
            elif fused and n > 64:
                out["kernels"] = {
                    "layer_fused": {"avg_us": gu_ms * 1e3, "launches": int(kcnt[0]), "share": float(kms[0] / ms_timed),
                                    "tflops": achieved},
                    "rmsnorm": {"avg_us": kms[2] / max(kcnt[2], 1) * 1e3, "launches": int(kcnt[2]), "share": float(kms[2] / ms_timed)},
                }
            else:
                out["kernels"] = {
                "gate_up": {"avg_us": gu_ms * 1e3, "launches": int(kcnt[0]), "share": float(kms[0] / ms_timed),
                            "tflops": float(np.mean(flops_gu)) / (gu_ms * 1e-3) / 1e12, "weight_gbs": float(np.mean(wbytes_gu)) / (gu_ms * 1e-3) / 1e9},
                "down": {"avg_us": dn_ms * 1e3, "launches": int(kcnt[1]), "share": float(kms[1] / ms_timed),
                         "tflops": float(np.mean(flops_dn)) / (dn_ms * 1e-3) / 1e12, "weight_gbs": float(np.mean(wbytes_dn)) / (dn_ms * 1e-3) / 1e9},
                "rmsnorm": {"avg_us": kms[2] / max(kcnt[2], 1) * 1e3, "launches": int(kcnt[2]), "share": float(kms[2] / ms_timed)},
            }
        else:
            out["roofline"] = None
        if out.get("roofline"):
            # context only: the same figure against the nominal peaks (2.25 PFLOP/s dense bf16, 8 TB/s HBM3e)
            nominal = 2250.0 if out["roofline"]["bound"] == "tensor" else 8000.0
            out["roofline"]["frac_of_nominal"] = out["roofline"]["achieved"] / nominal
        if world == 1 and not args.no_cpu_baseline and w["name"] == "qwen_stack":
            rows = 512
            tps, dt = time_oracle(w, rows, 3, 1)
            out["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                   "sample": f"first {rows} of {n} token rows through all {L} layers, 3 passes, numpy float64"}
        else:
            out["cpu_baseline"] = None
        print(json.dumps(out))
    for h in layers[1:] + layers[:1]:
        lib.mlpmoe_destroy(h)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--layers", type=int, default=None, help="fewer layers of the same stack (profiling captures only)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen_stack", choices=["qwen_stack", "llama_decode", "llama_layer_fade", "llama_prefill"],
                    help="the driver runs the default; the others measure the remaining configurations")
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--branches", type=int, default=None)
    ap.add_argument("--ratio", type=float, default=0.0)
    ap.add_argument("--prune-k", type=int, default=None)
    ap.add_argument("--kernel-events", type=int, default=1, help="record per-kernel CUDA events in the timed region")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
