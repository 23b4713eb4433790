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

CFG = 2
METRIC = "mlpmoe_mlp_tokens_per_s"
UNIT = "tokens/s"
WORKLOAD = ("configs[1]: 24-layer MLP-only stack, Qwen2.5-0.5B shapes (d_model=896, d_inter=4864), bf16, "
            "B=16 equal slices, Compensated Pruning 12 of 16 branches kept per layer (seeded), "
            "RMSNorm + residual, 4096 tokens")


def workload(layers=None):
    c = synth.CONFIGS[CFG]
    return dict(d=c["d_model"], I=c["d_inter"], B=c["B"], n=c["n"], L=layers or c["layers"], n_drop=c["n_drop"])


def layer_inputs(layer: int, w):
    """Seeded weights (bf16 bit patterns), partition and keep set of one layer."""
    bits = synth.layer_weights(CFG, layer, w["d"], w["I"], 0.02, bf16=True)
    d_b = synth.equal_partition(w["I"], w["B"])
    keep = synth.keep_set((synth.BASE_SEED, CFG, layer, synth.T_KEEP), w["B"], w["n_drop"])
    return bits, d_b, keep


# DRAM traffic of one gate|up launch from the ncu capture summarised in
# profiles/tc_pair_gemm_qwen_c2_2layers.md (dram__bytes_read.sum + dram__bytes_write.sum), valid
# only while the kernel's sources are the ones that were profiled.
GATEUP_TRAFFIC_BYTES = 20.70e6 + 0.12e6
GATEUP_SOURCES = ("tc_gemm2.cu", "tc_common.cuh", "ptx.cuh")
GATEUP_SOURCES_SHA = "b842eb5204afc5ef"


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
        bits, d_b, keep = layer_inputs(l, w)
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
    x = synth.tokens(CFG, w["n"], w["d"])[:rows]
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

    w = workload(args.layers)
    n, d, L = w["n"], w["d"], w["L"]
    stream = torch.cuda.current_stream()
    st = stream.cuda_stream
    layers, active = [], []
    for l in range(L):
        bits, d_b, keep = layer_inputs(l, w)
        dev = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).cuda() for b in bits]
        h = lib.mlpmoe_create(d, w["I"], d_b, dev[0], dev[1], dev[2], None, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, n, st)
        lib.mlpmoe_prune(h, keep, True, st)
        if layers:
            lib.mlpmoe_share_workspace(h, layers[0])
        layers.append(h)
        active.append(lib.mlpmoe_get_active_neurons(h))
        del dev
    torch.cuda.synchronize()

    x0_host = torch.from_numpy(synth.tokens(CFG, n, d, stream=rank)).pin_memory()     # each rank its own batch
    y_host = torch.empty((n, d), dtype=torch.float32).pin_memory()
    x0 = x0_host.cuda()
    xw = torch.empty_like(x0)

    def step():
        xw.copy_(x0, non_blocking=True)          # fresh residual stream; inputs already resident in HBM
        lib.mlpmoe_stack_forward(layers, xw, n, 1e-6, st)

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
        lib.mlpmoe_stack_forward_host(layers, x0_host, y_host, n, 1e-6, st)
    barrier()
    e2e_steps = max(3, min(args.steps, 10))
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        lib.mlpmoe_stack_forward_host(layers, x0_host, y_host, n, 1e-6, st)     # synchronises the stream itself
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
    if not np.isfinite(y_host.numpy()).all():
        raise RuntimeError("non-finite output")

    t = torch.tensor([ms_total, e2e_ms], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total, e2e_ms = float(t[0]), float(t[1])
    ms_step = ms_total / args.steps
    value = world * n * args.steps / (ms_total * 1e-3)

    if rank == 0:
        pk = peaks()
        flops_gu = [4.0 * n * d * a for a in active]              # algorithmic FLOPs of each gate|up launch
        flops_dn = [2.0 * n * d * a for a in active]
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": WORKLOAD if L == synth.CONFIGS[CFG]["layers"] else WORKLOAD + f" [REDUCED to {L} layers]", "l2": "inputs larger than L2: each step streams 0.47 GB of distinct weights",
                       "surviving_neurons_per_layer": int(np.mean(active)), "tokens_per_rank": n},
            "clocks": clocks,
            "e2e": {"value": world * n / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": n * d * 4,
                    "d2h_bytes_per_step": n * d * 4, "ms_per_step": e2e_ms},
            "gpu_launches": int(launches),
            "tflops": (sum(flops_gu) + sum(flops_dn)) / (ms_step * 1e-3) / 1e12,
        }
        if kcnt[0] > 0:
            gu_ms = kms[0] / kcnt[0]
            achieved = float(np.mean(flops_gu)) / (gu_ms * 1e-3) / 1e12
            out["roofline"] = {"bound": "tensor", "kernel": "gate|up GEMM + SiLU*up epilogue (tcgen05)",
                               "achieved": achieved, "peak": pk["tflops_sustained"], "unit": "TFLOP/s",
                               "frac": achieved / pk["tflops_sustained"], "traffic": gateup_traffic(),
                               "peak_source": pk["source"] + " (sustained bf16 matmul)", "avg_launch_us": gu_ms * 1e3}
            out["kernels"] = {
                "gate_up": {"avg_us": gu_ms * 1e3, "launches": int(kcnt[0]), "share": float(kms[0] / ms_total)},
                "down": {"avg_us": kms[1] / max(kcnt[1], 1) * 1e3, "launches": int(kcnt[1]), "share": float(kms[1] / ms_total),
                         "tflops": float(np.mean(flops_dn)) / (kms[1] / max(kcnt[1], 1) * 1e-3) / 1e12},
                "rmsnorm": {"avg_us": kms[2] / max(kcnt[2], 1) * 1e3, "launches": int(kcnt[2]), "share": float(kms[2] / ms_total)},
            }
        else:
            out["roofline"] = None
        if world == 1 and not args.no_cpu_baseline:
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
    ap.add_argument("--kernel-events", type=int, default=1, help="record per-kernel CUDA events in the timed region")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
