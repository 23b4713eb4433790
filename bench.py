#!/usr/bin/env python
"""Benchmark of the MLPMoE forward path on B200.

    python bench.py --gpus N --steps K --warmup W            (N > 1: launched once per rank by torchrun)
    python bench.py --impl reference --steps K --warmup W     (the CPU oracle, timed on the host cores)

Headline workload (configs[4] at its largest point, the largest single-GPU configuration): the
32-layer MLP-only stack with Llama-3-8B shapes (d_model 4096, d_inter 14336, bf16), B = 32 unequal
contiguous slices drawn from seed, Compensated Pruning of 20 % of the branches per layer (seeded
keep set), RMSNorm before and residual add after each layer, over 16384 tokens ~ N(0, 1).  One step
= one pass of the whole stack over one batch; every rank runs its own batch (token split, no
collective on the data path), so scaling is weak.

At one GPU the same run also measures, each with its own roofline block under "configs":
configs[1] (24-layer Qwen-shaped stack, 4096 tokens), configs[2] (one Llama-shaped layer with
Fractal Fade, 8192 tokens) and configs[3] (32-layer Llama-shaped decode at 1 / 8 / 32 / 64 tokens,
unpruned and with first-K pruning K = 51), and the pruned / unpruned time ratio of decode next to
the byte ratio.

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import hashlib
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
HEADLINE = dict(name="llama_prefill", tokens=16384, branches=32, ratio=0.2)


def workload(name="llama_prefill", layers=None, tokens=None, branches=None, ratio=None, prune_k=None):
    """Shapes and transform of one benchmark workload (synthetic stand-ins for the checkpoints the paper used)."""
    if name == "qwen_stack":
        c = synth.CONFIGS[2]
        n, L = tokens or c["n"], layers or c["layers"]
        return dict(name=name, cfg=2, d=c["d_model"], I=c["d_inter"], B=c["B"], n=n, L=L, n_drop=c["n_drop"], stack=True,
                    label=f"configs[1]: {L}-layer MLP-only stack, Qwen2.5-0.5B shapes (d_model=896, d_inter=4864), bf16, B=16 equal "
                          f"slices, Compensated Pruning 12 of 16 branches kept per layer (seeded), RMSNorm + residual, {n} tokens")
    c = synth.CONFIGS[4]
    d, I = c["d_model"], c["d_inter"]
    if name == "llama_decode":
        n, L = tokens or 64, layers or 32
        return dict(name=name, cfg=4, d=d, I=I, B=64, n=n, L=L, prune_k=prune_k, stack=True,
                    label=f"configs[3]: {L}-layer Llama-3-8B-shaped MLP stack, bf16, B=64 equal slices, decode, {n} tokens, "
                          + (f"first-K pruning K={prune_k}" if prune_k else "no pruning"))
    if name == "llama_layer_fade":
        n = tokens or 8192
        return dict(name=name, cfg=3, d=d, I=I, B=32, n=n, L=1, stack=False, fade=True,
                    label=f"configs[2]: single Llama-3-8B-shaped layer, bf16, B=32, Fractal Fade s_b=0.9b/B, alpha~U(0.8,1.2), {n} tokens")
    if name == "llama_prefill":
        n, B, L = tokens or HEADLINE["tokens"], branches or HEADLINE["branches"], layers or 32
        r = HEADLINE["ratio"] if ratio is None else ratio
        return dict(name=name, cfg=5, d=d, I=I, B=B, n=n, L=L, ratio=r, stack=True,
                    label=f"configs[4]: {L}-layer Llama-3-8B-shaped MLP stack (d_model=4096, d_inter=14336), bf16, B={B} unequal "
                          f"slices (seeded), {n} tokens, Compensated Pruning ratio {r} (seeded keep set per layer), RMSNorm + residual")
    raise ValueError(name)


def layer_inputs(layer: int, w, bits_cache=None):
    """Seeded inputs of one layer: (weights as bf16 bit patterns, partition, alpha or None, keep mask or None)."""
    cfg, B = w["cfg"], w["B"]
    wcfg = 4 if cfg == 5 else cfg          # the prefill sweep runs on the decode configuration's weights
    key = (wcfg, layer)
    if bits_cache is not None and key in bits_cache:
        bits = bits_cache[key]
    else:
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


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel of a
# workload, from the committed ncu summary under profiles/ named beside each figure; valid only while
# the kernel's sources are the ones that were profiled (hash of the files), else reported as null.
TRAFFIC = {
    # workload key: (bytes per launch, source files, sha256[:16] of their concatenation, profile)
    "llama_prefill": ((6234150144 + 627657728 + 5631617792 + 619579904) / 2, ('tc_layer.cu', 'tc_common.cuh', 'ptx.cuh'), "61d5a0e50491c749",
                      "profiles/tc_layer_kernel_llama_c5_16384tokens.md (mean of the two layers captured at the headline shape)"),
    "qwen_stack": (865387520 + 955156480, ('tc_stack.cu', 'tc_common.cuh', 'ptx.cuh'), "8fb514fda6c30732", "profiles/tc_stack_kernel_qwen_c2_24layers.md"),
    # decode: captured on 4 of the 32 layers; a launch streams its layers' weights once, so traffic scales with the layers
    "llama_decode_1": ((1470823936 + 4195840) * 8, ('decode_fused.cu', 'ptx.cuh'), "41ae9186018dac22", "profiles/decode_fused_kernel_llama_c4_4layers.md"),
    "llama_decode_8": ((1467553280 + 4698368) * 8, ('decode_fused.cu', 'ptx.cuh'), "41ae9186018dac22", "profiles/decode_fused_kernel_llama_c4_4layers.md"),
    "llama_decode_32": ((1413492992 + 10519040) * 8, ('decode_stack.cu', 'ptx.cuh'), "73796a8498fd42e1", "profiles/decode_stack_kernel_llama_c4_4layers.md"),
    "llama_decode_64": ((1416848384 + 15218944) * 8, ('decode_stack.cu', 'ptx.cuh'), "73796a8498fd42e1", "profiles/decode_stack_kernel_llama_c4_4layers.md"),
}


def sources_sha(files) -> str:
    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2511_21089_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def traffic_for(w):
    """DRAM bytes per launch of workload w's dominant kernel, if w is one of the captured shapes."""
    name = None
    if w["name"] == "llama_prefill" and (w["n"], w["B"], w["ratio"], w["L"]) == (HEADLINE["tokens"], HEADLINE["branches"], HEADLINE["ratio"], 32):
        name = "llama_prefill"
    elif w["name"] == "qwen_stack" and (w["n"], w["L"]) == (synth.CONFIGS[2]["n"], synth.CONFIGS[2]["layers"]):
        name = "qwen_stack"
    elif w["name"] == "llama_decode" and not w.get("prune_k") and w["L"] == 32:
        name = f"llama_decode_{w['n']}"
    if name not in TRAFFIC:
        return None
    nbytes, files, sha, _ = TRAFFIC[name]
    return float(nbytes) if sources_sha(files) == sha else None


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(tflops_burst=p["bf16_tflops"], tflops_sustained=p["bf16_tflops_sustained"], hbm_gbs=p["hbm_gbs"],
                    source="measured")
    return dict(tflops_burst=1590.0, tflops_sustained=1400.0, hbm_gbs=6650.0, source="fallback")


# ------------------------------------------------------------------ oracle leg --
def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i["num_threads"] for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def time_oracle(w, rows: int, n_layers: int, steps: int, warmup: int):
    """The oracle as it stands on a bounded sample of the workload: the first `rows` token rows (tokens are
    independent, so a row sample runs exactly the per-token work of the full batch) through the first
    `n_layers` layers of the stack (all layers have the same shape; the whole-stack time is the sample's
    time x L / n_layers).  Returns (tokens/s of the whole stack, seconds per sampled pass)."""
    import oracle
    layers = []
    for l in range(n_layers):
        bits, d_b, alpha, keep = layer_inputs(l, w)
        host = [synth.bf16_bits_to_f32(b) for b in bits]
        a = alpha if alpha is not None else [1.0] * w["B"]
        layers.append((host[0], host[1], host[2], d_b, oracle.prune_alpha(a, keep) if keep is not None else a))
    x = synth.tokens(w["cfg"], w["n"], w["d"])[:rows]
    for _ in range(warmup):
        oracle.stack_forward(x, layers, bf16_activations=True)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.stack_forward(x, layers, bf16_activations=True)
    dt = (time.perf_counter() - t0) / steps
    return rows / (dt * w["L"] / n_layers), dt


def oracle_sample(w, arm: str):
    """(rows, layers) of the CPU sample.  On Llama-shaped layers a pass costs about 0.3 s per layer (much of it the
    oracle widening the layer's weights to float64, whatever the row count): the one-pass baseline of the default
    run takes 64 rows through the whole stack, the reference arm (steps + warm-up passes) 32 rows through the first
    8 layers."""
    if w["d"] >= 4096:
        return (32, min(8, w["L"])) if arm == "reference" else (64, w["L"])
    return 256, w["L"]


def sample_text(w, rows, nl):
    return (f"first {rows} of {w['n']} token rows through the first {nl} of {w['L']} layers per pass "
            f"(tokens/s = rows / (pass time x {w['L']}/{nl})), numpy float64")


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload(args.workload, args.layers, args.tokens, args.branches, args.ratio, args.prune_k)
    rows, nl = oracle_sample(w, "reference")
    tps, dt = time_oracle(w, rows, nl, args.steps, args.warmup)
    cores = blas_threads()
    sample = sample_text(w, rows, nl)
    out = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": w["label"], "sample": sample},
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


def pick_frac(achieved: float, pk: dict, region_s: float):
    """Roofline fractions of a tensor-bound kernel against both measured bf16 peaks; `frac` takes the one
    that matches the length of the timed region (the burst figure was measured on a short run at boost
    clocks, the sustained one on a seconds-long loop under the power cap)."""
    fb, fs = achieved / pk["tflops_burst"], achieved / pk["tflops_sustained"]
    sustained = region_s >= 1.0
    return dict(frac=fs if sustained else fb, peak=pk["tflops_sustained"] if sustained else pk["tflops_burst"],
                frac_burst=fb, frac_sustained=fs,
                peak_source=f"{pk['source']} ({'sustained' if sustained else 'burst'} bf16 matmul: the timed region lasts {region_s:.2f} s)")


# ------------------------------------------------------------------- CUDA leg --
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str, period_ms: int = 20):
        self.path = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".csv", delete=False).name
        self.f = open(self.path, "w")
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                       "-lms", str(period_ms)], stdout=self.f, stderr=subprocess.DEVNULL)
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
        # the samples taken under load (power well above idle) are the ones that say what the kernels ran at
        busy = [s for s, p in zip(sm, power) if p >= 0.5 * max(power)] or sm
        return {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm), "samples_under_load": len(busy), "power_w_max": float(max(power))}


class Bench:
    """Device-side state shared by the workloads of one run."""

    def __init__(self, args):
        import torch
        import torch.distributed as dist
        from paper_2511_21089_b200 import build
        self.torch, self.dist, self.args = torch, dist, args
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
        torch.cuda.set_device(self.local_rank)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local_rank))
        if self.rank == 0:
            build.build()
        if self.world > 1:
            dist.barrier()
        from paper_2511_21089_b200 import binding
        self.lib = binding
        self.stream = torch.cuda.current_stream()
        self.st = self.stream.cuda_stream
        self.gpu_id = "GPU-" + str(torch.cuda.get_device_properties(self.local_rank).uuid)
        self.dev_weights = {}        # (weight config, layer) -> device tensors, shared by the workloads on the same weights
        self.pk = peaks()

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def weights(self, w, layer):
        torch = self.torch
        key = (4 if w["cfg"] == 5 else w["cfg"], layer)
        if key not in self.dev_weights:
            bits = layer_inputs(layer, w)[0]
            self.dev_weights[key] = [torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).cuda() for b in bits]
        return self.dev_weights[key]

    def drop_weights(self, wcfg=None):
        for k in [k for k in self.dev_weights if wcfg is None or k[0] == wcfg]:
            del self.dev_weights[k]
        self.torch.cuda.empty_cache()

    def create_layers(self, w):
        lib, st = self.lib, self.st
        layers = []
        for l in range(w["L"]):
            _, d_b, alpha, keep = layer_inputs(l, w, bits_cache={(4 if w["cfg"] == 5 else w["cfg"], l): None})
            dev = self.weights(w, l)
            h = lib.mlpmoe_create(w["d"], w["I"], d_b, dev[0], dev[1], dev[2], alpha, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, w["n_max"], st)
            if w.get("fade"):
                lib.mlpmoe_fade(h, None, st)
            if w.get("structured"):
                lib.mlpmoe_fade_structured(h, None, st)
            if keep is not None:
                lib.mlpmoe_prune(h, keep, True, st)
            if layers:
                lib.mlpmoe_share_workspace(h, layers[0])
            layers.append(h)
        self.torch.cuda.synchronize()
        return layers

    def destroy(self, layers):
        for h in layers[1:] + layers[:1]:
            self.lib.mlpmoe_destroy(h)

    def measure(self, w, layers, steps, warmup, e2e=True, kernel_events=True):
        """Times `steps` steps of workload w on the prepared handles; returns the result block."""
        torch, lib, st, args = self.torch, self.lib, self.st, self.args
        n, d, L = w["n"], w["d"], w["L"]
        active = [lib.mlpmoe_get_active_neurons(h) for h in layers]
        x_f32 = rank_batch(w["cfg"], n, d, self.rank)
        y_host = torch.empty((n, d), dtype=torch.float32).pin_memory()
        if w["stack"]:
            x0_host = torch.from_numpy(x_f32).pin_memory()
            x0 = x0_host.cuda()
            xw = torch.empty_like(x0)
            lib.mlpmoe_stack_prepare(layers, n, st)       # set-up (allocation, work sequences) outside the timed region

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

        warmup = max(warmup, 3)
        for _ in range(warmup):
            step()
        self.barrier()
        launches0 = sum(lib.mlpmoe_get_launch_count(h) for h in layers)
        for h in layers:
            lib.mlpmoe_set_timing(h, bool(kernel_events))     # allocates the event pools (set-up)
            lib.mlpmoe_get_timing(h)
            lib.mlpmoe_set_timing(h, False)
        sampler = ClockSampler(self.gpu_id)
        time.sleep(0.25)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # per-kernel events on every k-th step only: a record costs about a microsecond of stream time
        every = 8 if steps >= 16 else 1
        self.barrier()
        e0.record(self.stream)
        for i in range(steps):
            timed = bool(kernel_events) and i % every == 0
            if timed:
                for h in layers:
                    lib.mlpmoe_set_timing(h, True)
            step()
            if timed:
                for h in layers:
                    lib.mlpmoe_set_timing(h, False)
        e1.record(self.stream)
        self.barrier()
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
        # SM clock as the kernels saw it: cycle counter over wall clock inside the last launch of each layer's kernel
        probes = [lib.mlpmoe_get_kernel_clock(h) for h in (layers if not self.is_one_launch(w) else layers[:1])]
        probes = [p for p in probes if p[0] > 0]
        kernel_mhz = float(np.median([p[0] for p in probes])) if probes else None

        e2e_ms = None
        if e2e:
            # end to end through the host-buffer entry point: H2D of x and D2H of y inside the timed region
            for _ in range(2):
                step_host()
            self.barrier()
            e2e_steps = max(3, min(steps, 10))
            t0 = time.perf_counter()
            for _ in range(e2e_steps):
                step_host()                                  # synchronises the stream itself
            e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
            if not np.isfinite(y_host.numpy()).all():
                raise RuntimeError("non-finite output")
        ms_total, e2e_max = max_over_ranks([ms_total, e2e_ms or 0.0], device="cuda")
        ms_step = ms_total / steps
        region_s = ms_total * 1e-3
        pk = self.pk
        flops = [6.0 * n * d * a for a in active]                 # algorithmic FLOPs of each layer call (surviving neurons only)
        wbytes = [3.0 * d * a * 2 for a in active]                # weight bytes each layer call must stream
        weights_gb = sum(wbytes) / 1e9
        out = {
            "workload": w["label"], "value": job_throughput(self.world, n, steps, ms_total), "unit": UNIT, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_step, "timed_region_s": region_s, "gpu_launches": int(launches),
            "tflops": sum(flops) / (ms_step * 1e-3) / 1e12, "weight_gbs": weights_gb / (ms_step * 1e-3),
            "surviving_neurons_per_layer": int(np.mean(active)), "weights_gb_per_step": weights_gb,
            "clocks": dict(clocks, kernel_sm_mhz=kernel_mhz),
        }
        if e2e:
            out["e2e"] = {"value": self.world * n / (e2e_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": in_bytes,
                          "d2h_bytes_per_step": n * d * 4, "ms_per_step": e2e_max}
        if kcnt[0] > 0:
            timed_steps = len(range(0, steps, every))
            ms_timed = ms_total * timed_steps / steps
            main_ms = kms[0] / kcnt[0]
            share = float(kms[0] / ms_timed)
            if n <= 128 and w["stack"]:
                achieved = sum(wbytes) / (main_ms * 1e-3) / 1e9
                # the library's rule (plan_decode): the few-token kernel up to 13 tokens, fewer when few SMs own a neuron tile
                owners = float(np.mean([(a + 127) // 128 for a in active])) / self.torch.cuda.get_device_properties(0).multi_processor_count
                fused_max = 13 if owners > 0.71 else (12 if owners > 0.64 else (7 if owners > 0.38 else 0))
                kernel = ("decode_fused_kernel" if n <= fused_max else "decode_stack_kernel") + \
                    ": whole stack in one persistent launch (bulk-copy weight ring + tcgen05)"
                out["roofline"] = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
                                   "frac": achieved / pk["hbm_gbs"], "traffic": traffic_for(w),
                                   "peak_source": pk["source"] + " (copy bandwidth)", "avg_launch_us": main_ms * 1e3,
                                   "launches_timed": int(kcnt[0]), "share": share, "frac_of_nominal": achieved / 8000.0}
            elif n <= 64:
                achieved = float(np.mean(wbytes)) * 2.0 / 3.0 / (main_ms * 1e-3) / 1e9
                out["roofline"] = {"bound": "hbm", "kernel": "decode_gateup_kernel (TMA weight ring + tcgen05)", "achieved": achieved,
                                   "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": achieved / pk["hbm_gbs"], "traffic": None,
                                   "peak_source": pk["source"] + " (copy bandwidth)", "avg_launch_us": main_ms * 1e3,
                                   "launches_timed": int(kcnt[0]), "share": share, "frac_of_nominal": achieved / 8000.0}
            else:
                one_launch = self.is_one_launch(w)
                per_launch_flops = sum(flops) if one_launch else float(np.mean(flops))
                achieved = per_launch_flops / (main_ms * 1e-3) / 1e12
                kernel = ("tc_stack_kernel: per layer RMSNorm, gate|up GEMM + SiLU*up epilogue, down GEMM + residual add (tcgen05, CTA "
                          "pairs, all layers in one launch)" if one_launch else
                          "tc_layer_kernel: gate|up GEMM + SiLU*up epilogue, then down GEMM + residual add (tcgen05, CTA pairs, one "
                          "launch per layer)")
                rf = {"bound": "tensor", "kernel": kernel, "achieved": achieved, "unit": "TFLOP/s",
                      "traffic": traffic_for(w), "avg_launch_us": main_ms * 1e3, "launches_timed": int(kcnt[0]), "share": share,
                      "frac_of_nominal": achieved / 2250.0}
                rf.update(pick_frac(achieved, pk, region_s))
                if kernel_mhz:
                    # clock-normalised: FLOP per SM cycle against 8192 dense bf16 FLOP per SM cycle (148 SMs)
                    sms = torch.cuda.get_device_properties(self.local_rank).multi_processor_count
                    rf["flop_per_sm_cycle"] = achieved * 1e12 / (kernel_mhz * 1e6 * sms)
                    rf["frac_of_tensor_pipe_at_kernel_clock"] = rf["flop_per_sm_cycle"] / 8192.0
                out["roofline"] = rf
                if kcnt[2] > 0:
                    out["rmsnorm"] = {"avg_us": kms[2] / kcnt[2] * 1e3, "launches_timed": int(kcnt[2]), "share": float(kms[2] / ms_timed)}
        else:
            out["roofline"] = None
        return out

    def measure_fp32(self):
        """configs[0] (one Qwen-shaped fp32 layer, B = 8, all alpha 1): the plain fp32 FMA path against the fast fp32
        mode (six bf16 piece products per product on the tensor cores), at the configuration's 128 tokens and at 4096."""
        torch, lib, st = self.torch, self.lib, self.st
        c = synth.CONFIGS[1]
        d, I, B = c["d_model"], c["d_inter"], c["B"]
        w = synth.layer_weights(1, 0, d, I, 0.02, bf16=False)
        dev = [torch.from_numpy(np.ascontiguousarray(a)).cuda() for a in w]
        n_max = 4096
        h = lib.mlpmoe_create(d, I, synth.equal_partition(I, B), dev[0], dev[1], dev[2], None, lib.MLPMOE_FP32, lib.MLPMOE_LAYOUT_PAPER, n_max, st)
        out = {"workload": f"configs[0]: single Qwen2.5-0.5B-shaped layer, fp32 weights and activations, B={B}, alpha=1"}
        try:
            for n in (c["n"], n_max):
                x = torch.from_numpy(synth.tokens(1, n, d)).cuda()
                y = torch.empty((n, d), dtype=torch.float32, device="cuda")
                res = {}
                for mode in ("plain", "fast"):
                    lib.mlpmoe_set_fast_fp32(h, mode == "fast", st)
                    for _ in range(5):
                        lib.mlpmoe_forward(h, x, y, n, st)
                    steps = 50
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    torch.cuda.synchronize()
                    e0.record(self.stream)
                    for _ in range(steps):
                        lib.mlpmoe_forward(h, x, y, n, st)
                    e1.record(self.stream)
                    torch.cuda.synchronize()
                    ms = e0.elapsed_time(e1) / steps
                    res[mode] = {"ms_per_step": ms, "tokens_per_s": n / (ms * 1e-3), "tflops": 6.0 * n * d * I / (ms * 1e-3) / 1e12}
                res["speedup_fast_over_plain"] = res["plain"]["ms_per_step"] / res["fast"]["ms_per_step"]
                out[f"n{n}"] = res
        finally:
            lib.mlpmoe_destroy(h)
        return out

    def measure_routed(self, k=8):
        """configs[2]'s Llama-shaped layer (B = 32 equal slices, no Fade) under per-token branch selection, every token
        choosing k of the 32 branches uniformly by seed (a labelled extension: the paper names routing as future work
        only), against the plain forward of the same layer on the same tokens."""
        torch, lib, st = self.torch, self.lib, self.st
        w = workload("llama_layer_fade")
        w = dict(w, fade=False, n_max=w["n"])
        n, d, B = w["n"], w["d"], w["B"]
        hs = self.create_layers(w)
        h = hs[0]
        out = {"workload": f"configs[2] shapes: single Llama-3-8B-shaped layer, bf16, B={B} equal slices, {n} tokens, every token "
                           f"selects {k} of {B} branches (seeded), compensation sqrt(B/k)"}
        try:
            xb = synth.f32_to_bf16_bits(rank_batch(w["cfg"], n, d, self.rank))
            x = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).cuda()
            y = torch.empty((n, d), dtype=torch.float32, device="cuda")
            sel = torch.from_numpy(synth.route_select((synth.BASE_SEED, w["cfg"], synth.T_ROUTE), n, B, k)).cuda()
            res = {}
            for mode in ("dense", "routed"):
                def step():
                    if mode == "dense":
                        lib.mlpmoe_forward(h, x, y, n, st)
                    else:
                        lib.mlpmoe_forward_routed(h, x, y, n, sel, True, st)
                for _ in range(5):
                    step()
                steps = 50
                l0 = lib.mlpmoe_get_launch_count(h)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record(self.stream)
                for _ in range(steps):
                    step()
                e1.record(self.stream)
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / steps
                frac = 1.0 if mode == "dense" else k / B
                res[mode] = {"ms_per_step": ms, "tokens_per_s": n / (ms * 1e-3), "tflops": 6.0 * n * d * w["I"] * frac / (ms * 1e-3) / 1e12,
                             "gpu_launches_per_step": (lib.mlpmoe_get_launch_count(h) - l0) / steps}
            assert lib.mlpmoe_get_status(h) == lib.MLPMOE_OK
            res["flop_ratio_routed_over_dense"] = k / B
            res["time_ratio_routed_over_dense"] = res["routed"]["ms_per_step"] / res["dense"]["ms_per_step"]
            out.update(res)
        finally:
            self.destroy(hs)
        return out

    def is_one_launch(self, w):
        """Whether a stack call of workload w is one persistent launch (up to 128 tokens always; prefill when the layers stay in L2)."""
        if not w["stack"]:
            return False
        return w["n"] <= 128 or 3 * w["d"] * w["I"] * 2 <= (48 << 20)


def run_ours(args):
    b = Bench(args)
    lib = b.lib
    single = args.workload is not None
    if args.workload == "llama_layer_routed":
        out = b.measure_routed()
        if b.rank == 0:
            print(json.dumps({"configs": {"c3_llama_layer_routed": out}}))
        return
    if args.workload == "qwen_layer_fp32":
        # the fp32 block of the default line by itself (profiling captures of the fast fp32 kernels)
        out = b.measure_fp32()
        if b.rank == 0:
            print(json.dumps({"configs": {"c1_qwen_layer_fp32": out}}))
        return
    w = workload(args.workload or HEADLINE["name"], args.layers, args.tokens, args.branches, args.ratio, args.prune_k)
    w["n_max"] = w["n"]
    layers = b.create_layers(w)
    head = b.measure(w, layers, args.steps, args.warmup, e2e=True, kernel_events=bool(args.kernel_events))
    b.destroy(layers)
    extras = {}
    if b.world == 1 and not single and not args.no_extras:
        # configs[3]: decode on the same Llama-shaped weights, B = 64 equal slices, unpruned then first-K pruning K = 51
        dsteps = 200
        for K in (None, 51):
            wd = workload("llama_decode", tokens=64, prune_k=K)
            wd["n_max"] = 64
            hs = b.create_layers(wd)
            for n in (1, 8, 32, 64):
                wn = dict(wd, n=n, label=workload("llama_decode", tokens=n, prune_k=K)["label"])
                extras[f"c4_decode_n{n}" + ("_k51" if K else "")] = b.measure(wn, hs, dsteps, 20, e2e=(n == 64))
            b.destroy(hs)
        ratios = {}
        for n in (1, 8, 32, 64):
            full, pruned = extras[f"c4_decode_n{n}"], extras[f"c4_decode_n{n}_k51"]
            ratios[f"n{n}"] = {"time_ratio_pruned_over_unpruned": pruned["ms_per_step"] / full["ms_per_step"],
                               "byte_ratio": pruned["weights_gb_per_step"] / full["weights_gb_per_step"]}
        extras["c4_decode_pruning"] = ratios
        b.drop_weights()
        # configs[2]: one Llama-shaped layer with Fractal Fade
        wf = workload("llama_layer_fade")
        wf["n_max"] = wf["n"]
        hs = b.create_layers(wf)
        extras["c3_llama_layer_fade"] = b.measure(wf, hs, 300, 20)
        b.destroy(hs)
        # the same layer under the neuron-structured Fade variant (same schedule, whole neurons removed): the only
        # form of Fade that takes work off the dense tensor-core tiles
        ws = dict(wf, fade=False, structured=True,
                  label=wf["label"].replace("Fractal Fade s_b=0.9b/B", "neuron-structured Fade variant (labelled; not the paper's element-wise mask), s_b=0.9b/B"))
        hs = b.create_layers(ws)
        extras["c3_llama_layer_structured_fade"] = b.measure(ws, hs, 300, 20, e2e=False)
        extras["c3_llama_layer_structured_fade"]["time_ratio_over_elementwise_fade"] = \
            extras["c3_llama_layer_structured_fade"]["ms_per_step"] / extras["c3_llama_layer_fade"]["ms_per_step"]
        extras["c3_llama_layer_structured_fade"]["neuron_ratio"] = \
            extras["c3_llama_layer_structured_fade"]["surviving_neurons_per_layer"] / extras["c3_llama_layer_fade"]["surviving_neurons_per_layer"]
        b.destroy(hs)
        extras["c3_llama_layer_routed"] = b.measure_routed()
        b.drop_weights()
        extras["c1_qwen_layer_fp32"] = b.measure_fp32()
        # configs[1]: the 24-layer Qwen-shaped stack
        wq = workload("qwen_stack")
        wq["n_max"] = wq["n"]
        hs = b.create_layers(wq)
        extras["c2_qwen_stack"] = b.measure(wq, hs, 800, 20)
        b.destroy(hs)
        b.drop_weights()

    if b.rank == 0:
        default = (not single) and args.layers is None
        out = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": b.world, "steps": args.steps, "warmup": head["warmup"],
            "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": head["workload"] + ("" if default or single else f" [REDUCED to {w['L']} layers]"),
                       "l2": f"inputs larger than L2: each step streams {head['weights_gb_per_step']:.2f} GB of distinct weights",
                       "surviving_neurons_per_layer": head["surviving_neurons_per_layer"], "tokens_per_rank": w["n"]},
            "clocks": head["clocks"], "e2e": head.get("e2e"), "gpu_launches": head["gpu_launches"], "tflops": head["tflops"],
            "weight_gbs": head["weight_gbs"], "timed_region_s": head["timed_region_s"], "roofline": head["roofline"],
        }
        if "rmsnorm" in head:
            out["rmsnorm"] = head["rmsnorm"]
        if extras:
            out["configs"] = extras
        if b.world == 1 and not args.no_cpu_baseline:
            rows, nl = oracle_sample(w, "baseline")
            tps, dt = time_oracle(w, rows, nl, 1, 0)
            out["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                   "sample": sample_text(w, rows, nl) + f", one pass of {dt:.1f} s"}
        else:
            out["cpu_baseline"] = None
        print(json.dumps(out))
    if b.world > 1:
        b.dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--layers", type=int, default=None, help="fewer layers of the same stack (profiling captures only)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=None, choices=["qwen_stack", "llama_decode", "llama_layer_fade", "llama_prefill", "qwen_layer_fp32", "llama_layer_routed"],
                    help="measure this workload alone (default: the headline workload plus the other configurations)")
    ap.add_argument("--tokens", type=int, default=None)
    ap.add_argument("--branches", type=int, default=None)
    ap.add_argument("--ratio", type=float, default=None)
    ap.add_argument("--prune-k", type=int, default=None)
    ap.add_argument("--kernel-events", type=int, default=1, help="record per-kernel CUDA events in the timed region")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="headline workload only")
    args = ap.parse_args()
    if args.impl == "reference":
        args.workload = args.workload or HEADLINE["name"]
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
