"""Seeded synthetic inputs for the MLPMoE forward path.

This module only draws numbers: weights, activations, partitions, keep sets and
gate values with the shapes and value distributions of the workloads (Qwen2.5-
0.5B- and Llama-3-8B-shaped MLPs stand in for the checkpoints the paper used).
It contains none of the method's arithmetic and is the one module that both the
CPU oracle's tests and the CUDA path's callers may use.

Every tensor is addressed by a key (base seed, config, layer, tensor id) and is
filled in fixed-size blocks, each block from its own counter-based Philox stream,
so the values do not depend on how many host threads fill it.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from typing import List, Sequence

import numpy as np

BASE_SEED = 20251121

# tensor ids
T_GATE, T_UP, T_DOWN, T_X, T_ALPHA, T_KEEP, T_PARTITION, T_ROUTE = range(8)

_BLOCK = 1 << 20


def _rng(key: Sequence[int], block: int = 0) -> np.random.Generator:
    ss = np.random.SeedSequence(entropy=[int(k) & 0xFFFFFFFF for k in key] + [int(block)])
    return np.random.Generator(np.random.Philox(ss))


def normal_f32(key: Sequence[int], shape, std: float = 1.0, threads: int | None = None) -> np.ndarray:
    """float32 N(0, std^2) tensor of the given shape, reproducible from `key`."""
    total = int(np.prod(shape))
    out = np.empty(total, dtype=np.float32)
    nblocks = (total + _BLOCK - 1) // _BLOCK

    def fill(i: int) -> None:
        lo = i * _BLOCK
        hi = min(total, lo + _BLOCK)
        g = _rng(key, i)
        out[lo:hi] = g.standard_normal(hi - lo, dtype=np.float32)
        if std != 1.0:
            out[lo:hi] *= np.float32(std)

    if threads is None:
        threads = min(16, os.cpu_count() or 1)
    if nblocks > 1 and threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(nblocks)))
    else:
        for i in range(nblocks):
            fill(i)
    return out.reshape(shape)


def uniform_f64(key: Sequence[int], n: int, lo: float, hi: float) -> np.ndarray:
    return _rng(key).uniform(lo, hi, size=n)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((bits >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((bits + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to the float32 values they denote."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def equal_partition(d_inter: int, B: int) -> List[int]:
    if d_inter % B:
        raise ValueError("d_inter is not divisible by B")
    return [d_inter // B] * B


def random_partition(key: Sequence[int], d_inter: int, B: int, unit: int = 64) -> List[int]:
    """B unequal contiguous slices, each a positive multiple of `unit`: choose B-1
    distinct cut points among the interior unit boundaries."""
    units = d_inter // unit
    if d_inter % unit or B > units:
        raise ValueError("cannot cut d_inter into B multiples of unit")
    cuts = np.sort(_rng(key).choice(np.arange(1, units), size=B - 1, replace=False)) if B > 1 else np.array([], dtype=np.int64)
    edges = np.concatenate([[0], cuts, [units]]).astype(np.int64)
    return [int(w) * unit for w in np.diff(edges)]


def keep_set(key: Sequence[int], B: int, n_drop: int) -> List[bool]:
    """Keep mask with exactly n_drop branches dropped, chosen uniformly by seed."""
    if not (0 <= n_drop < B):
        raise ValueError("n_drop must lie in 0..B-1")
    keep = np.ones(B, dtype=bool)
    if n_drop:
        keep[_rng(key).choice(B, size=n_drop, replace=False)] = False
    return [bool(k) for k in keep]


def route_select(key: Sequence[int], n: int, B: int, k: int) -> np.ndarray:
    """Selection bytes [n, B] of a per-token routing: every token selects exactly k distinct
    branches, uniformly by seed (the k smallest of B independent uniform draws)."""
    if not (0 <= k <= B):
        raise ValueError("k must lie in 0..B")
    sel = np.zeros((n, B), dtype=np.uint8)
    if k:
        order = np.argsort(_rng(key).random((n, B)), axis=1, kind="stable")[:, :k]
        np.put_along_axis(sel, order, 1, axis=1)
    return sel


def n_drop_for_ratio(B: int, ratio: float) -> int:
    """Number of branches to drop for a pruning ratio: round half up."""
    return int(np.floor(ratio * B + 0.5))


def layer_weights(cfg: int, layer: int, d_model: int, d_inter: int, std: float = 0.02,
                  bf16: bool = True, seed: int = BASE_SEED):
    """(W_gate [d, I], W_up [d, I], W_down [I, d]) in the paper's stated shapes,
    row-major, entries ~ N(0, std^2).  With bf16=True the float32 draws are
    rounded to bfloat16 and returned as uint16 bit patterns."""
    wg = normal_f32((seed, cfg, layer, T_GATE), (d_model, d_inter), std)
    wu = normal_f32((seed, cfg, layer, T_UP), (d_model, d_inter), std)
    wd = normal_f32((seed, cfg, layer, T_DOWN), (d_inter, d_model), std)
    if bf16:
        return f32_to_bf16_bits(wg), f32_to_bf16_bits(wu), f32_to_bf16_bits(wd)
    return wg, wu, wd


def tokens(cfg: int, n: int, d_model: int, seed: int = BASE_SEED, stream: int = 0) -> np.ndarray:
    """x: [n, d_model] float32 ~ N(0, 1)."""
    return normal_f32((seed, cfg, stream, T_X), (n, d_model), 1.0)


# The five workload configurations (shapes only; see the bench and the tests
# for how each is run).
CONFIGS = {
    1: dict(name="qwen_fp32_single", d_model=896, d_inter=4864, B=8, n=128, layers=1, bf16=False),
    2: dict(name="qwen_stack_pruned", d_model=896, d_inter=4864, B=16, n=4096, layers=24, bf16=True, n_drop=4),
    3: dict(name="llama_single_fade", d_model=4096, d_inter=14336, B=32, n=8192, layers=1, bf16=True),
    4: dict(name="llama_decode", d_model=4096, d_inter=14336, B=64, n=(1, 8, 32, 64), layers=32, bf16=True, first_k=51),
    5: dict(name="llama_prefill_sweep", d_model=4096, d_inter=14336, B=(4, 8, 16, 32, 64, 128), n=(2048, 16384),
            layers=32, bf16=True, ratios=(0.0, 0.1, 0.2, 0.4)),
}
