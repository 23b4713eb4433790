"""Plain fp64 CPU oracle for the MLPMoE layer (arXiv 2511.21089).

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement
of what the CUDA library must compute.  It is written from the paper's
equations, uses numpy in float64 throughout, does no blocking, fusion or
reordering beyond what the equations state, and shares no code with the CUDA
path.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import it; the product never does.

Notation follows the paper (Section 3.1):
    d = d_model, I = d_inter, B branches of widths d_b (contiguous slices of I),
    W_gate, W_up in R^{d x I}, W_down in R^{I x d}, alpha_b one scalar per branch.
The paper writes "W x" for a matrix whose stated shape is d_model x d_inter; the
only dimensionally consistent reading is g_j = sum_k x_k W_gate[k, j] and
y_m = sum_j h_j W_down[j, m], which is what is computed here, with tokens as
rows of x (each token is independent of all others).

Branch indices are 0-based, as in the paper's Fade ("branch index i > 0") and
pruning ("b < K") formulas.

Pins (see tests/test_oracle_*.py): dense-SwiGLU identity at alpha = 1
(Section 3.1, last sentence), invariance to the partition (Section 2.2
identity), brute-force scalar evaluation of tiny cases, hand-computed golden
values, closed-form Fade zero counts and the paper's Table 1 / Table 2
non-zero parameter counts, top-k-by-magnitude brute force for the Fade mask,
exact sqrt(B/K) values and the variance-preservation claim of Section 3.3.
fade_structured / neuron_scores are a labelled variant of this build (no passage
of the paper defines them): pinned by a scalar brute force, the closed-form
count of removed neurons and exact small-integer cases.
routed_forward is a labelled extension too (the paper names dynamic routing as
future work only): pinned by its two special cases that the paper does define
(all branches selected = the layer; one shared set = Compensated Pruning,
Section 3.3), by a scalar brute force and by hand-computed values.
The paper's perplexity and generation-time figures need trained checkpoints
and an unpublished text mixture: parity unpinned for those (out of scope).
"""
from __future__ import annotations

import math
from fractions import Fraction
from typing import List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------- #
# Section 3.1: partition, branch forward, branch sum
# --------------------------------------------------------------------------- #
def branch_offsets(d_b: Sequence[int], d_inter: Optional[int] = None) -> List[int]:
    """Start offsets o_b of the contiguous slices, o_b = sum_{c<b} d_c (Section 3.1:
    d_inter = sum_b d_b).  Returns B+1 offsets; the last one is d_inter."""
    offs = [0]
    for w in d_b:
        w = int(w)
        if w <= 0:
            raise ValueError("every branch width d_b must be positive")
        offs.append(offs[-1] + w)
    if d_inter is not None and offs[-1] != int(d_inter):
        raise ValueError("branch widths must sum to d_inter")
    return offs


def silu(g: np.ndarray) -> np.ndarray:
    """phi(g) = g * sigmoid(g) = g / (1 + exp(-g)); the paper leaves phi generic
    (Section 3.1) and targets Qwen / Llama MLPs, whose gate activation is SiLU."""
    g = np.asarray(g, dtype=np.float64)
    with np.errstate(over="ignore"):
        return g / (1.0 + np.exp(-g))


def branch_forward(x, W_gate, W_up, W_down, lo: int, hi: int, alpha_b: float) -> np.ndarray:
    """branch_b(x) = alpha_b * W_down^(b) [ phi(W_gate^(b) x) (.) W_up^(b) x ]
    (Section 3.1, branch equation).  The sub-matrices are the column slice
    [lo, hi) of W_gate / W_up and the row slice [lo, hi) of W_down."""
    x = np.asarray(x, dtype=np.float64)
    Wg = np.asarray(W_gate)[:, lo:hi].astype(np.float64)
    Wu = np.asarray(W_up)[:, lo:hi].astype(np.float64)
    Wd = np.asarray(W_down)[lo:hi, :].astype(np.float64)
    g = x @ Wg
    u = x @ Wu
    h = silu(g) * u
    return float(alpha_b) * (h @ Wd)


def mlpmoe_forward(x, W_gate, W_up, W_down, d_b: Sequence[int],
                   alpha: Optional[Sequence[float]] = None) -> np.ndarray:
    """MLPMoE(x) = sum_b branch_b(x), summed in ascending b (Section 3.1, layer
    equation).  x: [n, d]; returns [n, d] float64.  alpha=None means all 1.0
    (the paper's initial value)."""
    x = np.asarray(x, dtype=np.float64)
    d, I = np.asarray(W_gate).shape
    if x.ndim != 2 or x.shape[1] != d:
        raise ValueError("x must be [n, d_model]")
    if np.asarray(W_up).shape != (d, I) or np.asarray(W_down).shape != (I, d):
        raise ValueError("weight shapes must be [d, I], [d, I], [I, d]")
    offs = branch_offsets(d_b, I)
    B = len(d_b)
    if alpha is None:
        alpha = [1.0] * B
    if len(alpha) != B:
        raise ValueError("alpha must have one entry per branch")
    y = np.zeros((x.shape[0], d), dtype=np.float64)
    for b in range(B):
        y = y + branch_forward(x, W_gate, W_up, W_down, offs[b], offs[b + 1], alpha[b])
    return y


# --------------------------------------------------------------------------- #
# Section 3.2: Fractal Fade
# --------------------------------------------------------------------------- #
def fade_schedule(B: int) -> List[Fraction]:
    """s_i = 0.9 * i / B for branch index i > 0; branch 0 is the dense backbone
    (s_0 = 0, never masked).  Kept as exact rationals 9 i / (10 B)."""
    return [Fraction(9 * i, 10 * B) for i in range(B)]


def _as_fraction(s) -> Fraction:
    # Fraction(float) is exact, so a schedule given in floating point is taken
    # at the exact value of the double.
    return s if isinstance(s, Fraction) else Fraction(s)


def fade_position(s, m: int) -> Tuple[int, Fraction]:
    """Position of the s-quantile among m sorted values (the usual linear
    definition): p = s (m - 1), split into the lower order statistic index
    lo = floor(p) and the fraction p - lo.  Exact arithmetic."""
    p = _as_fraction(s) * (m - 1)
    lo = p.numerator // p.denominator
    return int(lo), p - lo


def fade_mask(w: np.ndarray, s) -> np.ndarray:
    """Keep-mask of one projection of one branch under Fractal Fade (Section 3.2:
    magnitude pruning of the slice at sparsity ratio s), stated by rank: with the
    m magnitudes |w| (as float32) sorted ascending into a[0..m-1] and
    lo = floor(s (m - 1)) in exact rational arithmetic, an entry is kept iff
    |w| > a[lo].  Entries that tie with a[lo] go as well.

    This is the set that the s-quantile threshold of Section 4 (linear
    interpolation between a[lo] and a[lo+1], strict '>') selects: that threshold
    t satisfies a[lo] <= t < a[lo+1] when the two differ and t = a[lo] otherwise,
    so {|w| > t} = {|w| > a[lo]}; tests/test_oracle_fade_prune.py checks the
    equivalence with the threshold evaluated in exact rationals.
    s == 0 means "leave untouched" (the paper's branch 0)."""
    s = _as_fraction(s)
    if not (0 <= s < 1):
        raise ValueError("sparsity ratio must lie in [0, 1)")
    w = np.asarray(w)
    if s == 0:
        return np.ones(w.shape, dtype=bool)
    w_abs = np.abs(w.astype(np.float32))
    a = np.sort(w_abs, axis=None)
    lo, _ = fade_position(s, a.size)
    return w_abs > a[lo]


def fade(W_gate, W_up, d_b: Sequence[int], s: Optional[Sequence] = None):
    """Apply Fractal Fade to W_gate and W_up (W_down is not touched): for every
    branch b with s_b > 0, and for the gate and the up projection separately,
    zero the entries of that branch's slice that are not above the slice's own
    s_b-quantile of magnitudes.  Returns masked copies (same dtype)."""
    Wg = np.array(W_gate, copy=True)
    Wu = np.array(W_up, copy=True)
    B = len(d_b)
    offs = branch_offsets(d_b, Wg.shape[1])
    if s is None:
        s = fade_schedule(B)
    if len(s) != B:
        raise ValueError("schedule must have one entry per branch")
    for b in range(B):
        if _as_fraction(s[b]) == 0:
            continue
        for W in (Wg, Wu):
            sl = W[:, offs[b]:offs[b + 1]]
            keep = fade_mask(sl, s[b])
            sl *= keep.astype(W.dtype)
    return Wg, Wu


def neuron_scores(W_gate, W_up) -> np.ndarray:
    """score_j = sum_k W_gate[k, j]^2 + sum_k W_up[k, j]^2 in float64, the terms added
    one after the other in that order (the gate column first), so that any program
    adding the same terms in the same order gets the same bits (the products of
    float32 or bfloat16 values are exact in float64; the order fixes the sums)."""
    g = np.asarray(W_gate).astype(np.float64)
    u = np.asarray(W_up).astype(np.float64)
    terms = np.concatenate([(g * g).T, (u * u).T], axis=1)        # [I, 2 d]: neuron j's terms in order
    return np.cumsum(terms, axis=1)[:, -1]                        # a running sum is sequential by construction


def fade_structured_count(s, d_b: int) -> int:
    """q = floor(s * d_b) neurons leave a branch of width d_b (exact arithmetic)."""
    p = _as_fraction(s) * d_b
    return int(p.numerator // p.denominator)


def fade_structured(W_gate, W_up, d_b: Sequence[int], s: Optional[Sequence] = None):
    """Neuron-structured Fade, a labelled variant of Section 3.2 (NOT the paper's
    definition, which masks single weights): with the same schedule s_b, branch b
    loses its q_b = floor(s_b d_b) neurons of smallest neuron_scores, ties to the
    lower index first; their W_gate and W_up columns become zero, W_down stays.
    Returns masked copies."""
    Wg = np.array(W_gate, copy=True)
    Wu = np.array(W_up, copy=True)
    B = len(d_b)
    offs = branch_offsets(d_b, Wg.shape[1])
    if s is None:
        s = fade_schedule(B)
    if len(s) != B:
        raise ValueError("schedule must have one entry per branch")
    score = neuron_scores(Wg, Wu)
    for b in range(B):
        sb = _as_fraction(s[b])
        if not (0 <= sb < 1):
            raise ValueError("sparsity ratio must lie in [0, 1)")
        q = fade_structured_count(sb, int(d_b[b]))
        if sb == 0 or q == 0:
            continue
        order = np.argsort(score[offs[b]:offs[b + 1]], kind="stable")      # ascending, ties to the lower index
        gone = offs[b] + order[:q]
        Wg[:, gone] = 0
        Wu[:, gone] = 0
    return Wg, Wu


# --------------------------------------------------------------------------- #
# Section 3.3: Compensated Branch Pruning
# --------------------------------------------------------------------------- #
def first_k_keep(B: int, K: int) -> List[bool]:
    """The paper's rule: retain the first K branches (b < K)."""
    if not (1 <= K <= B):
        raise ValueError("K must lie in 1..B")
    return [b < K for b in range(B)]


def prune_alpha(alpha: Sequence[float], keep: Sequence[bool], compensate: bool = True) -> List[float]:
    """alpha_b <- alpha_b * sqrt(B / K) for kept branches and 0 for the others,
    K = number of kept branches (Section 3.3; with the paper's alpha = 1 this is
    exactly its piecewise formula).  compensate=False drops without rescaling."""
    B = len(alpha)
    if len(keep) != B:
        raise ValueError("keep must have one entry per branch")
    K = sum(1 for k in keep if k)
    if K == 0:
        raise ValueError("the keep set is empty")
    c = math.sqrt(B / K) if compensate else 1.0
    return [float(alpha[b]) * c if keep[b] else 0.0 for b in range(B)]


def mlpmoe_forward_h_bf16(x, W_gate, W_up, W_down, d_b: Sequence[int],
                          alpha: Optional[Sequence[float]] = None) -> np.ndarray:
    """The layer equation of Section 3.1 with ONE rounding added, the one a bf16
    implementation that keeps the intermediate in bf16 commits: per branch
    h = bf16(alpha_b * phi(W_gate^(b) x) (.) W_up^(b) x), then y = sum_b W_down^(b) h.
    Everything else stays float64.  Not the paper's arithmetic (the paper fixes no
    precision): a model of the stated storage format, used to check a bf16 kernel
    far more tightly than the paper-level tolerance allows.  |y - mlpmoe_forward|
    is bounded by 2^-9 * sum_j |h_j W_down[j, m]| (half an ulp per h)."""
    x = np.asarray(x, dtype=np.float64)
    d, I = np.asarray(W_gate).shape
    offs = branch_offsets(d_b, I)
    B = len(d_b)
    if alpha is None:
        alpha = [1.0] * B
    y = np.zeros((x.shape[0], d), dtype=np.float64)
    for b in range(B):
        lo, hi = offs[b], offs[b + 1]
        g = x @ np.asarray(W_gate)[:, lo:hi].astype(np.float64)
        u = x @ np.asarray(W_up)[:, lo:hi].astype(np.float64)
        h = round_to_bf16(float(alpha[b]) * (silu(g) * u))
        y = y + h @ np.asarray(W_down)[lo:hi, :].astype(np.float64)
    return y


def routed_forward(x, W_gate, W_up, W_down, d_b: Sequence[int], alpha: Sequence[float], select,
                   compensate: bool = True) -> np.ndarray:
    """Per-token branch selection, a labelled extension (NOT defined by the paper:
    Section 7, Limitation 2, and the outlook of Section 8 only name dynamic routing
    over branches as future work).  The rule, stated here: token t evaluates the
    branches S_t = {b : select[t, b] != 0 and alpha_b != 0} and nothing else,

        y_t = c_t * sum_{b in S_t} branch_b(x_t),   c_t = sqrt(B' / |S_t|),

    B' = number of branches with alpha_b != 0: Section 3.3's compensation with the
    token's own K = |S_t|.  |S_t| = 0 gives y_t = 0; compensate=False gives c_t = 1.
    With every available branch selected it is mlpmoe_forward; with one set S shared
    by all tokens and all alpha_b != 0 it is the layer after prune_alpha(alpha, S).
    The selection itself (a router) is an input: the paper defines none."""
    x = np.asarray(x, dtype=np.float64)
    sel = np.asarray(select)
    B = len(d_b)
    if sel.shape != (x.shape[0], B):
        raise ValueError("select must be [n_tokens x B]")
    offs = branch_offsets(d_b, np.asarray(W_gate).shape[1])
    avail = [b for b in range(B) if float(alpha[b]) != 0.0]
    chosen = np.zeros((x.shape[0], B), dtype=bool)
    for b in avail:
        chosen[:, b] = sel[:, b] != 0
    acc = np.zeros((x.shape[0], np.asarray(W_down).shape[1]), dtype=np.float64)
    for b in avail:                      # ascending b: every token's sum runs in the layer equation's order
        rows = np.nonzero(chosen[:, b])[0]
        if rows.size:
            acc[rows] += branch_forward(x[rows], W_gate, W_up, W_down, offs[b], offs[b + 1], float(alpha[b]))
    k = chosen.sum(axis=1)
    c = np.zeros(x.shape[0], dtype=np.float64)
    c[k > 0] = np.sqrt(len(avail) / k[k > 0]) if compensate else 1.0
    return c[:, None] * acc


# --------------------------------------------------------------------------- #
# Bookkeeping the scheduler must reproduce exactly
# --------------------------------------------------------------------------- #
def nnz_per_branch(W_gate, W_up, W_down, d_b: Sequence[int]):
    """Non-zero entries per branch of each projection (the paper's "Non-zero
    Params" column counts entries != 0)."""
    offs = branch_offsets(d_b, np.asarray(W_gate).shape[1])
    g = [int(np.count_nonzero(np.asarray(W_gate)[:, offs[b]:offs[b + 1]])) for b in range(len(d_b))]
    u = [int(np.count_nonzero(np.asarray(W_up)[:, offs[b]:offs[b + 1]])) for b in range(len(d_b))]
    dn = [int(np.count_nonzero(np.asarray(W_down)[offs[b]:offs[b + 1], :])) for b in range(len(d_b))]
    return g, u, dn


def live_neurons(W_gate, W_up, W_down) -> np.ndarray:
    """Neuron j can contribute to y only if column j of W_gate, column j of W_up
    and row j of W_down each hold a non-zero (silu(0) = 0, 0 * u = 0, h * 0 = 0)."""
    return (np.any(np.asarray(W_gate) != 0, axis=0)
            & np.any(np.asarray(W_up) != 0, axis=0)
            & np.any(np.asarray(W_down) != 0, axis=1))


def surviving_set(alpha: Sequence[float], W_gate, W_up, W_down, d_b: Sequence[int]):
    """Branches and neuron runs that still have to be computed: a branch
    survives iff alpha_b != 0 and it holds a live neuron; inside it, maximal runs
    of consecutive live neurons.  Returns (branches, segments) with segments a
    list of (start, length) in ascending order, never crossing a branch boundary."""
    offs = branch_offsets(d_b, np.asarray(W_gate).shape[1])
    live = live_neurons(W_gate, W_up, W_down)
    branches: List[int] = []
    segments: List[Tuple[int, int]] = []
    for b in range(len(d_b)):
        if float(alpha[b]) == 0.0:
            continue
        run_start = None
        found = False
        for j in range(offs[b], offs[b + 1]):
            if live[j]:
                found = True
                if run_start is None:
                    run_start = j
            elif run_start is not None:
                segments.append((run_start, j - run_start))
                run_start = None
        if run_start is not None:
            segments.append((run_start, offs[b + 1] - run_start))
        if found:
            branches.append(b)
    return branches, segments


def mlpmoe_forward_skiplist(x, W_gate, W_up, W_down, d_b, alpha) -> np.ndarray:
    """The layer evaluated over the surviving set only.  Must agree with
    mlpmoe_forward (which multiplies through the zeros) for finite inputs."""
    x = np.asarray(x, dtype=np.float64)
    offs = branch_offsets(d_b, np.asarray(W_gate).shape[1])
    _, segments = surviving_set(alpha, W_gate, W_up, W_down, d_b)
    y = np.zeros((x.shape[0], np.asarray(W_down).shape[1]), dtype=np.float64)
    for start, length in segments:
        b = max(i for i in range(len(d_b)) if offs[i] <= start)
        y = y + branch_forward(x, W_gate, W_up, W_down, start, start + length, alpha[b])
    return y


# --------------------------------------------------------------------------- #
# Stack harness: x <- x + MLPMoE_l(RMSNorm(x)) (not in the paper; the benchmark
# configurations wrap the layer this way)
# --------------------------------------------------------------------------- #
def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even) and return them
    as float64.  bfloat16 = the upper 16 bits of an IEEE float32."""
    f = np.asarray(a, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    bias = ((bits >> 16) & 1) + 0x7FFF
    r = ((bits + bias) >> 16) << 16
    return r.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


def rmsnorm(x: np.ndarray, eps: float = 1e-6) -> np.ndarray:
    """r = x / sqrt(mean(x^2) + eps) per token row, unit gain."""
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x, axis=1, keepdims=True) + eps)


def stack_forward(x, layers, bf16_activations: bool = True, eps: float = 1e-6,
                  return_layer_inputs: bool = False):
    """Pre-norm residual stack of MLPMoE layers.  `layers` is a sequence of
    (W_gate, W_up, W_down, d_b, alpha).  With bf16_activations the normalised
    input of every layer is rounded to bfloat16 (the layer's input dtype) first.
    The residual stream itself stays in float64."""
    x = np.asarray(x, dtype=np.float64)
    inputs = []
    for (Wg, Wu, Wd, d_b, alpha) in layers:
        if return_layer_inputs:
            inputs.append(x.copy())
        r = rmsnorm(x, eps)
        if bf16_activations:
            r = round_to_bf16(r)
        x = x + mlpmoe_forward(r, Wg, Wu, Wd, d_b, alpha)
    return (x, inputs) if return_layer_inputs else x
