"""Pins for the oracle's forward pass (Section 3.1), none of which re-use the
oracle's own formula: hand-computed goldens, a scalar brute force, the dense
SwiGLU identity evaluated with a different library (torch), invariance under
re-partitioning, linearity in alpha, and planted-mistake checks showing that the
pins catch the usual slips."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import mlpmoe_oracle as mo

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v) if "." in v else int(v)
    return out


def brute_force(x, Wg, Wu, Wd, d_b, alpha):
    """Literal scalar evaluation of the branch and layer equations."""
    n, d = len(x), len(x[0])
    y = [[0.0] * d for _ in range(n)]
    off = 0
    for b, w in enumerate(d_b):
        for t in range(n):
            for j in range(off, off + w):
                g = sum(x[t][k] * Wg[k][j] for k in range(d))
                u = sum(x[t][k] * Wu[k][j] for k in range(d))
                h = g * (1.0 / (1.0 + math.exp(-g))) * u
                for m in range(d):
                    y[t][m] += alpha[b] * h * Wd[j][m]
        off += w
    return np.array(y)


def rand_case(rng, n, d, I):
    return (rng.standard_normal((n, d)), rng.standard_normal((d, I)) * 0.5,
            rng.standard_normal((d, I)) * 0.5, rng.standard_normal((I, d)) * 0.5)


def test_golden_two_branches():
    g = read_golden("tiny_forward.txt")
    ln3 = math.log(3.0)
    x = [[1.0]]
    Wg = [[ln3, -ln3]]
    Wu = [[2.0, 4.0]]
    Wd = [[1.0], [1.0]]
    y = oracle.mlpmoe_forward(x, Wg, Wu, Wd, [1, 1], [1.0, 1.0])
    assert y.shape == (1, 1)
    assert y[0, 0] == pytest.approx(g["two_branches_alpha_1_1"], rel=1e-14)
    y = oracle.mlpmoe_forward(x, Wg, Wu, Wd, [1, 1], [2.0, 0.5])
    assert y[0, 0] == pytest.approx(g["two_branches_alpha_2_half"], rel=1e-14)


def test_golden_asymmetric():
    g = read_golden("tiny_forward.txt")
    ln3 = math.log(3.0)
    y = oracle.mlpmoe_forward([[1.0, 0.0]], [[ln3], [100.0]], [[2.0], [50.0]], [[1.0, 10.0]], [1])
    assert y[0, 0] == pytest.approx(g["asymmetric_y0"], rel=1e-14)
    assert y[0, 1] == pytest.approx(g["asymmetric_y1"], rel=1e-14)


@pytest.mark.parametrize("n,d,I,d_b", [(3, 4, 8, [2, 2, 2, 2]), (2, 3, 7, [1, 4, 2]), (1, 2, 5, [5]), (3, 4, 8, [1] * 8)])
def test_brute_force_tiny(n, d, I, d_b):
    rng = np.random.default_rng(7)
    x, Wg, Wu, Wd = rand_case(rng, n, d, I)
    alpha = list(rng.uniform(0.5, 1.5, size=len(d_b)))
    ref = brute_force(x.tolist(), Wg.tolist(), Wu.tolist(), Wd.tolist(), d_b, alpha)
    got = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, alpha)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-13)


def dense_swiglu_torch(x, Wg, Wu, Wd):
    """The dense SwiGLU MLP through torch's own silu / linear in float64."""
    X = torch.from_numpy(np.asarray(x, dtype=np.float64))
    gate = torch.nn.functional.linear(X, torch.from_numpy(Wg.T.copy()))
    up = torch.nn.functional.linear(X, torch.from_numpy(Wu.T.copy()))
    return torch.nn.functional.linear(torch.nn.functional.silu(gate) * up, torch.from_numpy(Wd.T.copy())).numpy()


@pytest.mark.parametrize("d_b", [[608] * 8, [304] * 16, [4864], [64, 4800], [1] * 64 + [4800]])
def test_identity_with_dense_ffn_at_init(d_b):
    """With alpha = 1 and no pruning the layer equals the dense FFN (Section 3.1):
    relative error <= 1e-6 required, float64 gives ~1e-14."""
    rng = np.random.default_rng(11)
    d, I, n = 96, 4864, 5
    x = rng.standard_normal((n, d))
    Wg = rng.standard_normal((d, I)) * 0.02
    Wu = rng.standard_normal((d, I)) * 0.02
    Wd = rng.standard_normal((I, d)) * 0.02
    ref = dense_swiglu_torch(x, Wg, Wu, Wd)
    got = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b)
    rel = np.max(np.abs(got - ref)) / np.sqrt(np.mean(ref ** 2))
    assert rel <= 1e-6
    assert rel <= 1e-12


def test_partition_invariance():
    rng = np.random.default_rng(13)
    n, d, I = 4, 16, 112
    x, Wg, Wu, Wd = rand_case(rng, n, d, I)
    base = oracle.mlpmoe_forward(x, Wg, Wu, Wd, [I])
    for d_b in ([56, 56], [16] * 7, [1] * I, [3, 100, 9], [111, 1]):
        y = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b)
        np.testing.assert_allclose(y, base, rtol=1e-12, atol=1e-12)


def test_alpha_linearity_and_uniform_scale():
    rng = np.random.default_rng(17)
    n, d, I, d_b = 3, 8, 24, [8, 4, 12]
    x, Wg, Wu, Wd = rand_case(rng, n, d, I)
    alpha = [0.3, -1.7, 2.5]
    parts = []
    for b in range(3):
        e = [0.0, 0.0, 0.0]
        e[b] = 1.0
        parts.append(oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, e))
    y = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, alpha)
    np.testing.assert_allclose(y, sum(a * p for a, p in zip(alpha, parts)), rtol=1e-12, atol=1e-12)
    c = 1.25
    np.testing.assert_allclose(oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, [c] * 3),
                               c * dense_swiglu_torch(x, Wg, Wu, Wd), rtol=1e-12, atol=1e-12)
    # a zero gate removes exactly that branch's slice
    off = oracle.branch_offsets(d_b)
    Wd2 = Wd.copy()
    Wd2[off[1]:off[2], :] = 0.0
    np.testing.assert_allclose(oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, [1.0, 0.0, 1.0]),
                               dense_swiglu_torch(x, Wg, Wu, Wd2), rtol=1e-12, atol=1e-12)


def test_special_values():
    # silu(0) = 0: a zero gate matrix silences the layer; known sigmoid values.
    rng = np.random.default_rng(19)
    x, Wg, Wu, Wd = rand_case(rng, 2, 4, 6)
    assert np.all(oracle.mlpmoe_forward(x, np.zeros_like(Wg), Wu, Wd, [3, 3]) == 0.0)
    assert oracle.silu(np.array([0.0]))[0] == 0.0
    assert oracle.silu(np.array([math.log(3.0)]))[0] == pytest.approx(0.75 * math.log(3.0), rel=1e-15)
    assert oracle.silu(np.array([-800.0]))[0] == 0.0          # no overflow to nan
    assert oracle.silu(np.array([50.0]))[0] == pytest.approx(50.0, rel=1e-15)


def test_argument_checks():
    rng = np.random.default_rng(23)
    x, Wg, Wu, Wd = rand_case(rng, 2, 4, 6)
    with pytest.raises(ValueError):
        oracle.mlpmoe_forward(x, Wg, Wu, Wd, [3, 2])
    with pytest.raises(ValueError):
        oracle.mlpmoe_forward(x, Wg, Wu, Wd, [6, 0])
    with pytest.raises(ValueError):
        oracle.mlpmoe_forward(x, Wg, Wu, Wd, [3, 3], [1.0])
    with pytest.raises(ValueError):
        oracle.mlpmoe_forward(x[:, :3], Wg, Wu, Wd, [3, 3])


# ---- planted mistakes: each must be caught by a pin above ------------------ #
def _pins_hold():
    rng = np.random.default_rng(29)
    n, d, I, d_b = 2, 3, 7, [1, 4, 2]
    x, Wg, Wu, Wd = rand_case(rng, n, d, I)
    alpha = [0.7, 1.3, -0.4]
    ref = brute_force(x.tolist(), Wg.tolist(), Wu.tolist(), Wd.tolist(), d_b, alpha)
    got = mo.mlpmoe_forward(x, Wg, Wu, Wd, d_b, alpha)
    return np.allclose(got, ref, rtol=1e-10, atol=1e-12)


def test_planted_mistakes_are_caught(monkeypatch):
    assert _pins_hold()
    # activation without the leading factor g
    monkeypatch.setattr(mo, "silu", lambda g: 1.0 / (1.0 + np.exp(-np.asarray(g, dtype=np.float64))))
    assert not _pins_hold()
    monkeypatch.undo()
    # dropped alpha
    orig = mo.branch_forward
    monkeypatch.setattr(mo, "branch_forward", lambda x, a, b, c, lo, hi, al: orig(x, a, b, c, lo, hi, 1.0))
    assert not _pins_hold()
    monkeypatch.undo()
    # gate and up swapped
    monkeypatch.setattr(mo, "branch_forward", lambda x, a, b, c, lo, hi, al: orig(x, b, a, c, lo, hi, al))
    assert not _pins_hold()
    monkeypatch.undo()
    # slice shifted by one neuron
    monkeypatch.setattr(mo, "branch_forward",
                        lambda x, a, b, c, lo, hi, al: orig(x, a, b, c, max(lo - 1, 0), hi, al))
    assert not _pins_hold()
    monkeypatch.undo()
    assert _pins_hold()


def test_bf16_intermediate_model_is_the_layer_plus_one_rounding():
    """mlpmoe_forward_h_bf16 (a model of a bf16 implementation's stored intermediate, not the paper's
    arithmetic): the rounding is done here by another library (torch's bfloat16 conversion), the
    result must agree exactly; and it stays within half a bf16 ulp per h of the unrounded layer."""
    rng = np.random.default_rng(11)
    d, d_b = 12, [16, 32, 16]
    I = sum(d_b)
    x, Wg, Wu, Wd = rng.normal(size=(9, d)), rng.normal(size=(d, I)), rng.normal(size=(d, I)), rng.normal(size=(I, d))
    alpha = [1.0, 0.7, 1.9]
    got = oracle.mlpmoe_forward_h_bf16(x, Wg, Wu, Wd, d_b, alpha)
    g, u = x @ Wg, x @ Wu
    scale = np.repeat(alpha, d_b)
    h = g / (1.0 + np.exp(-g)) * u * scale
    hb = torch.from_numpy(h.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_allclose(got, hb @ Wd, rtol=1e-13, atol=1e-13)
    plain = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, alpha)
    bound = 2.0 ** -9 * (np.abs(h) @ np.abs(Wd))
    assert np.all(np.abs(got - plain) <= bound + 1e-12)
    assert np.abs(got - plain).max() > 0          # the rounding is really there
