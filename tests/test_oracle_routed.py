"""Pins for oracle.routed_forward (per-token branch selection, a labelled extension: Section 7,
Limitation 2, and the outlook of Section 8 name dynamic routing as future work and define no
rule).  None re-uses its formula: the two special cases the paper does define (every branch
selected = the layer equation of Section 3.1; one shared set = Compensated Pruning, Section 3.3,
both computed by other oracle functions that have their own pins), closed-form values worked out
by hand, a scalar brute force, and planted mistakes that these must catch."""
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_case(seed, n=7, d=6, d_b=(4, 2, 6, 4)):
    rng = np.random.default_rng(seed)
    I = sum(d_b)
    return (rng.normal(size=(n, d)), rng.normal(size=(d, I)), rng.normal(size=(d, I)), rng.normal(size=(I, d)), list(d_b),
            list(rng.uniform(0.5, 1.5, size=len(d_b))))


def brute_force(x, Wg, Wu, Wd, d_b, alpha, sel, compensate=True):
    """Scalar loops: token by token, selected branch by selected branch, neuron by neuron."""
    n, d = x.shape
    offs = [0]
    for w in d_b:
        offs.append(offs[-1] + w)
    avail = [b for b in range(len(d_b)) if alpha[b] != 0.0]
    y = [[0.0] * d for _ in range(n)]
    for t in range(n):
        S = [b for b in avail if sel[t][b]]
        if not S:
            continue
        c = math.sqrt(len(avail) / len(S)) if compensate else 1.0
        for b in S:
            for j in range(offs[b], offs[b + 1]):
                g = sum(x[t, k] * Wg[k, j] for k in range(d))
                u = sum(x[t, k] * Wu[k, j] for k in range(d))
                h = g / (1.0 + math.exp(-g)) * u
                for m in range(d):
                    y[t][m] += c * alpha[b] * h * Wd[j, m]
    return np.array(y)


def test_every_branch_selected_is_the_layer_equation():
    x, Wg, Wu, Wd, d_b, alpha = small_case(1)
    y = oracle.routed_forward(x, Wg, Wu, Wd, d_b, alpha, np.ones((x.shape[0], len(d_b)), dtype=np.uint8))
    assert np.array_equal(y, oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, alpha))
    # a branch whose gate is zero is not available: selecting it changes nothing, and the
    # compensation counts the available branches only (c_t = 1 when all of those are selected)
    alpha0 = list(alpha)
    alpha0[2] = 0.0
    y0 = oracle.routed_forward(x, Wg, Wu, Wd, d_b, alpha0, np.ones((x.shape[0], len(d_b)), dtype=np.uint8))
    np.testing.assert_allclose(y0, oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, alpha0), rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("keep", [[True, False, True, False], [False, False, False, True], [True, True, True, False]])
def test_one_shared_set_is_compensated_pruning(keep):
    """Section 3.3: alpha_b <- sqrt(B / K) alpha_b on the kept branches, 0 elsewhere."""
    x, Wg, Wu, Wd, d_b, alpha = small_case(2)
    sel = np.tile(np.array(keep, dtype=np.uint8), (x.shape[0], 1))
    y = oracle.routed_forward(x, Wg, Wu, Wd, d_b, alpha, sel)
    want = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, oracle.prune_alpha(alpha, keep))
    np.testing.assert_allclose(y, want, rtol=1e-12, atol=1e-12)
    y1 = oracle.routed_forward(x, Wg, Wu, Wd, d_b, alpha, sel, compensate=False)
    want1 = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, oracle.prune_alpha(alpha, keep, compensate=False))
    np.testing.assert_allclose(y1, want1, rtol=1e-12, atol=1e-12)


def test_hand_computed_values():
    """tests/golden/tiny_routed.txt: d = 2, I = 4, two branches of two neurons, alpha = (2, 3), x = (ln 3, 1).
    Gate pre-activations (ln 3, 0 | -ln 3, 0), up (2, 1 | 4, 1): with sigmoid(ln 3) = 3/4 and sigmoid(-ln 3) = 1/4,
    h = (3/2 ln 3, 0 | -ln 3, 0); branch 0 gives alpha_0 (3/2 ln 3, 0), branch 1 gives alpha_1 (0, -2 ln 3)."""
    vals = {}
    with open(os.path.join(GOLDEN, "tiny_routed.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                vals[k] = float(v)
    L = math.log(3.0)
    x = np.tile(np.array([[L, 1.0]]), (4, 1))
    Wg = np.array([[1.0, 0.0, -1.0, 0.0], [0.0, 0.0, 0.0, 0.0]])
    Wu = np.array([[0.0, 0.0, 0.0, 0.0], [2.0, 1.0, 4.0, 1.0]])
    Wd = np.array([[1.0, 0.0], [5.0, 5.0], [0.0, 2.0], [7.0, 7.0]])
    sel = np.array([[1, 0], [0, 1], [1, 1], [0, 0]], dtype=np.uint8)
    y = oracle.routed_forward(x, Wg, Wu, Wd, [2, 2], [2.0, 3.0], sel)
    want = np.array([[vals["t0_y0"], vals["t0_y1"]], [vals["t1_y0"], vals["t1_y1"]], [vals["t2_y0"], vals["t2_y1"]],
                     [vals["t3_y0"], vals["t3_y1"]]])
    np.testing.assert_allclose(y, want, rtol=1e-14, atol=1e-14)
    # the file's numbers are the closed forms
    assert vals["t0_y0"] == pytest.approx(3.0 * math.sqrt(2.0) * L, rel=1e-15)
    assert vals["t1_y1"] == pytest.approx(-6.0 * math.sqrt(2.0) * L, rel=1e-15)
    assert vals["t2_y0"] == pytest.approx(3.0 * L, rel=1e-15) and vals["t2_y1"] == pytest.approx(-6.0 * L, rel=1e-15)


@pytest.mark.parametrize("seed", [3, 4])
def test_scalar_brute_force(seed):
    x, Wg, Wu, Wd, d_b, alpha = small_case(seed)
    rng = np.random.default_rng(100 + seed)
    sel = (rng.random((x.shape[0], len(d_b))) < 0.5).astype(np.uint8)
    sel[0] = 0                       # a token that selects nothing
    sel[1] = 1                       # one that selects everything
    alpha[1] = 0.0                   # an unavailable branch, selected by some tokens
    for comp in (True, False):
        y = oracle.routed_forward(x, Wg, Wu, Wd, d_b, alpha, sel, compensate=comp)
        np.testing.assert_allclose(y, brute_force(x, Wg, Wu, Wd, d_b, alpha, sel, comp), rtol=1e-11, atol=1e-12)
    assert np.all(y[0] == 0.0)


def test_tokens_are_independent_and_rows_can_be_permuted():
    x, Wg, Wu, Wd, d_b, alpha = small_case(5, n=9)
    rng = np.random.default_rng(6)
    sel = (rng.random((9, len(d_b))) < 0.6).astype(np.uint8)
    y = oracle.routed_forward(x, Wg, Wu, Wd, d_b, alpha, sel)
    perm = rng.permutation(9)
    yp = oracle.routed_forward(x[perm], Wg, Wu, Wd, d_b, alpha, sel[perm])
    np.testing.assert_allclose(yp, y[perm], rtol=1e-13, atol=1e-13)
    for t in range(9):
        one = oracle.routed_forward(x[t:t + 1], Wg, Wu, Wd, d_b, alpha, sel[t:t + 1])
        np.testing.assert_allclose(one[0], y[t], rtol=1e-13, atol=1e-13)


def test_planted_mistakes_are_caught():
    """What the pins above are for: each of these wrong rules fails one of them."""
    x, Wg, Wu, Wd, d_b, alpha = small_case(7)
    B = len(d_b)
    alpha[3] = 0.0
    rng = np.random.default_rng(8)
    sel = (rng.random((x.shape[0], B)) < 0.5).astype(np.uint8)
    sel[:, 0] = 1
    good = oracle.routed_forward(x, Wg, Wu, Wd, d_b, alpha, sel)
    ref = brute_force(x, Wg, Wu, Wd, d_b, alpha, sel)
    np.testing.assert_allclose(good, ref, rtol=1e-11, atol=1e-12)

    def wrong_counts_all_branches(t):       # c_t = sqrt(B / k) with the unavailable branch counted in B
        S = [b for b in range(B) if sel[t, b] and alpha[b] != 0.0]
        return math.sqrt(B / len(S))

    def wrong_counts_selected_unavailable(t):   # k counts a selected branch whose gate is zero
        S = [b for b in range(B) if sel[t, b]]
        return math.sqrt(sum(1 for a in alpha if a != 0.0) / len(S))

    offs = oracle.branch_offsets(d_b)
    for wrong in (wrong_counts_all_branches, wrong_counts_selected_unavailable):
        y = np.zeros_like(good)
        for t in range(x.shape[0]):
            for b in range(B):
                if sel[t, b] and alpha[b] != 0.0:
                    y[t] += wrong(t) * oracle.branch_forward(x[t:t + 1], Wg, Wu, Wd, offs[b], offs[b + 1], alpha[b])[0]
        assert np.abs(y - ref).max() > 1e-3 * np.abs(ref).max()
