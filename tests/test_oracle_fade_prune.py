"""Pins for the oracle's Fractal Fade (Section 3.2) and Compensated Pruning
(Section 3.3): the paper's printed parameter counts, closed-form zero counts,
torch.quantile on the paper's own fragment, a top-k brute force, exact
sqrt(B/K) values and the variance-preservation claim."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import mlpmoe_oracle as mo
from tests.test_oracle_forward import read_golden


# ---------------------------------------------------------------- Fade ------ #
def closed_form_zero_count(layers, d, I, B, first_index=0, include_down=False):
    """Zeros Fade leaves when all magnitudes in a slice are distinct: lo + 1 per
    (branch, projection), lo = floor(s (m - 1)), m = d * d_b."""
    sched = oracle.fade_schedule(B)
    m = d * (I // B)
    total = 0
    for b in range(B):
        i = b + first_index
        s = Fraction(9 * i, 10 * B)
        if first_index == 0:
            assert s == sched[b]
        if s == 0:
            continue
        lo, _ = oracle.fade_position(s, m)
        total += (3 if include_down else 2) * (lo + 1)
    return layers * total


@pytest.mark.parametrize("model", ["qwen", "llama"])
def test_paper_tables_nonzero_counts(model):
    """Tables 1 and 2: the Fade variant's zero count is reproduced to 0.2 % by the
    schedule s_i = 0.9 i / B with 0-based i, gate and up only; the small excess in
    the paper is what a strict '>' does to ties in 16-bit checkpoints.  A 1-based
    index or a faded W_down lands far outside."""
    g = read_golden("paper_tables.txt")
    B = g["tables_B"]
    L, d, I = g[f"{model}_layers"], g[f"{model}_d_model"], g[f"{model}_d_inter"]
    assert g[f"{model}_total_mlpmoe"] - g[f"{model}_total_dense"] == L * B      # one alpha per branch
    paper_zeros = g[f"{model}_total_mlpmoe"] - g[f"{model}_nonzero_fade"]
    ours = closed_form_zero_count(L, d, I, B)
    assert {"qwen": 88252464, "llama": 1585447040}[model] == ours
    assert 1.0 <= paper_zeros / ours <= 1.003
    assert paper_zeros / closed_form_zero_count(L, d, I, B, first_index=1) < 0.9
    assert paper_zeros / closed_form_zero_count(L, d, I, B, include_down=True) < 0.7


def test_schedule_values():
    s = oracle.fade_schedule(16)
    assert s[0] == 0 and s[1] == Fraction(9, 160) and s[15] == Fraction(135, 160)
    assert all(s[i] < s[i + 1] for i in range(15)) and s[-1] < Fraction(9, 10)
    assert float(oracle.fade_schedule(32)[31]) == pytest.approx(0.9 * 31 / 32)


def test_zero_counts_on_continuous_weights():
    rng = np.random.default_rng(3)
    d, d_b = 24, [16, 16, 32, 8]
    I = sum(d_b)
    Wg = rng.standard_normal((d, I)).astype(np.float32)
    Wu = rng.standard_normal((d, I)).astype(np.float32)
    Wd = rng.standard_normal((I, d)).astype(np.float32)
    Fg, Fu = oracle.fade(Wg, Wu, d_b)
    offs = oracle.branch_offsets(d_b)
    sched = oracle.fade_schedule(len(d_b))
    fracs = []
    for b in range(len(d_b)):
        for W, F in ((Wg, Fg), (Wu, Fu)):
            sl, fsl = W[:, offs[b]:offs[b + 1]], F[:, offs[b]:offs[b + 1]]
            zeros = int(np.sum(fsl == 0))
            if b == 0:
                assert np.array_equal(sl, fsl)                       # dense backbone
            else:
                lo, _ = oracle.fade_position(sched[b], sl.size)
                assert zeros == lo + 1
                assert np.array_equal(fsl[fsl != 0], sl[fsl != 0])   # survivors unchanged
        fracs.append(np.mean(Fg[:, offs[b]:offs[b + 1]] == 0))
    # equal-width branches 0,1 then check the trend over b where widths allow: s_b rises with b
    assert fracs[0] == 0 and fracs[1] < fracs[2] < fracs[3]
    g, u, dn = oracle.nnz_per_branch(Fg, Fu, Wd, d_b)
    assert dn == [d * w for w in d_b]
    assert g[0] == d * d_b[0] and u[0] == d * d_b[0]


def test_mask_is_top_k_by_magnitude():
    rng = np.random.default_rng(5)
    w = rng.standard_normal((7, 9)).astype(np.float32)
    for s in (Fraction(1, 10), Fraction(9, 32), Fraction(1, 2), Fraction(27, 32), 0.3):
        keep = oracle.fade_mask(w, s)
        m = w.size
        lo = int(math.floor(Fraction(s) * (m - 1)))
        order = np.argsort(np.abs(w), axis=None)
        expect = np.zeros(m, dtype=bool)
        expect[order[lo + 1:]] = True
        assert np.array_equal(keep.ravel(), expect)


@pytest.mark.parametrize("s", [0.5, 0.25, 0.75, 0.125])
def test_matches_the_papers_fragment_with_torch_quantile(s):
    """The 'Differential Sparsity Logic' fragment run literally through
    torch.quantile, on inputs where float32 interpolation is exact (small integers,
    with ties) and on random floats."""
    rng = np.random.default_rng(9)
    for w in (rng.integers(-20, 21, size=(6, 11)).astype(np.float32),
              rng.standard_normal((5, 13)).astype(np.float32)):
        t = torch.from_numpy(w.copy())
        w_abs = torch.abs(t).float()
        thr = torch.quantile(w_abs, s)
        expect = (w_abs > thr).numpy()
        assert np.array_equal(oracle.fade_mask(w, s), expect)


def test_rank_form_equals_interpolated_threshold_in_exact_arithmetic():
    """The rank form of fade_mask against the quantile threshold of Section 4 evaluated without
    rounding: t = a[lo] + frac (a[lo+1] - a[lo]) in rationals, keep = |w| > t.  Includes ratios
    whose double sits a hair below a rational (frac within 1e-16 of 1), where a float64
    interpolation would round t up to a[lo+1] and drop one entry too many."""
    rng = np.random.default_rng(11)
    w = rng.standard_normal((9, 11)).astype(np.float32)
    w[2, 3] = w[4, 5]                                            # a tie
    m = w.size
    a = np.sort(np.abs(w), axis=None)
    ratios = [Fraction(1, 7), Fraction(9, 32), 0.3, 0.7, float(np.nextafter(20 / (m - 1), 0.0)), float(np.nextafter(0.5, 0.0))]
    for s in ratios:
        lo, frac = oracle.fade_position(s, m)
        assert lo == (Fraction(s) * (m - 1)).__floor__()
        a_lo, a_hi = Fraction(float(a[lo])), Fraction(float(a[min(lo + 1, m - 1)]))
        t = a_lo + frac * (a_hi - a_lo)
        expect = np.array([Fraction(float(v)) > t for v in np.abs(w).ravel()]).reshape(w.shape)
        assert np.array_equal(oracle.fade_mask(w, s), expect), s
    lo, frac = oracle.fade_position(float(np.nextafter(20 / (m - 1), 0.0)), m)
    assert lo == 19 and 1 - frac < Fraction(1, 10 ** 12)         # the case a float64 interpolation gets wrong


def test_ties_and_idempotence():
    w = np.array([[1, -1, 1, 2, 2, -3, 3, 4, 5, 6]], dtype=np.float32)
    keep = oracle.fade_mask(w, Fraction(1, 3))           # lo = 3 -> a[lo] = 2: both 2s go too
    assert keep.tolist() == [[False, False, False, False, False, True, True, True, True, True]]
    rng = np.random.default_rng(21)
    d, d_b = 8, [16, 16, 16, 16]
    Wg = rng.standard_normal((d, 64)).astype(np.float32)
    Wu = rng.standard_normal((d, 64)).astype(np.float32)
    F1 = oracle.fade(Wg, Wu, d_b)
    F2 = oracle.fade(F1[0], F1[1], d_b)
    assert np.array_equal(F1[0], F2[0]) and np.array_equal(F1[1], F2[1])


def test_fade_leaves_inputs_and_down_untouched_and_checks_arguments():
    rng = np.random.default_rng(25)
    Wg = rng.standard_normal((4, 8)).astype(np.float32)
    Wu = rng.standard_normal((4, 8)).astype(np.float32)
    g0, u0 = Wg.copy(), Wu.copy()
    oracle.fade(Wg, Wu, [4, 4])
    assert np.array_equal(Wg, g0) and np.array_equal(Wu, u0)
    with pytest.raises(ValueError):
        oracle.fade(Wg, Wu, [4, 4], [0, 1.0])
    with pytest.raises(ValueError):
        oracle.fade(Wg, Wu, [4, 4], [0])
    # custom schedule: an entry of 0 means untouched, whatever the branch
    Fg, Fu = oracle.fade(Wg, Wu, [4, 4], [0.5, 0])
    assert np.array_equal(Fg[:, 4:], Wg[:, 4:]) and np.sum(Fg[:, :4] == 0) == int(0.5 * 15) + 1


def test_planted_fade_mistakes_are_caught(monkeypatch):
    rng = np.random.default_rng(27)
    w = rng.standard_normal((6, 10)).astype(np.float32)

    def top_k_ok():
        keep = mo.fade_mask(w, Fraction(1, 2))
        lo = (w.size - 1) // 2
        order = np.argsort(np.abs(w), axis=None)
        expect = np.zeros(w.size, dtype=bool)
        expect[order[lo + 1:]] = True
        return np.array_equal(keep.ravel(), expect)

    assert top_k_ok()
    orig = mo.fade_position
    monkeypatch.setattr(mo, "fade_position", lambda s, m: orig(s, m + 1))     # p = s*m instead of s*(m-1)
    assert not top_k_ok()
    monkeypatch.undo()
    monkeypatch.setattr(mo, "fade_position", lambda s, m: (orig(s, m)[0] + 1, orig(s, m)[1]))
    assert not top_k_ok()


# ------------------------------------------------ structured variant -------- #
def test_structured_fade_brute_force_and_counts():
    """The neuron-structured variant against a scalar restatement: per branch, sort the neurons by
    (score, index) with scores summed term by term in plain Python floats, drop the first floor(s d_b)."""
    rng = np.random.default_rng(41)
    d, d_b = 6, [4, 5, 7, 8]
    I = sum(d_b)
    Wg = rng.standard_normal((d, I)).astype(np.float32)
    Wu = rng.standard_normal((d, I)).astype(np.float32)
    Wg[:, 10] = Wg[:, 9]; Wu[:, 10] = Wu[:, 9]                     # a tie inside branch 2: the lower index goes first
    s = [0, Fraction(2, 5), 0.5, Fraction(7, 8)]
    Fg, Fu = oracle.fade_structured(Wg, Wu, d_b, s)
    offs = oracle.branch_offsets(d_b)
    for b in range(4):
        scores = []
        for j in range(offs[b], offs[b + 1]):
            acc = 0.0
            for k in range(d):
                acc += float(Wg[k, j]) * float(Wg[k, j])
            for k in range(d):
                acc += float(Wu[k, j]) * float(Wu[k, j])
            scores.append((acc, j))
        q = int(math.floor(Fraction(s[b]) * d_b[b]))
        assert q == oracle.fade_structured_count(s[b], d_b[b])
        gone = {j for _, j in sorted(scores)[:q]}
        for j in range(offs[b], offs[b + 1]):
            if j in gone:
                assert not Fg[:, j].any() and not Fu[:, j].any()
            else:
                assert np.array_equal(Fg[:, j], Wg[:, j]) and np.array_equal(Fu[:, j], Wu[:, j])
    assert 9 in {j for j in range(I) if not Fg[:, j].any()} or 10 not in {j for j in range(I) if not Fg[:, j].any()}
    # exact small integers: scores 2 k^2 for column k; the default schedule on B = 2 drops floor(0.45 * 4) = 1 of branch 1
    Wi = np.tile(np.arange(1, 9, dtype=np.float32), (3, 1))
    assert oracle.neuron_scores(Wi, Wi).tolist() == [6.0 * k * k for k in range(1, 9)]
    Gi, Ui = oracle.fade_structured(Wi, Wi, [4, 4])
    assert [j for j in range(8) if not Gi[:, j].any()] == [4]
    # idempotent, inputs untouched, dead neurons leave the schedule
    G2, U2 = oracle.fade_structured(Fg, Fu, d_b, s)
    assert np.array_equal(G2, Fg) and np.array_equal(U2, Fu)
    Wd = rng.standard_normal((I, d)).astype(np.float32)
    _, segs = oracle.surviving_set([1.0] * 4, Fg, Fu, Wd, d_b)
    assert sum(l for _, l in segs) == I - sum(oracle.fade_structured_count(s[b], d_b[b]) for b in range(4))
    x = rng.standard_normal((3, d))
    np.testing.assert_allclose(oracle.mlpmoe_forward(x, Fg, Fu, Wd, d_b), oracle.mlpmoe_forward_skiplist(x, Fg, Fu, Wd, d_b, [1.0] * 4),
                               rtol=1e-12, atol=1e-12)


# -------------------------------------------------------------- pruning ----- #
def test_compensation_values():
    a = oracle.prune_alpha([1.0] * 16, oracle.first_k_keep(16, 12))
    assert a[:12] == [math.sqrt(16 / 12)] * 12 and a[12:] == [0.0] * 4
    assert oracle.prune_alpha([1.0] * 4, [True] * 4) == [1.0] * 4                       # K = B: no-op
    assert oracle.prune_alpha([1.0] * 4, [True, False, False, False]) == [2.0, 0.0, 0.0, 0.0]  # sqrt(4/1)
    assert oracle.prune_alpha([0.5, 2.0, 1.0, 1.0], [False, True, True, False]) == \
        [0.0, 2.0 * math.sqrt(2.0), math.sqrt(2.0), 0.0]
    assert oracle.prune_alpha([1.0, 1.0], [True, False], compensate=False) == [1.0, 0.0]
    with pytest.raises(ValueError):
        oracle.prune_alpha([1.0, 1.0], [False, False])
    with pytest.raises(ValueError):
        oracle.first_k_keep(4, 0)


def test_variance_preservation():
    """Section 3.3: scaling the K kept branches by sqrt(B/K) keeps the output's
    variance magnitude.  On iid random weights the branch outputs are uncorrelated
    and equally distributed, so RMS(pruned) / RMS(full) -> 1."""
    rng = np.random.default_rng(31)
    n, d, I, B = 64, 128, 2048, 16
    x = rng.standard_normal((n, d))
    Wg = rng.standard_normal((d, I)) * 0.05
    Wu = rng.standard_normal((d, I)) * 0.05
    Wd = rng.standard_normal((I, d)) * 0.05
    d_b = [I // B] * B
    full = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b)
    for K in (12, 8, 4):
        a = oracle.prune_alpha([1.0] * B, oracle.first_k_keep(B, K))
        y = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, a)
        ratio = np.sqrt(np.mean(y ** 2) / np.mean(full ** 2))
        assert abs(ratio - 1.0) < 0.05
        y_raw = oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, oracle.prune_alpha([1.0] * B, oracle.first_k_keep(B, K), False))
        assert np.sqrt(np.mean(y_raw ** 2) / np.mean(full ** 2)) == pytest.approx(math.sqrt(K / B), abs=0.05)


def test_surviving_set_brute_force():
    rng = np.random.default_rng(33)
    d, d_b = 3, [4, 4, 4, 4]
    I = 16
    Wg = rng.standard_normal((d, I))
    Wu = rng.standard_normal((d, I))
    Wd = rng.standard_normal((I, d))
    Wg[:, 1] = 0          # dead through gate
    Wu[:, 5] = 0          # dead through up
    Wd[6, :] = 0          # dead through down
    Wg[:, 8:12] = 0       # a whole branch dead
    alpha = [1.0, 1.0, 1.0, 0.0]
    branches, segs = oracle.surviving_set(alpha, Wg, Wu, Wd, d_b)
    assert branches == [0, 1]
    assert segs == [(0, 1), (2, 2), (4, 1), (7, 1)]
    x = rng.standard_normal((5, d))
    np.testing.assert_allclose(oracle.mlpmoe_forward_skiplist(x, Wg, Wu, Wd, d_b, alpha),
                               oracle.mlpmoe_forward(x, Wg, Wu, Wd, d_b, alpha), rtol=1e-12, atol=1e-13)
    # nothing dead, nothing pruned: one segment per branch
    b2, s2 = oracle.surviving_set([1.0] * 4, np.ones((d, I)), np.ones((d, I)), np.ones((I, d)), d_b)
    assert b2 == [0, 1, 2, 3] and s2 == [(0, 4), (4, 4), (8, 4), (12, 4)]


# ---------------------------------------------------------------- stack ----- #
def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(35)
    a = np.concatenate([rng.standard_normal(4096).astype(np.float32) * 3,
                        np.array([1.0, 1.00390625, 1.001953125, 1.005859375, 0.0, -2.5], dtype=np.float32)])
    ref = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_to_bf16(a), ref)


def test_rmsnorm_and_stack():
    rng = np.random.default_rng(37)
    x = rng.standard_normal((6, 32)) * 3
    r = oracle.rmsnorm(x, eps=0.0)
    np.testing.assert_allclose(np.sqrt(np.mean(r ** 2, axis=1)), 1.0, rtol=1e-14)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (32,), eps=1e-6).numpy()
    np.testing.assert_allclose(oracle.rmsnorm(x), ref, rtol=1e-13)
    d, I, d_b = 32, 48, [16, 32]
    layers = []
    for _ in range(2):
        layers.append((rng.standard_normal((d, I)) * 0.1, rng.standard_normal((d, I)) * 0.1,
                       rng.standard_normal((I, d)) * 0.1, d_b, [1.0, 0.5]))
    y, inputs = oracle.stack_forward(x, layers, bf16_activations=False, return_layer_inputs=True)
    x1 = x + oracle.mlpmoe_forward(oracle.rmsnorm(x), *layers[0])
    x2 = x1 + oracle.mlpmoe_forward(oracle.rmsnorm(x1), *layers[1])
    np.testing.assert_allclose(y, x2, rtol=1e-13)
    np.testing.assert_allclose(inputs[1], x1, rtol=1e-13)
    # rows are independent: a subset of rows gives the same rows
    np.testing.assert_allclose(oracle.stack_forward(x[[1, 4]], layers), oracle.stack_forward(x, layers)[[1, 4]], rtol=1e-12)


def test_stack_with_bf16_activations_hand_computed():
    """Two layers of the pre-norm stack with the normalised input rounded to bfloat16, against values
    derived by hand in tests/golden/tiny_stack_bf16.txt (the rounding of 1/sqrt(2) and of the second
    layer's normalised input are where a missing or misplaced rounding shows)."""
    g = {}
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "tiny_stack_bf16.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                g[k] = float(v)
    c = math.log(3.0) * 128.0 / 181.0                        # bf16(sqrt 2) = 181/128, so the first gate pre-activation is ln 3
    layer = (np.array([[c], [c]]), np.array([[1.0], [0.0]]), np.array([[1.0, 2.0]]), [1], [1.0])
    x = np.array([[1.0, 0.0]])
    y1, inputs = oracle.stack_forward(x, [layer], bf16_activations=True, eps=0.0, return_layer_inputs=True)
    assert np.array_equal(inputs[0], x)
    np.testing.assert_allclose(y1, [[g["layer1_x0"], g["layer1_x1"]]], rtol=1e-14)
    y2 = oracle.stack_forward(x, [layer, layer], bf16_activations=True, eps=0.0)
    np.testing.assert_allclose(y2, [[g["layer2_x0"], g["layer2_x1"]]], rtol=1e-14)
    # without the rounding the layer's contribution moves in its 4th digit
    y1_exact = oracle.stack_forward(x, [layer], bf16_activations=False, eps=0.0)
    assert abs(y1_exact[0, 0] - g["layer1_x0"]) > 1e-4
