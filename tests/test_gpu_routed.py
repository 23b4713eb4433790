"""GPU parity of mlpmoe_forward_routed (per-token branch selection, a labelled extension: the paper
names dynamic routing over branches as future work only) against oracle.routed_forward, element by
element through the C ABI: bf16 layers (all branches in one launch of the stack kernel) and fp32
layers (one layer call per branch, with token counts that land in each of its kernel families),
tokens that select nothing, branches nobody selects, unavailable branches, several output passes,
Fade and pruning before routing."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21089_b200 import synth
from tests.helpers import TOL_BF16, TOL_FP32, Case, Guarded, rel_err, stream_ptr

pytestmark = pytest.mark.gpu


def run_routed(lib, h, xd, sel, n, d, compensate=True):
    y = Guarded((n, d), torch.float32)
    seld = torch.from_numpy(np.ascontiguousarray(sel)).cuda()
    lib.mlpmoe_forward_routed(h, xd, y.t, n, seld, compensate, stream_ptr())
    torch.cuda.synchronize()
    assert lib.mlpmoe_get_status(h) == lib.MLPMOE_OK
    y.check()
    return y.t.cpu().numpy()


@pytest.mark.parametrize("bf16", [True, False])
@pytest.mark.parametrize("n,k", [(1, 2), (13, 1), (70, 2), (300, 3), (700, 2)])
def test_small_layer_routed(lib, bf16, n, k):
    """d = 320, unequal branches (one of 16 neurons, so the padded widths differ), non-unit alpha with a negative gate.
    700 tokens with 2 of 5 branches put about 280 tokens (two 256-row blocks) on a branch, 300 x 3/5 = 180, 70 x 2/5 = 28."""
    d, d_b = 320, [64, 160, 16, 160, 112]
    I = sum(d_b)
    alpha = [1.0, 0.8, 1.2, -0.5, 0.9]
    c = Case((300, n, k), d, I, d_b, bf16=bf16, std=0.05, alpha=alpha)
    xh, xd = c.tokens((300, n, k), n)
    sel = synth.route_select((300, n, k, synth.T_ROUTE), n, len(d_b), k)
    if n > 2:
        sel[1] = 0                    # a token that selects nothing
        sel[2] = 1                    # a token that selects every branch
    h = c.create(lib, 1024)
    try:
        for comp in (True, False):
            y = run_routed(lib, h, xd, sel, n, d, comp)
            ref = oracle.routed_forward(xh, *c.host, d_b, c.alpha, sel, compensate=comp)
            assert rel_err(y, ref) <= (TOL_BF16 if bf16 else TOL_FP32)
            if n > 2:
                assert np.all(y[1] == 0.0)
    finally:
        lib.mlpmoe_destroy(h)


@pytest.mark.parametrize("bf16", [True, False])
def test_every_branch_selected_equals_forward_and_passes(lib, bf16):
    """B = 12 > 8 branches all selected by all 1024 = max_tokens tokens: 12 x 1024 selected rows against room for
    8 x 1024 + 12 x 256, so the branch outputs take two passes through the buffers; the result is the plain layer
    (Section 3.1) at the bf16 tolerance."""
    d, B = 256, 12
    d_b = [32] * B
    c = Case((301,), d, 32 * B, d_b, bf16=bf16, std=0.05, alpha=list(np.linspace(0.7, 1.3, B)))
    tol = TOL_BF16 if bf16 else TOL_FP32
    n = 1024
    xh, xd = c.tokens((301,), n)
    h = c.create(lib, n)
    try:
        sel = np.ones((n, B), dtype=np.uint8)
        y = run_routed(lib, h, xd, sel, n, d)
        ref = oracle.mlpmoe_forward(xh, *c.host, d_b, c.alpha)
        assert rel_err(y, ref) <= tol
        # a routing that leaves branches 3 and 7 to nobody
        sel2 = synth.route_select((301, synth.T_ROUTE), n, B, 5)
        sel2[:, 3] = 0
        sel2[:, 7] = 0
        y2 = run_routed(lib, h, xd, sel2, n, d)
        ref2 = oracle.routed_forward(xh, *c.host, d_b, c.alpha, sel2)
        assert rel_err(y2, ref2) <= tol
    finally:
        lib.mlpmoe_destroy(h)


def test_routed_after_fade_and_prune(lib):
    """Routing runs on the layer as it stands: Fade changes the branches' weights, a static prune makes branches
    unavailable (selected or not, they add nothing and do not count in |S_t|) and rescales the rest; the per-branch
    layers are rebuilt after each."""
    d, B = 320, 8
    d_b = [48] * B
    c = Case((302,), d, 48 * B, d_b, bf16=True, std=0.05, alpha=list(np.linspace(0.8, 1.2, B)))
    n = 333
    xh, xd = c.tokens((302,), n)
    sel = synth.route_select((302, synth.T_ROUTE), n, B, 3)
    h = c.create(lib, 512)
    try:
        y0 = run_routed(lib, h, xd, sel, n, d)
        assert rel_err(y0, oracle.routed_forward(xh, *c.host, d_b, c.alpha, sel)) <= TOL_BF16
        lib.mlpmoe_fade(h, None, stream_ptr())
        wg, wu = oracle.fade(c.host[0], c.host[1], d_b)
        y1 = run_routed(lib, h, xd, sel, n, d)
        assert rel_err(y1, oracle.routed_forward(xh, wg, wu, c.host[2], d_b, c.alpha, sel)) <= TOL_BF16
        keep = [True, True, False, True, False, True, True, False]
        lib.mlpmoe_prune(h, keep, True, stream_ptr())
        alpha_p = [float(np.float32(a)) for a in oracle.prune_alpha(c.alpha, keep)]
        y2 = run_routed(lib, h, xd, sel, n, d)
        assert rel_err(y2, oracle.routed_forward(xh, wg, wu, c.host[2], d_b, alpha_p, sel)) <= TOL_BF16
        # all available branches selected: the pruned layer itself
        y3 = run_routed(lib, h, xd, np.ones((n, B), dtype=np.uint8), n, d)
        assert rel_err(y3, oracle.mlpmoe_forward(xh, wg, wu, c.host[2], d_b, alpha_p)) <= TOL_BF16
    finally:
        lib.mlpmoe_destroy(h)


def test_routed_argument_errors(lib):
    d, d_b = 128, [64, 64]
    c = Case((303,), d, 128, d_b, bf16=True)
    xh, xd = c.tokens((303,), 8)
    h = c.create(lib, 8)
    try:
        y = torch.empty((8, d), dtype=torch.float32, device="cuda")
        sel = torch.ones((8, 2), dtype=torch.uint8, device="cuda")
        with pytest.raises(lib.MlpmoeError):
            lib.mlpmoe_forward_routed(h, xd, y, 9, sel, True, stream_ptr())        # more tokens than max_tokens
        with pytest.raises(lib.MlpmoeError):
            lib.mlpmoe_forward_routed(h, xd, y, 8, None, True, stream_ptr())       # no selection
        lib.mlpmoe_forward_routed(h, xd, y, 0, sel, True, stream_ptr())            # nothing to do
        lib.mlpmoe_forward_routed(h, xd, y, 8, sel, True, stream_ptr())
        torch.cuda.synchronize()
        assert rel_err(y.cpu().numpy(), oracle.mlpmoe_forward(xh, *c.host, d_b, None)) <= TOL_BF16
    finally:
        lib.mlpmoe_destroy(h)
