"""GPU edge cases, guard bands and the give-up path of the bounded waits.

Guard bands stand in for a memory checker: every caller-owned buffer of a call sits between
poisoned margins, and the library's activation workspace is poisoned beyond the rows the call may
use; after the call the poison must be intact.  Shapes are chosen so that every kernel family runs
with ragged tails: d_model = 328 is a multiple of 8 but not of the 64-wide K-step (the zero-filled
K tail of the tensor tiles) nor of any output tile width.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21089_b200 import synth
from tests.helpers import (TOL_BF16, TOL_FP32, Case, Guarded, check_workspace, dev_bf16, dev_f32, poison_workspace, rel_err,
                           stream_ptr)

pytestmark = pytest.mark.gpu

TOKEN_COUNTS = [1, 13, 14, 64, 65, 128, 129, 300]


@pytest.mark.parametrize("n", TOKEN_COUNTS)
def test_odd_width_layer_with_guard_bands(lib, n):
    """d_model = 328, unequal branches, non-unit alpha; x, y and the residual between guard bands."""
    d, I, d_b = 328, 400, [64, 160, 16, 160]
    c = Case((400, n), d, I, d_b, bf16=True, std=0.05, alpha=[1.0, 0.8, 1.2, -0.5])
    xh, xd = c.tokens((400, n), n)
    h = c.create(lib, 320)
    try:
        ref = oracle.mlpmoe_forward(xh, *c.host, d_b, c.alpha)
        gx = Guarded((n, d), torch.bfloat16, xd)
        gy = Guarded((n, d), torch.float32)
        ws = poison_workspace(lib, h)
        lib.mlpmoe_forward(h, gx.t, gy.t, n, stream_ptr())
        torch.cuda.synchronize()
        assert rel_err(gy.t.cpu().numpy(), ref) <= TOL_BF16
        gx.check(); gy.check()
        check_workspace(lib, h, ws, n, d, 2, used_xnorm=False)
        # residual added in place (the K slices of the down projection accumulate into y)
        r = synth.normal_f32((400, n, 9), (n, d), 1.0)
        gr = Guarded((n, d), torch.float32, dev_f32(r))
        lib.mlpmoe_forward_ex(h, gx.t, gr.t, n, gr.t, lib.MLPMOE_FP32, stream_ptr())
        torch.cuda.synchronize()
        assert rel_err(gr.t.cpu().numpy().astype(np.float64) - r, ref) <= TOL_BF16
        gr.check(); gx.check()
        # bf16 output
        gb = Guarded((n, d), torch.bfloat16)
        lib.mlpmoe_forward_ex(h, gx.t, gb.t, n, None, lib.MLPMOE_BF16, stream_ptr())
        torch.cuda.synchronize()
        yb = gb.t.float().cpu().numpy().astype(np.float64)
        assert np.max(np.abs(yb - ref) - np.abs(ref) * 2.0 ** -8) <= TOL_BF16 * np.sqrt(np.mean(ref ** 2))
        gb.check()
        assert lib.mlpmoe_get_status(h) == lib.MLPMOE_OK
    finally:
        lib.mlpmoe_destroy(h)


@pytest.mark.parametrize("n,kernel", [(n, 0) for n in TOKEN_COUNTS] + [(1, 1), (13, 1)])
def test_odd_width_stack_with_guard_bands(lib, n, kernel):
    """Three layers with d_model = 328 as a pre-norm stack (decode-fused, decode-stack, 65..128-token and
    prefill-stack kernels by token count), the residual stream between guard bands, the workspace poisoned."""
    d, I, d_b, L = 328, 384, [128, 64, 192], 3
    handles, layers = [], []
    try:
        for l in range(L):
            c = Case((401, l), d, I, d_b, bf16=True, std=0.05, alpha=[1.0, 0.9, 1.1])
            h = c.create(lib, 320)
            if handles:
                lib.mlpmoe_share_workspace(h, handles[0])
            handles.append(h)
            layers.append((*c.host, d_b, c.alpha))
        lib.mlpmoe_debug_set_decode_kernel(handles[0], kernel)      # 1: the few-token kernel (the rule picks the other one on layers this small)
        x = synth.normal_f32((401, 9, n), (n, d), 1.0)
        ref = oracle.stack_forward(x, layers, bf16_activations=True)
        lib.mlpmoe_stack_prepare(handles, n, stream_ptr())
        torch.cuda.synchronize()
        gx = Guarded((n, d), torch.float32, dev_f32(x))
        ws = poison_workspace(lib, handles[0])
        free_before = torch.cuda.mem_get_info()[0]
        lib.mlpmoe_stack_forward(handles, gx.t, n, 1e-6, stream_ptr())
        assert torch.cuda.mem_get_info()[0] >= free_before          # prepared: the forward call allocates nothing
        torch.cuda.synchronize()
        assert rel_err(gx.t.cpu().numpy(), ref) <= TOL_BF16
        gx.check()
        check_workspace(lib, handles[0], ws, n, d, 2)
        assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
    finally:
        for h in handles[1:] + handles[:1]:
            lib.mlpmoe_destroy(h)


@pytest.mark.parametrize("bf16", [True, False])
@pytest.mark.parametrize("n", [5, 40, 100, 260])
def test_single_branch_and_narrow_survivors(lib, bf16, n):
    """B = 1 (the layer is the dense SwiGLU MLP), and a layer whose surviving width after pruning and
    Fade is below one 128-neuron group (64 neurons of a Faded branch)."""
    d = 128
    c1 = Case((402, int(bf16)), d, 256, [256], bf16=bf16, std=0.05)
    xh, xd = c1.tokens((402, n), n)
    h = c1.create(lib, 512)
    try:
        y = torch.empty((n, d), dtype=torch.float32, device="cuda")
        lib.mlpmoe_forward(h, xd, y, n, stream_ptr())
        torch.cuda.synchronize()
        assert lib.mlpmoe_get_klist(h, 1, 256) == ([0], [(0, 256)])
        assert rel_err(y.cpu().numpy(), oracle.mlpmoe_forward(xh, *c1.host, [256])) <= (TOL_BF16 if bf16 else TOL_FP32)
        lib.mlpmoe_prune_first_k(h, 1, stream_ptr())                 # K = B = 1: sqrt(1/1), nothing changes
        assert lib.mlpmoe_get_alpha(h, 1).tolist() == [1.0]
    finally:
        lib.mlpmoe_destroy(h)
    d_b = [64, 64, 128]
    c2 = Case((403, int(bf16)), d, 256, d_b, bf16=bf16, std=0.05, alpha=[1.0, 1.1, 0.9])
    xh, xd = c2.tokens((403, n), n)
    h = c2.create(lib, 512)
    try:
        lib.mlpmoe_fade(h, None, stream_ptr())
        keep = [False, True, False]
        lib.mlpmoe_prune(h, keep, True, stream_ptr())
        Fg, Fu = oracle.fade(c2.host[0], c2.host[1], d_b)
        alpha = oracle.prune_alpha(c2.alpha, keep)
        assert lib.mlpmoe_get_active_neurons(h) == 64
        assert lib.mlpmoe_get_klist(h, 3, 256) == oracle.surviving_set(alpha, Fg, Fu, c2.host[2], d_b)
        y = torch.empty((n, d), dtype=torch.float32, device="cuda")
        lib.mlpmoe_forward(h, xd, y, n, stream_ptr())
        torch.cuda.synchronize()
        assert rel_err(y.cpu().numpy(), oracle.mlpmoe_forward(xh, Fg, Fu, c2.host[2], d_b, alpha)) <= (TOL_BF16 if bf16 else TOL_FP32)
        if bf16:
            xs = synth.normal_f32((403, 9, n), (n, d), 1.0)
            xsd = dev_f32(xs)
            lib.mlpmoe_stack_forward([h, h], xsd, n, 1e-6, stream_ptr())
            torch.cuda.synchronize()
            ref = oracle.stack_forward(xs, [(Fg, Fu, c2.host[2], d_b, alpha)] * 2, bf16_activations=True)
            assert rel_err(xsd.cpu().numpy(), ref) <= TOL_BF16
        assert lib.mlpmoe_get_status(h) == lib.MLPMOE_OK
    finally:
        lib.mlpmoe_destroy(h)


@pytest.mark.parametrize("n,stack,kernel", [(4, True, 1), (4, True, 2), (40, True, 0), (100, True, 0), (300, True, 0), (300, False, 0)])
def test_bounded_wait_runs_out_and_the_handle_recovers(lib, n, stack, kernel):
    """The give-up path of the kernels whose CTAs wait for one another (few-token decode stack, the other decode-stack
    kernel in its 64-row and 128-row builds, prefill stack, single-layer prefill): with the wait limit cut to 3 ms and every
    cross-CTA target raised by one arrival (a count that is never reached) the call must return, the
    status must read DEVICE_TIMEOUT, and, once that has been reported, the same handles must compute
    the right result again.  Nothing traps or faults: the kernels leave their loops and free their TMEM."""
    d, I, d_b, L = 256, 512, [128, 128, 64, 192], 2
    cases, handles = [], []
    try:
        for l in range(L):
            c = Case((404, l), d, I, d_b, bf16=True, std=0.05)
            h = c.create(lib, 512)
            if handles:
                lib.mlpmoe_share_workspace(h, handles[0])
            cases.append(c)
            handles.append(h)
        ones = [1.0] * len(d_b)
        lib.mlpmoe_debug_set_decode_kernel(handles[0], kernel)
        if stack:
            x = synth.normal_f32((404, 9, n), (n, d), 1.0)
            ref = oracle.stack_forward(x, [(*c.host, d_b, ones) for c in cases], bf16_activations=True)

            def run():
                xd = dev_f32(x)
                lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
                torch.cuda.synchronize()
                return xd.cpu().numpy()
        else:
            xh, xdev = cases[0].tokens((404, n), n)
            ref = oracle.mlpmoe_forward(xh, *cases[0].host, d_b, ones)

            def run():
                y = torch.empty((n, d), dtype=torch.float32, device="cuda")
                lib.mlpmoe_forward(handles[0], xdev, y, n, stream_ptr())
                torch.cuda.synchronize()
                return y.cpu().numpy()
        assert rel_err(run(), ref) <= TOL_BF16
        lib.mlpmoe_debug_set_wait(handles[0], 3_000_000, 1)
        run()                                                        # returns; its output is undefined
        assert lib.mlpmoe_get_status(handles[0]) == lib.MLPMOE_ERR_DEVICE_TIMEOUT
        assert lib.mlpmoe_get_status(handles[0]) == lib.MLPMOE_OK    # reported once, and the handle is re-armed
        lib.mlpmoe_debug_set_wait(handles[0], 0, 0)
        for _ in range(2):
            assert rel_err(run(), ref) <= TOL_BF16
        assert lib.mlpmoe_get_status(handles[0]) == lib.MLPMOE_OK
    finally:
        for h in handles[1:] + handles[:1]:
            lib.mlpmoe_destroy(h)
    # a fresh handle afterwards is fine too (the context is intact)
    c = Case((405, 0), d, I, d_b, bf16=True, std=0.05)
    xh, xdev = c.tokens((405, 1), 130)
    h = c.create(lib, 256)
    try:
        y = torch.empty((130, d), dtype=torch.float32, device="cuda")
        lib.mlpmoe_forward(h, xdev, y, 130, stream_ptr())
        torch.cuda.synchronize()
        assert rel_err(y.cpu().numpy(), oracle.mlpmoe_forward(xh, *c.host, d_b)) <= TOL_BF16
    finally:
        lib.mlpmoe_destroy(h)


def test_a_recreated_layer_is_not_served_from_a_stale_stack_plan(lib):
    """Destroying and re-creating a layer of a stack (new weights, often the same host address for the
    handle) must make the next stack call plan again: the cached set-up is keyed on a per-handle id that
    is never reused."""
    d, I, d_b, n = 256, 512, [128, 128, 64, 192], 300
    ones = [1.0] * len(d_b)
    c0 = Case((406, 0), d, I, d_b, bf16=True, std=0.05)
    h0 = c0.create(lib, 512)
    h1 = None
    try:
        x = synth.normal_f32((406, 9, n), (n, d), 1.0)
        for seed in (1, 2, 3):
            c1 = Case((406, seed), d, I, d_b, bf16=True, std=0.05)
            h1 = c1.create(lib, 512)
            lib.mlpmoe_share_workspace(h1, h0)
            xd = dev_f32(x)
            lib.mlpmoe_stack_forward([h0, h1], xd, n, 1e-6, stream_ptr())
            torch.cuda.synchronize()
            ref = oracle.stack_forward(x, [(*c0.host, d_b, ones), (*c1.host, d_b, ones)], bf16_activations=True)
            assert rel_err(xd.cpu().numpy(), ref) <= TOL_BF16
            lib.mlpmoe_destroy(h1)
            h1 = None
    finally:
        if h1 is not None:
            lib.mlpmoe_destroy(h1)
        lib.mlpmoe_destroy(h0)
