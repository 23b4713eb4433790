"""GPU parity of the pre-norm residual stack x <- x + MLPMoE_l(RMSNorm(x)) against the oracle:
a small stack compared element by element, and the full-size benchmark workload (24 layers,
Qwen2.5-0.5B shapes, 4096 tokens, 12 of 16 branches kept) compared on sampled token rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21089_b200 import synth
from tests.helpers import TOL_BF16, TOL_FP32, Case, dev_bf16, dev_f32, layer_rms, rel_err, rms_err, stack_tolerance, stream_ptr

pytestmark = pytest.mark.gpu


def test_rmsnorm_kernel(lib):
    x = synth.normal_f32((200, 0), (300, 320), 3.0)
    xd = dev_f32(x)
    ref = oracle.rmsnorm(x)
    r32 = torch.empty((300, 320), dtype=torch.float32, device="cuda")
    lib.mlpmoe_rmsnorm(xd, r32, 300, 320, 1e-6, lib.MLPMOE_FP32, stream_ptr())
    rb = torch.empty((300, 320), dtype=torch.bfloat16, device="cuda")
    lib.mlpmoe_rmsnorm(xd, rb, 300, 320, 1e-6, lib.MLPMOE_BF16, stream_ptr())
    torch.cuda.synchronize()
    np.testing.assert_allclose(r32.cpu().numpy(), ref, rtol=2e-6, atol=1e-7)
    # bf16 output: the rounding of a value within 2e-6 of the exact one, i.e. at most one bf16 step away
    got = rb.float().cpu().numpy().astype(np.float64)
    assert np.max(np.abs(got - oracle.round_to_bf16(ref)) / np.maximum(np.abs(ref), 1e-30)) <= 2.0 ** -7
    assert np.mean(got != oracle.round_to_bf16(ref)) < 1e-3


# (tokens, decode kernel): 1 = the few-token kernel, 2 = the kernel with the H exchange, 0 = the library's rule
# (on layers as small as these the rule always picks kernel 2 for at most 64 tokens)
SMALL_STACK_CASES = [(1, 1), (1, 2), (5, 1), (5, 2), (12, 1), (13, 1), (13, 2), (16, 1), (14, 0), (24, 0), (64, 0), (100, 0), (129, 0),
                     (300, 0), (512, 0)]


@pytest.mark.parametrize("bf16,n,kernel", [(True, n, k) for n, k in SMALL_STACK_CASES] +
                         [(False, n, 0) for n in sorted({n for n, _ in SMALL_STACK_CASES})])
def test_small_stack(lib, bf16, n, kernel):
    d, I, d_b, L = 256, 384, [128, 64, 192], 3
    cases, handles, layers = [], [], []
    try:
        for l in range(L):
            c = Case((201, l, int(bf16)), d, I, d_b, bf16=bf16, std=0.05, alpha=[1.0, 0.9, 1.1])
            h = c.create(lib, 512)
            keep = [True, l != 1, True]
            lib.mlpmoe_prune(h, keep, True, stream_ptr())
            if handles:
                lib.mlpmoe_share_workspace(h, handles[0])
            handles.append(h)
            layers.append((*c.host, d_b, oracle.prune_alpha(c.alpha, keep)))
        lib.mlpmoe_debug_set_decode_kernel(handles[0], kernel)
        x = synth.normal_f32((201, 9, n), (n, d), 1.0)
        xd = dev_f32(x)
        lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
        torch.cuda.synchronize()
        ref = oracle.stack_forward(x, layers, bf16_activations=bf16)
        assert rel_err(xd.cpu().numpy(), ref) <= (TOL_BF16 if bf16 else TOL_FP32)
        # host-buffer entry point
        yh = torch.empty((n, d), dtype=torch.float32)
        lib.mlpmoe_stack_forward_host(handles, torch.from_numpy(x), yh, n, 1e-6, stream_ptr())
        # Same numbers up to the order in which K slices are added into the fp32 stream.  In bf16 a
        # last-bit difference of x can also flip the rounding of one normalised input of the next
        # layer, which moves that token's row by a bf16 step of one product: far inside the parity
        # tolerance, far outside fp32 round-off.
        assert rel_err(yh.numpy(), ref) <= (TOL_BF16 if bf16 else TOL_FP32)
        if bf16:
            assert rel_err(yh.numpy(), xd.cpu().numpy().astype(np.float64)) <= TOL_BF16 / 4
        else:
            np.testing.assert_allclose(yh.numpy(), xd.cpu().numpy(), rtol=1e-5, atol=1e-5)
        assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
    finally:
        for h in handles[1:] + handles[:1]:
            lib.mlpmoe_destroy(h)


def test_config2_full_size_sampled_rows(lib):
    """The benchmark's workload in the benchmark's launch configuration; the oracle runs the
    sampled rows through all 24 layers (rows are independent)."""
    cfg = synth.CONFIGS[2]
    d, I, B, n, L = cfg["d_model"], cfg["d_inter"], cfg["B"], cfg["n"], cfg["layers"]
    d_b = synth.equal_partition(I, B)
    handles, layers = [], []
    try:
        for l in range(L):
            bits = synth.layer_weights(2, l, d, I, 0.02, bf16=True)
            keep = synth.keep_set((synth.BASE_SEED, 2, l, synth.T_KEEP), B, cfg["n_drop"])
            dev = [dev_bf16(b) for b in bits]
            h = lib.mlpmoe_create(d, I, d_b, dev[0], dev[1], dev[2], None, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, n, stream_ptr())
            lib.mlpmoe_prune(h, keep, True, stream_ptr())
            if handles:
                lib.mlpmoe_share_workspace(h, handles[0])
            handles.append(h)
            alpha = oracle.prune_alpha([1.0] * B, keep)
            host = [synth.bf16_bits_to_f32(b) for b in bits]
            layers.append((*host, d_b, alpha))
            # the schedule is bit-exact: kept branches, one full segment each
            assert np.array_equal(lib.mlpmoe_get_alpha(h, B).view(np.uint32), np.array(alpha).astype(np.float32).view(np.uint32))
            assert lib.mlpmoe_get_klist(h, B, I) == oracle.surviving_set(alpha, *host, d_b)
            assert lib.mlpmoe_get_active_neurons(h) == 12 * 304
        x = synth.tokens(2, n, d)
        xd = dev_f32(x)
        lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
        torch.cuda.synchronize()
        rows = sorted(set([0, 1, 127, 128, 255, 256, 2047, 2048, n - 129, n - 1] +
                          list(np.random.default_rng(5).integers(0, n, size=38))))
        ref, inputs = oracle.stack_forward(x[rows], layers, bf16_activations=True, return_layer_inputs=True)
        got = xd.cpu().numpy()
        assert np.isfinite(got).all()
        # End to end over 24 layers: the worst element sits at about 2e-2 RMS (bf16 rounding of H adds up like a
        # random walk), so the bound is 3e-2 on the worst element and 2e-2 / 4 on the bulk (RMS) of the error.
        e_max, e_rms = rel_err(got[rows], ref), rms_err(got[rows], ref)
        print(f"config 2 end to end: max|delta|/RMS = {e_max:.4f}, RMS(delta)/RMS = {e_rms:.5f}, "
              f"first-order bound {stack_tolerance(inputs, ref):.4f}")
        assert e_max <= 3e-2
        assert e_rms <= TOL_BF16 / 4
        # every layer on its own, fed the oracle's input of that layer, at the layer tolerance
        xs = inputs + [ref]
        worst = 0.0
        for l in range(L):
            xin = np.zeros((n, d), dtype=np.float32)
            xin[:len(rows)] = xs[l].astype(np.float32)
            xin_d = dev_f32(xin)
            lib.mlpmoe_stack_forward(handles[l:l + 1], xin_d, n, 1e-6, stream_ptr())
            torch.cuda.synchronize()
            delta_got = xin_d.cpu().numpy()[:len(rows)].astype(np.float64) - xin[:len(rows)].astype(np.float64)
            e = rel_err(delta_got, xs[l + 1] - xs[l])
            worst = max(worst, e)
            assert e <= TOL_BF16, l
        print(f"config 2 layer by layer: worst max|delta|/RMS(y_l) = {worst:.4f}")
        assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
    finally:
        for h in handles[1:] + handles[:1]:
            lib.mlpmoe_destroy(h)


def test_two_full_width_layers_every_row(lib):
    """What the one-launch prefill-stack kernel adds over a single layer, at full width and checked on
    EVERY row: 2 layers of the Qwen shape over 4096 tokens = 16 token blocks, so the down items trail
    their block's gate|up tiles by 7 blocks across the layer boundary, the norm warps race the GEMM
    pipeline, and every (layer, block) dependency counter is in use.  A K slice dropped or added twice,
    or a block normalised before its down items are in, moves whole rows by far more than the bound."""
    cfg = synth.CONFIGS[2]
    d, I, B, n, L = cfg["d_model"], cfg["d_inter"], cfg["B"], cfg["n"], 2
    d_b = synth.equal_partition(I, B)
    handles, layers = [], []
    try:
        for l in range(L):
            bits = synth.layer_weights(2, l, d, I, 0.02, bf16=True)
            keep = synth.keep_set((synth.BASE_SEED, 2, l, synth.T_KEEP), B, cfg["n_drop"])
            dev = [dev_bf16(b) for b in bits]
            h = lib.mlpmoe_create(d, I, d_b, dev[0], dev[1], dev[2], None, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, n, stream_ptr())
            lib.mlpmoe_prune(h, keep, True, stream_ptr())
            if handles:
                lib.mlpmoe_share_workspace(h, handles[0])
            handles.append(h)
            layers.append((*[synth.bf16_bits_to_f32(b) for b in bits], d_b, oracle.prune_alpha([1.0] * B, keep)))
        x = synth.tokens(2, n, d)
        ref, inputs = oracle.stack_forward(x, layers, bf16_activations=True, return_layer_inputs=True)
        bound = stack_tolerance(inputs, ref)           # first order: TOL_BF16 * (RMS(y_0) + RMS(y_1)) / RMS(x_out)
        for rep in range(3):                           # arrival order differs from run to run
            xd = dev_f32(x)
            lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
            torch.cuda.synchronize()
            got = xd.cpu().numpy()
            e_max, e_rms = rel_err(got, ref), rms_err(got, ref)
            print(f"2 Qwen layers, all {n} rows, run {rep}: max|delta|/RMS = {e_max:.5f} (bound {bound:.5f}), RMS(delta)/RMS = {e_rms:.6f}")
            assert e_max <= bound
            # measured against the layers' own contribution (what the kernel computes), the bulk of the error is tiny
            y_got = got.astype(np.float64) - x
            assert rms_err(y_got, ref - x) <= TOL_BF16 / 4
        assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
    finally:
        for h in handles[1:] + handles[:1]:
            lib.mlpmoe_destroy(h)


@pytest.mark.parametrize("n,kernel", [(4, 1), (4, 2), (40, 0), (300, 0)])
def test_stack_follows_a_later_prune_and_fade(lib, n, kernel):
    """The stack kernels cache per-stack set-up (work sequences, layer records, the decode kernel's
    tiled weight copy): a prune or a Fade between two calls must show in the second call."""
    d, I, d_b, L = 256, 512, [128, 128, 64, 192], 2
    cases, handles = [], []
    try:
        for l in range(L):
            c = Case((207, l), d, I, d_b, bf16=True, std=0.05)
            h = c.create(lib, 512)
            if handles:
                lib.mlpmoe_share_workspace(h, handles[0])
            cases.append(c)
            handles.append(h)
        lib.mlpmoe_debug_set_decode_kernel(handles[0], kernel)
        x = synth.normal_f32((207, 9, n), (n, d), 1.0)
        ones = [1.0] * len(d_b)

        def run_and_check(layers):
            xd = dev_f32(x)
            lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
            torch.cuda.synchronize()
            ref = oracle.stack_forward(x, layers, bf16_activations=True)
            assert rel_err(xd.cpu().numpy(), ref) <= TOL_BF16

        run_and_check([(*c.host, d_b, ones) for c in cases])
        keep = [True, False, True, True]
        for h in handles:
            lib.mlpmoe_prune(h, keep, True, stream_ptr())
        run_and_check([(*c.host, d_b, oracle.prune_alpha(ones, keep)) for c in cases])
        for h in handles:
            lib.mlpmoe_fade(h, None, stream_ptr())
        faded = [oracle.fade(c.host[0], c.host[1], d_b) for c in cases]
        run_and_check([(Fg, Fu, c.host[2], d_b, oracle.prune_alpha(ones, keep)) for c, (Fg, Fu) in zip(cases, faded)])
        assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
    finally:
        for h in handles[1:] + handles[:1]:
            lib.mlpmoe_destroy(h)
