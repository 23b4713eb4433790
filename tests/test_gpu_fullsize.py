"""Full-size parity runs on Llama-3-8B-shaped MLPs (d_model 4096, d_inter 14336), in the launch
configurations the library uses at these sizes, against the oracle on sampled token rows
(rows are independent, so the oracle runs exactly those rows):

  config 3: one layer, B = 32 x 448, 8192 tokens, alpha ~ U(0.8, 1.2), Fractal Fade s_b = 0.9 b / B
  config 4: 32-layer stack, B = 64 x 224, decode token counts 1 / 8 / 32 / 64, unpruned and
            first-K pruning with K = 51
  config 5: 32-layer stack, prefill, unequal seeded partitions, Compensated Pruning by ratio
            (a sample of the sweep's corners: B = 4 / 128, tokens = 2048 / 16384)
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21089_b200 import synth
from tests.helpers import TOL_BF16, bits_of, dev_bf16, dev_f32, rel_err, rms_err, stack_tolerance, stream_ptr

pytestmark = pytest.mark.gpu

D, I, L = 4096, 14336, 32


def test_config3_fade_full_size(lib):
    B, n = 32, 8192
    d_b = synth.equal_partition(I, B)
    bits = synth.layer_weights(3, 0, D, I, 0.02, bf16=True)
    host = [synth.bf16_bits_to_f32(b) for b in bits]
    alpha = synth.uniform_f64((synth.BASE_SEED, 3, 0, synth.T_ALPHA), B, 0.8, 1.2).astype(np.float32)
    dev = [dev_bf16(b) for b in bits]
    h = lib.mlpmoe_create(D, I, d_b, dev[0], dev[1], dev[2], alpha.tolist(), lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, n, stream_ptr())
    try:
        lib.mlpmoe_fade(h, None, stream_ptr())
        Fg, Fu = oracle.fade(host[0], host[1], d_b)
        wg = torch.empty_like(dev[0]); wu = torch.empty_like(dev[1])
        lib.mlpmoe_get_weights(h, wg, wu, None, stream_ptr())
        torch.cuda.synchronize()
        assert np.array_equal(synth.bf16_bits_to_f32(bits_of(wg)), Fg)          # masks bit-exact, 58.7 M entries each
        assert np.array_equal(synth.bf16_bits_to_f32(bits_of(wu)), Fu)
        nnz = lib.mlpmoe_nnz(h, B)
        assert nnz == oracle.nnz_per_branch(Fg, Fu, host[2], d_b)
        # sparsity rises with the branch index; branch 0 dense; about 43.6 % of gate+up zeroed at B = 32
        frac = [1.0 - g / (D * 448) for g in nnz[0]]
        assert frac[0] < 1e-3 and all(frac[b] < frac[b + 1] for b in range(B - 1))
        assert abs(sum(frac) / B - 0.9 * (B - 1) / (2 * B)) < 5e-3
        assert lib.mlpmoe_get_klist(h, B, I) == oracle.surviving_set(alpha, Fg, Fu, host[2], d_b)
        xb = synth.f32_to_bf16_bits(synth.tokens(3, n, D))
        xd = dev_bf16(xb)
        y = torch.empty((n, D), dtype=torch.float32, device="cuda")
        lib.mlpmoe_forward(h, xd, y, n, stream_ptr())
        torch.cuda.synchronize()
        assert lib.mlpmoe_get_status(h) == lib.MLPMOE_OK
        rows = sorted(set([0, 127, 128, 255, 256, 4095, 4096, n - 1] + list(np.random.default_rng(3).integers(0, n, size=40))))
        ref = oracle.mlpmoe_forward(synth.bf16_bits_to_f32(xb[rows]), Fg, Fu, host[2], d_b, alpha)
        got = y.cpu().numpy()
        assert np.isfinite(got).all()
        assert rel_err(got[rows], ref) <= TOL_BF16
    finally:
        lib.mlpmoe_destroy(h)


def test_config3_structured_fade_full_size(lib):
    """The neuron-structured variant at the Llama-shaped layer of configs[2]: the set of removed neurons is decided by
    float64 scores that both sides must add up identically (14336 neurons x 8192 terms), so it is compared exactly."""
    B, n = 32, 2048
    d_b = synth.equal_partition(I, B)
    bits = synth.layer_weights(3, 0, D, I, 0.02, bf16=True)
    host = [synth.bf16_bits_to_f32(b) for b in bits]
    dev = [dev_bf16(b) for b in bits]
    h = lib.mlpmoe_create(D, I, d_b, dev[0], dev[1], dev[2], None, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, n, stream_ptr())
    try:
        lib.mlpmoe_fade_structured(h, None, stream_ptr())
        Fg, Fu = oracle.fade_structured(host[0], host[1], d_b)
        assert lib.mlpmoe_get_klist(h, B, I) == oracle.surviving_set([1.0] * B, Fg, Fu, host[2], d_b)
        left = lib.mlpmoe_get_active_neurons(h)
        assert left == I - sum((9 * b * 448) // (10 * B) for b in range(B))
        xb = synth.f32_to_bf16_bits(synth.tokens(3, n, D))
        y = torch.empty((n, D), dtype=torch.float32, device="cuda")
        lib.mlpmoe_forward(h, dev_bf16(xb), y, n, stream_ptr())
        torch.cuda.synchronize()
        rows = [0, 255, 256, 1000, n - 1]
        ref = oracle.mlpmoe_forward(synth.bf16_bits_to_f32(xb[rows]), Fg, Fu, host[2], d_b)
        assert rel_err(y.cpu().numpy()[rows], ref) <= TOL_BF16
        # and far tighter against the layer with the kernel's one extra rounding (H kept in bf16)
        ref_b = oracle.mlpmoe_forward_h_bf16(synth.bf16_bits_to_f32(xb[rows]), Fg, Fu, host[2], d_b)
        assert rel_err(y.cpu().numpy()[rows], ref_b) <= 4e-3
    finally:
        lib.mlpmoe_destroy(h)


def test_config3_routed_full_size(lib):
    """Per-token branch selection (labelled extension) at the Llama-shaped layer of configs[2], in the launch
    configuration the bench times: 8192 tokens, every token 8 of 32 branches (2048 rows, 8 blocks per branch, 256 blocks
    and about 5000 work items in the one grouped launch), non-unit alpha.  Rows are independent, so the oracle runs on a
    sample of them; a second call with another selection reuses the handle's buffers."""
    B, n, k = 32, 8192, 8
    d_b = synth.equal_partition(I, B)
    bits = synth.layer_weights(3, 0, D, I, 0.02, bf16=True)
    host = [synth.bf16_bits_to_f32(b) for b in bits]
    dev = [dev_bf16(b) for b in bits]
    alpha = [float(np.float32(a)) for a in synth.uniform_f64((synth.BASE_SEED, 3, 0, synth.T_ALPHA), B, 0.8, 1.2)]
    h = lib.mlpmoe_create(D, I, d_b, dev[0], dev[1], dev[2], alpha, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, n, stream_ptr())
    try:
        xb = synth.f32_to_bf16_bits(synth.tokens(3, n, D))
        xd = dev_bf16(xb)
        y = torch.empty((n, D), dtype=torch.float32, device="cuda")
        rows = [0, 1, 255, 256, 3000, 4095, 4096, 8000, n - 1]
        for trial, kk in enumerate((k, 3)):
            sel = synth.route_select((synth.BASE_SEED, 3, trial, synth.T_ROUTE), n, B, kk)
            sel[255] = 0
            sel[256] = 1
            lib.mlpmoe_forward_routed(h, xd, y, n, torch.from_numpy(sel).cuda(), True, stream_ptr())
            torch.cuda.synchronize()
            assert lib.mlpmoe_get_status(h) == lib.MLPMOE_OK
            got = y.cpu().numpy()
            ref = oracle.routed_forward(synth.bf16_bits_to_f32(xb[rows]), host[0], host[1], host[2], d_b, alpha, sel[rows])
            assert rel_err(got[rows], ref) <= TOL_BF16
            assert np.all(got[255] == 0.0) and np.isfinite(got).all()
    finally:
        lib.mlpmoe_destroy(h)


@pytest.fixture(scope="module")
def llama_stack():
    """Seeded bf16 weights of the 32 Llama-shaped layers: bit patterns on the host, tensors on the device."""
    host_bits, dev = [], []
    for l in range(L):
        bits = synth.layer_weights(4, l, D, I, 0.02, bf16=True)
        host_bits.append(bits)
        dev.append([dev_bf16(b) for b in bits])
    yield host_bits, dev
    del dev
    torch.cuda.empty_cache()


class LazyLayers:
    """Sequence of oracle layer tuples that widens one layer's weights at a time."""

    def __init__(self, host_bits, d_b, alphas):
        self.host_bits, self.d_b, self.alphas = host_bits, d_b, alphas

    def __iter__(self):
        for bits, alpha in zip(self.host_bits, self.alphas):
            yield (*[synth.bf16_bits_to_f32(b) for b in bits], self.d_b, alpha)


def make_handles(lib, dev, d_b, max_tokens, prune=None):
    handles = []
    for l in range(L):
        h = lib.mlpmoe_create(D, I, d_b, dev[l][0], dev[l][1], dev[l][2], None, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER,
                              max_tokens, stream_ptr())
        if handles:
            lib.mlpmoe_share_workspace(h, handles[0])
        handles.append(h)
        if prune is not None:
            prune(l, h)
    torch.cuda.synchronize()
    return handles


def check_layers_one_by_one(lib, handles, which, inputs, out, n_launch):
    """Each GPU layer, fed the oracle's input of that layer, must reproduce the oracle's contribution
    of that layer within the layer tolerance.  The first rows of an n_launch-row batch carry the
    sampled rows (the rest are zero), so the kernels run in their n_launch-token configuration."""
    xs = list(inputs) + [out]
    rows = xs[0].shape[0]
    for l in which:
        xin = np.zeros((n_launch, D), dtype=np.float32)
        xin[:rows] = xs[l].astype(np.float32)
        xd = dev_f32(xin)
        lib.mlpmoe_stack_forward([handles[l]], xd, n_launch, 1e-6, stream_ptr())
        torch.cuda.synchronize()
        got = xd.cpu().numpy()[:rows].astype(np.float64) - xin[:rows].astype(np.float64)
        assert rel_err(got, xs[l + 1] - xs[l]) <= TOL_BF16, l


def destroy(lib, handles):
    for h in handles[1:] + handles[:1]:
        lib.mlpmoe_destroy(h)


@pytest.mark.parametrize("n", [65, 128])
def test_llama_shape_decode_stack_65_to_128_tokens(lib, llama_stack, n):
    """The 128-row build of the persistent decode kernel (65 to 128 tokens) at the Llama shape: three layers, every
    token row real, against the oracle end to end (3 layers: first-order bound) and on the bulk of the error."""
    host_bits, dev = llama_stack
    B, nl = 64, 3
    d_b = synth.equal_partition(I, B)
    x = synth.tokens(4, 128, D, stream=7)[:n]
    handles = []
    try:
        for l in range(nl):
            h = lib.mlpmoe_create(D, I, d_b, dev[l][0], dev[l][1], dev[l][2], None, lib.MLPMOE_BF16, lib.MLPMOE_LAYOUT_PAPER, 128,
                                  stream_ptr())
            if handles:
                lib.mlpmoe_share_workspace(h, handles[0])
            handles.append(h)
        layers = [tuple(synth.bf16_bits_to_f32(b) for b in host_bits[l]) + (d_b, [1.0] * B) for l in range(nl)]
        ref, inputs = oracle.stack_forward(x, layers, bf16_activations=True, return_layer_inputs=True)
        xd = dev_f32(x)
        lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
        torch.cuda.synchronize()
        assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
        got = xd.cpu().numpy()
        tol = stack_tolerance(inputs, ref)
        e_max, e_rms = rel_err(got, ref), rms_err(got, ref)
        print(f"{n} tokens, 3 Llama-shaped layers: max|delta|/RMS = {e_max:.4f} (bound {tol:.4f}), RMS(delta)/RMS = {e_rms:.5f}")
        assert e_max <= tol and e_rms <= 5e-3
    finally:
        destroy(lib, handles)


def test_config4_decode_stack(lib, llama_stack):
    host_bits, dev = llama_stack
    B = 64
    d_b = synth.equal_partition(I, B)
    x = synth.tokens(4, 64, D)
    handles = make_handles(lib, dev, d_b, 64)
    try:
        for K in (None, 51):
            if K is not None:
                for h in handles:
                    lib.mlpmoe_prune_first_k(h, K, stream_ptr())
                alpha = oracle.prune_alpha([1.0] * B, oracle.first_k_keep(B, K))
                assert lib.mlpmoe_get_active_neurons(handles[0]) == K * 224
                assert lib.mlpmoe_get_klist(handles[-1], B, I) == (list(range(K)), [(224 * b, 224) for b in range(K)])
            else:
                alpha = [1.0] * B
            ref, inputs = oracle.stack_forward(x, LazyLayers(host_bits, d_b, [alpha] * L), bf16_activations=True,
                                               return_layer_inputs=True)
            check_layers_one_by_one(lib, handles, range(L), inputs, ref, 64)
            check_layers_one_by_one(lib, handles, (0, L - 1), [v[:1] for v in inputs], ref[:1], 1)
            # End to end over 32 layers: first-order sum of the per-layer allowances on the worst element
            # (about 0.09 of RMS(x_out) here), 2e-2 on the bulk (RMS) of the error.
            tol = stack_tolerance(inputs, ref)
            assert tol < 0.12
            for n in (1, 8, 32, 64):
                xd = dev_f32(x[:n])
                lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
                torch.cuda.synchronize()
                e_max, e_rms = rel_err(xd.cpu().numpy(), ref[:n]), rms_err(xd.cpu().numpy(), ref[:n])
                print(f"config 4 end to end, K={K}, n={n}: max|delta|/RMS = {e_max:.4f} (bound {tol:.4f}), RMS(delta)/RMS = {e_rms:.5f}")
                assert e_max <= tol, (K, n)
                assert e_rms <= TOL_BF16, (K, n)
            assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
    finally:
        destroy(lib, handles)


@pytest.mark.parametrize("B,n,ratio", [(128, 2048, 0.4), (4, 16384, 0.1), (16, 2048, 0.2)])
def test_config5_prefill_sweep_corners(lib, llama_stack, B, n, ratio):
    host_bits, dev = llama_stack
    d_b = synth.random_partition((synth.BASE_SEED, 5, B, synth.T_PARTITION), I, B, 64)
    n_drop = synth.n_drop_for_ratio(B, ratio)
    keeps = [synth.keep_set((synth.BASE_SEED, 5, B, l, synth.T_KEEP), B, n_drop) for l in range(L)]
    alphas = [oracle.prune_alpha([1.0] * B, k) for k in keeps]
    handles = make_handles(lib, dev, d_b, n, prune=lambda l, h: lib.mlpmoe_prune(h, keeps[l], True, stream_ptr()))
    try:
        offs = oracle.branch_offsets(d_b)
        for l in (0, L - 1):
            kept = [b for b in range(B) if keeps[l][b]]
            assert lib.mlpmoe_get_klist(handles[l], B, I) == (kept, [(offs[b], d_b[b]) for b in kept])
            assert np.array_equal(lib.mlpmoe_get_alpha(handles[l], B).view(np.uint32),
                                  np.array(alphas[l]).astype(np.float32).view(np.uint32))
        x = synth.tokens(5, n, D, stream=B)
        xd = dev_f32(x)
        lib.mlpmoe_stack_forward(handles, xd, n, 1e-6, stream_ptr())
        torch.cuda.synchronize()
        rows = sorted(set([0, 255, 256, n - 1] + list(np.random.default_rng(B).integers(0, n, size=8))))
        ref, inputs = oracle.stack_forward(x[rows], LazyLayers(host_bits, d_b, alphas), bf16_activations=True,
                                           return_layer_inputs=True)
        got = xd.cpu().numpy()
        assert np.isfinite(got).all()
        tol = stack_tolerance(inputs, ref)
        e_max, e_rms = rel_err(got[rows], ref), rms_err(got[rows], ref)
        print(f"config 5 end to end, B={B}, n={n}, ratio={ratio}: max|delta|/RMS = {e_max:.4f} (bound {tol:.4f}), RMS(delta)/RMS = {e_rms:.5f}")
        assert tol < 0.12
        assert e_max <= tol
        assert e_rms <= TOL_BF16
        check_layers_one_by_one(lib, handles, list(range(0, L, 4)) + [L - 1], inputs, ref, n)
        assert all(lib.mlpmoe_get_status(h) == lib.MLPMOE_OK for h in handles)
    finally:
        destroy(lib, handles)
