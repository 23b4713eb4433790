"""The allocation-free Fade entry point against the handle-based one.

mlpmoe_fade_buffers_static serves callers that cannot allocate device memory at the moment
they need the masking step (all memory already given to an arena, or no tolerance for
cudaMalloc's device-wide synchronisation): its scratch is a fixed array inside the library.
This file is collected last on purpose, so a failure here cannot hide another test's result.
The check: the same slices and ratios through mlpmoe_fade (scratch allocated at create) and
through the static entry point give bit-identical masked weights, on two calls in a row -
the second call proves that what the first left in the shared array does no harm.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_21089_b200 import synth
from tests.helpers import Case, bits_of, stream_ptr

pytestmark = pytest.mark.gpu


def _handle_fade(lib, c, s):
    h = c.create(lib, 64)
    try:
        lib.mlpmoe_fade(h, s, stream_ptr())
        wg = torch.empty_like(c.dev[0])
        wu = torch.empty_like(c.dev[1])
        lib.mlpmoe_get_weights(h, wg, wu, None, stream_ptr())
        torch.cuda.synchronize()
        return wg, wu
    finally:
        lib.mlpmoe_destroy(h)


@pytest.mark.parametrize("bf16", [True, False])
def test_static_fade_matches_handle_fade_twice(lib, bf16):
    d, d_b = 128, [64, 192, 128, 128]
    I = sum(d_b)
    offs = oracle.branch_offsets(d_b)
    dtype = lib.MLPMOE_BF16 if bf16 else lib.MLPMOE_FP32
    schedules = ([0.0, 0.225, 0.45, 0.675], [0.5, 0.0, 0.875, 0.0625])
    for call, s in enumerate(schedules):                      # two calls in a row, different data and ratios
        c = Case((300, call, int(bf16)), d, I, d_b, bf16=bf16, std=0.02)
        ref_g, ref_u = _handle_fade(lib, c, s)
        slices, ratios = [], []
        for W in (c.dev[0], c.dev[1]):
            for b in range(len(d_b)):
                slices.append(W[:, offs[b]:offs[b + 1]].contiguous())
                ratios.append(s[b])
        # cudaMalloc inside the library would not show in torch's caching allocator: watch the device's free memory
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        lib.mlpmoe_fade_buffers_static(slices, ratios, dtype, stream_ptr())
        assert torch.cuda.mem_get_info()[0] >= free_before
        for k, (W, ref) in enumerate(((c.dev[0], ref_g), (c.dev[1], ref_u))):
            for b in range(len(d_b)):
                got = slices[k * len(d_b) + b]
                want = ref[:, offs[b]:offs[b + 1]]
                if bf16:
                    assert np.array_equal(bits_of(got), bits_of(want.contiguous()))
                else:
                    assert np.array_equal(got.cpu().numpy(), want.cpu().numpy())
                if s[b] == 0.0:
                    assert torch.equal(got, W[:, offs[b]:offs[b + 1]])
        # and both agree with the oracle
        Fg, _ = oracle.fade(c.host[0], c.host[1], d_b, s)
        got_g = torch.cat(slices[:len(d_b)], dim=1)
        got_g = synth.bf16_bits_to_f32(bits_of(got_g)) if bf16 else got_g.cpu().numpy()
        assert np.array_equal(got_g, Fg)


def test_static_fade_rejects_bad_arguments(lib):
    import ctypes
    x = torch.zeros(64, device="cuda", dtype=torch.float32)
    with pytest.raises(lib.MlpmoeError) as e:
        lib.mlpmoe_fade_buffers_static([x] * 257, [0.5] * 257, lib.MLPMOE_FP32, stream_ptr())
    assert e.value.status == lib.MLPMOE_ERR_UNSUPPORTED                 # more slices than the fixed scratch holds
    with pytest.raises(lib.MlpmoeError) as e:
        lib.mlpmoe_fade_buffers_static([x], [1.0], lib.MLPMOE_FP32, stream_ptr())
    assert e.value.status == lib.MLPMOE_ERR_BAD_SCHEDULE
    assert lib.lib.mlpmoe_fade_buffers_static(None, None, None, 3, 1, None) == lib.MLPMOE_ERR_INVALID_ARG
    # a slice that is not aligned to its element size is refused on the host (nothing is launched)
    for dtype, off in ((lib.MLPMOE_FP32, 2), (lib.MLPMOE_FP32, 1), (lib.MLPMOE_BF16, 1)):
        ptrs = (ctypes.c_void_p * 1)(x.data_ptr() + off)
        m = (ctypes.c_int64 * 1)(8)
        s = (ctypes.c_double * 1)(0.5)
        assert lib.lib.mlpmoe_fade_buffers_static(ptrs, m, s, 1, dtype, None) == lib.MLPMOE_ERR_INVALID_ARG
    lib.mlpmoe_fade_buffers_static([], [], lib.MLPMOE_FP32, stream_ptr())   # nothing to do
    assert float(x.abs().sum()) == 0.0
