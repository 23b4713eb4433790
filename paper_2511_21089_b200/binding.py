"""Thin ctypes binding over the C-ABI library (include/mlpmoe.h): argument marshalling only.

Every function has the name of the C entry point it calls.  Device buffers are passed as
torch CUDA tensors (their data_ptr() is what crosses the boundary) or as raw integer
addresses; host arrays as Python sequences / numpy arrays.  There is no fallback: if the
shared library has not been built the import of this module raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_double, c_float, c_int32, c_int64, c_uint8, c_void_p
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("MLPMOE_LIB_PATH") or os.path.join(_HERE, "libmlpmoe_b200.so")

MLPMOE_OK = 0
MLPMOE_ERR_INVALID_ARG = 1
MLPMOE_ERR_BAD_PARTITION = 2
MLPMOE_ERR_EMPTY_KEEP_SET = 3
MLPMOE_ERR_BAD_SCHEDULE = 4
MLPMOE_ERR_UNSUPPORTED = 5
MLPMOE_ERR_ALLOC = 6
MLPMOE_ERR_CUDA = 7
MLPMOE_ERR_DEVICE_TIMEOUT = 8
MLPMOE_BF16 = 0
MLPMOE_FP32 = 1
MLPMOE_LAYOUT_PAPER = 0
MLPMOE_LAYOUT_LINEAR = 1

# name -> (restype, argtypes): every symbol include/mlpmoe.h declares
SIGNATURES = {
    "mlpmoe_create": (c_int32, [POINTER(c_void_p), c_int64, c_int64, c_int32, POINTER(c_int64), c_void_p, c_void_p,
                                c_void_p, POINTER(c_float), c_int32, c_int32, c_int64, c_void_p]),
    "mlpmoe_destroy": (None, [c_void_p]),
    "mlpmoe_share_workspace": (c_int32, [c_void_p, c_void_p]),
    "mlpmoe_fade": (c_int32, [c_void_p, POINTER(c_double), c_void_p]),
    "mlpmoe_set_fast_fp32": (c_int32, [c_void_p, c_int32, c_void_p]),
    "mlpmoe_fade_structured": (c_int32, [c_void_p, POINTER(c_double), c_void_p]),
    "mlpmoe_prune": (c_int32, [c_void_p, POINTER(c_uint8), c_int32, c_void_p]),
    "mlpmoe_prune_first_k": (c_int32, [c_void_p, c_int32, c_void_p]),
    "mlpmoe_forward": (c_int32, [c_void_p, c_void_p, c_void_p, c_int64, c_void_p]),
    "mlpmoe_forward_ex": (c_int32, [c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_int32, c_void_p]),
    "mlpmoe_forward_routed": (c_int32, [c_void_p, c_void_p, c_void_p, c_int64, c_void_p, c_int32, c_void_p]),
    "mlpmoe_forward_host": (c_int32, [c_void_p, c_void_p, c_void_p, c_int64, c_void_p]),
    "mlpmoe_rmsnorm": (c_int32, [c_void_p, c_void_p, c_int64, c_int64, c_float, c_int32, c_void_p]),
    "mlpmoe_stack_prepare": (c_int32, [POINTER(c_void_p), c_int32, c_int64, c_void_p]),
    "mlpmoe_debug_set_wait": (c_int32, [c_void_p, ctypes.c_uint64, ctypes.c_uint32]),
    "mlpmoe_debug_set_decode_kernel": (c_int32, [c_void_p, c_int32]),
    "mlpmoe_get_workspace": (c_int32, [c_void_p, POINTER(c_void_p), POINTER(c_int64), POINTER(c_void_p), POINTER(c_int64),
                                       POINTER(c_void_p), POINTER(c_int64), POINTER(c_int64)]),
    "mlpmoe_stack_forward": (c_int32, [POINTER(c_void_p), c_int32, c_void_p, c_int64, c_float, c_void_p]),
    "mlpmoe_stack_forward_host": (c_int32, [POINTER(c_void_p), c_int32, c_void_p, c_void_p, c_int64, c_float, c_void_p]),
    "mlpmoe_get_klist": (c_int32, [c_void_p, POINTER(c_int32), POINTER(c_int32), POINTER(c_int64), POINTER(c_int64),
                                   POINTER(c_int32)]),
    "mlpmoe_get_alpha": (c_int32, [c_void_p, POINTER(c_float)]),
    "mlpmoe_get_active_neurons": (c_int32, [c_void_p, POINTER(c_int64)]),
    "mlpmoe_nnz": (c_int32, [c_void_p, POINTER(c_int64), POINTER(c_int64), POINTER(c_int64)]),
    "mlpmoe_get_weights": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "mlpmoe_get_status": (c_int32, [c_void_p]),
    "mlpmoe_get_kernel_clock": (c_int32, [c_void_p, POINTER(c_double), POINTER(c_double)]),
    "mlpmoe_get_launch_count": (c_int32, [c_void_p, POINTER(c_int64)]),
    "mlpmoe_status_string": (c_char_p, [c_int32]),
    "mlpmoe_set_timing": (c_int32, [c_void_p, c_int32]),
    "mlpmoe_get_timing": (c_int32, [c_void_p, POINTER(c_double), POINTER(c_int64)]),
    "mlpmoe_fade_buffers_static": (c_int32, [POINTER(c_void_p), POINTER(c_int64), POINTER(c_double), c_int32, c_int32, c_void_p]),
    "mlpmoe_host_fade_position": (c_int32, [c_double, c_int64, POINTER(c_int64)]),
    "mlpmoe_host_fade_position_default": (c_int32, [c_int32, c_int32, c_int64, POINTER(c_int64)]),
    "mlpmoe_host_prune_alpha": (c_int32, [c_int32, POINTER(c_float), POINTER(c_uint8), c_int32, POINTER(c_float)]),
    "mlpmoe_host_tile_schedule": (c_int32, [c_int64, c_int64, c_int64, c_int32, c_int32, c_int32, POINTER(c_int32), POINTER(c_int32),
                                            POINTER(c_int32)]),
    "mlpmoe_host_stack_schedule": (c_int32, [c_int64, c_int64, c_int32, POINTER(c_int64), POINTER(c_int32), c_int32, c_int32,
                                             POINTER(c_int32), c_int64, POINTER(c_int64), POINTER(c_int32)]),
    "mlpmoe_host_group_schedule": (c_int32, [POINTER(c_int32), c_int32, c_int64, c_int32, POINTER(c_int64), c_int32, c_int32,
                                             POINTER(c_int32), c_int64, POINTER(c_int64), POINTER(c_int32)]),
    "mlpmoe_host_schedule": (c_int32, [c_int32, POINTER(c_int64), POINTER(c_float), POINTER(c_uint8), POINTER(c_int32),
                                       POINTER(c_int32), POINTER(c_int64), POINTER(c_int64), POINTER(c_int32),
                                       POINTER(c_int64)]),
}

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_21089_b200.build` "
                      "(there is no CPU or PyTorch fallback)")
lib = ctypes.CDLL(LIB_PATH)
for _name, (_res, _args) in SIGNATURES.items():
    _f = getattr(lib, _name)
    _f.restype = _res
    _f.argtypes = _args


class MlpmoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {mlpmoe_status_string(status)} (status {status})")


def _check(status: int, where: str) -> None:
    if status != MLPMOE_OK:
        raise MlpmoeError(status, where)


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor / numpy array / raw int, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return None
    return stream if isinstance(stream, int) else stream.cuda_stream


def _arr(values, ctype):
    if values is None:
        return None
    values = list(values)
    return (ctype * len(values))(*values)


def mlpmoe_status_string(status: int) -> str:
    return lib.mlpmoe_status_string(status).decode()


def mlpmoe_create(d_model: int, d_inter: int, d_b: Sequence[int], W_gate, W_up, W_down, alpha=None,
                  dtype: int = MLPMOE_BF16, layout: int = MLPMOE_LAYOUT_PAPER, max_tokens: int = 4096, stream=None) -> int:
    out = c_void_p()
    st = lib.mlpmoe_create(ctypes.byref(out), d_model, d_inter, len(d_b), _arr(d_b, c_int64), _ptr(W_gate), _ptr(W_up),
                           _ptr(W_down), _arr(alpha, c_float), dtype, layout, max_tokens, _stream(stream))
    _check(st, "mlpmoe_create")
    return out.value


def mlpmoe_destroy(h: int) -> None:
    lib.mlpmoe_destroy(h)


def mlpmoe_share_workspace(h: int, donor: int) -> None:
    _check(lib.mlpmoe_share_workspace(h, donor), "mlpmoe_share_workspace")


def mlpmoe_fade(h: int, s: Optional[Sequence[float]] = None, stream=None) -> None:
    _check(lib.mlpmoe_fade(h, _arr(s, c_double), _stream(stream)), "mlpmoe_fade")


def mlpmoe_set_fast_fp32(h: int, enable: bool = True, stream=None) -> None:
    _check(lib.mlpmoe_set_fast_fp32(h, 1 if enable else 0, _stream(stream)), "mlpmoe_set_fast_fp32")


def mlpmoe_fade_structured(h: int, s: Optional[Sequence[float]] = None, stream=None) -> None:
    _check(lib.mlpmoe_fade_structured(h, _arr(s, c_double), _stream(stream)), "mlpmoe_fade_structured")


def mlpmoe_prune(h: int, keep: Sequence[bool], compensate: bool = True, stream=None) -> None:
    _check(lib.mlpmoe_prune(h, _arr([1 if k else 0 for k in keep], c_uint8), 1 if compensate else 0, _stream(stream)),
           "mlpmoe_prune")


def mlpmoe_prune_first_k(h: int, K: int, stream=None) -> None:
    _check(lib.mlpmoe_prune_first_k(h, K, _stream(stream)), "mlpmoe_prune_first_k")


def mlpmoe_forward(h: int, x, y, n_tokens: int, stream=None) -> None:
    _check(lib.mlpmoe_forward(h, _ptr(x), _ptr(y), n_tokens, _stream(stream)), "mlpmoe_forward")


def mlpmoe_forward_ex(h: int, x, y, n_tokens: int, residual=None, y_dtype: int = MLPMOE_FP32, stream=None) -> None:
    _check(lib.mlpmoe_forward_ex(h, _ptr(x), _ptr(y), n_tokens, _ptr(residual), y_dtype, _stream(stream)), "mlpmoe_forward_ex")


def mlpmoe_forward_routed(h: int, x, y, n_tokens: int, select, compensate: bool = True, stream=None) -> None:
    """select: device uint8 [n_tokens x B]."""
    _check(lib.mlpmoe_forward_routed(h, _ptr(x), _ptr(y), n_tokens, _ptr(select), 1 if compensate else 0, _stream(stream)),
           "mlpmoe_forward_routed")


def mlpmoe_forward_host(h: int, x_host, y_host, n_tokens: int, stream=None) -> None:
    _check(lib.mlpmoe_forward_host(h, _ptr(x_host), _ptr(y_host), n_tokens, _stream(stream)), "mlpmoe_forward_host")


def mlpmoe_rmsnorm(x, r, n_tokens: int, d_model: int, eps: float = 1e-6, out_dtype: int = MLPMOE_BF16, stream=None) -> None:
    _check(lib.mlpmoe_rmsnorm(_ptr(x), _ptr(r), n_tokens, d_model, eps, out_dtype, _stream(stream)), "mlpmoe_rmsnorm")


def mlpmoe_stack_forward(layers: Sequence[int], x, n_tokens: int, eps: float = 1e-6, stream=None) -> None:
    arr = (c_void_p * len(layers))(*layers)
    _check(lib.mlpmoe_stack_forward(arr, len(layers), _ptr(x), n_tokens, eps, _stream(stream)), "mlpmoe_stack_forward")


def mlpmoe_stack_prepare(layers: Sequence[int], n_tokens: int, stream=None) -> None:
    arr = (c_void_p * len(layers))(*layers)
    _check(lib.mlpmoe_stack_prepare(arr, len(layers), n_tokens, _stream(stream)), "mlpmoe_stack_prepare")


def mlpmoe_debug_set_decode_kernel(h: int, kernel: int) -> None:
    _check(lib.mlpmoe_debug_set_decode_kernel(h, kernel), "mlpmoe_debug_set_decode_kernel")


def mlpmoe_debug_set_wait(h: int, limit_ns: int = 0, extra_arrivals: int = 0) -> None:
    _check(lib.mlpmoe_debug_set_wait(h, limit_ns, extra_arrivals), "mlpmoe_debug_set_wait")


def mlpmoe_get_workspace(h: int) -> dict:
    """Addresses and byte sizes of the handle's activation workspace, and the padded neuron count."""
    H, xn, yr = c_void_p(), c_void_p(), c_void_p()
    hb, xb, yb, ip = c_int64(), c_int64(), c_int64(), c_int64()
    _check(lib.mlpmoe_get_workspace(h, ctypes.byref(H), ctypes.byref(hb), ctypes.byref(xn), ctypes.byref(xb), ctypes.byref(yr),
                                    ctypes.byref(yb), ctypes.byref(ip)), "mlpmoe_get_workspace")
    return dict(H=H.value, H_bytes=hb.value, xnorm=xn.value, xnorm_bytes=xb.value, yres=yr.value, yres_bytes=yb.value,
                n_active_pad=ip.value)


def mlpmoe_stack_forward_host(layers: Sequence[int], x_host, y_host, n_tokens: int, eps: float = 1e-6, stream=None) -> None:
    arr = (c_void_p * len(layers))(*layers)
    _check(lib.mlpmoe_stack_forward_host(arr, len(layers), _ptr(x_host), _ptr(y_host), n_tokens, eps, _stream(stream)),
           "mlpmoe_stack_forward_host")


def mlpmoe_get_klist(h: int, B: int, d_inter: int):
    """Returns (branches, [(start, length), ...])."""
    br = (c_int32 * B)()
    nb = c_int32()
    ss = (c_int64 * d_inter)()
    sl = (c_int64 * d_inter)()
    ns = c_int32()
    _check(lib.mlpmoe_get_klist(h, br, ctypes.byref(nb), ss, sl, ctypes.byref(ns)), "mlpmoe_get_klist")
    return list(br[:nb.value]), [(ss[i], sl[i]) for i in range(ns.value)]


def mlpmoe_get_alpha(h: int, B: int) -> np.ndarray:
    a = (c_float * B)()
    _check(lib.mlpmoe_get_alpha(h, a), "mlpmoe_get_alpha")
    return np.array(a[:], dtype=np.float32)


def mlpmoe_get_active_neurons(h: int) -> int:
    v = c_int64()
    _check(lib.mlpmoe_get_active_neurons(h, ctypes.byref(v)), "mlpmoe_get_active_neurons")
    return v.value


def mlpmoe_nnz(h: int, B: int):
    g, u, d = (c_int64 * B)(), (c_int64 * B)(), (c_int64 * B)()
    _check(lib.mlpmoe_nnz(h, g, u, d), "mlpmoe_nnz")
    return list(g), list(u), list(d)


def mlpmoe_get_weights(h: int, W_gate=None, W_up=None, W_down=None, stream=None) -> None:
    _check(lib.mlpmoe_get_weights(h, _ptr(W_gate), _ptr(W_up), _ptr(W_down), _stream(stream)), "mlpmoe_get_weights")


def mlpmoe_get_status(h: int) -> int:
    return lib.mlpmoe_get_status(h)


def mlpmoe_get_kernel_clock(h: int):
    """(SM MHz, kernel lifetime in microseconds) of the handle's last persistent-kernel launch."""
    mhz, us = c_double(), c_double()
    _check(lib.mlpmoe_get_kernel_clock(h, ctypes.byref(mhz), ctypes.byref(us)), "mlpmoe_get_kernel_clock")
    return mhz.value, us.value


def mlpmoe_get_launch_count(h: int) -> int:
    v = c_int64()
    _check(lib.mlpmoe_get_launch_count(h, ctypes.byref(v)), "mlpmoe_get_launch_count")
    return v.value


def mlpmoe_set_timing(h: int, enable: bool) -> None:
    _check(lib.mlpmoe_set_timing(h, 1 if enable else 0), "mlpmoe_set_timing")


def mlpmoe_get_timing(h: int):
    """Returns ([ms gate|up, ms down, ms rmsnorm], [launch counts]) since the last call."""
    ms = (c_double * 3)()
    cnt = (c_int64 * 3)()
    _check(lib.mlpmoe_get_timing(h, ms, cnt), "mlpmoe_get_timing")
    return list(ms), list(cnt)


def mlpmoe_fade_buffers_static(slices: Sequence, s: Sequence[float], dtype: int = MLPMOE_BF16, stream=None) -> None:
    """Mask caller-owned device buffers in place (one contiguous tensor per slice) with the library's
    built-in scratch; allocates nothing.  `slices` are torch CUDA tensors or (address, n_elements) pairs."""
    ptrs, sizes = [], []
    for t in slices:
        if isinstance(t, tuple):
            ptrs.append(t[0]); sizes.append(t[1])
        else:
            ptrs.append(t.data_ptr()); sizes.append(t.numel())
    n = len(ptrs)
    _check(lib.mlpmoe_fade_buffers_static((c_void_p * n)(*ptrs), (c_int64 * n)(*sizes), (c_double * n)(*s), n, dtype,
                                          _stream(stream)), "mlpmoe_fade_buffers_static")


def mlpmoe_host_fade_position(s: float, m: int) -> int:
    lo = c_int64()
    _check(lib.mlpmoe_host_fade_position(s, m, ctypes.byref(lo)), "mlpmoe_host_fade_position")
    return lo.value


def mlpmoe_host_fade_position_default(b: int, B: int, m: int) -> int:
    lo = c_int64()
    _check(lib.mlpmoe_host_fade_position_default(b, B, m, ctypes.byref(lo)), "mlpmoe_host_fade_position_default")
    return lo.value


def mlpmoe_host_prune_alpha(alpha: Sequence[float], keep: Sequence[bool], compensate: bool = True) -> np.ndarray:
    B = len(alpha)
    out = (c_float * B)()
    _check(lib.mlpmoe_host_prune_alpha(B, _arr(alpha, c_float), _arr([1 if k else 0 for k in keep], c_uint8),
                                       1 if compensate else 0, out), "mlpmoe_host_prune_alpha")
    return np.array(out[:], dtype=np.float32)


def mlpmoe_host_schedule(d_b: Sequence[int], alpha_eff: Sequence[float], live=None):
    """Returns (branches, [(start, length), ...], n_active)."""
    B = len(d_b)
    I = int(sum(d_b))
    br = (c_int32 * B)()
    nb = c_int32()
    ss = (c_int64 * I)()
    sl = (c_int64 * I)()
    ns = c_int32()
    na = c_int64()
    live_arr = None if live is None else _arr([1 if v else 0 for v in live], c_uint8)
    _check(lib.mlpmoe_host_schedule(B, _arr(d_b, c_int64), _arr(alpha_eff, c_float), live_arr, br, ctypes.byref(nb), ss, sl,
                                    ctypes.byref(ns), ctypes.byref(na)), "mlpmoe_host_schedule")
    return list(br[:nb.value]), [(ss[i], sl[i]) for i in range(ns.value)], na.value


def mlpmoe_host_tile_schedule(n_tokens: int, d_model: int, n_active_pad: int, bn: int, ksplit: int = 1, num_sms: int = 148):
    """Returns one list of (is_down, column_tile [* ksplit + slice], token_block) per CTA pair."""
    cap = ((n_tokens + 255) // 256) * (n_active_pad // 128 + ksplit * ((d_model + bn - 1) // bn))
    tiles = (c_int32 * cap)()
    n_tiles = c_int32()
    offs = (c_int32 * (num_sms // 2 + 1))()
    _check(lib.mlpmoe_host_tile_schedule(n_tokens, d_model, n_active_pad, bn, ksplit, num_sms, tiles, ctypes.byref(n_tiles), offs),
           "mlpmoe_host_tile_schedule")
    out = []
    for c in range(num_sms // 2):
        out.append([((t >> 31) & 1, (t >> 16) & 0x7FFF, t & 0xFFFF) for t in tiles[offs[c]:offs[c + 1]]])
    return out


def mlpmoe_host_stack_schedule(n_tokens: int, d_model: int, n_active_pad: Sequence[int], ksplit: Sequence[int], bn: int,
                               num_sms: int = 148):
    """Returns (gemm, norm): for each CTA pair its sequence of GEMM items and its sequence of norm
    parts, as (type, column, token_block, layer); type 0 = gate|up tile, 1 = down item, 2 = norm part."""
    L = len(n_active_pad)
    m_pairs = (n_tokens + 255) // 256
    pairs = num_sms // 2
    cap = sum(m_pairs * (16 + ip // 128 + ks * ((d_model + bn - 1) // bn)) for ip, ks in zip(n_active_pad, ksplit))
    items = (c_int32 * (2 * cap))()
    n_items = c_int64()
    offs = (c_int32 * (2 * (pairs + 1)))()
    _check(lib.mlpmoe_host_stack_schedule(n_tokens, d_model, L, (c_int64 * L)(*n_active_pad), (c_int32 * L)(*ksplit), bn, num_sms,
                                          items, cap, ctypes.byref(n_items), offs), "mlpmoe_host_stack_schedule")

    def seq(lo, hi):
        return [((items[2 * i] >> 30) & 3, (items[2 * i] >> 16) & 0x3FFF, items[2 * i] & 0xFFFF, items[2 * i + 1]) for i in range(lo, hi)]
    gemm = [seq(offs[c], offs[c + 1]) for c in range(pairs)]
    norm = [seq(offs[pairs + 1 + c], offs[pairs + 2 + c]) for c in range(pairs)]
    return gemm, norm


def mlpmoe_host_group_schedule(block_branch: Sequence[int], d_model: int, n_active_pad: Sequence[int], bn: int, num_sms: int = 148):
    """For each CTA pair its sequence of items (type, column, block, branch) of the grouped launch of the routed
    forward; type 0 = gate|up tile, 1 = down item."""
    nb, B = len(block_branch), len(n_active_pad)
    pairs = num_sms // 2
    n2 = (d_model + bn - 1) // bn
    cap = sum(n_active_pad[b] // 128 + n2 for b in block_branch) + 1
    items = (c_int32 * (2 * cap))()
    n_items = c_int64()
    offs = (c_int32 * (2 * (pairs + 1)))()
    _check(lib.mlpmoe_host_group_schedule((c_int32 * max(nb, 1))(*block_branch), nb, d_model, B, (c_int64 * B)(*n_active_pad), bn, num_sms,
                                          items, cap, ctypes.byref(n_items), offs), "mlpmoe_host_group_schedule")
    assert all(offs[pairs + 1 + c] == n_items.value for c in range(pairs + 1))      # the norm sequences are empty
    return [[((items[2 * i] >> 30) & 3, (items[2 * i] >> 16) & 0x3FFF, items[2 * i] & 0xFFFF, items[2 * i + 1])
             for i in range(offs[c], offs[c + 1])] for c in range(pairs)]
