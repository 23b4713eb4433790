"""Shared helpers of the GPU parity tests: moving seeded inputs to the device and the
error measure the tolerances are stated in."""
import numpy as np
import torch

from paper_2511_21089_b200 import synth

TOL_BF16 = 2e-2     # max|delta| <= 2e-2 * RMS(y_ref), bf16 layers
TOL_FP32 = 1e-4     # max|delta| <= 1e-4 * RMS(y_ref), fp32 layers


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bfloat16 tensor of the same shape."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def dev_f32(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def bits_of(t: torch.Tensor) -> np.ndarray:
    """CUDA bfloat16 tensor -> uint16 bit patterns on the host."""
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


def rel_err(y: np.ndarray, ref: np.ndarray) -> float:
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(np.asarray(y, dtype=np.float64) - ref)) / np.sqrt(np.mean(ref ** 2)))


def stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream


class Case:
    """One synthetic layer: weights on the host (exact values as float arrays for the oracle)
    and on the device (for the library)."""

    def __init__(self, key, d, I, d_b, bf16=True, std=0.02, alpha=None):
        self.d, self.I, self.d_b, self.bf16 = d, I, list(d_b), bf16
        wg = synth.normal_f32((*key, synth.T_GATE), (d, I), std)
        wu = synth.normal_f32((*key, synth.T_UP), (d, I), std)
        wd = synth.normal_f32((*key, synth.T_DOWN), (I, d), std)
        if bf16:
            self.bits = [synth.f32_to_bf16_bits(w) for w in (wg, wu, wd)]
            self.host = [synth.bf16_bits_to_f32(b) for b in self.bits]
            self.dev = [dev_bf16(b) for b in self.bits]
        else:
            self.host = [wg, wu, wd]
            self.dev = [dev_f32(w) for w in self.host]
        self.alpha = None if alpha is None else [float(np.float32(a)) for a in alpha]

    def tokens(self, key, n):
        """(host values as float32 exactly as the device sees them, device tensor)."""
        x = synth.normal_f32((*key, synth.T_X), (n, self.d), 1.0)
        if self.bf16:
            b = synth.f32_to_bf16_bits(x)
            return synth.bf16_bits_to_f32(b), dev_bf16(b)
        return x, dev_f32(x)

    def create(self, lib, max_tokens, layout=0):
        dtype = lib.MLPMOE_BF16 if self.bf16 else lib.MLPMOE_FP32
        wg, wu, wd = self.dev
        if layout == lib.MLPMOE_LAYOUT_LINEAR:
            wg, wu, wd = wg.t().contiguous(), wu.t().contiguous(), wd.t().contiguous()
        h = lib.mlpmoe_create(self.d, self.I, self.d_b, wg, wu, wd, self.alpha, dtype, layout, max_tokens, stream_ptr())
        torch.cuda.synchronize()
        return h


def layer_rms(inputs, out):
    """RMS of every layer's own contribution y_l = x_{l+1} - x_l in the oracle's run."""
    xs = list(inputs) + [out]
    return [float(np.sqrt(np.mean((xs[l + 1] - xs[l]) ** 2))) for l in range(len(inputs))]


def rms_err(y: np.ndarray, ref: np.ndarray) -> float:
    """RMS of the error over the RMS of the reference (the bulk of the error, not its worst element)."""
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.sqrt(np.mean((np.asarray(y, dtype=np.float64) - ref) ** 2)) / np.sqrt(np.mean(ref ** 2)))


def stack_tolerance(inputs, out):
    """End-to-end bound on max|delta| for a deep stack, as a multiple of RMS(output): every layer's
    contribution may be off by TOL_BF16 * RMS(y_l) and the stack output is the sum of the
    contributions, so to first order its error is bounded by the sum of those allowances."""
    return TOL_BF16 * sum(layer_rms(inputs, out)) / float(np.sqrt(np.mean(out ** 2)))


class RawCuda:
    """A raw device address as a byte array (through __cuda_array_interface__)."""

    def __init__(self, ptr: int, nbytes: int):
        self.__cuda_array_interface__ = {"shape": (int(nbytes),), "typestr": "|u1", "data": (int(ptr), False), "version": 2}


def raw_bytes(ptr: int, nbytes: int) -> torch.Tensor:
    """uint8 view of nbytes of device memory at ptr (memory owned by someone else)."""
    return torch.as_tensor(RawCuda(ptr, nbytes), device="cuda")


GUARD_BYTES = 4096
POISON = 0xA5


class Guarded:
    """A device buffer with poisoned margins on both sides: `t` is the interior (what a call is given),
    check() asserts that nothing outside it was written."""

    def __init__(self, shape, dtype, fill=None):
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((nbytes + 2 * GUARD_BYTES,), POISON, dtype=torch.uint8, device="cuda")
        self.nbytes = nbytes
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(*shape)
        if fill is not None:
            self.t.copy_(fill)

    def check(self):
        assert bool((self.raw[:GUARD_BYTES] == POISON).all()) and bool((self.raw[GUARD_BYTES + self.nbytes:] == POISON).all()), \
            "a write outside the buffer"


def poison_workspace(lib, h):
    """Fill the handle's activation workspace with the poison byte; returns what check_workspace needs."""
    ws = lib.mlpmoe_get_workspace(h)
    for name in ("H", "xnorm"):
        raw_bytes(ws[name], ws[name + "_bytes"]).fill_(POISON)
    torch.cuda.synchronize()
    return ws


def check_workspace(lib, h, ws, n, d, elem_size, used_xnorm=True):
    """After an n-token call: H beyond n rows of the current padded width, and the normalised-input
    buffer beyond n rows, still hold the poison."""
    ipad = lib.mlpmoe_get_workspace(h)["n_active_pad"]
    torch.cuda.synchronize()
    tail = raw_bytes(ws["H"], ws["H_bytes"])[n * ipad * elem_size:]
    assert bool((tail == POISON).all()), "a write past the H rows of the call"
    tail = raw_bytes(ws["xnorm"], ws["xnorm_bytes"])[(n * d * elem_size if used_xnorm else 0):]
    assert bool((tail == POISON).all()), "a write past the normalised rows of the call"
