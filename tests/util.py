"""Helpers shared by the GPU parity tests: host<->device marshalling and the acceptance metrics."""
import numpy as np
import torch

MAX_ERR_FACTOR = 2e-2   # max|out - ref| <= 2e-2 * max|ref|
REL_FRO = 5e-3          # ||out - ref||_F / ||ref||_F <= 5e-3
TOPK_W_ATOL = 1e-6


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev_f16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.float16)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host_bf16_bits(t):
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def host_bf16_f64(t):
    return t.detach().to(torch.float64).cpu().numpy()


def errors(out, ref):
    out = np.asarray(out, np.float64); ref = np.asarray(ref, np.float64)
    mx = float(np.max(np.abs(out - ref))) if out.size else 0.0
    rmax = float(np.max(np.abs(ref))) if ref.size else 0.0
    fro = float(np.linalg.norm(out - ref) / max(np.linalg.norm(ref), 1e-300)) if out.size else 0.0
    return mx, rmax, fro


def assert_close(out, ref, what=""):
    mx, rmax, fro = errors(out, ref)
    assert np.all(np.isfinite(out)), f"{what}: non-finite output"
    assert mx <= MAX_ERR_FACTOR * rmax, f"{what}: max err {mx:.3e} > 2e-2 * {rmax:.3e}"
    assert fro <= REL_FRO, f"{what}: rel Frobenius {fro:.3e} > 5e-3"
    return mx, rmax, fro


SENTINEL16 = 0x7B5A     # a finite bf16 pattern (about 1.1e36) no kernel output takes


class Guarded:
    """A tensor placed inside a larger buffer filled with a sentinel, at a 16-byte-aligned offset with a head and a
    tail of `pad` elements.  `intact()` tells whether a kernel wrote outside the tensor."""

    def __init__(self, shape, dtype, pad=4096, fill_inside=True):
        n = int(np.prod(shape))
        esz = torch.empty((), dtype=dtype).element_size()
        assert (pad * esz) % 16 == 0
        self.pad, self.n = pad, n
        self.bits = {2: torch.int16, 4: torch.int32}[esz]
        self.sent = SENTINEL16 if esz == 2 else 0x7B5A7B5A
        self.buf = torch.full((n + 2 * pad,), self.sent, dtype=self.bits, device="cuda")
        self.t = self.buf[pad:pad + n].view(dtype).view(*shape)
        if not fill_inside:
            self.t.zero_()

    def intact(self):
        head = self.buf[:self.pad]
        tail = self.buf[self.pad + self.n:]
        return bool((head == self.sent).all().item()) and bool((tail == self.sent).all().item())

    def untouched_inside(self):
        """Mask of elements of the tensor itself that still hold the sentinel."""
        return self.buf[self.pad:self.pad + self.n].view(self.t.shape) == self.sent
