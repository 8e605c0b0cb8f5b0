"""Torch-side plumbing for the GPU tests: uploads and calls through the C-ABI binding."""
import numpy as np
import torch

from paper_2310_08041_b200 import binding as B
from paper_2310_08041_b200 import synth

DEV = "cuda:0"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def dev_x(x_np):
    """float32 array or uint16 bf16 bit patterns -> device tensor of the right dtype."""
    if x_np.dtype == np.uint16:
        return torch.from_numpy(x_np.view(np.int16)).to(DEV).view(torch.bfloat16)
    return dev(x_np)


def bf16_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


class Guarded:
    """An output tensor placed in the middle of a larger buffer filled with a canary pattern: check() fails when a
    kernel wrote a byte before or behind the tensor it was given."""
    PAD = 4096                                           # bytes on either side (keeps the 16-byte alignment)

    def __init__(self, shape, dtype, fill):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((n + 2 * self.PAD,), 0x5C, dtype=torch.uint8, device=DEV)
        self.n = n
        self.t = self.raw[self.PAD:self.PAD + n].view(dtype).view(*shape)
        self.t.fill_(fill)

    def check(self, what="output"):
        r = self.raw.cpu().numpy()
        before, after = r[:self.PAD], r[self.PAD + self.n:]
        assert (before == 0x5C).all(), f"{what}: {int((before != 0x5C).sum())} bytes written in front of the tensor"
        assert (after == 0x5C).all(), f"{what}: {int((after != 0x5C).sum())} bytes written behind the tensor"


def run_reassemble_quant(x_np, gamma, beta, eps, ptr, src, coef, bits, want_rowsum=True):
    x = dev_x(x_np)
    M, C = x.shape
    row = C // 2 if bits == 4 else C
    g_codes = Guarded((M, row), torch.uint8, 0xAB)
    g_scale = Guarded((M,), torch.float32, -1.0)
    g_zero = Guarded((M,), torch.float32, -1e9)
    g_rowsum = Guarded((M,), torch.int32, -7) if want_rowsum else None
    codes, a_scale, a_zero = g_codes.t, g_scale.t, g_zero.t
    a_rowsum = g_rowsum.t if want_rowsum else None
    B.qllm_reassemble_quant(x, None if gamma is None else dev(gamma), None if beta is None else dev(beta), dev(ptr), dev(src), dev(coef),
                            bits, codes, a_scale, a_zero, a_rowsum, ln_eps=eps)
    torch.cuda.synchronize()
    g_codes.check("codes"); g_scale.check("a_scale"); g_zero.check("a_zero")
    if g_rowsum is not None:
        g_rowsum.check("a_rowsum")
    stored = codes.cpu().numpy()
    return dict(stored=stored, codes=synth.unpack_nibbles(stored) if bits == 4 else stored,
                scale=a_scale.cpu().numpy(), zero=a_zero.cpu().numpy(),
                rowsum=None if a_rowsum is None else a_rowsum.cpu().numpy(),
                dev=dict(codes=codes, a_scale=a_scale, a_zero=a_zero, a_rowsum=a_rowsum))


def store_codes(codes_np, bits):
    return synth.pack_nibbles(codes_np) if bits == 4 else np.ascontiguousarray(codes_np)
