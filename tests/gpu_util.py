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


def run_reassemble_quant(x_np, gamma, beta, eps, ptr, src, coef, bits, want_rowsum=True):
    x = dev_x(x_np)
    M, C = x.shape
    row = C // 2 if bits == 4 else C
    codes = torch.full((M, row), 0xAB, dtype=torch.uint8, device=DEV)
    a_scale = torch.full((M,), -1.0, dtype=torch.float32, device=DEV)
    a_zero = torch.full((M,), -1e9, dtype=torch.float32, device=DEV)
    a_rowsum = torch.full((M,), -7, dtype=torch.int32, device=DEV) if want_rowsum else None
    B.qllm_reassemble_quant(x, None if gamma is None else dev(gamma), None if beta is None else dev(beta), dev(ptr), dev(src), dev(coef),
                            bits, codes, a_scale, a_zero, a_rowsum, ln_eps=eps)
    torch.cuda.synchronize()
    stored = codes.cpu().numpy()
    return dict(stored=stored, codes=synth.unpack_nibbles(stored) if bits == 4 else stored,
                scale=a_scale.cpu().numpy(), zero=a_zero.cpu().numpy(),
                rowsum=None if a_rowsum is None else a_rowsum.cpu().numpy(),
                dev=dict(codes=codes, a_scale=a_scale, a_zero=a_zero, a_rowsum=a_rowsum))


def store_codes(codes_np, bits):
    return synth.pack_nibbles(codes_np) if bits == 4 else np.ascontiguousarray(codes_np)
