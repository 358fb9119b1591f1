"""Seeded payload generation on the device for workloads too large to draw on the host.

Only random draws; none of the method's arithmetic.  Values do not influence timing or
checks (the cipher is data independent), they only give the buffers the dtype and
distribution the workload names.
"""
from __future__ import annotations

import torch


def fill_bf16_normal(buf_u8: torch.Tensor, seed: int, std: float = 1.0, chunk_elems: int = 1 << 27):
    """Overwrite a uint8 CUDA buffer (even length) with bf16 N(0, std) values, chunk by chunk."""
    assert buf_u8.dtype == torch.uint8 and buf_u8.is_cuda and buf_u8.numel() % 2 == 0
    gen = torch.Generator(device=buf_u8.device)
    gen.manual_seed(seed)
    view = buf_u8.view(torch.bfloat16)
    n = view.numel()
    for lo in range(0, n, chunk_elems):
        hi = min(n, lo + chunk_elems)
        tmp = torch.randn(hi - lo, generator=gen, device=buf_u8.device, dtype=torch.float32)
        view[lo:hi] = (tmp * std).to(torch.bfloat16)
        del tmp
    return buf_u8


def fill_bytes(buf_u8: torch.Tensor, seed: int, chunk: int = 1 << 28):
    """Overwrite a uint8 CUDA buffer with uniform random bytes."""
    gen = torch.Generator(device=buf_u8.device)
    gen.manual_seed(seed)
    n = buf_u8.numel()
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        buf_u8[lo:hi] = torch.randint(0, 256, (hi - lo,), generator=gen, device=buf_u8.device, dtype=torch.uint8)
    return buf_u8
