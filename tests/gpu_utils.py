"""Helpers for the GPU parity tests: numpy <-> device tensors, BF16 bit views."""
import numpy as np
import torch


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


def bf16_dev(bits_u16):
    """uint16 BF16 bit patterns -> torch.bfloat16 tensor on the device."""
    return torch.from_numpy(np.ascontiguousarray(bits_u16).view(np.int16)).view(torch.bfloat16).cuda()


def bf16_bits(t):
    """torch.bfloat16 tensor -> numpy uint16 bit patterns."""
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def weights_to_dev(codes, gscale, gzero, s_w):
    return (dev(codes), bf16_dev(gscale), None if gzero is None else dev(gzero), dev(s_w))
