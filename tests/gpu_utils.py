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


def hessian_upper_cholesky_dev(H, perm=None, damp=0.01):
    """The factor U that w4a8_dpq_quantize takes as an INPUT (Sec. 3.3, as in GPTQ), computed with
    torch.linalg in float64 on the device: permute H to processing order, give dead columns a unit
    diagonal, add damp * mean(diag), invert, return the upper Cholesky factor of the inverse as
    float32.  The library has no entry point for this step: U is the caller's."""
    H = H.to(torch.float64)
    if perm is not None:
        idx = perm.to(torch.int64)
        H = H[idx][:, idx]
    H = H.clone()
    d = torch.diagonal(H)
    d[d == 0] = 1.0
    d += damp * d.mean()
    Hinv = torch.cholesky_inverse(torch.linalg.cholesky(H))
    Hinv = 0.5 * (Hinv + Hinv.T)
    return torch.linalg.cholesky(Hinv, upper=True).to(torch.float32).contiguous()


class Guarded:
    """A device buffer with poisoned guard bands in front of and behind it: `t` is the usable part
    (a view of `shape` / `dtype`, 256-byte aligned), check() asserts that the bands still hold the
    poison -- a kernel that wrote outside the buffer it was given has changed them."""
    BAND = 4096
    POISON = 0xA5

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.nbytes = n
        self.raw = torch.full((n + 2 * self.BAND,), self.POISON, dtype=torch.uint8, device="cuda")
        assert self.raw.data_ptr() % 256 == 0
        self.t = self.raw[self.BAND:self.BAND + n].view(dtype).view(shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self):
        torch.cuda.synchronize()
        front = self.raw[:self.BAND]
        back = self.raw[self.BAND + self.nbytes:]
        assert bool((front == self.POISON).all()), "bytes in front of the buffer were overwritten"
        assert bool((back == self.POISON).all()), "bytes behind the buffer were overwritten"
