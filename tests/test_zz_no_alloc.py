"""The allocation-free entry point, w4a8_linear_static_scratch, against w4a8_linear_ex.

Some callers cannot give the library a workspace: an engine plugin that only receives its input
and output tensors, a serving loop that must not trigger an allocation (which would stall the
device), a process whose memory pool is already fully handed out.  For them the split-K partial
sums live in an array inside the library image.  The array is shared by every call and keeps
whatever the previous call left in it, so the check runs the entry point twice in a row (with
different shapes in between) and compares each result with the ordinary entry point, which uses a
caller-provided workspace.  This file sorts last so that a failure here cannot hide another one.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, dev, weights_to_dev
from helpers import bf16_gate
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _case(M, N, K, seed):
    W = inputs.make_weight(N, K, 0.02, seed)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    xb = inputs.make_activation(M, K, seed, 0.01, 20.0)
    x8, s_x = oracle.quantize_act(xb)
    return x8, s_x, wq


def test_static_scratch_matches_the_workspace_entry_point_twice_in_a_row():
    for call, (M, N, K, split_k) in enumerate([(16, 1024, 2048, 4), (5, 272, 1024, 8), (16, 1024, 2048, 4)]):
        x8, s_x, wq = _case(M, N, K, seed=40 + call)
        xd, sd, wd = dev(x8), dev(s_x), weights_to_dev(*wq)
        for out_dtype in (binding.OUT_FP32, binding.OUT_BF16):
            want = binding.linear(xd, sd, *wd, out_dtype=out_dtype, algo=binding.ALGO_UMMA, split_k=split_k)
            out = torch.full_like(want, 7.0)
            got = binding.linear_static_scratch(xd, sd, *wd, out_dtype=out_dtype, out=out, split_k=split_k)
            torch.cuda.synchronize()
            assert binding.query_device_status() == 0
            # same kernels, same summation order: the two entry points agree bit for bit
            assert torch.equal(got, want), (call, out_dtype)
        ref = oracle.linear(x8, s_x, oracle.dequant_weight(*wq[:3]), wq[3])
        ok, dist = bf16_gate(bf16_bits(got), ref["y64"])
        assert ok, dist


def test_static_scratch_rejects_problems_beyond_its_size_and_bad_arguments():
    L = binding.lib()
    p = ctypes.c_void_p(0x1000)
    f = L.w4a8_linear_static_scratch
    # 16 x 14336 outputs in 8 K slices need 7.3 MB of partial sums: more than the built-in 4 MiB
    assert 8 * 16 * 14336 * 4 > binding.STATIC_SCRATCH_BYTES
    assert f(p, 4096, p, 16, p, p, None, p, 0, 14336, 4096, 128, p, 14336, 0, 8, None) == binding.ERR_WORKSPACE_TOO_SMALL
    assert f(p, 4096, p, 0, p, p, None, p, 0, 14336, 4096, 128, p, 14336, 0, 2, None) == binding.ERR_INVALID_ARG
    assert f(p, 4096, p, 16, p, p, None, p, 0, 14336, 4000, 128, p, 14336, 0, 2, None) == binding.ERR_BAD_SHAPE
    assert f(p, 4096, p, 16, p, p, None, p, 0, 14336, 4096, 128, p, 14336, 0, 5, None) == binding.ERR_BAD_SHAPE
