"""GPU: every kernel family of w4a8_linear, launched several times on FRESH zero-filled workspaces and
fresh outputs, must return the same bits every time, and the first launch must be right (checked
against a float32 product of the dequantized operands, which is exact enough to expose a tile that
was summed from stale or missing data).  A repeat on a USED workspace cannot show such an error: a
kernel that reads partial sums too early finds the previous launch's identical values there.  (This
is how a barrier-phase hazard in the expansion groups showed up: wrong sums in a few tiles of the
first launch of a process only.)  Shapes: one per kernel and plan -- split-N with and without a
K cut, the persistent kernel with 64-, 128- and 256-token tiles as equal slices, as whole CTAs per
tile and as whole tiles, the 256 x 256 tiles, the two-CTA kernel, the cluster plan (K cut between two to eight CTAs of a cluster,
with a ragged last tile, with as few as two k-blocks per CTA, with the largest number of clusters
that fits)."""
import numpy as np
import pytest
import torch

from gpu_utils import Guarded
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu

SHAPES = [(8, 4096, 4096), (16, 14336, 4096), (48, 4096, 4096), (128, 6144, 4096), (128, 4096, 14336),
          (17, 2048, 4096), (64, 1024, 1024), (100, 2064, 8192), (33, 4096, 384), (128, 9472, 1024),
          (100, 512, 8192), (200, 4096, 4096), (256, 4096, 14336), (512, 4096, 4096), (512, 6144, 4096),
          (700, 10576, 640), (1061, 16384, 1024), (2048, 4096, 4096)]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_fresh_workspace_launches_agree_and_are_right(M, N, K):
    dev = torch.device("cuda")
    W = torch.from_numpy(inputs.make_weight(N, K, 0.02, seed=M + N)).to(dev)
    codes, gs, gz, sw = binding.quantize_weight_rtn(W, symmetric=True)
    del W
    w8 = binding.dequant_weight(codes, gs, gz)
    tw = binding.prepack_weight(codes, gs, gz, sw)
    xb = inputs.make_activation(M, K, M + K, 0.01, 20.0)
    x8, s_x = binding.quantize_act(torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev))
    ref = (x8.view(torch.float8_e4m3fn).float() @ w8.view(torch.float8_e4m3fn).float().t()) * s_x[:, None] * sw
    outs = []
    for _ in range(4):
        ws = binding.new_workspace(M, N, K, tw.fmt, dev)          # zero-filled, never used
        outs.append(binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32, workspace=ws))
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for o in outs[1:]:
        assert torch.equal(o.view(torch.int32), outs[0].view(torch.int32))
    # float32 sums of K exact products: agreement to ~1e-5 of the output scale; a misplaced or missing
    # k-slice of a tile is off by a good fraction of it
    scale = float(ref.abs().max())
    assert float((outs[0] - ref).abs().max()) <= 1e-3 * scale


def test_one_workspace_shared_by_layers_of_different_shapes_and_kernels():
    # One workspace of the largest size, used by calls of different shapes one after the other -- split-N
    # with and without a K cut, the persistent kernel as equal slices and as whole CTAs per tile, the
    # 256 x 256 tiles: whatever a call leaves behind in the data part of the workspace, the next call's
    # counters must be zero.  Every result must equal the one computed on a fresh workspace of its own.
    dev = torch.device("cuda")
    shapes = [(128, 4096, 14336), (128, 28672, 4096), (128, 4096, 4096), (16, 4096, 14336), (300, 640, 8192),
              (128, 6144, 4096), (512, 4096, 4096), (700, 10576, 640), (8, 4096, 4096), (256, 4096, 14336)]
    cases = []
    for (M, N, K) in shapes:
        W = torch.from_numpy(inputs.make_weight(N, K, 0.02, seed=7 * M + N)).to(dev)
        tw = binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True))
        del W
        xb = inputs.make_activation(M, K, M + 3 * K, 0.01, 20.0)
        x8, s_x = binding.quantize_act(torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev))
        own = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32,
                                   workspace=binding.new_workspace(M, N, K, tw.fmt, dev))
        cases.append((tw, x8, s_x, own))
    need = max(binding.linear_workspace_bytes(M, N, K, weight_format=binding.FMT_TILED_SIGNMAG) for (M, N, K) in shapes)
    shared = torch.zeros((need,), dtype=torch.uint8, device=dev)
    for _ in range(2):
        for tw, x8, s_x, own in cases:
            got = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32, workspace=shared)
            assert torch.equal(got.view(torch.int32), own.view(torch.int32))
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    # the control area is left zero-filled (but for the generation word of the split-N kernel's placement state,
    # in its last kilobyte)
    assert bool((shared[:65536 - 1024] == 0).all())


@pytest.mark.parametrize("M,N,K,pad", [(16, 4096, 14336, 8), (128, 4096, 4096, 8), (100, 512, 8192, 8), (300, 640, 8192, 8),
                                       (700, 10576, 640, 8), (1061, 16384, 1024, 8), (512, 6144, 1024, 8),
                                       (100, 2064, 8192, 2), (37, 4096, 4096, 6), (128, 6144, 4096, 8)])
def test_linear_kernels_write_only_their_outputs_and_their_workspace(M, N, K, pad):
    # poisoned guard bands in front of and behind Y (with padding columns between its rows, which must
    # stay untouched too) and around a workspace of exactly the size the library asks for: no kernel
    # family of w4a8_linear may write a byte outside them
    dev = torch.device("cuda")
    W = torch.from_numpy(inputs.make_weight(N, K, 0.02, seed=M + 2 * N)).to(dev)
    tw = binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True))
    del W
    xb = inputs.make_activation(M, K, 5 * M + K, 0.01, 20.0)
    x8, s_x = binding.quantize_act(torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev))
    need = binding.linear_workspace_bytes(M, N, K, weight_format=tw.fmt)
    gws = Guarded((need,), torch.uint8, fill=0)
    ldy = N + pad   # (a row stride that is no multiple of four elements: the scalar store path of the cluster plan)
    gy = Guarded((M, ldy), torch.bfloat16, fill=7.0)
    ref = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_BF16, workspace=binding.new_workspace(M, N, K, tw.fmt, dev))
    for _ in range(2):
        binding.linear_tiled(x8, s_x, tw, out=gy.t[:, :N], workspace=gws.t)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    gy.check()
    gws.check()
    assert torch.equal(gy.t[:, :N].contiguous().view(torch.int16), ref.view(torch.int16))
    assert bool((gy.t[:, N:] == 7.0).all())


def test_seeded_random_shapes_through_every_route():
    # 72 seeded shapes across the routing rules of w4a8_linear on prepacked weights (token counts around
    # 16 / 64 / 128 / 512, one to many tiles, one to many k-blocks, ragged last tiles), both tiled formats in
    # turn, BF16 and FP32 outputs in turn: every result against the float32 product of the dequantized
    # operands, and a second launch on a fresh workspace bit for bit equal to the first
    rng = np.random.default_rng(20250611)
    dev = torch.device("cuda")
    ms = [1, 7, 16, 17, 31, 64, 65, 100, 128, 129, 300, 513, 700]
    for t in range(72):
        M = int(ms[t % len(ms)]) if t % 3 else int(rng.integers(1, 600))
        N = 16 * int(rng.integers(1, 260))
        K = 128 * int(rng.integers(1, 17 if M > 128 else 40))
        asym = bool(t % 2)
        W = torch.from_numpy(inputs.make_weight(N, K, 0.02, seed=900 + t)).to(dev)
        codes, gs, gz, sw = binding.quantize_weight_rtn(W, symmetric=not asym)
        del W
        w8 = binding.dequant_weight(codes, gs, gz)
        tw = binding.prepack_weight(codes, gs, gz, sw)
        xb = inputs.make_activation(M, K, 1000 + t, 0.01, 20.0)
        x8, s_x = binding.quantize_act(torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev))
        ref = (x8.view(torch.float8_e4m3fn).float() @ w8.view(torch.float8_e4m3fn).float().t()) * s_x[:, None] * sw
        od = binding.OUT_FP32 if t % 4 < 2 else binding.OUT_BF16
        a = binding.linear_tiled(x8, s_x, tw, out_dtype=od, workspace=binding.new_workspace(M, N, K, tw.fmt, dev))
        b = binding.linear_tiled(x8, s_x, tw, out_dtype=od, workspace=binding.new_workspace(M, N, K, tw.fmt, dev))
        torch.cuda.synchronize()
        assert binding.query_device_status() == 0, (M, N, K)
        assert torch.equal(a, b), (M, N, K)
        scale = float(ref.abs().max())
        tol = 1e-3 if od == binding.OUT_FP32 else 6e-3      # (BF16: half a unit in the last place of the largest output)
        assert float((a.float() - ref).abs().max()) <= tol * scale, (M, N, K, asym)


def test_cluster_plan_needs_no_workspace():
    # 17..128 tokens on a layer with few tiles: the call succeeds without any workspace and equals the
    # call with one bit for bit
    dev = torch.device("cuda")
    M, N, K = 48, 528, 1024
    W = torch.from_numpy(inputs.make_weight(N, K, 0.02, seed=77)).to(dev)
    tw = binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True))
    xb = inputs.make_activation(M, K, 78, 0.01, 20.0)
    x8, s_x = binding.quantize_act(torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev))
    with_ws = binding.linear_tiled(x8, s_x, tw, out_dtype=binding.OUT_FP32)
    y = torch.empty((M, N), dtype=torch.float32, device=dev)
    rc = binding.lib().w4a8_linear(x8.data_ptr(), x8.stride(0), s_x.data_ptr(), M, tw.buf.data_ptr(), None, None, tw.fmt,
                                   tw.s_w.data_ptr(), 0 if tw.s_w.numel() == 1 else 1, N, K, 128, y.data_ptr(), y.stride(0),
                                   binding.OUT_FP32, None, 0, torch.cuda.current_stream().cuda_stream)
    assert rc == 0
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert torch.equal(y, with_ws)
