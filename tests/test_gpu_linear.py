"""GPU parity: w4a8_linear against the oracle (Sec. 3 flow: Eq. 13 -> Eq. 10 -> FP8 matmul ->
Eq. 4 / Eq. 11).  FP8 operands must be bit-exact (checked in the other GPU tests); the output
gate is max relative error 2e-3 before the BF16 cast and 1 BF16 step after it."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, bf16_dev, dev, weights_to_dev
from helpers import bf16_gate, e4m3_value_table, fp32_gate, pack_codes
from helpers import unpack_codes as helpers_unpack
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu

ALGOS = [binding.ALGO_UMMA, binding.ALGO_SIMT, "tiled"]


def _gpu_linear(x8, s_x, wq, out_dtype, algo=binding.ALGO_AUTO, split_k=0):
    """algo "tiled": prepack (sign-magnitude format when the storage is symmetric, generic tiled
    otherwise) and run the persistent kernel; "tiled_generic" forces the generic tiled format."""
    wd = weights_to_dev(*wq)
    if algo in ("tiled", "tiled_generic"):
        fmt = binding.FMT_TILED if (algo == "tiled_generic" or wq[2] is not None) else binding.FMT_TILED_SIGNMAG
        tw = binding.prepack_weight(*wd, weight_format=fmt)
        y = binding.linear_tiled(dev(x8), dev(s_x), tw, out_dtype=out_dtype)
    else:
        y = binding.linear(dev(x8), dev(s_x), *wd, out_dtype=out_dtype, algo=algo, split_k=split_k)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    return y


def _check(x8, s_x, wq, algo=binding.ALGO_AUTO, split_k=0, cols=None):
    codes, gs, gz, s_w = wq
    w8 = oracle.dequant_weight(codes, gs, gz)
    ref = oracle.linear(x8, s_x, w8, s_w, cols=cols)
    y32 = _gpu_linear(x8, s_x, wq, binding.OUT_FP32, algo, split_k).cpu().numpy()
    ybf = bf16_bits(_gpu_linear(x8, s_x, wq, binding.OUT_BF16, algo, split_k))
    if cols is not None:
        y32, ybf = y32[:, cols], ybf[:, cols]
    worst, _ = fp32_gate(y32, ref["y64"], rel=2e-3)
    assert worst <= 2e-3, worst
    ok, dist = bf16_gate(ybf, ref["y64"])
    assert ok, dist
    return worst


def _gaussian_case(M, N, K, seed, asym=False, per_channel=False, frac=0.01, mult=20.0, sigma=0.02):
    W = inputs.make_weight(N, K, sigma, seed)
    wq = oracle.quantize_weight_rtn(W, symmetric=not asym, per_channel=per_channel)
    xb = inputs.make_activation(M, K, seed, frac, mult)
    x8, s_x = oracle.quantize_act(xb)
    return x8, s_x, wq


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("M,N,K", [(1, 16, 128), (3, 16, 256), (16, 128, 512), (5, 144, 384),
                                   (17, 256, 1024), (40, 272, 640), (100, 128, 256), (130, 384, 512),
                                   (300, 512, 1024)])
def test_exact_integer_inputs_are_bit_exact(algo, M, N, K):
    # group scales 1 and small-integer operands: every partial sum fits in 24 bits, so fp32
    # accumulation in any order is exact and the result must equal the oracle bit for bit.
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    tab = e4m3_value_table()
    ints = {int(v): c for c, v in enumerate(tab) if np.isfinite(v) and v == int(v) and abs(v) <= 6}
    xv = rng.integers(-6, 7, size=(M, K))
    x8 = np.vectorize(lambda v: ints[int(v)])(xv).astype(np.uint8)
    s_x = np.ones(M, dtype=np.float32)
    u = rng.integers(1, 16, size=(N, K)).astype(np.uint8)
    codes = pack_codes(u)
    gs = inputs.f32_to_bf16_bits(np.ones((N, K // 128), dtype=np.float32))
    gz = rng.integers(4, 12, size=(N, K // 128)).astype(np.uint8)
    s_w = np.ones(1, dtype=np.float32)
    for wq in ((codes, gs, gz, s_w), (codes, gs, None, s_w)):
        ref = oracle.linear(x8, s_x, oracle.dequant_weight(*wq[:3]), s_w)
        y = _gpu_linear(x8, s_x, wq, binding.OUT_FP32, algo).cpu().numpy()
        assert np.array_equal(y, ref["y32"])
        assert np.array_equal(y.astype(np.float64), ref["y64"])
        if algo == "tiled" and wq[2] is None:
            y = _gpu_linear(x8, s_x, wq, binding.OUT_FP32, "tiled_generic").cpu().numpy()
            assert np.array_equal(y, ref["y32"])


@pytest.mark.parametrize("M,N,K,asym,pc", [(16, 1024, 1024, False, False),      # config c1
                                           (1, 256, 4096, True, True),
                                           (4, 1040, 2048, False, True),
                                           (33, 640, 1536, True, False),
                                           (128, 512, 2048, False, False),
                                           (200, 400, 1024, True, True),
                                           (515, 272, 1152, False, False)])
def test_gaussian_inputs_within_gates(M, N, K, asym, pc):
    x8, s_x, wq = _gaussian_case(M, N, K, seed=M + N + K, asym=asym, per_channel=pc)
    _check(x8, s_x, wq)
    _check(x8, s_x, wq, algo="tiled")
    if not asym:
        _check(x8, s_x, wq, algo="tiled_generic")


@pytest.mark.parametrize("M,N,K", [(16, 128, 128), (1, 16, 14336), (16, 4096, 4096), (8, 6144, 4096),
                                   (32, 4096, 14336), (64, 1024, 2048), (128, 2048, 1024), (512, 1024, 1024),
                                   (300, 640, 8192), (100, 512, 8192), (65, 4096, 4096), (128, 14336, 1024)])
def test_persistent_kernel_split_tiles_and_reuse_of_workspace(M, N, K):
    # shapes whose tiles are split between CTAs in many ways (equal slices in the persistent kernel, K
    # chunks in the split-N kernel with 16-token tiles, clusters of two to eight CTAs per tile); the workspace is shared by
    # consecutive calls (the kernel leaves its counters zeroed) and results repeat bit for bit
    x8, s_x, wq = _gaussian_case(M, N, K, seed=M * 3 + N + K)
    w8 = oracle.dequant_weight(*wq[:3])
    rng = np.random.default_rng(M + N)
    cols = np.unique(np.concatenate([rng.choice(N, min(N, 64), replace=False), [0, N - 1]]))
    ref = oracle.linear(x8, s_x, w8, wq[3], cols=cols)
    tw = binding.prepack_weight(*weights_to_dev(*wq))
    ws = binding.new_workspace(M, N, K, tw.fmt)
    xd, sd = dev(x8), dev(s_x)
    outs = []
    for _ in range(3):
        outs.append(binding.linear_tiled(xd, sd, tw, out_dtype=binding.OUT_FP32, workspace=ws).clone())
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])
    worst, _ = fp32_gate(outs[0].cpu().numpy()[:, cols], ref["y64"])
    assert worst <= 2e-3, worst
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    if 16 < M <= 128 and ((N + 127) // 128) * 2 <= sms and K >= 512:
        # 17..128 tokens on a layer with few tiles: K is cut inside thread-block clusters, which exchange
        # their partial sums through shared memory -- the workspace is not touched at all
        assert not bool(ws.any())
    else:
        persistent = M > 128
        n_counter_bytes = 8 * ((M + 255) // 256) * ((N + 127) // 128) if persistent else 1024
        # tile counters (persistent kernel: start of the 64 KB control area; split-N: its last 2 KB) are back to zero
        first = 0 if persistent else 65536 - 2048
        assert np.all(ws[first:first + n_counter_bytes].cpu().numpy() == 0)


def test_sign_magnitude_prepack_flags_code_zero():
    codes, gs, _ = inputs.random_codes(128, 256, seed=1)          # random nibbles include code 0
    cd, gd = dev(codes), bf16_dev(gs)
    binding.prepack_weight(cd, gd, None, None, weight_format=binding.FMT_TILED_SIGNMAG)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 2
    assert binding.query_device_status() == 0                     # reading clears it
    binding.prepack_weight(cd, gd, None, None, weight_format=binding.FMT_TILED)
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0


def test_tiled_formats_see_the_same_fp8_weights_as_eq10():
    # one-hot FP8 activations (value 1.0, s_x = 1) read the dequantized weights back through the
    # GEMM: Y[m][n] = w8[n][k_m] exactly, for every code, zero-point and a spread of scales
    N, K = 256, 512
    codes, gs, gz = inputs.random_codes(N, K, seed=21, asymmetric=True)
    M = 64
    ks = (np.arange(M) * 37) % K
    x8 = np.zeros((M, K), dtype=np.uint8)
    x8[np.arange(M), ks] = 0x38                                    # 1.0
    s_x = np.ones(M, dtype=np.float32)
    s_w = np.ones(1, dtype=np.float32)
    tab = e4m3_value_table()
    w8 = oracle.dequant_weight(codes, gs, gz)
    y = _gpu_linear(x8, s_x, (codes, gs, gz, s_w), binding.OUT_FP32, "tiled").cpu().numpy()
    assert np.array_equal(y.astype(np.float64), tab[w8][:, ks].T)
    sym_u = np.clip(helpers_unpack(codes), 1, 15)
    codes_s = pack_codes(sym_u.astype(np.uint8))
    w8s = oracle.dequant_weight(codes_s, gs, None)
    for algo in ("tiled", "tiled_generic"):
        y = _gpu_linear(x8, s_x, (codes_s, gs, None, s_w), binding.OUT_FP32, algo).cpu().numpy()
        assert np.array_equal(y.astype(np.float64), tab[w8s][:, ks].T), algo


@pytest.mark.parametrize("split_k", [1, 2, 4, 8])
def test_split_k_variants(split_k):
    x8, s_x, wq = _gaussian_case(16, 512, 2048, seed=77)
    _check(x8, s_x, wq, algo=binding.ALGO_UMMA, split_k=split_k)
    # deterministic: two runs give identical bits
    a = _gpu_linear(x8, s_x, wq, binding.OUT_FP32, binding.ALGO_UMMA, split_k).cpu().numpy()
    b = _gpu_linear(x8, s_x, wq, binding.OUT_FP32, binding.ALGO_UMMA, split_k).cpu().numpy()
    assert np.array_equal(a, b)


def test_simt_and_umma_agree_closely():
    x8, s_x, wq = _gaussian_case(48, 384, 1024, seed=5, asym=True)
    a = _gpu_linear(x8, s_x, wq, binding.OUT_FP32, binding.ALGO_UMMA).cpu().numpy()
    b = _gpu_linear(x8, s_x, wq, binding.OUT_FP32, binding.ALGO_SIMT).cpu().numpy()
    assert np.allclose(a, b, rtol=1e-4, atol=1e-5 * np.abs(b).max())


def test_outputs_outside_the_problem_are_untouched():
    # ragged M and N: guard bands around Y must keep their poison
    M, N, K = 19, 144, 256
    x8, s_x, wq = _gaussian_case(M, N, K, seed=8)
    ldy = N + 16
    buf = torch.full((M + 2, ldy), 7.0, dtype=torch.bfloat16, device="cuda")
    out = buf[1:M + 1, :N]
    binding.linear(dev(x8), dev(s_x), *weights_to_dev(*wq), out=out)
    torch.cuda.synchronize()
    full = buf.float().cpu().numpy()
    assert np.all(full[0] == 7.0) and np.all(full[-1] == 7.0) and np.all(full[:, N:] == 7.0)
    ref = oracle.linear(x8, s_x, oracle.dequant_weight(*wq[:3]), wq[3])
    ok, dist = bf16_gate(bf16_bits(out), ref["y64"])
    assert ok, dist


@pytest.mark.parametrize("M", [1, 4, 16])
def test_config_c2_decode_full(M):
    K, N = 4096, 14336
    x8, s_x, wq = _gaussian_case(M, N, K, seed=2)
    _check(x8, s_x, wq)
    _check(x8, s_x, wq, algo="tiled")


def test_config_c3_prefill_sampled_columns():
    M, K, N = 2048, 4096, 4096
    x8, s_x, wq = _gaussian_case(M, N, K, seed=3)
    rng = np.random.default_rng(3)
    cols = np.unique(np.concatenate([rng.choice(N, 96, replace=False),
                                     np.array([0, 127, 128, 255, 256, 2047, 2048, N - 129, N - 128, N - 1])]))
    _check(x8, s_x, wq, cols=cols)
    _check(x8, s_x, wq, algo="tiled", cols=cols)


def test_whole_path_from_bf16_activations():
    # act quant and linear chained on the device, against the oracle's whole forward
    M, K, N = 24, 1024, 512
    W = inputs.make_weight(N, K, 0.02, 12)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    xb = inputs.make_activation(M, K, 12, 0.01, 20.0)
    x8, s_x = binding.quantize_act(bf16_dev(xb))
    y = binding.linear(x8, s_x, *weights_to_dev(*wq), out_dtype=binding.OUT_BF16)
    torch.cuda.synchronize()
    ref = oracle.forward(xb, *wq)
    assert np.array_equal(x8.cpu().numpy(), ref["x8"])
    ok, dist = bf16_gate(bf16_bits(y), ref["y64"])
    assert ok, dist


def test_host_forward_entry_point():
    M, K, N = 16, 1024, 1024
    W = inputs.make_weight(N, K, 0.02, 13)
    wq = oracle.quantize_weight_rtn(W, symmetric=True)
    xb = inputs.make_activation(M, K, 13, 0.01, 20.0)
    ref = oracle.forward(xb, *wq)
    x_host = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()
    wd = weights_to_dev(*wq)
    # pinned input: the kernels read and write the host buffers themselves; pageable input: copies
    x_pageable = torch.from_numpy(xb.view(np.int16).copy()).view(torch.bfloat16)
    assert not x_pageable.is_pinned()
    for weight in (wd, binding.prepack_weight(*wd)):
        for xh in (x_host, x_pageable):
            fwd = binding.HostForward(M, weight)
            fwd.y_host.fill_(7.0)
            y_host = fwd(xh)
            torch.cuda.synchronize()
            assert binding.query_device_status() == 0
            ok, dist = bf16_gate(bf16_bits(y_host), ref["y64"])
            assert ok, dist
            assert np.array_equal(fwd.x8.cpu().numpy(), ref["x8"])                       # Eq. 13, bit for bit
            assert np.array_equal(fwd.s_x.cpu().numpy().view(np.uint32), ref["s_x"].view(np.uint32))
            assert fwd.h2d_bytes == M * K * 2 and fwd.d2h_bytes == M * N * 2
            if xh is x_host:
                # later calls with the same buffers must see what the buffers hold NOW (new
                # activations in the same pinned buffer)
                xb2 = inputs.make_activation(M, K, 99, 0.01, 20.0)
                ref2 = oracle.forward(xb2, *wq)
                keep = x_host.clone()
                for _ in range(3):
                    x_host.copy_(torch.from_numpy(xb2.view(np.int16)).view(torch.bfloat16))
                    fwd.y_host.fill_(7.0)
                    y2 = fwd(x_host)
                    torch.cuda.synchronize()
                    ok, dist = bf16_gate(bf16_bits(y2), ref2["y64"])
                    assert ok, dist
                    assert np.array_equal(fwd.x8.cpu().numpy(), ref2["x8"])
                x_host.copy_(keep)


def test_host_forward_many_tokens_takes_the_copy_path():
    M, K, N = 200, 512, 256
    wq = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 14), symmetric=True)
    xb = inputs.make_activation(M, K, 15)
    ref = oracle.forward(xb, *wq)
    x_host = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).pin_memory()
    fwd = binding.HostForward(M, binding.prepack_weight(*weights_to_dev(*wq)))
    y_host = fwd(x_host)
    torch.cuda.synchronize()
    ok, dist = bf16_gate(bf16_bits(y_host), ref["y64"])
    assert ok, dist
