"""GPU parity: w4a8_linear_chain (a chain of decode-sized layers in one persistent launch) against
the oracle's forward pass (Sec. 3 flow: Eq. 13 -> Eq. 10 -> FP8 matmul -> Eq. 4 / Eq. 11).  The FP8
activations and scales the chain used are read back and must be bit-exact; the output gate is max
relative error 2e-3 before the BF16 cast and one BF16 step after it.  Where the chain does not cut K
(whole 96-row blocks per CTA) its outputs must also equal those of the per-launch path
(w4a8_quantize_act + w4a8_linear) bit for bit: same operands, same accumulation order."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from gpu_utils import Guarded, bf16_bits, bf16_dev, dev, weights_to_dev
from helpers import bf16_gate, fp32_gate
from paper_2505_14638_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _weights(N, K, seed, asym=False, sigma=0.02):
    W = inputs.make_weight(N, K, sigma, seed)
    wq = oracle.quantize_weight_rtn(W, symmetric=not asym, per_channel=asym)
    fmt = binding.FMT_TILED if asym else binding.FMT_TILED_SIGNMAG
    tw = binding.prepack_weight(*weights_to_dev(*wq), weight_format=fmt)
    return wq, tw


def _oracle_layer(xb, wq, pow2=False):
    x8, s_x = oracle.quantize_act(xb, scale_mode=1 if pow2 else 0)
    ref = oracle.linear(x8, s_x, oracle.dequant_weight(*wq[:3]), wq[3])
    return x8, s_x, ref


def _per_launch(x, tw, out_dtype):
    """The two-kernel path on the same weights, K never cut (a workspace too small for partial sums)."""
    tiny = torch.zeros((16,), dtype=torch.uint8, device="cuda")
    x8, s_x = binding.quantize_act(x)
    return binding.linear_tiled(x8, s_x, tw, out_dtype=out_dtype, workspace=tiny)


@pytest.mark.parametrize("groups", [0, 2, 4])
@pytest.mark.parametrize("asym", [False, True])
def test_independent_problems_match_oracle_and_per_launch_path(groups, asym):
    # problems of different token counts and shapes in one launch (all with fewer 96-row blocks than
    # SMs, so every block is cut along K and summed by the CTA that arrives last): a short last
    # block, an odd number of k-blocks, fewer items than CTAs, M <= 8 and M > 8
    shapes = [(1, 2368, 640), (4, 4736, 384), (16, 1024, 1024), (7, 48, 256), (9, 16, 128)]
    probs, refs = [], []
    for i, (M, N, K) in enumerate(shapes):
        wq, tw = _weights(N, K, 50 + i, asym)
        xb = inputs.make_activation(M, K, 60 + i, 0.01, 20.0)
        x = bf16_dev(xb)
        y = torch.full((M, N), 7.0, dtype=torch.float32, device="cuda")
        x8o = torch.full((M, K), 0xAA, dtype=torch.uint8, device="cuda")
        sxo = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
        probs.append(dict(x=x, weight=tw, y=y, x8_out=x8o, s_x_out=sxo))
        refs.append((xb, wq))
    chain = binding.LinearChain(probs, groups=groups)
    chain()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for d, (xb, wq) in zip(probs, refs):
        x8, s_x, ref = _oracle_layer(xb, wq)
        assert np.array_equal(d["s_x_out"].cpu().numpy().view(np.uint32), s_x.astype(np.float32).view(np.uint32))
        assert np.array_equal(d["x8_out"].cpu().numpy(), x8)
        worst, _ = fp32_gate(d["y"].cpu().numpy(), ref["y64"], rel=2e-3)
        assert worst <= 2e-3, worst


def test_exact_integer_problem_is_bit_exact():
    # group scales 1, small integer activations: every partial sum is an exact integer below 2^24,
    # so any accumulation order gives the oracle's value bit for bit -- a layout test of the
    # activation tiles (token row, swizzled 16-byte chunks) and of the row ranges
    rng = np.random.default_rng(3)
    M, N, K = 13, 2368, 512
    codes_u = rng.integers(1, 16, size=(N, K), dtype=np.int32)
    from helpers import pack_codes
    codes = pack_codes(codes_u)
    gscale = np.full((N, K // 128), 0x3F80, dtype=np.uint16)     # BF16 1.0
    s_w = np.ones((1,), dtype=np.float32)
    tw = binding.prepack_weight(dev(codes), bf16_dev(gscale), None, dev(s_w), weight_format=binding.FMT_TILED_SIGNMAG)
    xi = rng.integers(-3, 4, size=(M, K)).astype(np.float32)
    xi[:, 5] = 4.0                                               # every row's absmax is 4: s_x = 4 / 448 exactly
    xb = (xi.view(np.uint32) >> 16).astype(np.uint16)
    x8, s_x = oracle.quantize_act(xb)
    ref = oracle.linear(x8, s_x, oracle.dequant_weight(codes, gscale, None), s_w)
    y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    chain = binding.LinearChain([dict(x=bf16_dev(xb), weight=tw, y=y)])
    chain()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert np.array_equal(y.cpu().numpy(), ref["y32"])


def test_whole_blocks_match_the_per_launch_path_bit_for_bit():
    # N = (number of SMs) x 96 x rounds: every CTA owns whole blocks and walks all of K, one block
    # (rounds = 1), two at a time (2) or two and one (3); plus a short remainder cut along K
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for rounds, extra, M, K in ((1, 0, 16, 384), (2, 0, 5, 256), (3, 128, 9, 128)):
        N = sms * 96 * rounds + extra
        wq, tw = _weights(N, K, 100 + rounds)
        xb = inputs.make_activation(M, K, 110 + rounds, 0.01, 20.0)
        x = bf16_dev(xb)
        y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        binding.LinearChain([dict(x=x, weight=tw, y=y)])()
        want = _per_launch(x, tw, binding.OUT_FP32)
        torch.cuda.synchronize()
        assert binding.query_device_status() == 0
        whole = sms * 96 * rounds
        assert torch.equal(y[:, :whole], want[:, :whole]), rounds
        _, _, ref = _oracle_layer(xb, wq)
        worst, _ = fp32_gate(y.cpu().numpy(), ref["y64"], rel=2e-3)
        assert worst <= 2e-3, (rounds, worst)


def test_dependent_chain_and_gated_block():
    # x -> gate_up (BF16) -> silu(gate) * up quantized in the chain -> down (BF16) -> next layer on
    # the down projection's output: every hand-over goes through the chain's counters.  Each stage is
    # checked against the oracle on the input that stage saw (the chain's own previous output).
    M, H, F = 5, 1024, 1408
    wq_gu, tw_gu = _weights(2 * F, H, 70)
    wq_dn, tw_dn = _weights(H, F, 71)
    wq_nx, tw_nx = _weights(2304, H, 72)
    xb = inputs.make_activation(M, H, 73, 0.01, 20.0)
    x = bf16_dev(xb)
    gu = torch.zeros((M, 2 * F), dtype=torch.bfloat16, device="cuda")
    dn = torch.zeros((M, H), dtype=torch.bfloat16, device="cuda")
    nx = torch.zeros((M, 2304), dtype=torch.float32, device="cuda")
    x8_dn = torch.zeros((M, F), dtype=torch.uint8, device="cuda")
    sx_dn = torch.zeros((M,), dtype=torch.float32, device="cuda")
    x8_nx = torch.zeros((M, H), dtype=torch.uint8, device="cuda")
    sx_nx = torch.zeros((M,), dtype=torch.float32, device="cuda")
    chain = binding.LinearChain([
        dict(x=x, weight=tw_gu, y=gu),
        dict(x=gu, weight=tw_dn, y=dn, kind=binding.CHAIN_INPUT_SILU_MUL, depends_on=0, x8_out=x8_dn, s_x_out=sx_dn),
        dict(x=dn, weight=tw_nx, y=nx, depends_on=1, x8_out=x8_nx, s_x_out=sx_nx),
    ])
    chain()
    torch.cuda.synchronize()
    first = [t.clone() for t in (gu, dn, nx, x8_dn, sx_dn)]
    for _ in range(3):     # repeated launches: the counters reset themselves, the results repeat
        gu.zero_(); dn.zero_(); nx.zero_()
        chain()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for a, b in zip(first, (gu, dn, nx, x8_dn, sx_dn)):
        assert torch.equal(a, b)
    # layer 1 against the oracle
    _, _, ref = _oracle_layer(xb, wq_gu)
    ok, dist = bf16_gate(bf16_bits(gu), ref["y64"])
    assert ok, dist
    # the gated activation + quantization: the same arithmetic as w4a8_silu_mul_quantize on the same input
    h8, s_h = binding.silu_mul_quantize(gu)
    torch.cuda.synchronize()
    assert torch.equal(x8_dn, h8) and torch.equal(sx_dn, s_h)
    # layer 2 on the FP8 activations it used
    ref2 = oracle.linear(x8_dn.cpu().numpy(), sx_dn.cpu().numpy(), oracle.dequant_weight(*wq_dn[:3]), wq_dn[3])
    ok, dist = bf16_gate(bf16_bits(dn), ref2["y64"])
    assert ok, dist
    # layer 3: Eq. 13 of the chain's own BF16 output, bit-exact, then the product
    d8, s_d = oracle.quantize_act(bf16_bits(dn))
    assert np.array_equal(x8_nx.cpu().numpy(), d8)
    assert np.array_equal(sx_nx.cpu().numpy().view(np.uint32), s_d.astype(np.float32).view(np.uint32))
    ref3 = oracle.linear(d8, s_d, oracle.dequant_weight(*wq_nx[:3]), wq_nx[3])
    worst, _ = fp32_gate(nx.cpu().numpy(), ref3["y64"], rel=2e-3)
    assert worst <= 2e-3, worst


def test_two_row_blocks_per_cta_and_graph_replay():
    # N = 28672: two whole 96-row blocks per CTA plus a remainder cut along K; replayed from a CUDA graph many times
    M, N, K = 3, 28672, 256
    wq, tw = _weights(N, K, 80)
    xb = inputs.make_activation(M, K, 81)
    x = bf16_dev(xb)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    y2 = torch.zeros((16, 1024), dtype=torch.bfloat16, device="cuda")
    wq2, tw2 = _weights(1024, K, 82)
    xb2 = inputs.make_activation(16, K, 83)
    chain = binding.LinearChain([dict(x=x, weight=tw, y=y), dict(x=bf16_dev(xb2), weight=tw2, y=y2)])
    chain()
    torch.cuda.synchronize()
    first = (y.clone(), y2.clone())
    _, _, ref = _oracle_layer(xb, wq)
    ok, dist = bf16_gate(bf16_bits(y), ref["y64"])
    assert ok, dist
    _, _, ref2 = _oracle_layer(xb2, wq2)
    ok, dist = bf16_gate(bf16_bits(y2), ref2["y64"])
    assert ok, dist
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(4):
                chain()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(10):
        y.zero_(); y2.zero_()
        g.replay()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    assert torch.equal(y, first[0]) and torch.equal(y2, first[1])


def test_pow2_and_static_scales():
    M, N, K = 6, 512, 512
    wq, tw = _weights(N, K, 90)
    xb = inputs.make_activation(M, K, 91, 0.01, 20.0)
    x = bf16_dev(xb)
    ss = dev(np.array([0.05], dtype=np.float32))
    outs = [torch.zeros((M, N), dtype=torch.float32, device="cuda") for _ in range(2)]
    x8s = [torch.zeros((M, K), dtype=torch.uint8, device="cuda") for _ in range(2)]
    sxs = [torch.zeros((M,), dtype=torch.float32, device="cuda") for _ in range(2)]
    chain = binding.LinearChain([
        dict(x=x, weight=tw, y=outs[0], scale_mode=binding.SCALE_POW2, x8_out=x8s[0], s_x_out=sxs[0]),
        dict(x=x, weight=tw, y=outs[1], static_scale=ss, x8_out=x8s[1], s_x_out=sxs[1]),
    ])
    chain()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for k, kw in enumerate((dict(scale_mode=1), dict(static_scale=0.05))):
        x8, s_x = oracle.quantize_act(xb, **kw)
        assert np.array_equal(x8s[k].cpu().numpy(), x8)
        assert np.array_equal(sxs[k].cpu().numpy().view(np.uint32), s_x.astype(np.float32).view(np.uint32))
        ref = oracle.linear(x8, s_x, oracle.dequant_weight(*wq[:3]), wq[3])
        worst, _ = fp32_gate(outs[k].cpu().numpy(), ref["y64"], rel=2e-3)
        assert worst <= 2e-3, worst


def test_chain_writes_only_its_outputs_and_its_workspace():
    # poisoned guard bands around every buffer the chain writes: Y (with padding columns between the
    # rows: ldy > N), the optional copies of the FP8 activations and scales, and a workspace of
    # exactly the size the library asks for; shapes with whole blocks, a K-cut remainder and a short
    # last block
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    shapes = [(16, sms * 96 + 176, 384), (3, 2000, 640), (8, 48, 128)]
    probs, guards, pads = [], [], []
    for i, (M, N, K) in enumerate(shapes):
        wq, tw = _weights(N, K, 120 + i)
        x = bf16_dev(inputs.make_activation(M, K, 130 + i, 0.01, 20.0))
        ldy = N + 24
        gy = Guarded((M, ldy), torch.bfloat16, fill=7.0)
        g8 = Guarded((M, K), torch.uint8)
        gs = Guarded((M,), torch.float32)
        guards += [gy, g8, gs]
        pads.append(gy)
        probs.append(dict(x=x, weight=tw, y=gy.t[:, :N], x8_out=g8.t, s_x_out=gs.t))
    probe = binding.LinearChain(probs)
    gw = Guarded((probe.need,), torch.uint8, fill=0)
    chain = binding.LinearChain(probs, workspace=gw.t)
    for _ in range(3):
        chain()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for g in guards + [gw]:
        g.check()
    for gy, (M, N, K) in zip(pads, shapes):
        assert bool((gy.t[:, N:] == 7.0).all()), "padding columns of Y were written"
        assert not bool((gy.t[:, :N] == 7.0).all())
    # the counters are left zero for the next launch
    assert int(gw.t[:1024].view(torch.int32).abs().sum().item()) == 0


def test_chain_argument_errors():
    M, N, K = 4, 256, 256
    wq, tw = _weights(N, K, 95)
    x = bf16_dev(inputs.make_activation(M, K, 96))
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    good = binding.LinearChain([dict(x=x, weight=tw, y=y)])
    L = binding.lib()
    arr = good.arr
    ws = ctypes.c_void_p(good.ws.data_ptr())
    assert L.w4a8_linear_chain(arr, 0, ws, good.need, 0, None) == binding.ERR_INVALID_ARG
    assert L.w4a8_linear_chain(arr, 25, ws, good.need, 0, None) == binding.ERR_INVALID_ARG
    assert L.w4a8_linear_chain(arr, 1, ws, good.need - 1, 0, None) == binding.ERR_WORKSPACE_TOO_SMALL
    assert L.w4a8_linear_chain(arr, 1, ws, good.need, 7, None) == binding.ERR_INVALID_ARG
    arr[0].depends_on = 0
    assert L.w4a8_linear_chain(arr, 1, ws, good.need, 0, None) == binding.ERR_INVALID_ARG
    arr[0].depends_on = -1
    arr[0].M = 17
    assert L.w4a8_linear_chain(arr, 1, ws, good.need, 0, None) == binding.ERR_BAD_SHAPE
    arr[0].M = M
    arr[0].ldx = K - 8
    assert L.w4a8_linear_chain(arr, 1, ws, good.need, 0, None) == binding.ERR_BAD_SHAPE
    arr[0].ldx = K
    assert L.w4a8_linear_chain(arr, 1, ctypes.c_void_p(good.ws.data_ptr() + 16), good.need, 0, None) == \
        binding.ERR_BAD_ALIGNMENT
    good()     # still launches after the rejected calls
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0


def test_a_dependent_problem_may_not_read_an_fp32_output():
    M, N, K = 4, 256, 256
    wq, tw = _weights(N, K, 95)
    wq2, tw2 = _weights(128, N, 96)
    x = bf16_dev(inputs.make_activation(M, K, 97))
    y32 = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    y2 = torch.zeros((M, 128), dtype=torch.float32, device="cuda")
    probs = [dict(x=x, weight=tw, y=y32), dict(x=y32.view(torch.bfloat16)[:, :N], weight=tw2, y=y2, depends_on=0)]
    with pytest.raises(binding.W4A8Error):
        binding.LinearChain(probs)()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_library_carries_on():
    # one CTA waits, with a limit of one millisecond, on a barrier nobody arrives on: the kernel
    # returns by itself, the status word carries the time-out bit, the query reports and clears it,
    # and the next ordinary call is correct
    took = binding.selftest_bounded_wait(1_000_000)
    assert 1_000_000 <= took < 50_000_000, took
    flags = ctypes.c_uint(0)
    assert binding.lib().w4a8_query_device_status(ctypes.byref(flags)) == binding.ERR_TIMEOUT
    assert flags.value & 1
    assert binding.query_device_status() == 0      # cleared by the query
    M, N, K = 4, 512, 256
    wq, tw = _weights(N, K, 97)
    xb = inputs.make_activation(M, K, 98)
    y = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    binding.LinearChain([dict(x=bf16_dev(xb), weight=tw, y=y)])()
    torch.cuda.synchronize()
    _, _, ref = _oracle_layer(xb, wq)
    worst, _ = fp32_gate(y.cpu().numpy(), ref["y64"], rel=2e-3)
    assert worst <= 2e-3 and binding.query_device_status() == 0


@pytest.mark.parametrize("dtype,pad", [(torch.bfloat16, 3), (torch.float32, 1), (torch.bfloat16, 24)])
def test_output_rows_that_are_not_16_byte_aligned(dtype, pad):
    # Y as a view of a wider buffer: with an odd row pitch the kernel cannot store 16-byte pieces and
    # takes its two-byte path; the values must be those of a contiguous output bit for bit, and the
    # padding columns must stay untouched.  Whole blocks (N > 96 * SMs is not needed: the path is
    # the same for blocks cut along K) and a short last block.
    probs, wide = [], []
    for i, (M, N, K) in enumerate([(5, 208, 256), (16, 1040, 384), (1, 96, 128)]):
        wq, tw = _weights(N, K, 300 + i)
        x = bf16_dev(inputs.make_activation(M, K, 310 + i, 0.01, 20.0))
        buf = torch.full((M, N + pad), 7.0, dtype=dtype, device="cuda")
        yc = torch.zeros((M, N), dtype=dtype, device="cuda")
        probs.append(dict(x=x, weight=tw, y=buf[:, :N]))
        probs.append(dict(x=x, weight=tw, y=yc))
        wide.append((buf, yc, N))
    binding.LinearChain(probs)()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for buf, yc, N in wide:
        assert torch.equal(buf[:, :N].contiguous().view(torch.uint8), yc.view(torch.uint8))
        assert bool((buf[:, N:] == 7.0).all())
        assert bool(torch.isfinite(yc.float()).all()) and float(yc.float().abs().max()) > 0


def test_w8a8_comparison_scheme_in_the_chain_kernel():
    # FP8 weights (the dequantized weights of the same layers, tiled by w4a8_prepack_fp8) through the same
    # launch, partition and MMAs, the expansion replaced by a copy: outputs must equal those of the INT4
    # problems bit for bit (same FP8 operands, same accumulation order), and match the oracle.
    shapes = [(1, 2368, 640), (16, 1024, 1024), (7, 48, 256), (4, 14336, 512)]
    p4, p8, refs = [], [], []
    for i, (M, N, K) in enumerate(shapes):
        wq, tw = _weights(N, K, 400 + i)
        wd = weights_to_dev(*wq)
        tw8 = binding.prepack_fp8(binding.dequant_weight(*wd[:3]), wd[3])
        xb = inputs.make_activation(M, K, 410 + i, 0.01, 20.0)
        x = bf16_dev(xb)
        p4.append(dict(x=x, weight=tw, y=torch.zeros((M, N), dtype=torch.float32, device="cuda")))
        p8.append(dict(x=x, weight=tw8, y=torch.zeros((M, N), dtype=torch.float32, device="cuda")))
        refs.append((xb, wq))
    binding.LinearChain(p4)()
    binding.LinearChain(p8)()
    torch.cuda.synchronize()
    assert binding.query_device_status() == 0
    for a, b, (xb, wq) in zip(p4, p8, refs):
        assert torch.equal(a["y"].view(torch.int32), b["y"].view(torch.int32))
        _, _, ref = _oracle_layer(xb, wq)
        worst, _ = fp32_gate(b["y"].cpu().numpy(), ref["y64"], rel=2e-3)
        assert worst <= 2e-3, worst
    # formats may not be mixed within a launch
    with pytest.raises(binding.W4A8Error):
        binding.LinearChain([p4[0], p8[1]])()


@pytest.mark.parametrize("M", [1, 5, 16])
def test_rows_quantized_in_chunks_by_several_ctas(M):
    # Long rows are cut into chunks that different CTAs quantize; the chunk maxima meet in the workspace
    # before any chunk is converted.  Plain input with K = 8192 and 16384 (two and four chunks; 16384 is the
    # largest K), the gated kind with F = 4096 and 6144 (two and three chunks), dynamic, power-of-two and
    # static scales; FP8 bytes and scales bit-exact against the oracle (plain) and against
    # w4a8_silu_mul_quantize (gated), outputs within the gate; three launches on the same workspace (the
    # maxima and chunk counts must be back to zero after every launch).
    N = 208
    ss = dev(np.array([0.07], dtype=np.float32))
    probs, checks = [], []
    for i, (K, kw, okw) in enumerate([(8192, {}, {}), (16384, dict(scale_mode=binding.SCALE_POW2), dict(scale_mode=1)),
                                      (8192, dict(static_scale=ss), dict(static_scale=0.07))]):
        wq, tw = _weights(N, K, 500 + i)
        xb = inputs.make_activation(M, K, 510 + i, 0.01, 20.0)
        d = dict(x=bf16_dev(xb), weight=tw, y=torch.zeros((M, N), dtype=torch.float32, device="cuda"),
                 x8_out=torch.zeros((M, K), dtype=torch.uint8, device="cuda"),
                 s_x_out=torch.zeros((M,), dtype=torch.float32, device="cuda"), **kw)
        probs.append(d)
        checks.append(("plain", xb, wq, okw))
    for i, F in enumerate([4096, 6144]):
        wq, tw = _weights(N, F, 520 + i)
        gu = bf16_dev(inputs.make_activation(M, 2 * F, 530 + i, 0.0, 1.0))
        d = dict(x=gu, weight=tw, y=torch.zeros((M, N), dtype=torch.float32, device="cuda"),
                 kind=binding.CHAIN_INPUT_SILU_MUL, x8_out=torch.zeros((M, F), dtype=torch.uint8, device="cuda"),
                 s_x_out=torch.zeros((M,), dtype=torch.float32, device="cuda"))
        probs.append(d)
        checks.append(("gated", gu, wq, None))
    chain = binding.LinearChain(probs)
    for _ in range(3):
        for d in probs:
            d["y"].zero_(); d["x8_out"].zero_(); d["s_x_out"].zero_()
        chain()
        torch.cuda.synchronize()
        assert binding.query_device_status() == 0
        for d, (kind, src, wq, okw) in zip(probs, checks):
            if kind == "plain":
                x8, s_x = oracle.quantize_act(src, **okw)
                assert np.array_equal(d["x8_out"].cpu().numpy(), x8)
                assert np.array_equal(d["s_x_out"].cpu().numpy().view(np.uint32), s_x.astype(np.float32).view(np.uint32))
            else:
                h8, s_h = binding.silu_mul_quantize(src)
                torch.cuda.synchronize()
                assert torch.equal(d["x8_out"], h8) and torch.equal(d["s_x_out"], s_h)
                x8, s_x = h8.cpu().numpy(), s_h.cpu().numpy()
            ref = oracle.linear(x8, s_x, oracle.dequant_weight(*wq[:3]), wq[3])
            worst, _ = fp32_gate(d["y"].cpu().numpy(), ref["y64"], rel=2e-3)
            assert worst <= 2e-3, worst
