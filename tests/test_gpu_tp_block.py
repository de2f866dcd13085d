"""GPU parity of the tensor-parallel MLP block with the ranks run one after the other on one
device (no rank waits on another: each rank's partial output is complete before the next starts,
and the sum over ranks is taken on the host).  Every stage of every rank is checked against the
oracle on the inputs that stage saw on the GPU: activations bit-exact, linear outputs within the
output gates, the gated activation by the rules of its own test; the summed output is compared
with the oracle block run on the same shards."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import bf16_bits, bf16_dev, dev
from helpers import bf16_gate, bf16_ulp_distance, fp32_gate
from paper_2505_14638_b200 import binding, inputs, tp
from tp_ops import OracleOps

pytestmark = pytest.mark.gpu


def _host(w):
    g = lambda t: None if t is None else t.cpu().numpy()
    return tp.Weights(g(w.codes), bf16_bits(w.gscale), g(w.gzero), g(w.s_w))


class CheckedCudaOps(tp.CudaOps):
    """The CUDA steps, each compared with the oracle on the inputs it was given."""

    def __init__(self):
        super().__init__()
        self.ref = OracleOps()
        self.host = {}
        self.checked = {"quantize_act": 0, "linear": 0, "silu_mul_quantize": 0}

    def prepare(self, w):
        p = super().prepare(w)
        self.host[id(p)] = self.ref.prepare(_host(w))
        return p

    def quantize_act(self, x):
        x8, s_x = super().quantize_act(x)
        r8, rs = self.ref.quantize_act(bf16_bits(x))
        assert np.array_equal(x8.cpu().numpy(), r8)
        assert np.array_equal(s_x.cpu().numpy().view(np.uint32), rs.view(np.uint32))
        self.checked["quantize_act"] += 1
        return x8, s_x

    def linear(self, x8, s_x, prepared, fp32_out):
        y = super().linear(x8, s_x, prepared, fp32_out)
        w8, s_w = self.host[id(prepared)]
        ref = oracle.linear(x8.cpu().numpy(), s_x.cpu().numpy(), w8, s_w, want=("y64",))["y64"]
        if fp32_out:
            worst, _ = fp32_gate(y.cpu().numpy(), ref, rel=2e-3)
            assert worst <= 2e-3, worst
        else:
            ok, dist = bf16_gate(bf16_bits(y), ref)
            assert ok, dist
        self.checked["linear"] += 1
        return y

    def silu_mul_quantize(self, gate_up):
        x8, s_x = super().silu_mul_quantize(gate_up)
        gu = bf16_bits(gate_up)
        h_ref = oracle.silu_mul(gu)
        r8, rs = oracle.quantize_act(h_ref)
        x8n, sn = x8.cpu().numpy(), s_x.cpu().numpy()
        assert np.all(np.abs(sn - rs) <= 2.0 ** -7 * rs)
        hv = oracle.bf16_to_f32(h_ref).astype(np.float64)
        got = oracle.e4m3_decode_array(x8n).astype(np.float64) * sn[:, None].astype(np.float64)
        step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(hv), 1e-30))) - 7)
        assert np.all(np.abs(got - hv) <= np.abs(hv) * 2.0 ** -4 + sn[:, None] * 2.0 ** -10 + step * (1 + 2.0 ** -3))
        assert (x8n != r8).mean() <= 1e-2
        self.checked["silu_mul_quantize"] += 1
        return x8, s_x


def _weights(N, K, seed):
    codes, gscale, gzero, s_w = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.03, seed), symmetric=True)
    return tp.Weights(codes, gscale, gzero, s_w)


def _to_dev(w):
    return tp.Weights(dev(w.codes), bf16_dev(w.gscale), None if w.gzero is None else dev(w.gzero), dev(w.s_w))


@pytest.mark.parametrize("world,M,H,F", [(1, 4, 512, 1024), (2, 1, 1024, 2048), (2, 16, 512, 1280), (4, 7, 512, 1024),
                                         (8, 3, 4096, 14336)])
def test_ranks_in_sequence_every_stage_against_the_oracle(world, M, H, F):
    gu_h, down_h = _weights(2 * F, H, 21), _weights(H, F, 22)
    gu_d, down_d = _to_dev(gu_h), _to_dev(down_h)
    xb = inputs.make_activation(M, H, 23, 0.01, 20.0)
    x = bf16_dev(xb)
    ops = CheckedCudaOps()
    total = np.zeros((M, H), dtype=np.float64)
    ref_total = np.zeros((M, H), dtype=np.float64)
    for r in range(world):
        blk = tp.TPMlpBlock(gu_d, down_d, r, world, ops=ops, exchange=tp.Exchange(world=world), reduce_fp32=True)
        part = blk.partial(x)
        torch.cuda.synchronize()
        assert part.shape == (M, H) and part.dtype == torch.float32
        total += part.cpu().numpy().astype(np.float64)
        ref_blk = tp.TPMlpBlock(gu_h, down_h, r, world, ops=ops.ref, exchange=tp.Exchange(world=world), reduce_fp32=True)
        ref_total += ref_blk.partial(xb).numpy().astype(np.float64)
    assert binding.query_device_status() == 0
    assert ops.checked == {"quantize_act": world, "linear": 2 * world, "silu_mul_quantize": world}
    # the whole block: the oracle's h can differ from the GPU's by one BF16 step on a few elements
    # (exp of the math library), which moves a few FP8 codes of the down projection's input
    rms = np.sqrt(np.mean(ref_total ** 2))
    assert np.abs(total - ref_total).max() <= 2e-2 * rms
    assert np.sqrt(np.mean((total - ref_total) ** 2)) <= 2e-3 * rms


def test_world_of_one_with_bf16_output_equals_the_plain_block():
    M, H, F = 5, 512, 1024
    gu_d, down_d = _to_dev(_weights(2 * F, H, 31)), _to_dev(_weights(H, F, 32))
    x = bf16_dev(inputs.make_activation(M, H, 33))
    y = tp.TPMlpBlock(gu_d, down_d, 0, 1, exchange=tp.Exchange(world=1)).forward(x)
    x8, s_x = binding.quantize_act(x)
    g = binding.linear_tiled(x8, s_x, binding.prepack_weight(gu_d.codes, gu_d.gscale, None, gu_d.s_w))
    h8, s_h = binding.silu_mul_quantize(g)
    want = binding.linear_tiled(h8, s_h, binding.prepack_weight(down_d.codes, down_d.gscale, None, down_d.s_w))
    torch.cuda.synchronize()
    assert y.dtype == torch.bfloat16 and torch.equal(y, want)
