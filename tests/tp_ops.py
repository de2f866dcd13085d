"""Test-side stand-in for the CUDA steps of the tensor-parallel block: the same four methods on the
CPU oracle (numpy in, numpy or torch out), so that sharding and exchange can run without a GPU and
GPU results have something to be compared with.  Activations travel as BF16 bit patterns (uint16)."""
import numpy as np
import torch

import oracle


class OracleOps:
    def prepare(self, w):
        return oracle.dequant_weight(np.asarray(w.codes), np.asarray(w.gscale),
                                     None if w.gzero is None else np.asarray(w.gzero)), np.asarray(w.s_w)

    def quantize_act(self, x_bits):
        return oracle.quantize_act(np.ascontiguousarray(x_bits))

    def linear(self, x8, s_x, prepared, fp32_out):
        w8, s_w = prepared
        out = oracle.linear(x8, s_x, w8, s_w, want=("y32", "ybf16"))
        if fp32_out:
            return torch.from_numpy(out["y32"])
        return torch.from_numpy(out["ybf16"].view(np.int16)).view(torch.bfloat16)

    def silu_mul_quantize(self, gate_up):
        bits = gate_up.view(torch.int16).numpy().view(np.uint16) if isinstance(gate_up, torch.Tensor) else gate_up
        return oracle.quantize_act(oracle.silu_mul(np.ascontiguousarray(bits)))


def bf16_tensor_bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
