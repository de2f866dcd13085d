"""Pins of the per-column-group-index dequantization (activation-ordered quantization, the W4A8*
rows of Table 3; appendix "Activation Reordering")."""
import numpy as np
import pytest

import oracle
from helpers import e4m3_value_table, unpack_codes
from paper_2505_14638_b200 import inputs


def test_consecutive_groups_reduce_to_eq10():
    # g_idx[k] = k / 128 is the ordinary grouping: Eq. 10 / Eq. 14 exactly
    rng = np.random.default_rng(0)
    N, K = 12, 512
    wq = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 1), symmetric=False)
    g_idx = (np.arange(K) // 128).astype(np.int32)
    assert np.array_equal(oracle.dequant_weight_gidx(wq[0], wq[1], wq[2], g_idx), oracle.dequant_weight(*wq[:3]))
    wq = oracle.quantize_weight_rtn(inputs.make_weight(N, K, 0.02, 2), symmetric=True)
    assert np.array_equal(oracle.dequant_weight_gidx(wq[0], wq[1], None, g_idx), oracle.dequant_weight(*wq[:3]))
    del rng


def test_permuted_columns_follow_their_groups():
    # quantize a column-permuted matrix with ordinary groups, then put the codes back: column c of the
    # original order must dequantize with the group of its permuted position
    rng = np.random.default_rng(3)
    N, K = 8, 384
    W = inputs.make_weight(N, K, 0.02, 3)
    perm = rng.permutation(K)
    codes_p, gs, gz, s_w = oracle.quantize_weight_rtn(W[:, perm], symmetric=False)
    u_p = unpack_codes(codes_p)
    u = np.empty_like(u_p)
    u[:, perm] = u_p
    g_idx = np.empty(K, dtype=np.int32)
    g_idx[perm] = np.arange(K) // 128
    codes = (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)
    w8 = oracle.dequant_weight_gidx(codes, gs, gz, g_idx)
    w8_p = oracle.dequant_weight(codes_p, gs, gz)
    assert np.array_equal(w8[:, perm], w8_p)
    # direct formula on a few elements
    tab = e4m3_value_table()
    scale = (gs.astype(np.uint32) << 16).view(np.float32)
    for (n, k) in [(0, 0), (3, 200), (7, 383)]:
        g = g_idx[k]
        exact = (float(u[n, k]) - float(gz[n, g])) * float(scale[n, g])
        assert abs(tab[w8[n, k]] - exact) <= 0.5 * 32 + 1e-9      # within half the widest E4M3 step


def test_rejects_bad_group_index():
    wq = oracle.quantize_weight_rtn(inputs.make_weight(2, 256, 0.02, 4), symmetric=False)
    g_idx = np.zeros(256, dtype=np.int32)
    g_idx[5] = 2
    with pytest.raises(ValueError):
        oracle.dequant_weight_gidx(wq[0], wq[1], wq[2], g_idx)
