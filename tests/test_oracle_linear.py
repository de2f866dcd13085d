"""Pins for the oracle's FP8 matmul with Eq. 4 / Eq. 11 scaling, and for the whole Sec. 3 flow."""
import os

import numpy as np

import oracle
from helpers import e4m3_value_table, pack_codes
from paper_2505_14638_b200 import inputs

G = 128
GOLD = os.path.join(os.path.dirname(__file__), "golden", "linear_tiny.txt")


def _case(M, N, K, seed, asym=False):
    W = inputs.make_weight(N, K, 0.02, seed)
    codes, gs, gz, s_w = oracle.quantize_weight_rtn(W, G, symmetric=not asym)
    xb = inputs.make_activation(M, K, seed, 0.01, 20.0)
    return xb, codes, gs, gz, s_w


def test_against_float64_library_matmul_and_int64_fixed_point():
    xb, codes, gs, gz, s_w = _case(9, 48, 512, seed=1, asym=True)
    out = oracle.forward(xb, codes, gs, gz, s_w, G)
    tab = e4m3_value_table()
    xd, wd = tab[out["x8"]], tab[out["w8"]]
    ref = (xd @ wd.T) * out["s_x"][:, None].astype(np.float64) * np.float64(s_w[0])
    assert np.array_equal(out["y64"], ref)
    # fixed point: every FP8 value is an integer multiple of 2^-9
    xi = np.round(xd * 512).astype(np.int64)
    wi = np.round(wd * 512).astype(np.int64)
    assert np.array_equal(xi / 512.0, xd) and np.array_equal(wi / 512.0, wd)
    acc = (xi @ wi.T).astype(np.float64) / (512.0 * 512.0)
    assert np.array_equal(out["y64"], acc * out["s_x"][:, None].astype(np.float64) * np.float64(s_w[0]))
    assert np.array_equal(out["y32"], out["y64"].astype(np.float32))
    assert np.array_equal(out["ybf16"], inputs.f32_to_bf16_bits(out["y32"]))
    assert np.all(out["yabs"] >= np.abs(out["y64"]) - 1e-12)


def test_hand_computed_tiny_case():
    gold = {}
    with open(GOLD) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            gold[k] = [float(t) for t in v]
    K = 128
    x = np.zeros((1, K), dtype=np.float32)
    x[0, :3] = [7.0, -3.5, 0.4375]
    u = np.full((2, K), 8, dtype=np.uint8)
    u[0, :3] = [15, 1, 10]
    u[1, :3] = [13, 8, 11]
    gs = inputs.f32_to_bf16_bits(np.array([[0.5], [3.0]], dtype=np.float32))
    s_w = np.array([0.25], dtype=np.float32)
    out = oracle.forward(inputs.f32_to_bf16_bits(x), pack_codes(u), gs, None, s_w, G)
    assert out["s_x"][0] == gold["s_x"][0]
    tab = e4m3_value_table()
    acc = tab[out["x8"]] @ tab[out["w8"]].T
    assert acc[0].tolist() == gold["acc"]
    assert out["y64"][0].tolist() == gold["y"]
    assert inputs.bf16_bits_to_f32(out["ybf16"])[0].tolist() == gold["ybf16"]


def test_one_hot_weights_select_activation_columns():
    M, K, N = 5, 256, 16
    xb = inputs.make_activation(M, K, 3)
    u = np.full((N, K), 8, dtype=np.uint8)
    pick = np.arange(N) * 13 % K
    u[np.arange(N), pick] = 9                         # (9 - 8) * 1.0 = 1
    gs = inputs.f32_to_bf16_bits(np.ones((N, K // G), dtype=np.float32))
    out = oracle.forward(xb, pack_codes(u), gs, None, np.array([1.0], dtype=np.float32), G)
    tab = e4m3_value_table()
    xhat = tab[out["x8"]] * out["s_x"][:, None].astype(np.float64)      # Eq. 4
    assert np.array_equal(out["y64"], xhat[:, pick])


def test_column_subset_and_per_channel_scale():
    xb, codes, gs, gz, _ = _case(4, 64, 256, seed=2)
    s_w = (np.arange(64, dtype=np.float32) + 1) / 64
    full = oracle.forward(xb, codes, gs, gz, s_w, G)
    cols = np.array([63, 0, 17, 17, 5])
    sub = oracle.forward(xb, codes, gs, gz, s_w, G, cols=cols)
    for key in ("y64", "y32", "ybf16", "yabs"):
        assert np.array_equal(sub[key], full[key][:, cols])
    one = oracle.forward(xb, codes, gs, gz, np.array([1.0], dtype=np.float32), G)
    assert np.allclose(full["y64"], one["y64"] * s_w[None, :].astype(np.float64), rtol=1e-15)


def test_transposed_operand_or_dropped_scale_would_show():
    # asymmetric shapes and distinct scales: the result differs if x/w are swapped or a scale is lost
    xb, codes, gs, gz, s_w = _case(3, 32, 384, seed=4)
    out = oracle.forward(xb, codes, gs, gz, s_w, G)
    assert out["y64"].shape == (3, 32)
    x = inputs.bf16_bits_to_f32(xb).astype(np.float64)
    W = inputs.make_weight(32, 384, 0.02, 4).astype(np.float64)
    dense = x @ W.T
    rel = np.linalg.norm(out["y64"] - dense) / np.linalg.norm(dense)
    assert rel < 0.2                                  # INT4 + FP8 noise, but the same linear map
