"""Pins for the oracle's INT4 -> FP8 dequantization (Eq. 10, vectorised per group in Eq. 14)."""
import numpy as np

import oracle
from helpers import e4m3_encode_search, e4m3_value_table, pack_codes, unpack_codes, bf16_bits_to_f64
from paper_2505_14638_b200 import inputs

G = 128


def _enumeration_matrix(scale_bits):
    """One row per (zero-point, scale): all 16 codes repeated along a 128-wide group."""
    rows_u, rows_s, rows_z = [], [], []
    u_row = np.tile(np.arange(16, dtype=np.uint8), G // 16)
    for z in range(16):
        for sb in scale_bits:
            rows_u.append(u_row)
            rows_s.append(sb)
            rows_z.append(z)
    u = np.stack(rows_u)
    return pack_codes(u), np.array(rows_s, dtype=np.uint16)[:, None], np.array(rows_z, dtype=np.uint8)[:, None], u


def test_power_of_two_scales_land_on_the_grid_exactly():
    # (u - z) * 2^e is representable for |u - z| <= 15 and e in [-9, 4]: the stored format
    # then dequantizes with no rounding at all.
    tab = e4m3_value_table()
    for e in range(-9, 5):
        sb = inputs.f32_to_bf16_bits(np.array([2.0 ** e], dtype=np.float32))
        codes, gs, gz, u = _enumeration_matrix(sb)
        w8 = oracle.dequant_weight(codes, gs, gz, G)
        exact = (u.astype(np.float64) - gz.astype(np.float64)) * 2.0 ** e
        assert np.array_equal(tab[w8], exact), e


def test_symmetric_storage_means_zero_point_eight():
    rng = np.random.default_rng(0)
    codes, gs, _ = inputs.random_codes(8, 512, seed=3)
    a = oracle.dequant_weight(codes, gs, None, G)
    b = oracle.dequant_weight(codes, gs, np.full((8, 4), 8, dtype=np.uint8), G)
    assert np.array_equal(a, b)
    assert rng is not None


def test_saturation_and_underflow():
    big = inputs.f32_to_bf16_bits(np.array([100.0], dtype=np.float32))   # 15*100 > 448
    tiny = inputs.f32_to_bf16_bits(np.array([2.0 ** -14], dtype=np.float32))  # 15*2^-14 < 2^-10
    codes, gs, gz, u = _enumeration_matrix(np.array([big[0], tiny[0]], dtype=np.uint16))
    w8 = oracle.dequant_weight(codes, gs, gz, G)
    d = (u.astype(np.int32) - gz.astype(np.int32))
    rows_big = np.arange(0, 32, 2)
    rows_tiny = np.arange(1, 32, 2)
    wb, db = w8[rows_big], d[rows_big]
    assert np.all(wb[db >= 5] == 0x7E) and np.all(wb[db <= -5] == 0xFE)
    wt, dt = w8[rows_tiny], d[rows_tiny]
    assert np.all(wt[dt > 0] == 0x00) and np.all(wt[dt < 0] == 0x80) and np.all(wt[dt == 0] == 0x00)


def test_brute_force_all_codes_all_zero_points_all_bf16_scales():
    # 16 codes x 16 zero-points x every finite BF16 scale bit pattern, against an independent
    # encoder (nearest search over the value table, tie -> even code) fed the exact real product.
    bits = np.arange(65536, dtype=np.uint32)
    s32 = (bits << 16).view(np.float32)
    fin = np.isfinite(s32)
    sb = bits[fin].astype(np.uint16)
    s = s32[fin].astype(np.float64)
    u_row = np.tile(np.arange(16, dtype=np.uint8), G // 16)
    codes = pack_codes(np.broadcast_to(u_row, (sb.size, G)).copy())
    for z in range(16):
        gz = np.full((sb.size, 1), z, dtype=np.uint8)
        w8 = oracle.dequant_weight(codes, sb[:, None], gz, G)[:, :16]
        d = (np.arange(16) - z).astype(np.float64)
        # fp32 product as the definition states: exact unless it leaves the fp32 range
        with np.errstate(over="ignore"):
            prod = (d[None, :].astype(np.float32) * s[:, None].astype(np.float32)).astype(np.float64)
        exact = d[None, :] * s[:, None]
        inrange = np.abs(exact) < 3.0e38
        assert np.array_equal(prod[inrange], exact[inrange])  # the product really is exact
        ref = e4m3_encode_search(prod)
        assert np.array_equal(w8, ref), z


def test_nibble_order_and_group_layout():
    # element k lives in byte k/2, even k in the low nibble; group g covers k in [128g, 128g+128)
    N, K = 2, 256
    u = np.full((N, K), 8, dtype=np.uint8)
    u[0, 0], u[0, 1], u[0, 129], u[1, 255] = 9, 10, 11, 12
    codes = pack_codes(u)
    assert codes[0, 0] == (10 << 4 | 9) and codes[0, 64] == (11 << 4 | 8) and codes[1, 127] == (12 << 4 | 8)
    gs = inputs.f32_to_bf16_bits(np.array([[1.0, 2.0], [4.0, 8.0]], dtype=np.float32))
    w8 = oracle.dequant_weight(codes, gs, None, G)
    val = e4m3_value_table()[w8]
    assert val[0, 0] == 1.0 and val[0, 1] == 2.0 and val[0, 129] == 6.0 and val[1, 255] == 32.0
    assert np.count_nonzero(val) == 4
    assert np.array_equal(unpack_codes(codes), u)


def test_matches_plain_formula_on_random_weights():
    codes, gs, gz = inputs.random_codes(64, 1024, seed=11, asymmetric=True)
    w8 = oracle.dequant_weight(codes, gs, gz, G)
    u = unpack_codes(codes).astype(np.float64)
    s = np.repeat(bf16_bits_to_f64(gs), G, axis=1)
    z = np.repeat(gz.astype(np.float64), G, axis=1)
    assert np.array_equal(w8, e4m3_encode_search((u - z) * s))
