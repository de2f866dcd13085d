"""Pins for the oracle's E4M3 codec (Sec. 2.2 / Eq. 3 "nearest_Z", +-448 range of Sec. 4.1)."""
import os

import numpy as np
import pytest

import oracle
from helpers import e4m3_encode_search, e4m3_value_table

GOLD = os.path.join(os.path.dirname(__file__), "golden", "e4m3_grid.txt")


def test_decode_closed_form_all_codes():
    tab = oracle.e4m3_decode_table().astype(np.float64)
    ref = e4m3_value_table()
    assert np.array_equal(np.isnan(tab), np.isnan(ref))
    fin = ~np.isnan(ref)
    assert np.array_equal(tab[fin], ref[fin])
    assert np.isnan(tab[0x7F]) and np.isnan(tab[0xFF])
    assert tab[0x7E] == 448.0 and tab[0xFE] == -448.0
    assert np.signbit(tab[0x80]) and tab[0x80] == 0.0
    assert fin.sum() == 254


def test_decode_matches_library_dtypes():
    torch = pytest.importorskip("torch")
    codes = torch.arange(256, dtype=torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).float().numpy()
    tab = oracle.e4m3_decode_table()
    assert np.array_equal(np.isnan(tab), np.isnan(lib))
    assert np.array_equal(tab[~np.isnan(tab)], lib[~np.isnan(lib)])
    ml = pytest.importorskip("ml_dtypes")
    lib2 = np.arange(256, dtype=np.uint8).view(ml.float8_e4m3fn).astype(np.float32)
    assert np.array_equal(tab[~np.isnan(tab)], lib2[~np.isnan(lib2)])


def test_golden_grid_points():
    n = 0
    with open(GOLD) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            val, code = line.split()[:2]
            got = oracle.e4m3_encode(float(val))
            assert got == int(code, 16), (val, hex(got), code)
            n += 1
    assert n >= 15


def test_roundtrip_all_finite_codes():
    tab = oracle.e4m3_decode_table()
    for c in range(256):
        if c in (0x7F, 0xFF):
            continue
        assert oracle.e4m3_encode(float(tab[c])) == c


def test_nan_and_inf():
    assert oracle.e4m3_encode(float("nan")) == 0x7F
    assert oracle.e4m3_encode(float("inf")) == 0x7E
    assert oracle.e4m3_encode(float("-inf")) == 0xFE


def test_idempotent_and_monotone():
    rng = np.random.default_rng(1)
    v = np.concatenate([
        rng.standard_normal(200000).astype(np.float32) * 100,
        rng.standard_normal(200000).astype(np.float32) * 0.01,
        np.float32(2.0) ** rng.uniform(-14, 10, 200000).astype(np.float32),
    ]).astype(np.float32)
    c = oracle.e4m3_encode_array(v)
    d = oracle.e4m3_decode_array(c)
    assert np.array_equal(oracle.e4m3_encode_array(d), c)
    order = np.argsort(v, kind="stable")
    assert np.all(np.diff(d[order].astype(np.float64)) >= 0)
    # nearest: no other grid point is closer
    tab = e4m3_value_table()
    fin = tab[~np.isnan(tab)]
    sample = v[:5000].astype(np.float64)
    best = np.abs(sample[:, None] - fin[None, :]).min(axis=1)
    clipped = np.clip(sample, -448, 448)
    assert np.allclose(np.abs(clipped - d[:5000]), np.abs(clipped[:, None] - fin[None, :]).min(axis=1), rtol=0, atol=0)
    assert best.shape == (5000,)


def test_against_table_search_encoder_all_bf16_patterns():
    bits = np.arange(65536, dtype=np.uint32)
    v = (bits << 16).view(np.float32)
    fin = np.isfinite(v)
    got = oracle.e4m3_encode_array(v[fin])
    ref = e4m3_encode_search(v[fin].astype(np.float64))
    assert np.array_equal(got, ref)


def test_against_table_search_encoder_random_fp32_patterns():
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 2 ** 32, size=4_000_000, dtype=np.uint64).astype(np.uint32)
    v = bits.view(np.float32)
    v = v[np.isfinite(v)]
    assert np.array_equal(oracle.e4m3_encode_array(v), e4m3_encode_search(v.astype(np.float64)))
    # dense sweep of the range where the grid lives, including every midpoint neighbourhood
    tab = e4m3_value_table()[:0x7F]
    mids = (tab[:-1] + tab[1:]) / 2
    near = np.concatenate([np.nextafter(mids.astype(np.float32), np.float32(0)),
                           mids.astype(np.float32),
                           np.nextafter(mids.astype(np.float32), np.float32(1e9))])
    near = np.concatenate([near, -near])
    assert np.array_equal(oracle.e4m3_encode_array(near), e4m3_encode_search(near.astype(np.float64)))


def test_in_range_agrees_with_library_casts():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(3)
    v = (rng.standard_normal(1_000_000) * 120).astype(np.float32)
    v = v[np.abs(v) <= 448]
    lib = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(oracle.e4m3_encode_array(v), lib)
    ml = pytest.importorskip("ml_dtypes")
    lib2 = v.astype(ml.float8_e4m3fn).view(np.uint8)
    assert np.array_equal(oracle.e4m3_encode_array(v), lib2)


def test_bf16_helpers():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(20000) * 3).astype(np.float32)
    x[:4] = [1.00390625, 1.01171875, 0.0, -0.0]  # two exact ties, signed zeros
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.f32_to_bf16(x), lib)
    assert np.array_equal(oracle.bf16_to_f32(lib), torch.from_numpy(x).to(torch.bfloat16).float().numpy())
