"""Test-only helpers: a second, independent E4M3 encoder (table search) and tolerance gates.

Nothing here is used by the oracle or by the CUDA library."""
import numpy as np


def e4m3_value_table():
    """Closed-form value of every E4M3 code (OCP fn variant); NaN for 0x7F / 0xFF."""
    vals = np.empty(256, dtype=np.float64)
    for c in range(256):
        s, e, m = c >> 7, (c >> 3) & 15, c & 7
        if e == 15 and m == 7:
            v = np.nan
        elif e == 0:
            v = (m / 8.0) * 2.0 ** -6
        else:
            v = (1 + m / 8.0) * 2.0 ** (e - 7)
        vals[c] = -v if s else v
    return vals


_POS = e4m3_value_table()[:0x7F]  # codes 0x00..0x7E, increasing magnitudes


def e4m3_encode_search(v):
    """Nearest representable magnitude by searching the 127-entry table; a tie goes to the even
    code; magnitudes beyond 448 saturate; the sign bit of the input is kept.  Works on float64
    arrays holding exact values."""
    v = np.asarray(v, dtype=np.float64)
    a = np.abs(v)
    sign = np.signbit(v).astype(np.uint8) << 7
    hi = np.searchsorted(_POS, a, side="left")  # first index with table >= a
    hi = np.clip(hi, 0, 0x7E)
    lo = np.clip(hi - 1, 0, 0x7E)
    dlo = np.abs(a - _POS[lo])
    dhi = np.abs(_POS[hi] - a)
    pick_hi = (dhi < dlo) | ((dhi == dlo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    code = np.where(a >= 448.0, 0x7E, code).astype(np.uint8)
    out = code | sign
    out = np.where(np.isnan(v), 0x7F, out).astype(np.uint8)
    return out


def unpack_codes(codes):
    """[N, K/2] packed bytes -> [N, K] integer codes, even k in the low nibble."""
    codes = np.asarray(codes, dtype=np.uint8)
    N, Kh = codes.shape
    u = np.empty((N, Kh * 2), dtype=np.int32)
    u[:, 0::2] = codes & 0x0F
    u[:, 1::2] = codes >> 4
    return u


def pack_codes(u):
    u = np.asarray(u, dtype=np.uint8)
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)


def bf16_bits_to_f64(b):
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_ulp_distance(a_bits, b_bits):
    """Distance in BF16 steps between two arrays of BF16 bit patterns (sign-magnitude aware)."""
    def key(x):
        x = np.asarray(x, dtype=np.uint16).astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7FFF), x & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def fp32_gate(y, ref64, rel=2e-3):
    """Every element within rel * max(|ref|, tau_m), tau_m = 1e-2 * rms of the reference row."""
    ref64 = np.asarray(ref64, dtype=np.float64)
    tau = 1e-2 * np.sqrt(np.mean(ref64 ** 2, axis=1, keepdims=True))
    denom = np.maximum(np.abs(ref64), tau)
    err = np.abs(np.asarray(y, dtype=np.float64) - ref64) / np.where(denom == 0, 1.0, denom)
    return float(err.max()), err


def bf16_gate(y_bits, ref64):
    """BF16 output within 1 BF16 step of the correctly rounded reference where |ref| >= tau_m;
    below the floor the absolute error is at most one BF16 step of tau_m."""
    ref64 = np.asarray(ref64, dtype=np.float64)
    ref_bits = _f32_to_bf16(ref64.astype(np.float32))
    tau = 1e-2 * np.sqrt(np.mean(ref64 ** 2, axis=1, keepdims=True))
    big = np.abs(ref64) >= tau
    dist = bf16_ulp_distance(y_bits, ref_bits)
    ok_big = dist <= 1
    y = bf16_bits_to_f64(y_bits)
    tau_safe = np.where(tau > 0, tau, 1.0)
    ulp_tau = 2.0 ** (np.floor(np.log2(tau_safe)) - 7)
    ok_small = np.abs(y - ref64) <= ulp_tau
    ok = np.where(big, ok_big, ok_small)
    return bool(ok.all()), int(dist[big].max()) if big.any() else 0


def _f32_to_bf16(x):
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)
