"""numpy front-end of the CPU oracle (plain C, see w4a8_oracle.c / w4a8_oracle.h).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's CPU-baseline
leg are the only callers.  Nothing here imports or is imported by the CUDA package.

BF16 tensors are numpy uint16 arrays of bit patterns; E4M3 tensors are uint8 arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "w4a8_oracle.c")
_SRC_DPQ = os.path.join(_HERE, "w4a8_dpq_oracle.c")
_HDR = os.path.join(_HERE, "w4a8_oracle.h")
_LIB = os.path.join(_HERE, "liboracle_w4a8.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction). Returns the .so path."""
    stale = (
        force
        or not os.path.exists(_LIB)
        or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_DPQ), os.path.getmtime(_HDR))
    )
    if stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        cmd = [
            "gcc", "-std=c11", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
            "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC, _SRC_DPQ, "-lm",
        ]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c = ctypes
    p = c.c_void_p
    i64 = c.c_int64
    lib.oracle_e4m3_decode.restype = c.c_float
    lib.oracle_e4m3_decode.argtypes = [c.c_uint8]
    lib.oracle_e4m3_encode.restype = c.c_uint8
    lib.oracle_e4m3_encode.argtypes = [c.c_float]
    lib.oracle_e4m3_encode_n.restype = None
    lib.oracle_e4m3_encode_n.argtypes = [p, i64, p]
    lib.oracle_e4m3_decode_n.restype = None
    lib.oracle_e4m3_decode_n.argtypes = [p, i64, p]
    lib.oracle_bf16_to_f32.restype = c.c_float
    lib.oracle_bf16_to_f32.argtypes = [c.c_uint16]
    lib.oracle_f32_to_bf16.restype = c.c_uint16
    lib.oracle_f32_to_bf16.argtypes = [c.c_float]
    lib.oracle_quantize_weight_rtn.restype = c.c_int
    lib.oracle_quantize_weight_rtn.argtypes = [p, i64, i64, c.c_int, c.c_int, c.c_int, c.c_int, p, p, p, p]
    lib.oracle_dpq_quantize.restype = c.c_int
    lib.oracle_dpq_quantize.argtypes = [p, i64, i64, c.c_int, p, p, c.c_int, c.c_int, c.c_int, p, p, p, p, p, p]
    lib.oracle_dequant_weight_gidx.restype = c.c_int
    lib.oracle_dequant_weight_gidx.argtypes = [p, p, p, p, i64, i64, i64, p]
    lib.oracle_dequant_weight.restype = c.c_int
    lib.oracle_dequant_weight.argtypes = [p, p, p, i64, i64, c.c_int, p]
    lib.oracle_quantize_act.restype = c.c_int
    lib.oracle_quantize_act.argtypes = [p, i64, i64, i64, p, i64, p, c.c_int, p]
    lib.oracle_linear.restype = c.c_int
    lib.oracle_linear.argtypes = [p, i64, p, i64, p, p, c.c_int, i64, i64, p, i64, p, p, p, p]
    lib.oracle_num_threads.restype = c.c_int
    lib.oracle_num_threads.argtypes = []
    _lib = lib
    return lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


# ----------------------------------------------------------------------------- scalar codec

def e4m3_decode(code: int) -> float:
    return float(_load().oracle_e4m3_decode(int(code) & 0xFF))


def e4m3_encode(v: float) -> int:
    return int(_load().oracle_e4m3_encode(float(np.float32(v))))


def e4m3_encode_array(v) -> np.ndarray:
    """Element-wise oracle encoder over an fp32 array."""
    lib = _load()
    v = np.ascontiguousarray(v, dtype=np.float32)
    out = np.empty(v.shape, dtype=np.uint8)
    lib.oracle_e4m3_encode_n(_ptr(v), v.size, _ptr(out))
    return out


def e4m3_decode_array(c) -> np.ndarray:
    """Element-wise oracle decoder over a uint8 array."""
    lib = _load()
    c = np.ascontiguousarray(c, dtype=np.uint8)
    out = np.empty(c.shape, dtype=np.float32)
    lib.oracle_e4m3_decode_n(_ptr(c), c.size, _ptr(out))
    return out


def e4m3_decode_table() -> np.ndarray:
    return e4m3_decode_array(np.arange(256, dtype=np.uint8))


def bf16_to_f32(bits) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(x) -> np.ndarray:
    """Round-to-nearest-even fp32 -> BF16 bit patterns, through the C routine's definition."""
    lib = _load()
    x = np.asarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    fo, fx = out.reshape(-1), x.reshape(-1)
    f = lib.oracle_f32_to_bf16
    for i in range(fx.size):
        fo[i] = f(float(fx[i]))
    return out


# ----------------------------------------------------------------------------- tensor routines

def quantize_weight_rtn(W, group=128, symmetric=True, pow2=False, per_channel=False):
    """Eq. 6-9 round-to-nearest.  Returns (codes[N,K/2] u8, gscale[N,K/g] u16 bf16 bits,
    gzero[N,K/g] u8 or None when symmetric, s_w fp32[N or 1])."""
    lib = _load()
    W = _c(W, np.float32)
    N, K = W.shape
    G = K // group
    codes = np.zeros((N, K // 2), dtype=np.uint8)
    gscale = np.zeros((N, G), dtype=np.uint16)
    gzero = np.zeros((N, G), dtype=np.uint8)
    s_w = np.zeros(N if per_channel else 1, dtype=np.float32)
    rc = lib.oracle_quantize_weight_rtn(_ptr(W), N, K, group, int(symmetric), int(pow2),
                                        int(per_channel), _ptr(codes), _ptr(gscale), _ptr(gzero),
                                        _ptr(s_w))
    if rc != 0:
        raise ValueError("oracle_quantize_weight_rtn: bad arguments")
    return codes, gscale, (None if symmetric else gzero), s_w


def gar_permutation(diag, group=128):
    """Group-Aware Reordering (Sec. 3.2, appendix): processing order from the Hessian diagonal.
    Inside each group the columns go by descending diagonal; the groups go by descending maximum
    diagonal (the ranking the paper used).  Ties keep the original order.  Returns int32 [K]:
    position p handles original column perm[p]."""
    d = np.asarray(diag, dtype=np.float64)
    K = d.size
    assert K % group == 0
    G = K // group
    within = []
    gmax = np.empty(G)
    for g in range(G):
        idx = np.arange(g * group, (g + 1) * group)
        order = idx[np.argsort(-d[idx], kind="stable")]
        within.append(order)
        gmax[g] = d[idx].max()
    gorder = np.argsort(-gmax, kind="stable")
    return np.concatenate([within[g] for g in gorder]).astype(np.int32)


def hessian(x_bf16) -> np.ndarray:
    """The layer Hessian of Sec. 3.1 (up to the constant factor that cancels in the update of
    Eq. 12): H = X^T X over the calibration tokens, X given as BF16 bits [T, K]; float64."""
    X = bf16_to_f32(x_bf16).astype(np.float64)
    return X.T @ X


def hessian_prepare(H, perm=None, damp=0.01) -> np.ndarray:
    """Sec. 3.3 (as in GPTQ), float64: the Hessian in processing order, a unit diagonal for columns
    whose diagonal entry is zero, damp * mean(diag) added to the diagonal."""
    H = np.array(H, dtype=np.float64)
    if perm is not None:
        H = H[np.ix_(perm, perm)]
    d = np.diag(H).copy()
    dead = d == 0
    H[dead, dead] = 1.0
    H[np.diag_indices_from(H)] += damp * np.mean(np.diag(H))
    return H


def hessian_upper_cholesky(H, perm=None, damp=0.01):
    """What Sec. 3.3 takes from GPTQ, in float64: the prepared Hessian (hessian_prepare) inverted,
    and the upper Cholesky factor U of the inverse (H^-1 = U^T U) as float32."""
    H = hessian_prepare(H, perm, damp)
    Hinv = np.linalg.inv(H)
    Hinv = 0.5 * (Hinv + Hinv.T)
    L = np.linalg.cholesky(Hinv)          # Hinv = L L^T
    return np.ascontiguousarray(L.T).astype(np.float32)


def dpq_quantize(W, U, perm=None, group=128, symmetric=False, mse_steps=0, per_channel=False, debug=False):
    """Algorithm 1 (DPQ).  W fp32 [N,K]; U fp32 [K,K] upper Cholesky factor in processing order;
    perm int32 [K] or None.  Returns (codes, gscale, gzero or None, s_w) in the original column
    order, plus (err, what) in processing order when debug is set."""
    lib = _load()
    W = _c(W, np.float32)
    U = _c(U, np.float32)
    N, K = W.shape
    assert U.shape == (K, K)
    G = K // group
    pm = None if perm is None else _c(perm, np.int32)
    codes = np.zeros((N, K // 2), dtype=np.uint8)
    gscale = np.zeros((N, G), dtype=np.uint16)
    gzero = np.zeros((N, G), dtype=np.uint8)
    s_w = np.zeros(N if per_channel else 1, dtype=np.float32)
    err = np.zeros((N, K), dtype=np.float32) if debug else None
    what = np.zeros((N, K), dtype=np.float32) if debug else None
    rc = lib.oracle_dpq_quantize(_ptr(W), N, K, group, _ptr(U), _ptr(pm), int(symmetric), int(mse_steps),
                                 int(per_channel), _ptr(codes), _ptr(gscale), _ptr(gzero), _ptr(s_w),
                                 _ptr(err), _ptr(what))
    if rc != 0:
        raise ValueError("oracle_dpq_quantize: bad arguments")
    out = (codes, gscale, (None if symmetric else gzero), s_w)
    return out + (err, what) if debug else out


def dequant_weight(codes, gscale, gzero=None, group=128):
    """Eq. 10: E4M3 bytes [N,K]."""
    lib = _load()
    codes = _c(codes, np.uint8)
    gscale = _c(gscale, np.uint16)
    N, Kh = codes.shape
    K = Kh * 2
    if gzero is not None:
        gzero = _c(gzero, np.uint8)
    w8 = np.empty((N, K), dtype=np.uint8)
    rc = lib.oracle_dequant_weight(_ptr(codes), _ptr(gscale), _ptr(gzero), N, K, group, _ptr(w8))
    if rc != 0:
        raise ValueError("oracle_dequant_weight: bad arguments")
    return w8


def dequant_weight_gidx(codes, gscale, gzero, g_idx):
    """Eq. 10 with a per-column group index g_idx int32 [K]: E4M3 bytes [N,K]."""
    lib = _load()
    codes = _c(codes, np.uint8)
    gscale = _c(gscale, np.uint16)
    g_idx = _c(g_idx, np.int32)
    N, Kh = codes.shape
    K = Kh * 2
    G = gscale.shape[1]
    if gzero is not None:
        gzero = _c(gzero, np.uint8)
    w8 = np.empty((N, K), dtype=np.uint8)
    rc = lib.oracle_dequant_weight_gidx(_ptr(codes), _ptr(gscale), _ptr(gzero), _ptr(g_idx), N, K, G, _ptr(w8))
    if rc != 0:
        raise ValueError("oracle_dequant_weight_gidx: bad arguments")
    return w8


def quantize_act(x_bf16, scale_mode=0, static_scale=None):
    """Eq. 13 per token.  x_bf16: uint16 [M,K].  Returns (x8 u8 [M,K], s_x fp32 [M])."""
    lib = _load()
    x = _c(x_bf16, np.uint16)
    M, K = x.shape
    x8 = np.empty((M, K), dtype=np.uint8)
    s_x = np.empty(M, dtype=np.float32)
    ss = None if static_scale is None else np.array([static_scale], dtype=np.float32)
    rc = lib.oracle_quantize_act(_ptr(x), M, K, K, _ptr(x8), K, _ptr(s_x), int(scale_mode), _ptr(ss))
    if rc != 0:
        raise ValueError("oracle_quantize_act: bad arguments")
    return x8, s_x


def dequant_weight_bf16(codes, gscale, gzero=None, group=128) -> np.ndarray:
    """W4A16 comparison scheme (Sec. 4.3): W16 = BF16_RNE((u - z) * s_g), the product formed exactly
    (a small integer times a BF16 value) and rounded once.  Returns BF16 bit patterns uint16 [N, K]."""
    codes = _c(codes, np.uint8)
    N, Kh = codes.shape
    K = 2 * Kh
    u = np.empty((N, K), dtype=np.int64)
    u[:, 0::2] = codes & 0x0F
    u[:, 1::2] = codes >> 4
    s = bf16_to_f32(_c(gscale, np.uint16)).astype(np.float64)           # [N, K/group]
    z = np.full(s.shape, 8, dtype=np.int64) if gzero is None else _c(gzero, np.uint8).astype(np.int64)
    prod = (u - np.repeat(z, group, axis=1)).astype(np.float64) * np.repeat(s, group, axis=1)
    return f64_to_bf16(prod)


def linear_w4a16(x_bf16, w16_bf16, s_w, cols=None) -> np.ndarray:
    """Y = s_w * X W16^T in double precision (every BF16 x BF16 product is exact in double; the sum of
    K of them is rounded at the 53rd bit at worst).  Returns float64 [M, N or len(cols)]."""
    x = bf16_to_f32(_c(x_bf16, np.uint16)).astype(np.float64)
    w = bf16_to_f32(_c(w16_bf16, np.uint16)).astype(np.float64)
    s_w = _c(s_w, np.float32).astype(np.float64)
    if cols is not None:
        w = w[np.asarray(cols)]
        sw = s_w if s_w.size == 1 else s_w[np.asarray(cols)]
    else:
        sw = s_w
    return (x @ w.T) * (sw[None, :] if sw.size > 1 else sw[0])


def silu_mul_f64(gate_up_bf16) -> np.ndarray:
    """The gated-MLP activation by its definition, in double precision:
    h = silu(G) * U, silu(g) = g / (1 + exp(-g)); G = first half of each row, U = second half.
    gate_up_bf16: uint16 [M, 2F] (BF16 bit patterns).  Returns float64 [M, F] (not rounded)."""
    gu = bf16_to_f32(_c(gate_up_bf16, np.uint16)).astype(np.float64)
    F = gu.shape[1] // 2
    g, u = gu[:, :F], gu[:, F:]
    return g / (1.0 + np.exp(-g)) * u


def f64_to_bf16(x) -> np.ndarray:
    """Round-to-nearest-even of doubles to BF16 bit patterns in ONE rounding (normal range only:
    the magnitudes here are far from the BF16 subnormals and from overflow; zero maps to zero)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    b = x.view(np.uint64)
    sign = (b >> np.uint64(63)).astype(np.uint64)
    exp = ((b >> np.uint64(52)) & np.uint64(0x7FF)).astype(np.int64)
    man = b & np.uint64((1 << 52) - 1)
    keep = (man >> np.uint64(45)).astype(np.int64)            # 7 mantissa bits
    rem = man & np.uint64((1 << 45) - 1)
    half = np.uint64(1 << 44)
    up = (rem > half) | ((rem == half) & ((keep & 1) == 1))
    keep = keep + up.astype(np.int64)
    carry = keep == 128
    keep = np.where(carry, 0, keep)
    e8 = exp - 1023 + 127 + carry.astype(np.int64)
    zero = (exp == 0)
    if np.any(~zero & ((e8 <= 0) | (e8 >= 255))):
        raise ValueError("f64_to_bf16: value outside the normal BF16 range")
    out = (sign.astype(np.int64) << 15) | (e8 << 7) | keep
    out = np.where(zero, sign.astype(np.int64) << 15, out)
    return out.astype(np.uint16)


def silu_mul(gate_up_bf16) -> np.ndarray:
    """h = BF16_RNE(silu(G) * U): the activations that enter the down projection.  uint16 [M, F]."""
    return f64_to_bf16(silu_mul_f64(gate_up_bf16))


def linear(x8, s_x, w8, s_w, cols=None, want=("y64", "y32", "ybf16", "yabs")):
    """Exact FP8 dot products with Eq. 4 / Eq. 11 scales.  Returns a dict of [M, N or len(cols)]."""
    lib = _load()
    x8 = _c(x8, np.uint8)
    w8 = _c(w8, np.uint8)
    s_x = _c(s_x, np.float32)
    s_w = _c(s_w, np.float32)
    M, K = x8.shape
    N = w8.shape[0]
    assert w8.shape[1] == K
    sw_stride = 0 if s_w.size == 1 else 1
    if sw_stride:
        assert s_w.size == N
    if cols is not None:
        cols = _c(cols, np.int64)
        NC = cols.size
    else:
        NC = N
    out = {}
    if "y64" in want:
        out["y64"] = np.empty((M, NC), dtype=np.float64)
    if "y32" in want:
        out["y32"] = np.empty((M, NC), dtype=np.float32)
    if "ybf16" in want:
        out["ybf16"] = np.empty((M, NC), dtype=np.uint16)
    if "yabs" in want:
        out["yabs"] = np.empty((M, NC), dtype=np.float64)
    rc = lib.oracle_linear(_ptr(x8), K, _ptr(s_x), M, _ptr(w8), _ptr(s_w), sw_stride, N, K,
                           _ptr(cols), NC, _ptr(out.get("y64")), _ptr(out.get("y32")),
                           _ptr(out.get("ybf16")), _ptr(out.get("yabs")))
    if rc != 0:
        raise ValueError("oracle_linear: bad arguments")
    return out


def forward(x_bf16, codes, gscale, gzero, s_w, group=128, scale_mode=0, cols=None):
    """Whole inference path of Sec. 3: Eq. 13 -> Eq. 10 -> FP8 matmul -> Eq. 4/11."""
    x8, s_x = quantize_act(x_bf16, scale_mode)
    w8 = dequant_weight(codes, gscale, gzero, group)
    out = linear(x8, s_x, w8, s_w, cols)
    out["x8"], out["s_x"], out["w8"] = x8, s_x, w8
    return out


def num_threads() -> int:
    return int(_load().oracle_num_threads())
