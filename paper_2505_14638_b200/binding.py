"""ctypes binding of the C-ABI library declared in include/w4a8.h.

Argument marshalling only: every step of the W4A8 path (Eq. 13 activation quantization, Eq. 10
weight dequantization, FP8 matmul, Eq. 4 / Eq. 11 epilogue) runs in the library's CUDA kernels.
PyTorch supplies device buffers and the current stream.  There is no CPU fallback: if the
library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libw4a8_b200.so")

OK = 0
ERR_INVALID_ARG, ERR_BAD_SHAPE, ERR_BAD_ALIGNMENT, ERR_WORKSPACE_TOO_SMALL = -1, -2, -3, -4
ERR_UNSUPPORTED_DEVICE, ERR_CUDA, ERR_TIMEOUT = -5, -6, -7
SCALE_EXACT, SCALE_POW2 = 0, 1
OUT_BF16, OUT_FP32 = 0, 1
ALGO_AUTO, ALGO_SIMT, ALGO_UMMA = 0, 1, 2
FMT_CANONICAL, FMT_TILED, FMT_TILED_SIGNMAG, FMT_TILED_FP8 = 0, 1, 2, 3
GROUP = 128

# Every symbol include/w4a8.h declares.
EXPORTS = (
    "w4a8_quantize_act", "w4a8_dequant_weight", "w4a8_linear", "w4a8_linear_workspace_bytes",
    "w4a8_prepack_bytes", "w4a8_prepack_weight",
    "w4a8_linear_ex", "w4a8_linear_ex_workspace_bytes", "w4a8_linear_static_scratch",
    "w4a8_linear_w8a8", "w4a8_dequant_weight_gidx", "w4a8_linear_gidx", "w4a8_prepack_fp8",
    "w4a8_hessian_accumulate", "w4a8_hessian_prepare",
    "w4a8_silu_mul_quantize", "w4a8_linear_w4a16", "w4a8_linear_w4a16_workspace_bytes", "w4a8_linear_w4a16_tiled",
    "w4a8_quantize_weight_rtn",
    "w4a8_gar_workspace_bytes", "w4a8_gar_permutation", "w4a8_dpq_workspace_bytes", "w4a8_dpq_quantize",
    "w4a8_forward_host", "w4a8_query_device_status", "w4a8_launch_count", "w4a8_status_string",
    "w4a8_linear_chain", "w4a8_linear_chain_workspace_bytes", "w4a8_selftest_bounded_wait",
    "w4a8_host_buffer_device_pointer",
)

CHAIN_INPUT_PLAIN, CHAIN_INPUT_SILU_MUL = 0, 1
CHAIN_MAX_PROBLEMS, CHAIN_MAX_M = 24, 16


class ChainProblem(ctypes.Structure):
    """struct w4a8_chain_problem of include/w4a8.h, field for field."""
    _fields_ = [
        ("x_bf16", ctypes.c_void_p), ("ldx", ctypes.c_int64),
        ("input_kind", ctypes.c_int32), ("depends_on", ctypes.c_int32),
        ("scale_mode", ctypes.c_int32), ("weight_format", ctypes.c_int32),
        ("static_scale", ctypes.c_void_p), ("weights", ctypes.c_void_p), ("s_w", ctypes.c_void_p),
        ("sw_stride", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
        ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
        ("y", ctypes.c_void_p), ("ldy", ctypes.c_int64),
        ("x8_out", ctypes.c_void_p), ("ldx8_out", ctypes.c_int64), ("s_x_out", ctypes.c_void_p),
    ]

_lib = None


class W4A8Error(RuntimeError):
    def __init__(self, fn, status):
        self.status = status
        super().__init__("%s failed: %d (%s)" % (fn, status, status_string(status)))


def lib():
    """The loaded shared library with argument types set.  Raises when it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "CUDA library %s is missing: build it with "
            "`python -m paper_2505_14638_b200.build` (there is no fallback path)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    c = ctypes
    p, i64, i32, sz = c.c_void_p, c.c_int64, c.c_int, c.c_size_t
    L.w4a8_quantize_act.restype = i32
    L.w4a8_quantize_act.argtypes = [p, i64, i64, i64, p, i64, p, i32, p, p]
    L.w4a8_linear_w4a16.restype = i32
    L.w4a8_linear_w4a16.argtypes = [p, i64, i64, p, p, p, p, i32, i64, i64, p, i64, i32, p, sz, p]
    L.w4a8_linear_w4a16_tiled.restype = i32
    L.w4a8_linear_w4a16_tiled.argtypes = [p, i64, i64, p, i32, p, i32, i64, i64, p, i64, i32, p]
    L.w4a8_linear_w4a16_workspace_bytes.restype = sz
    L.w4a8_linear_w4a16_workspace_bytes.argtypes = [i64, i64, i64]
    L.w4a8_silu_mul_quantize.restype = i32
    L.w4a8_silu_mul_quantize.argtypes = [p, i64, i64, i64, p, i64, p, i32, p, p, i64, p]
    L.w4a8_dequant_weight.restype = i32
    L.w4a8_dequant_weight.argtypes = [p, p, p, i64, i64, i32, p, p]
    L.w4a8_linear.restype = i32
    L.w4a8_linear.argtypes = [p, i64, p, i64, p, p, p, i32, p, i32, i64, i64, i32, p, i64, i32, p, sz, p]
    L.w4a8_linear_workspace_bytes.restype = sz
    L.w4a8_linear_workspace_bytes.argtypes = [i64, i64, i64, i32]
    L.w4a8_prepack_bytes.restype = sz
    L.w4a8_prepack_bytes.argtypes = [i64, i64, i32]
    L.w4a8_prepack_weight.restype = i32
    L.w4a8_prepack_weight.argtypes = [p, p, p, i64, i64, i32, i32, p, sz, p]
    L.w4a8_linear_ex.restype = i32
    L.w4a8_linear_ex.argtypes = [p, i64, p, i64, p, p, p, p, i32, i64, i64, i32, p, i64, i32, p, sz,
                                 i32, i32, p]
    L.w4a8_linear_static_scratch.restype = i32
    L.w4a8_linear_static_scratch.argtypes = [p, i64, p, i64, p, p, p, p, i32, i64, i64, i32, p, i64, i32, i32, p]
    L.w4a8_dequant_weight_gidx.restype = i32
    L.w4a8_dequant_weight_gidx.argtypes = [p, p, p, p, i64, i64, i64, p, p]
    L.w4a8_hessian_accumulate.restype = i32
    L.w4a8_hessian_accumulate.argtypes = [p, i64, i64, i64, p, i32, p]
    L.w4a8_hessian_prepare.restype = i32
    L.w4a8_hessian_prepare.argtypes = [p, i64, p, ctypes.c_float, p, p, p]
    L.w4a8_prepack_fp8.restype = i32
    L.w4a8_prepack_fp8.argtypes = [p, i64, i64, p, sz, p]
    L.w4a8_linear_gidx.restype = i32
    L.w4a8_linear_gidx.argtypes = [p, i64, p, i64, p, p, p, p, p, i32, i64, i64, i32, p, i64, i32, p, sz, p]
    L.w4a8_linear_w8a8.restype = i32
    L.w4a8_linear_w8a8.argtypes = [p, i64, p, i64, p, p, i32, i64, i64, p, i64, i32, p, sz, p]
    L.w4a8_linear_ex_workspace_bytes.restype = sz
    L.w4a8_linear_ex_workspace_bytes.argtypes = [i64, i64, i64, i32, i32]
    L.w4a8_quantize_weight_rtn.restype = i32
    L.w4a8_quantize_weight_rtn.argtypes = [p, i64, i64, i32, i32, i32, i32, p, p, p, p, p]
    L.w4a8_gar_workspace_bytes.restype = sz
    L.w4a8_gar_workspace_bytes.argtypes = [i64]
    L.w4a8_gar_permutation.restype = i32
    L.w4a8_gar_permutation.argtypes = [p, i64, i32, p, p, sz, p]
    L.w4a8_dpq_workspace_bytes.restype = sz
    L.w4a8_dpq_workspace_bytes.argtypes = [i64, i64]
    L.w4a8_dpq_quantize.restype = i32
    L.w4a8_dpq_quantize.argtypes = [p, i64, i64, i32, p, p, i32, i32, i32, p, p, p, p, p, sz, p]
    L.w4a8_forward_host.restype = i32
    L.w4a8_forward_host.argtypes = [p, i64, p, p, p, i32, p, i32, i64, i64, i32, p, p, p, p, p, p, sz, p]
    L.w4a8_linear_chain_workspace_bytes.restype = sz
    L.w4a8_linear_chain_workspace_bytes.argtypes = [c.POINTER(ChainProblem), i32]
    L.w4a8_linear_chain.restype = i32
    L.w4a8_linear_chain.argtypes = [c.POINTER(ChainProblem), i32, p, sz, i32, p]
    L.w4a8_host_buffer_device_pointer.restype = i32
    L.w4a8_host_buffer_device_pointer.argtypes = [p, c.POINTER(c.c_void_p)]
    L.w4a8_selftest_bounded_wait.restype = i32
    L.w4a8_selftest_bounded_wait.argtypes = [c.c_uint64, p, p]
    L.w4a8_query_device_status.restype = i32
    L.w4a8_query_device_status.argtypes = [c.POINTER(c.c_uint)]
    L.w4a8_launch_count.restype = c.c_uint64
    L.w4a8_launch_count.argtypes = []
    L.w4a8_status_string.restype = c.c_char_p
    L.w4a8_status_string.argtypes = [i32]
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().w4a8_status_string(int(status)).decode()


def launch_count() -> int:
    return int(lib().w4a8_launch_count())


def query_device_status() -> int:
    """Synchronises; returns the device status bit mask (0 = clean) and clears it."""
    flags = ctypes.c_uint(0)
    rc = lib().w4a8_query_device_status(ctypes.byref(flags))
    if rc not in (OK, ERR_TIMEOUT, ERR_BAD_SHAPE):
        raise W4A8Error("w4a8_query_device_status", rc)
    return int(flags.value)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    """Handle of torch's current CUDA stream on the current device (the raw getter when this torch
    has it: the Stream object route costs about ten microseconds per call)."""
    import torch
    raw = getattr(torch._C, "_cuda_getCurrentRawStream", None)
    if raw is not None:
        return ctypes.c_void_p(raw(torch.cuda.current_device()))
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(fn, rc):
    if rc != OK:
        raise W4A8Error(fn, rc)


def quantize_act(x, scale_mode=SCALE_EXACT, static_scale=None, out=None):
    """w4a8_quantize_act: x BF16 [M, K] (row stride in elements = x.stride(0)).
    Returns (x8 uint8 [M, K], s_x float32 [M])."""
    import torch
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    if out is None:
        x8 = torch.empty((M, K), dtype=torch.uint8, device=x.device)
        s_x = torch.empty((M,), dtype=torch.float32, device=x.device)
    else:
        x8, s_x = out
    rc = lib().w4a8_quantize_act(_ptr(x), M, K, x.stride(0), _ptr(x8), x8.stride(0), _ptr(s_x),
                                 int(scale_mode), _ptr(static_scale), _stream())
    _check("w4a8_quantize_act", rc)
    return x8, s_x


def linear_w4a16(x, codes, gscale, gzero, s_w, out=None, out_dtype=OUT_BF16, workspace=None):
    """w4a8_linear_w4a16: x BF16 [M, K]; canonical device weights.  Returns Y [M, N]."""
    import torch
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    N = codes.shape[0]
    if out is None:
        dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
        out = torch.empty((M, N), dtype=dt, device=x.device)
    nb = int(lib().w4a8_linear_w4a16_workspace_bytes(M, N, K))
    if workspace is None:
        workspace = torch.empty((max(nb, 16),), dtype=torch.uint8, device=x.device)
    rc = lib().w4a8_linear_w4a16(_ptr(x), x.stride(0), M, _ptr(codes), _ptr(gscale), _ptr(gzero), _ptr(s_w),
                                 0 if s_w.numel() == 1 else 1, N, K, _ptr(out), out.stride(0), int(out_dtype),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(), _stream())
    _check("w4a8_linear_w4a16", rc)
    return out


def linear_w4a16_tiled(x, tw, out=None, out_dtype=OUT_BF16):
    """w4a8_linear_w4a16_tiled: x BF16 [M, K]; tw a TiledWeight in the sign-magnitude format.  Returns Y [M, N]."""
    import torch
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    assert K == tw.K
    if out is None:
        dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
        out = torch.empty((M, tw.N), dtype=dt, device=x.device)
    rc = lib().w4a8_linear_w4a16_tiled(_ptr(x), x.stride(0), M, _ptr(tw.buf), tw.fmt, _ptr(tw.s_w),
                                       0 if tw.s_w.numel() == 1 else 1, tw.N, K, _ptr(out), out.stride(0),
                                       int(out_dtype), _stream())
    _check("w4a8_linear_w4a16_tiled", rc)
    return out


def silu_mul_quantize(gate_up, scale_mode=SCALE_EXACT, static_scale=None, out=None, h_out=None):
    """w4a8_silu_mul_quantize: gate_up BF16 [M, 2F] (gate first, up second).
    Returns (x8 uint8 [M, F], s_x float32 [M]); h_out (BF16 [M, F]) optionally receives h."""
    import torch
    assert gate_up.is_cuda and gate_up.dtype == torch.bfloat16 and gate_up.dim() == 2 and gate_up.stride(1) == 1
    M, F2 = gate_up.shape
    F = F2 // 2
    if out is None:
        x8 = torch.empty((M, F), dtype=torch.uint8, device=gate_up.device)
        s_x = torch.empty((M,), dtype=torch.float32, device=gate_up.device)
    else:
        x8, s_x = out
    rc = lib().w4a8_silu_mul_quantize(_ptr(gate_up), M, F, gate_up.stride(0), _ptr(x8), x8.stride(0), _ptr(s_x),
                                      int(scale_mode), _ptr(static_scale), _ptr(h_out),
                                      0 if h_out is None else h_out.stride(0), _stream())
    _check("w4a8_silu_mul_quantize", rc)
    return x8, s_x


def dequant_weight(codes, gscale, gzero=None, out=None):
    """w4a8_dequant_weight: codes uint8 [N, K/2], gscale BF16 [N, K/128], gzero uint8 or None.
    Returns E4M3 bytes uint8 [N, K]."""
    import torch
    N, Kh = codes.shape
    K = Kh * 2
    w8 = out if out is not None else torch.empty((N, K), dtype=torch.uint8, device=codes.device)
    rc = lib().w4a8_dequant_weight(_ptr(codes), _ptr(gscale), _ptr(gzero), N, K, GROUP, _ptr(w8),
                                   _stream())
    _check("w4a8_dequant_weight", rc)
    return w8


def linear_workspace_bytes(M, N, K, algo=ALGO_AUTO, split_k=0, weight_format=FMT_CANONICAL) -> int:
    if weight_format != FMT_CANONICAL or (algo == ALGO_AUTO and split_k == 0):
        return int(lib().w4a8_linear_workspace_bytes(M, N, K, weight_format))
    return int(lib().w4a8_linear_ex_workspace_bytes(M, N, K, algo, split_k))


class TiledWeight:
    """Weights re-laid out by w4a8_prepack_weight (FMT_TILED or FMT_TILED_SIGNMAG)."""

    def __init__(self, buf, fmt, N, K, s_w):
        self.buf, self.fmt, self.N, self.K, self.s_w = buf, fmt, N, K, s_w


def prepack_weight(codes, gscale, gzero, s_w, weight_format=None):
    """w4a8_prepack_weight: canonical device arrays -> TiledWeight.  Default format: the
    sign-magnitude one for symmetric storage (gzero None), the generic tiled one otherwise."""
    import torch
    if weight_format is None:
        weight_format = FMT_TILED_SIGNMAG if gzero is None else FMT_TILED
    N, Kh = codes.shape
    K = Kh * 2
    nbytes = int(lib().w4a8_prepack_bytes(N, K, weight_format))
    buf = torch.empty((nbytes,), dtype=torch.uint8, device=codes.device)
    rc = lib().w4a8_prepack_weight(_ptr(codes), _ptr(gscale), _ptr(gzero), N, K, GROUP,
                                   int(weight_format), _ptr(buf), nbytes, _stream())
    _check("w4a8_prepack_weight", rc)
    return TiledWeight(buf, weight_format, N, K, s_w)


def hessian_accumulate(x, H=None):
    """w4a8_hessian_accumulate: x BF16 [T, K] on the device; returns H float32 [K, K] (H = X^T X, added to H if given)."""
    import torch
    T, K = x.shape
    acc = H is not None
    if H is None:
        H = torch.empty((K, K), dtype=torch.float32, device=x.device)
    _check("w4a8_hessian_accumulate", lib().w4a8_hessian_accumulate(_ptr(x), T, K, x.stride(0), _ptr(H), int(acc), _stream()))
    return H


def hessian_prepare(H, perm=None, damp=0.01):
    """w4a8_hessian_prepare: the Hessian in processing order with the dead-feature rule and the dampening."""
    import torch
    K = H.shape[0]
    out = torch.empty_like(H)
    scratch = torch.empty((1,), dtype=torch.float32, device=H.device)
    _check("w4a8_hessian_prepare", lib().w4a8_hessian_prepare(_ptr(H), K, _ptr(perm), ctypes.c_float(damp), _ptr(out),
                                                             _ptr(scratch), _stream()))
    return out


def prepack_fp8(w8, s_w):
    """w4a8_prepack_fp8: FP8 E4M3 weights [N, K] (uint8) -> TiledWeight of format FMT_TILED_FP8, the W8A8
    comparison scheme for LinearChain."""
    import torch
    N, K = w8.shape
    buf = torch.empty((N * K,), dtype=torch.uint8, device=w8.device)
    _check("w4a8_prepack_fp8", lib().w4a8_prepack_fp8(_ptr(w8), N, K, _ptr(buf), N * K, _stream()))
    return TiledWeight(buf, FMT_TILED_FP8, N, K, s_w)


def new_workspace(M, N, K, weight_format=FMT_CANONICAL, device="cuda"):
    """Zero-filled workspace of the size w4a8_linear needs (at least 16 bytes)."""
    import torch
    need = linear_workspace_bytes(M, N, K, weight_format=weight_format)
    return torch.zeros((max(need, 16),), dtype=torch.uint8, device=device)


def linear(x8, s_x, codes, gscale, gzero, s_w, out_dtype=OUT_BF16, out=None, workspace=None,
           algo=ALGO_AUTO, split_k=0):
    """w4a8_linear / w4a8_linear_ex on canonical weights: returns Y [M, N] (BF16 or FP32)."""
    import torch
    M, K = x8.shape
    N = codes.shape[0]
    if out is None:
        dt = torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32
        out = torch.empty((M, N), dtype=dt, device=x8.device)
    need = linear_workspace_bytes(M, N, K, algo, split_k)
    if need and (workspace is None or workspace.numel() * workspace.element_size() < need):
        workspace = torch.empty((need,), dtype=torch.uint8, device=x8.device)
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    sw_stride = 0 if s_w.numel() == 1 else 1
    L = lib()
    if algo == ALGO_AUTO and split_k == 0:
        rc = L.w4a8_linear(_ptr(x8), x8.stride(0), _ptr(s_x), M, _ptr(codes), _ptr(gscale),
                           _ptr(gzero), FMT_CANONICAL, _ptr(s_w), sw_stride, N, K, GROUP, _ptr(out),
                           out.stride(0), int(out_dtype), _ptr(workspace), wbytes, _stream())
        _check("w4a8_linear", rc)
    else:
        rc = L.w4a8_linear_ex(_ptr(x8), x8.stride(0), _ptr(s_x), M, _ptr(codes), _ptr(gscale),
                              _ptr(gzero), _ptr(s_w), sw_stride, N, K, GROUP, _ptr(out),
                              out.stride(0), int(out_dtype), _ptr(workspace), wbytes, int(algo),
                              int(split_k), _stream())
        _check("w4a8_linear_ex", rc)
    return out


STATIC_SCRATCH_BYTES = 4 << 20


def linear_static_scratch(x8, s_x, codes, gscale, gzero, s_w, out_dtype=OUT_BF16, out=None, split_k=0):
    """w4a8_linear_static_scratch: the canonical-weight linear whose split-K partial sums live in
    an array built into the library, for callers that may not allocate or pass a workspace.
    `out` should be supplied by such callers; one is created here only as a convenience."""
    import torch
    M, K = x8.shape
    N = codes.shape[0]
    if out is None:
        dt = torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32
        out = torch.empty((M, N), dtype=dt, device=x8.device)
    rc = lib().w4a8_linear_static_scratch(
        _ptr(x8), x8.stride(0), _ptr(s_x), M, _ptr(codes), _ptr(gscale), _ptr(gzero), _ptr(s_w),
        0 if s_w.numel() == 1 else 1, N, K, GROUP, _ptr(out), out.stride(0), int(out_dtype),
        int(split_k), _stream())
    _check("w4a8_linear_static_scratch", rc)
    return out


def linear_tiled(x8, s_x, tw, out_dtype=OUT_BF16, out=None, workspace=None):
    """w4a8_linear on a TiledWeight.  `workspace` must come from new_workspace (zero-filled once);
    one is created when none is given."""
    import torch
    M, K = x8.shape
    assert K == tw.K
    if out is None:
        dt = torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32
        out = torch.empty((M, tw.N), dtype=dt, device=x8.device)
    if workspace is None:
        workspace = new_workspace(M, tw.N, K, tw.fmt, x8.device)
    rc = lib().w4a8_linear(_ptr(x8), x8.stride(0), _ptr(s_x), M, _ptr(tw.buf), None, None, tw.fmt,
                           _ptr(tw.s_w), 0 if tw.s_w.numel() == 1 else 1, tw.N, K, GROUP, _ptr(out),
                           out.stride(0), int(out_dtype), _ptr(workspace),
                           workspace.numel() * workspace.element_size(), _stream())
    _check("w4a8_linear", rc)
    return out


def dequant_weight_gidx(codes, gscale, gzero, g_idx, out=None):
    """w4a8_dequant_weight_gidx: per-column group index g_idx int32 [K]; returns E4M3 bytes [N, K]."""
    import torch
    N, Kh = codes.shape
    K = Kh * 2
    w8 = out if out is not None else torch.empty((N, K), dtype=torch.uint8, device=codes.device)
    rc = lib().w4a8_dequant_weight_gidx(_ptr(codes), _ptr(gscale), _ptr(gzero), _ptr(g_idx), N, K,
                                        gscale.shape[1], _ptr(w8), _stream())
    _check("w4a8_dequant_weight_gidx", rc)
    return w8


def linear_gidx(x8, s_x, codes, gscale, gzero, g_idx, s_w, out_dtype=OUT_BF16, out=None):
    """w4a8_linear_gidx: the linear layer on activation-ordered weights (per-column group index) in one kernel."""
    import torch
    M, K = x8.shape
    N = codes.shape[0]
    if out is None:
        dt = torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32
        out = torch.empty((M, N), dtype=dt, device=x8.device)
    nb = linear_workspace_bytes(M, N, K, ALGO_UMMA, 0)
    ws = torch.empty((max(nb, 16),), dtype=torch.uint8, device=x8.device)
    rc = lib().w4a8_linear_gidx(_ptr(x8), x8.stride(0), _ptr(s_x), M, _ptr(codes), _ptr(gscale), _ptr(gzero),
                                _ptr(g_idx), _ptr(s_w), 0 if s_w.numel() == 1 else 1, N, K, GROUP, _ptr(out),
                                out.stride(0), int(out_dtype), _ptr(ws), nb, _stream())
    _check("w4a8_linear_gidx", rc)
    return out


def linear_w8a8(x8, s_x, w8, s_w, out_dtype=OUT_BF16, out=None):
    """w4a8_linear_w8a8: FP8 activations [M, K] x FP8 weights [N, K] (uint8 E4M3 bytes)."""
    import torch
    M, K = x8.shape
    N = w8.shape[0]
    if out is None:
        dt = torch.bfloat16 if out_dtype == OUT_BF16 else torch.float32
        out = torch.empty((M, N), dtype=dt, device=x8.device)
    nb = linear_workspace_bytes(M, N, K, ALGO_UMMA, 0)
    ws = torch.empty((max(nb, 16),), dtype=torch.uint8, device=x8.device)
    rc = lib().w4a8_linear_w8a8(_ptr(x8), x8.stride(0), _ptr(s_x), M, _ptr(w8), _ptr(s_w),
                                0 if s_w.numel() == 1 else 1, N, K, _ptr(out), out.stride(0), int(out_dtype),
                                _ptr(ws), nb, _stream())
    _check("w4a8_linear_w8a8", rc)
    return out


def quantize_weight_rtn(W, symmetric=True, pow2=False, per_channel=False):
    """w4a8_quantize_weight_rtn: W float32 [N, K] on the device.
    Returns (codes, gscale BF16, gzero or None, s_w)."""
    import torch
    N, K = W.shape
    dev = W.device
    codes = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
    gscale = torch.empty((N, K // GROUP), dtype=torch.bfloat16, device=dev)
    gzero = None if symmetric else torch.empty((N, K // GROUP), dtype=torch.uint8, device=dev)
    s_w = torch.empty((N if per_channel else 1,), dtype=torch.float32, device=dev)
    rc = lib().w4a8_quantize_weight_rtn(_ptr(W), N, K, GROUP, int(symmetric), int(pow2),
                                        int(per_channel), _ptr(codes), _ptr(gscale), _ptr(gzero),
                                        _ptr(s_w), _stream())
    _check("w4a8_quantize_weight_rtn", rc)
    return codes, gscale, gzero, s_w


def gar_permutation(hdiag):
    """w4a8_gar_permutation: hdiag float32 [K] on the device -> int32 [K] processing order."""
    import torch
    K = hdiag.numel()
    perm = torch.empty((K,), dtype=torch.int32, device=hdiag.device)
    ws = torch.empty((lib().w4a8_gar_workspace_bytes(K),), dtype=torch.uint8, device=hdiag.device)
    rc = lib().w4a8_gar_permutation(_ptr(hdiag), K, GROUP, _ptr(perm), _ptr(ws), ws.numel(), _stream())
    _check("w4a8_gar_permutation", rc)
    return perm


def dpq_quantize(W, U, perm=None, symmetric=False, mse_steps=0, per_channel=False):
    """w4a8_dpq_quantize: W float32 [N, K], U float32 [K, K] (processing order), perm int32 [K] or
    None, all on the device.  Returns (codes, gscale BF16, gzero or None, s_w)."""
    import torch
    N, K = W.shape
    dev = W.device
    codes = torch.empty((N, K // 2), dtype=torch.uint8, device=dev)
    gscale = torch.empty((N, K // GROUP), dtype=torch.bfloat16, device=dev)
    gzero = None if symmetric else torch.empty((N, K // GROUP), dtype=torch.uint8, device=dev)
    s_w = torch.empty((N if per_channel else 1,), dtype=torch.float32, device=dev)
    ws = torch.empty((lib().w4a8_dpq_workspace_bytes(N, K),), dtype=torch.uint8, device=dev)
    rc = lib().w4a8_dpq_quantize(_ptr(W), N, K, GROUP, _ptr(U), _ptr(perm), int(symmetric), int(mse_steps),
                                 int(per_channel), _ptr(codes), _ptr(gscale), _ptr(gzero), _ptr(s_w), _ptr(ws),
                                 ws.numel(), _stream())
    _check("w4a8_dpq_quantize", rc)
    return codes, gscale, gzero, s_w


def host_buffer_device_pointer(t):
    """w4a8_host_buffer_device_pointer: device-side address of a pinned host tensor."""
    out = ctypes.c_void_p(0)
    _check("w4a8_host_buffer_device_pointer",
           lib().w4a8_host_buffer_device_pointer(ctypes.c_void_p(t.data_ptr()), ctypes.byref(out)))
    return out.value


def _addr(t):
    """Address a kernel can use: the tensor's own for device tensors, the mapped one for pinned host tensors."""
    if t is None:
        return None
    return t.data_ptr() if t.is_cuda else host_buffer_device_pointer(t)


class LinearChain:
    """w4a8_linear_chain: a list of decode-sized layers run by ONE persistent launch.

    Build it once from problem descriptions (dicts with the keys x, weight, y and optionally
    kind, depends_on, scale_mode, static_scale, x8_out, s_x_out), call it as often as wanted: the
    argument array and the zero-filled workspace are kept.  x: BF16 [M, K] (or [M, 2K] for the
    gated kind), weight: TiledWeight, y: BF16 or FP32 [M, N]; on one device, except that x and y may
    be pinned host tensors (the kernel then reads / writes them over the bus)."""

    def __init__(self, problems, groups=0, workspace=None):
        import torch
        n = len(problems)
        self.arr = (ChainProblem * n)()
        self.keep = problems          # keeps the tensors alive
        for i, d in enumerate(problems):
            x, tw, y = d["x"], d["weight"], d["y"]
            kind = d.get("kind", CHAIN_INPUT_PLAIN)
            assert x.dtype == torch.bfloat16 and x.stride(1) == 1 and y.stride(1) == 1
            q = self.arr[i]
            q.x_bf16, q.ldx = _addr(x), x.stride(0)
            q.input_kind, q.depends_on = kind, d.get("depends_on", -1)
            q.scale_mode, q.weight_format = d.get("scale_mode", SCALE_EXACT), tw.fmt
            q.static_scale = _addr(d.get("static_scale"))
            q.weights, q.s_w = tw.buf.data_ptr(), tw.s_w.data_ptr()
            q.sw_stride = 0 if tw.s_w.numel() == 1 else 1
            q.out_dtype = OUT_FP32 if y.dtype == torch.float32 else OUT_BF16
            q.M, q.N, q.K = x.shape[0], tw.N, tw.K
            q.y, q.ldy = _addr(y), y.stride(0)
            x8o = d.get("x8_out")
            q.x8_out, q.ldx8_out = _addr(x8o), (0 if x8o is None else x8o.stride(0))
            q.s_x_out = _addr(d.get("s_x_out"))
        self.n = n
        self.groups = int(groups)
        need = int(lib().w4a8_linear_chain_workspace_bytes(self.arr, n))
        if need == 0:
            _check("w4a8_linear_chain", lib().w4a8_linear_chain(self.arr, n, None, 0, self.groups, None))
        self.need = need
        dev = problems[0]["x"].device if problems[0]["x"].is_cuda else problems[0]["weight"].buf.device
        self.ws = workspace if workspace is not None else torch.zeros((need,), dtype=torch.uint8, device=dev)
        self._fn = lib().w4a8_linear_chain
        self._wsp = ctypes.c_void_p(self.ws.data_ptr())
        self._wsn = self.ws.numel()

    def __call__(self):
        rc = self._fn(self.arr, self.n, self._wsp, self._wsn, self.groups, _stream())
        if rc != 0:
            _check("w4a8_linear_chain", rc)


def selftest_bounded_wait(limit_ns):
    """w4a8_selftest_bounded_wait: returns the device-measured duration (ns) of a wait that runs out."""
    import torch
    out = torch.zeros((1,), dtype=torch.int64, device="cuda")
    _check("w4a8_selftest_bounded_wait", lib().w4a8_selftest_bounded_wait(int(limit_ns), _ptr(out), _stream()))
    torch.cuda.synchronize()
    return int(out.item())


class HostForward:
    """w4a8_forward_host with its device scratch buffers allocated once: activations come from
    and results go to pinned host memory, weights stay on the device.  `weight` is either a
    TiledWeight or a tuple (codes, gscale, gzero, s_w) of canonical device arrays."""

    def __init__(self, M, weight):
        import torch
        self.M = M
        self.set_weight(weight)
        dev = self.wbuf.device
        self.x_dev = torch.empty((M, self.K), dtype=torch.bfloat16, device=dev)
        self.x8 = torch.empty((M, self.K), dtype=torch.uint8, device=dev)
        self.s_x = torch.empty((M,), dtype=torch.float32, device=dev)
        self.y_dev = torch.empty((M, self.N), dtype=torch.bfloat16, device=dev)
        self.ws = new_workspace(M, self.N, self.K, self.fmt, dev)
        self.y_host = torch.empty((M, self.N), dtype=torch.bfloat16).pin_memory()
        self.h2d_bytes = M * self.K * 2
        self.d2h_bytes = M * self.N * 2

    def set_weight(self, weight):
        self._args = None
        if isinstance(weight, TiledWeight):
            self.wbuf, self.gscale, self.gzero, self.s_w = weight.buf, None, None, weight.s_w
            self.fmt, self.N, self.K = weight.fmt, weight.N, weight.K
        else:
            self.wbuf, self.gscale, self.gzero, self.s_w = weight
            self.fmt = FMT_CANONICAL
            self.N, self.K = self.wbuf.shape[0], self.wbuf.shape[1] * 2

    def __call__(self, x_host):
        """x_host: pinned BF16 [M, K] host tensor.  Enqueues everything; returns the pinned
        output tensor, valid after the current stream is synchronised."""
        if self._args is None:   # everything but the input pointer and the stream is fixed per weight
            self._args = (self.M, _ptr(self.wbuf), _ptr(self.gscale), _ptr(self.gzero), self.fmt, _ptr(self.s_w),
                          0 if self.s_w.numel() == 1 else 1, self.N, self.K, GROUP,
                          ctypes.c_void_p(self.y_host.data_ptr()), _ptr(self.x_dev), _ptr(self.x8), _ptr(self.s_x),
                          _ptr(self.y_dev), _ptr(self.ws), self.ws.numel())
            self._fn = lib().w4a8_forward_host
        rc = self._fn(ctypes.c_void_p(x_host.data_ptr()), *self._args, _stream())
        if rc != 0:
            _check("w4a8_forward_host", rc)
        return self.y_host
