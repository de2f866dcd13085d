"""Host-side checks of the C-ABI library: it loads, exports what include/w4a8.h declares, and
rejects bad arguments before touching a device (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2505_14638_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return binding.lib()


def test_exports_every_declared_symbol(L):
    hdr = open(os.path.join(ROOT, "include", "w4a8.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(w4a8_[a-z0-9_]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name
    assert 'extern "C"' in open(os.path.join(ROOT, "include", "w4a8.h")).read()


def test_status_strings(L):
    assert binding.status_string(0) == "ok"
    for code in range(-7, 0):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert binding.status_string(-99) == "unknown status"


def test_workspace_and_prepack_size_queries_are_host_only(L):
    assert L.w4a8_prepack_bytes(14336, 4096, binding.FMT_TILED_SIGNMAG) == 14336 * 32 * 66
    assert L.w4a8_prepack_bytes(14336 + 16, 4096, binding.FMT_TILED) == (14336 + 16) * 32 * 68
    assert L.w4a8_prepack_bytes(14336, 4096, binding.FMT_CANONICAL) == 0
    assert binding.linear_workspace_bytes(16, 14336, 4096, weight_format=binding.FMT_TILED_SIGNMAG) == 65536 + 160 * 128 * 128 * 4   # control area of fixed size (counters, placement state), partial tiles
    ws = binding.linear_workspace_bytes(2048, 4096, 4096, weight_format=binding.FMT_TILED_SIGNMAG)
    assert ws >= 2 * 8 * 32 * 4 + 2 * 148 * 256 * 128 * 4
    assert binding.linear_workspace_bytes(2048, 4096, 4096) == 0          # large M: no split
    ws = binding.linear_workspace_bytes(16, 14336, 4096)
    assert ws % (16 * 14336 * 4) == 0 and ws > 0                          # S partial tiles
    assert binding.linear_workspace_bytes(16, 14336, 4096, binding.ALGO_UMMA, 4) == 4 * 16 * 14336 * 4
    assert binding.linear_workspace_bytes(16, 14336, 4096, binding.ALGO_SIMT, 0) == 0
    assert binding.linear_workspace_bytes(16, 14336, 100) == 0            # invalid K


def _fake(addr=0x1000):
    return ctypes.c_void_p(addr)


def test_quantize_act_rejects_bad_arguments(L):
    p = _fake()
    f = L.w4a8_quantize_act
    assert f(None, 4, 128, 128, p, 128, p, 0, None, None) == binding.ERR_INVALID_ARG
    assert f(p, 0, 128, 128, p, 128, p, 0, None, None) == binding.ERR_INVALID_ARG
    assert f(p, 4, 128, 128, p, 128, p, 7, None, None) == binding.ERR_INVALID_ARG
    assert f(p, 4, 100, 128, p, 128, p, 0, None, None) == binding.ERR_BAD_SHAPE
    assert f(p, 4, 128, 64, p, 128, p, 0, None, None) == binding.ERR_BAD_SHAPE
    assert f(_fake(0x1004), 4, 128, 128, p, 128, p, 0, None, None) == binding.ERR_BAD_ALIGNMENT
    assert f(p, 4, 128, 132, p, 128, p, 0, None, None) == binding.ERR_BAD_ALIGNMENT


def test_dequant_rejects_bad_arguments(L):
    p = _fake()
    f = L.w4a8_dequant_weight
    assert f(None, p, None, 16, 128, 128, p, None) == binding.ERR_INVALID_ARG
    assert f(p, p, None, 16, 128, 64, p, None) == binding.ERR_BAD_SHAPE
    assert f(p, p, None, 16, 192, 128, p, None) == binding.ERR_BAD_SHAPE
    assert f(_fake(0x1008), p, None, 16, 128, 128, p, None) == binding.ERR_BAD_ALIGNMENT


def test_linear_rejects_bad_arguments(L):
    p = _fake()
    f = L.w4a8_linear

    def call(x8=p, ldx8=4096, s_x=p, M=16, codes=p, gs=p, gz=None, fmt=0, s_w=p, sws=0, N=14336, K=4096,
             group=128, y=p, ldy=14336, od=0, ws=p, wsb=1 << 30):
        return f(x8, ldx8, s_x, M, codes, gs, gz, fmt, s_w, sws, N, K, group, y, ldy, od, ws, wsb, None)

    assert call(fmt=3) == binding.ERR_INVALID_ARG
    assert call(gs=None) == binding.ERR_INVALID_ARG
    assert call(fmt=2, gs=None, M=512, ws=None, wsb=0) == binding.ERR_WORKSPACE_TOO_SMALL
    assert call(fmt=1, gs=None, M=512, wsb=1024) == binding.ERR_WORKSPACE_TOO_SMALL

    assert call(x8=None) == binding.ERR_INVALID_ARG
    assert call(M=0) == binding.ERR_INVALID_ARG
    assert call(sws=2) == binding.ERR_INVALID_ARG
    assert call(od=5) == binding.ERR_INVALID_ARG
    assert call(K=4000) == binding.ERR_BAD_SHAPE
    assert call(group=64) == binding.ERR_BAD_SHAPE
    assert call(N=14337, ldy=14352) == binding.ERR_BAD_SHAPE
    assert call(ldx8=2048) == binding.ERR_BAD_SHAPE
    assert call(ldy=1024) == binding.ERR_BAD_SHAPE
    assert call(x8=_fake(0x1001)) == binding.ERR_BAD_ALIGNMENT
    assert call(ldx8=4100) == binding.ERR_BAD_ALIGNMENT
    assert call(ws=None, wsb=0) == binding.ERR_WORKSPACE_TOO_SMALL
    assert call(wsb=16) == binding.ERR_WORKSPACE_TOO_SMALL
    g = L.w4a8_linear_ex
    assert g(p, 4096, p, 16, p, p, None, p, 0, 14336, 4096, 128, p, 14336, 0, p, 1 << 30, 9, 0, None) \
        == binding.ERR_INVALID_ARG
    assert g(p, 4096, p, 16, p, p, None, p, 0, 14336, 4096, 128, p, 14336, 0, p, 1 << 30, 2, 5, None) \
        == binding.ERR_BAD_SHAPE                                            # 5 does not divide K/128


def test_rtn_and_host_forward_reject_bad_arguments(L):
    p = _fake()
    f = L.w4a8_quantize_weight_rtn
    assert f(None, 16, 128, 128, 1, 0, 0, p, p, None, p, None) == binding.ERR_INVALID_ARG
    assert f(p, 16, 128, 128, 0, 0, 0, p, p, None, p, None) == binding.ERR_INVALID_ARG   # asymmetric needs gzero
    assert f(p, 16, 130, 128, 1, 0, 0, p, p, None, p, None) == binding.ERR_BAD_SHAPE
    h = L.w4a8_forward_host
    assert h(None, 4, p, p, None, 0, p, 0, 16, 128, 128, p, p, p, p, p, None, 0, None) == binding.ERR_INVALID_ARG
    assert h(p, 4, p, p, None, 0, p, 0, 16, 100, 128, p, p, p, p, p, None, 0, None) == binding.ERR_BAD_SHAPE
    assert h(p, 4, p, p, None, 9, p, 0, 16, 128, 128, p, p, p, p, p, None, 0, None) == binding.ERR_INVALID_ARG
    k = L.w4a8_prepack_weight
    assert k(None, p, None, 16, 128, 128, 1, p, 1 << 20, None) == binding.ERR_INVALID_ARG
    assert k(p, p, None, 16, 128, 128, 0, p, 1 << 20, None) == binding.ERR_INVALID_ARG      # canonical is not a target
    assert k(p, p, p, 16, 128, 128, 2, p, 1 << 20, None) == binding.ERR_INVALID_ARG          # sign-magnitude needs z = 8
    assert k(p, p, None, 16, 100, 128, 1, p, 1 << 20, None) == binding.ERR_BAD_SHAPE
    assert k(p, p, None, 16, 128, 128, 1, _fake(0x1010), 1 << 20, None) == binding.ERR_BAD_ALIGNMENT
    assert k(p, p, None, 16, 128, 128, 1, p, 100, None) == binding.ERR_WORKSPACE_TOO_SMALL
    assert L.w4a8_query_device_status(None) == binding.ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
