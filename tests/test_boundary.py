"""The C ABI without a GPU: the library loads, exports every symbol the header declares, and its
host-side argument checks return the documented status codes before anything is launched."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_05003_b200 import build, _lib
    build.build()
    return _lib.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "quest.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(quest_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2502_05003_b200 import _lib
    names = declared_functions()
    assert set(names) == set(_lib.EXPORTS), (names, _lib.EXPORTS)
    for n in names:
        assert getattr(lib, n) is not None


def test_python_binding_has_the_same_entry_points():
    import paper_2502_05003_b200 as quest
    for n in ("quest_quantize", "quest_trust_mask", "quest_lowbit_gemm", "quest_linear_fwd",
              "quest_workspace_bytes", "quest_codes_bytes", "quest_alpha_star", "quest_device_status"):
        assert callable(getattr(quest, n))


def test_size_helpers_and_table(lib):
    assert lib.quest_codes_bytes(4096, 2048, 4) == 4096 * 2048 // 2
    assert lib.quest_codes_bytes(8, 128, 1) == 8 * 16
    assert lib.quest_codes_bytes(8, 128, 3) == 8 * 64
    assert lib.quest_codes_bytes(8, 128, 8) == 8 * 128
    assert lib.quest_codes_bytes(8, 128, 9) == 0
    ws = lib.quest_workspace_bytes(4096, 2048, 2048, 4, 4)
    assert ws >= 4096 * 2048 + 2048 * 2048 and ws % 256 == 0
    assert lib.quest_workspace_bytes(16, 16, 48, 4, 4) == 0          # K % 32 != 0
    assert lib.quest_workspace_bytes(16, 16, 33056, 8, 8) == 0       # would overflow int32
    assert abs(lib.quest_alpha_star(1) - 0.7978846) < 1e-7
    assert abs(lib.quest_alpha_star(4) - 2.5140045) < 1e-6
    assert lib.quest_alpha_star(0) == 0.0
    assert lib.quest_status_string(0) == b"ok"
    assert b"bits" in lib.quest_status_string(3)


FAKE = ctypes.c_void_p(0x10000)      # aligned, never dereferenced: every case below fails validation first
F = ctypes.c_float


@pytest.mark.parametrize("kwargs,expected", [
    (dict(x=None), 1), (dict(dtype=7), 5), (dict(bits=0), 3), (dict(bits=9), 3),
    (dict(cols=0), 2), (dict(cols=12), 2), (dict(cols=32768), 2), (dict(rows=-1), 2), (dict(ld=64), 2),
    (dict(g=3), 4), (dict(g=256), 4), (dict(g=0), 4),
    (dict(trust=-0.5), 7), (dict(trust=float("inf")), 7), (dict(trust=float("nan")), 7),
    (dict(x=ctypes.c_void_p(0x10004)), 6), (dict(ld=132, dtype=1), 6), (dict(codes=ctypes.c_void_p(0x10001)), 6),
])
def test_quantize_argument_errors(lib, kwargs, expected):
    a = dict(x=FAKE, dtype=0, rows=4, cols=128, ld=128, bits=4, g=128, trust=1.0, codes=FAKE, scales=FAKE, mask=FAKE)
    a.update(kwargs)
    st = lib.quest_quantize(a["x"], a["dtype"], a["rows"], a["cols"], a["ld"], a["bits"], a["g"], F(a["trust"]),
                            a["codes"], a["scales"], a["mask"], None)
    assert st == expected
    if a["mask"] is not None:
        st = lib.quest_trust_mask(a["x"], a["dtype"], a["rows"], a["cols"], a["ld"], a["bits"], a["g"],
                                  F(a["trust"]), a["mask"], None)
        assert st == (expected if "codes" not in kwargs else st)


def test_trust_mask_requires_mask(lib):
    assert lib.quest_trust_mask(FAKE, 0, 4, 128, 128, 4, 128, F(1.0), None, None) == 1


@pytest.mark.parametrize("kwargs,expected", [
    (dict(xq=None), 1), (dict(y=None, acc=None), 1), (dict(sx=None), 1),
    (dict(bits_x=0), 3), (dict(bits_w=12), 3), (dict(K=16), 2), (dict(K=100), 2), (dict(M=-1), 2),
    (dict(K=33056, bits_x=8, bits_w=8), 9), (dict(K=1 << 20), 2), (dict(y_dtype=5), 5), (dict(ldy=8), 2),
    (dict(ws=None), 8), (dict(ws_bytes=16), 8), (dict(ws=ctypes.c_void_p(0x10010)), 8),
    (dict(xq=ctypes.c_void_p(0x10008)), 6),
])
def test_gemm_argument_errors(lib, kwargs, expected):
    a = dict(xq=FAKE, sx=FAKE, bits_x=4, wq=FAKE, sw=FAKE, bits_w=4, M=64, N=64, K=128, y=FAKE, y_dtype=1, ldy=64,
             acc=FAKE, ws=FAKE, ws_bytes=1 << 20)
    a.update(kwargs)
    st = lib.quest_lowbit_gemm(a["xq"], a["sx"], a["bits_x"], a["wq"], a["sw"], a["bits_w"], a["M"], a["N"], a["K"],
                               a["y"], a["y_dtype"], a["ldy"], a["acc"], a["ws"], a["ws_bytes"], None)
    assert st == expected


def test_linear_fwd_argument_errors(lib):
    def call(**kw):
        a = dict(x=FAKE, w=FAKE, dtype=1, M=64, N=64, K=128, bits=4, g=128, trust=1.0, y=FAKE, y_dtype=1,
                 xq=FAKE, sx=FAKE, mx=FAKE, wq=FAKE, sw=FAKE, mw=FAKE, cached=0, ws=FAKE, ws_bytes=1 << 20)
        a.update(kw)
        return lib.quest_linear_fwd(a["x"], a["w"], a["dtype"], a["M"], a["N"], a["K"], a["bits"], a["g"],
                                    F(a["trust"]), a["y"], a["y_dtype"], a["xq"], a["sx"], a["mx"], a["wq"],
                                    a["sw"], a["mw"], a["cached"], a["ws"], a["ws_bytes"], None)
    assert call(y=None) == 1 and call(xq=None) == 1 and call(w=None) == 1
    assert call(bits=0) == 3 and call(g=96) == 4 and call(K=48) == 2 and call(trust=-1.0) == 7
    assert call(ws_bytes=0) == 8 and call(y_dtype=3) == 5 and call(dtype=4) == 5


def test_valid_call_without_a_gpu_reports_an_error_not_a_crash(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    st = lib.quest_quantize(FAKE, 0, 4, 128, 128, 4, 128, F(1.0), FAKE, FAKE, FAKE, None)
    assert st in (10, 11)
    assert lib.quest_status_string(st)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2502_05003_b200 import _lib
    monkeypatch.setattr(_lib, "_lib", None)
    monkeypatch.setattr(_lib, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        _lib.load()


def test_backward_argument_errors(lib):
    def call(**kw):
        a = dict(dy=FAKE, M=64, N=64, K=128, bits=4, g=128, xq=FAKE, sx=FAKE, mx=FAKE, wq=FAKE, sw=FAKE, mw=FAKE,
                 dx=FAKE, dw=FAKE, out=0, ws=FAKE, ws_bytes=1 << 30)
        a.update(kw)
        return lib.quest_linear_bwd(a["dy"], a["M"], a["N"], a["K"], a["bits"], a["g"], a["xq"], a["sx"], a["mx"],
                                    a["wq"], a["sw"], a["mw"], a["dx"], a["dw"], a["out"], a["ws"], a["ws_bytes"], None)
    assert call(dy=None) == 1 and call(mx=None) == 1 and call(dx=None, dw=None) == 1
    assert call(bits=9) == 3 and call(M=60) == 2 and call(N=0) == 2 and call(K=48) == 2 and call(K=32768) == 2
    assert call(g=96) == 4 and call(g=256) == 4 and call(out=7) == 5
    assert call(dy=ctypes.c_void_p(0x10002)) == 6 and call(ws_bytes=16) == 8 and call(ws=None) == 8
    # the dequantised bfloat16 operands of w and x plus the two masked binary32 products
    assert lib.quest_bwd_workspace_bytes(4096, 2048, 2048) >= (2048 * 2048 + 4096 * 2048) * 2 + (4096 + 2048) * 2048 * 4
    assert lib.quest_bwd_workspace_bytes(60, 64, 128) == 0


def test_fp4_entry_points_validate_on_the_host(lib):
    assert abs(lib.quest_alpha_star_fp4() - 2.9224751) < 1e-6
    q = lambda **kw: lib.quest_quantize_fp4(kw.get("x", FAKE), kw.get("dtype", 1), kw.get("rows", 4), kw.get("cols", 128),
                                            kw.get("ld", 128), kw.get("g", 128), F(kw.get("trust", 1.0)), FAKE, FAKE, FAKE, None)
    assert q(x=None) == 1 and q(dtype=9) == 5 and q(cols=40, ld=40, g=8) == 2 and q(g=48) == 4 and q(trust=-1.0) == 7
    g = lambda **kw: lib.quest_lowbit_gemm_fp4(kw.get("xq", FAKE), FAKE, FAKE, FAKE, kw.get("M", 64), 64, kw.get("K", 128),
                                               FAKE, kw.get("yd", 1), 64, None, kw.get("ws", FAKE), kw.get("wsb", 1 << 20), None)
    assert g(xq=None) == 1 and g(K=100) == 2 and g(yd=4) == 5
    # the packed codes are read by TMA: 16-byte alignment; the scratch arguments are unused (no workspace error)
    assert g(xq=ctypes.c_void_p(FAKE.value + 8)) == 6 and g(ws=None) != 8
