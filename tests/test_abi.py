"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and rejects
bad arguments before touching the device (no compute calls here)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2605_08692_b200 import build, binding
    build.build()
    return binding.lib()


def test_every_declared_symbol_is_exported(L):
    hdr = open(os.path.join(ROOT, "include", "aaac.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(aaac_[a-z_0-9]+)\s*\(", hdr))
    assert {"aaac_act_stats", "aaac_fit_layer", "aaac_pack", "aaac_dequant"} <= names
    from paper_2605_08692_b200 import binding
    assert names == set(binding.EXPORTS)
    for n in names:
        assert hasattr(L, n), n


def test_status_strings(L):
    assert L.aaac_status_string(0) == b"ok"
    for code in range(1, 9):
        assert len(L.aaac_status_string(code)) > 3
    assert b"unknown" in L.aaac_status_string(99)


def test_workspace_sizes(L):
    a = L.aaac_workspace_bytes(0, 512, 512, 256)
    b = L.aaac_workspace_bytes(1, 4096, 4096, 4096)
    assert 0 < a < b
    assert a % 256 == 0 and b % 256 == 0
    assert L.aaac_workspace_bytes(7, 512, 512, 0) == 0
    assert L.aaac_host_workspace_bytes(1, 4096, 4096, 4096) > b + 4096 * 4096 * 4


def test_argument_validation_happens_on_the_host(L):
    P = C.c_void_p
    ok = P(1 << 20)           # non-null, 256-aligned, never dereferenced: every call below fails validation
    odd = P((1 << 20) + 2)
    big = C.c_size_t(1 << 40)
    # aaac_act_stats
    assert L.aaac_act_stats(None, 8, 256, 256, ok, 0, None, ok, big, None) == 1
    assert L.aaac_act_stats(ok, 0, 256, 256, ok, 0, None, ok, big, None) == 3
    assert L.aaac_act_stats(ok, 8, 252, 252, ok, 0, None, ok, big, None) == 3
    assert L.aaac_act_stats(odd, 8, 256, 256, ok, 0, None, ok, big, None) == 4
    assert L.aaac_act_stats(ok, 8, 256, 256, ok, 0, None, ok, C.c_size_t(16), None) == 5
    # aaac_fit_layer
    fit = lambda **kw: L.aaac_fit_layer(kw.get("W", ok), kw.get("N", 64), kw.get("K", 256), kw.get("ldw", 256),
                                        kw.get("mode", 0), kw.get("group", 128), kw.get("I", ok), None, 0, 0,
                                        kw.get("n_outer", 2), kw.get("n_inner", 1), kw.get("init", 1), ok, ok, ok,
                                        None, None, kw.get("ws", ok), kw.get("wsb", big), None)
    assert fit(W=None) == 1
    assert fit(mode=3) == 2
    assert fit(group=64) == 2
    assert fit(mode=1, group=128) == 2
    assert fit(K=192, ldw=192) == 3
    assert fit(ldw=128) == 3
    assert fit(N=0) == 3
    assert fit(n_outer=-1) == 3
    assert fit(init=9) == 2
    assert fit(W=odd) == 4
    assert fit(n_inner=0) == 3
    assert fit(n_outer=1 << 16, n_inner=1 << 8) == 3
    assert fit(I=None) == 1
    assert fit(wsb=C.c_size_t(1024)) == 5
    assert fit(ws=P((1 << 20) + 64)) == 4
    # selection group apart from the scale group: S = g, or S = 16 inside INT4's g = 128
    fits = lambda mode, group, sel: L.aaac_fit_layer_sel(ok, 64, 256, 256, mode, group, sel, ok, None, 0, 0, 2, 1, 1, ok,
                                                         ok, ok, None, None, ok, C.c_size_t(16), None)
    assert fits(0, 128, 16) == 5 and fits(0, 128, 128) == 5 and fits(1, 16, 16) == 5     # pass the checks up to the workspace size
    assert fits(0, 128, 32) == 2 and fits(1, 16, 8) == 2 and fits(1, 16, 128) == 2
    assert L.aaac_pack_sel(ok, 64, 256, 256, 0, 128, 16, ok, ok, ok, ok, ok, ok, None, None, None, ok, big, None) == 1
    assert L.aaac_dequant_sel(ok, ok, None, ok, ok, 64, 256, 0, 128, 16, ok, 256, None) == 1
    assert L.aaac_dequant_sel(ok, ok, ok, ok, ok, 64, 256, 0, 128, 64, ok, 256, None) == 2
    # aaac_prescale_columns
    pre = lambda **kw: L.aaac_prescale_columns(kw.get("W", ok), 64, kw.get("K", 256), 256, kw.get("a", ok), ok, 256,
                                               kw.get("I", None), kw.get("Io", None), None, None)
    assert pre(W=None) == 1 and pre(a=None) == 1 and pre(I=ok) == 1
    assert pre(K=100) == 3 and pre(W=odd) == 4
    # aaac_pack / aaac_dequant
    assert L.aaac_pack(ok, 64, 256, 256, 0, 128, None, ok, ok, ok, ok, ok, None, None, ok, big, None) == 1
    assert L.aaac_pack(ok, 64, 256, 256, 1, 16, ok, ok, ok, ok, None, ok, None, None, ok, big, None) == 1
    assert L.aaac_pack(ok, 64, 250, 256, 0, 128, ok, ok, ok, ok, ok, ok, None, None, ok, big, None) == 3
    assert L.aaac_dequant(None, ok, ok, ok, 64, 256, 0, 128, ok, 256, None) == 1
    assert L.aaac_dequant(ok, ok, ok, ok, 64, 256, 0, 16, ok, 256, None) == 2
    assert L.aaac_dequant(ok, ok, ok, ok, 64, 256, 0, 128, ok, 128, None) == 3
    assert L.aaac_dequant(ok, ok, ok, ok, 64, 256, 0, 128, odd, 256, None) == 4
    # host entry point
    assert L.aaac_quantize_layer_host(None, 64, 256, 0, 128, ok, 8, 2, 0, ok, ok, ok, ok, ok, None, ok, big, None) == 1
    assert L.aaac_quantize_layer_host(ok, 64, 256, 0, 128, ok, 8, 2, 0, ok, ok, ok, ok, ok, None, ok,
                                      C.c_size_t(4096), None) == 5


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2605_08692_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(binding.AaacError):
        binding.workspace_bytes(0, 512, 512)


def test_product_path_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2605_08692_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "aaac_oracle" not in src, f
