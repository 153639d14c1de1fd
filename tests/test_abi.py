"""The C-ABI library loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes as C
import os
import re

from paper_2604_26209_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "hpd.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b((?:hpd|std)_[a-z0-9_]+)\s*\(", src)
    return sorted(set(names))


def test_library_builds_and_exports_all_declared_symbols():
    build.build()
    lib = binding.load()
    decl = _declared()
    assert set(binding.EXPORTS) <= set(decl)
    for name in decl:
        assert hasattr(lib, name), name


def test_argument_checks_need_no_device():
    lib = binding.load()
    bad = binding.HpdGeom(32, 8, 96, 10000.0, 0.1, 16)            # D = 96 is not supported
    assert lib.hpd_rope(C.byref(bad), 4, None, None, None, None, None) == -2
    good = binding.HpdGeom(32, 8, 128, 10000.0, 0.1, 16)
    assert lib.hpd_rope(C.byref(good), 4, None, None, None, None, None) == -1     # null pointers
    assert lib.hpd_rope(C.byref(good), 0, None, None, None, None, None) == 0      # nothing to do
    assert lib.hpd_kv_append(C.byref(good), -1, 0, *([None] * 9)) == -1
    assert b"geometry" in lib.hpd_strerror(-2)
    odd = binding.HpdGeom(12, 4, 128, 10000.0, 0.1, 16)           # G = 3
    assert lib.hpd_workspace_bytes(C.byref(odd), 1, 1, 1) == 0
    assert lib.hpd_workspace_bytes(C.byref(good), 256, 6144, 131072) > 0


def test_attention_rejects_slabs_beyond_its_16_bit_column_index():
    """hpd_attn_decode packs up to 128/G branches of round4(suffix_cap) columns each and indexes them with 16 bits:
    larger slabs are refused before anything is launched (no pointer is looked at)."""
    lib = binding.load()
    nulls = [None] * 12
    tail = [1, None, None, None, 0, None, None]
    for Hq, Hkv, cap, want in ((8, 1, 4092, -1), (8, 1, 4093, -4), (32, 8, 2044, -1), (32, 8, 2045, -4),
                               (4, 4, 508, -1), (4, 4, 512, -4)):
        g = binding.HpdGeom(Hq, Hkv, 128, 10000.0, 0.1, cap)
        assert lib.hpd_attn_decode(C.byref(g), 1, 1, 1, 1, *nulls, *tail) == want, (Hq, Hkv, cap)
    assert b"suffix_cap" in lib.hpd_strerror(-4)


def test_missing_library_is_an_error(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    try:
        binding.load()
        assert False, "expected HpdError"
    except binding.HpdError as e:
        assert "no CPU fallback" in str(e)
