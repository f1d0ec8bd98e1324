"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol include/hero.h declares."""
import ctypes
import os
import re

from paper_2310_17723_b200 import build as B
from paper_2310_17723_b200 import hero

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    with open(os.path.join(ROOT, "include", "hero.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(hero_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = B.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"hero_layernorm_quant", "hero_w8a8_linear", "hero_int8_attention", "hero_layer_forward"} <= set(names)
    for n in names:
        assert hasattr(lib, n), "libhero.so does not export %s" % n
    assert set(hero.EXPORTS) <= set(names)


def test_mode_presets_follow_table1_without_a_gpu():
    # host-only entry point: Table 1 rows as (qkv, attn, attn_out, fc1, fc2), 0 = INT8, 1 = FP
    B.build()
    with open(os.path.join(ROOT, "tests", "golden", "mode_presets.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for name, _emb, *flags in rows:
        got = hero.mode_preset({"M1": hero.PRESET_M1, "M2": hero.PRESET_M2, "M3": hero.PRESET_M3}[name])
        assert got == [hero.MODE_INT8 if f == "1" else hero.MODE_FP for f in flags]
    assert hero.mode_preset(hero.PRESET_FP) == [hero.MODE_FP] * 5


def test_struct_layouts_match_the_header_sizes():
    # sizes the C compiler gives the same structs (x86-64 SysV): guards against a drifted ctypes mirror
    assert ctypes.sizeof(hero.Tensor) == 48
    assert ctypes.sizeof(hero.LinearParams) == 32
