"""The C-ABI library loads without a GPU and exports every symbol the headers declare."""
import ctypes
import glob
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    for h in glob.glob(os.path.join(ROOT, "include", "*.h")):
        text = re.sub(r"/\*.*?\*/", "", open(h).read(), flags=re.S)
        names.update(re.findall(r"\b(sifar_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2607_08973_b200 import build
    path = build.build()
    L = ctypes.CDLL(path)
    syms = _declared_symbols()
    assert len(syms) >= 16
    missing = [s for s in syms if not hasattr(L, s)]
    assert not missing, missing


def test_geometry_helpers_need_no_gpu():
    from paper_2607_08973_b200 import binding as sf
    assert sf.sifar_slot_count(sf.BF16, 4096) == 683 and sf.sifar_slot_count(sf.F32, 4096) == 1366
    assert sf.sifar_slot_count(sf.BF16, 0) == 0 and sf.sifar_slot_count(sf.BF16, 1) == 1
    # bytes = P reads of the partial + one write of the result + the flag words of the mode
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, 4096, sf.SPECULATIVE) == 8 * 683 * 16 + 8192
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, 4096, sf.DUALBUF) == 9 * 8192 + 32
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, 4096, sf.BARRIER_ONESHOT) == 9 * 8192 + 64


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2607_08973_b200 import binding as sf
    monkeypatch.setattr(sf, "_lib", None)
    monkeypatch.setattr(sf, "_LIB_PATH", str(tmp_path / "nope.so"))
    try:
        sf.sifar_slot_count(0, 1)
    except RuntimeError as e:
        assert "no CPU fallback" in str(e)
    else:
        raise AssertionError("binding did not raise")
