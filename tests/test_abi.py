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


def test_size_adaptive_mode_choice_needs_no_gpu():
    import pytest
    from paper_2607_08973_b200 import binding as sf
    # speculative while all P partials together stay below 16 MiB, dual-buffered from there on
    assert sf.sifar_mode_for_payload(8, sf.BF16, 4096) == sf.SPECULATIVE
    assert sf.sifar_mode_for_payload(8, sf.BF16, (1 << 20) - 1) == sf.SPECULATIVE
    assert sf.sifar_mode_for_payload(8, sf.BF16, 1 << 20) == sf.DUALBUF            # 8 x 2 MiB
    assert sf.sifar_mode_for_payload(2, sf.BF16, (1 << 22) - 1) == sf.SPECULATIVE
    assert sf.sifar_mode_for_payload(2, sf.BF16, 1 << 22) == sf.DUALBUF            # 2 x 8 MiB
    assert sf.sifar_mode_for_payload(8, sf.F32, (1 << 19) - 1) == sf.SPECULATIVE
    assert sf.sifar_mode_for_payload(8, sf.F32, 1 << 19) == sf.DUALBUF
    assert sf.sifar_mode_for_payload(1, sf.BF16, 0) == sf.SPECULATIVE
    for bad in ((0, sf.BF16, 1), (9, sf.BF16, 1), (2, 7, 1)):
        with pytest.raises(sf.SifarError):
            sf.sifar_mode_for_payload(*bad)


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
