"""The C-ABI library loads without a GPU and exports every symbol the headers declare."""
import ctypes
import glob
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols(header):
    text = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", header)).read(), flags=re.S)
    return sorted(set(re.findall(r"\b(sifar_[a-z0-9_]+)\s*\(", text)))


def test_libraries_build_load_and_export_every_declared_symbol():
    from paper_2607_08973_b200 import build
    build.build()
    core = ctypes.CDLL(build.LIB)
    bench = ctypes.CDLL(build.LIB_BENCH)
    assert sorted(os.path.basename(h) for h in glob.glob(os.path.join(ROOT, "include", "*.h"))) == \
        ["sifar.h", "sifar_workload.h"]
    core_syms, bench_syms = _declared_symbols("sifar.h"), _declared_symbols("sifar_workload.h")
    assert len(core_syms) >= 16 and len(bench_syms) >= 16
    assert {"sifar_create", "sifar_allreduce", "sifar_destroy"} <= set(core_syms)
    missing = [s for s in core_syms if not hasattr(core, s)] + [s for s in bench_syms if not hasattr(bench, s)]
    assert not missing, missing


def test_core_library_keeps_the_chain_and_probe_exports_out():
    """The measurement surface (decode-step chains, generator probes) lives in the second library only."""
    import subprocess
    from paper_2607_08973_b200 import build
    build.build()
    out = subprocess.run(["nm", "-D", "--defined-only", build.LIB], capture_output=True, text=True, check=True).stdout
    exported = set(re.findall(r"\bT (sifar_[a-z0-9_]+)$", out, flags=re.M))
    assert exported == set(_declared_symbols("sifar.h")), exported ^ set(_declared_symbols("sifar.h"))


def test_geometry_helpers_need_no_gpu():
    from paper_2607_08973_b200 import binding as sf
    assert sf.sifar_slot_count(sf.BF16, 4096) == 683 and sf.sifar_slot_count(sf.F32, 4096) == 1366
    assert sf.sifar_slot_count(sf.BF16, 0) == 0 and sf.sifar_slot_count(sf.BF16, 1) == 1
    # bytes = P reads of the partial + one write of the result + the flag words of the mode
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, 4096, sf.SPECULATIVE) == 8 * 683 * 16 + 8192
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, 4096, sf.DUALBUF) == 9 * 8192 + 32
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, 4096, sf.BARRIER_ONESHOT) == 9 * 8192 + 64


def test_speculative_format_choice_needs_no_gpu():
    import pytest
    from paper_2607_08973_b200 import binding as sf
    # tagged slots while all P partials together stay below 8 MiB, flagged tiles of plain data from there on
    assert sf.sifar_spec_format(8, sf.BF16, 4096) == sf.FORMAT_SLOTS
    assert sf.sifar_spec_format(8, sf.BF16, (1 << 19) - 1) == sf.FORMAT_SLOTS
    assert sf.sifar_spec_format(8, sf.BF16, 1 << 19) == sf.FORMAT_TILES            # 8 x 1 MiB
    assert sf.sifar_spec_format(2, sf.BF16, (1 << 21) - 1) == sf.FORMAT_SLOTS
    assert sf.sifar_spec_format(2, sf.BF16, 1 << 21) == sf.FORMAT_TILES            # 2 x 4 MiB
    assert sf.sifar_spec_format(8, sf.F32, (1 << 18) - 1) == sf.FORMAT_SLOTS
    assert sf.sifar_spec_format(8, sf.F32, 1 << 18) == sf.FORMAT_TILES
    assert sf.sifar_spec_format(1, sf.BF16, 0) == sf.FORMAT_SLOTS
    for bad in ((0, sf.BF16, 1), (9, sf.BF16, 1), (2, 7, 1)):
        with pytest.raises(sf.SifarError):
            sf.sifar_spec_format(*bad)
    # the bytes the method must move follow the format: no tag bytes, one 4-byte flag per 16 KiB block and rank
    n = 8 << 20
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, n, sf.SPECULATIVE) == 9 * n * 2 + 8 * 4 * (n * 2 // 16384)
    assert sf.sifar_algorithmic_bytes(8, sf.BF16, n, sf.DUALBUF) == 9 * n * 2 + 32


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
