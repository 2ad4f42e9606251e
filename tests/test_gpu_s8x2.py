"""The fallback slot format (two self-validating 8-byte halves per slot, libsifar_s8x2.so): same C ABI, same
results.  It relies on 64-bit single-copy atomicity only and is kept building for the day a 16-byte access is
seen torn; the default library is what everything else tests."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import build, synth

from gpu_util import BF16, F32, assert_bits_equal, canary_ok, empty_out, out_to_numpy, to_device

SPECULATIVE = 2


def _lib():
    build.build()
    L = ctypes.CDLL(build.LIB_S8X2)
    vp, sz, ci, cu = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint
    for name, res, args in (("sifar_create", vp, [ci, sz, ci]), ("sifar_destroy", ci, [vp]),
                            ("sifar_pack", ci, [vp, ci, vp, sz, ci, vp]), ("sifar_allreduce", ci, [vp, vp, vp, sz, ci, vp]),
                            ("sifar_status", ci, [vp]), ("sifar_slot_count", sz, [ci, sz]),
                            ("sifar_algorithmic_bytes", sz, [ci, ci, sz, ci]), ("sifar_set_timeout_us", ci, [vp, cu]),
                            ("sifar_get_stats", ci, [vp, ctypes.POINTER(ctypes.c_ulonglong)])):
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    return L


def test_fallback_format_geometry_needs_no_gpu():
    L = _lib()
    # 8 data bytes per slot: four bf16 or two fp32 elements
    assert L.sifar_slot_count(BF16, 4096) == 1024 and L.sifar_slot_count(F32, 4096) == 2048
    assert L.sifar_slot_count(BF16, 5) == 2 and L.sifar_slot_count(BF16, 0) == 0
    assert L.sifar_algorithmic_bytes(8, BF16, 4096, SPECULATIVE) == 8 * 1024 * 16 + 8192


@pytest.mark.gpu
@pytest.mark.parametrize("P,n,dtype", [(8, 4096, BF16), (8, 4099, BF16), (3, 1, BF16), (2, 7, F32), (8, 100_003, BF16),
                                       (5, 70_001, F32), (8, 400_000, BF16)])
def test_fallback_format_matches_the_oracle_with_late_producers(oracle, P, n, dtype):
    L = _lib()
    ctx = L.sifar_create(P, n, dtype)
    assert ctx
    try:
        L.sifar_set_timeout_us(ctx, 2_000_000)
        xs = synth.rank_inputs(P, n, dtype, 4000 + n, "gauss")
        xd = [to_device(x) for x in xs]
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        from paper_2607_08973_b200 import binding as sf
        for call in range(3):
            out = empty_out(n, dtype)
            torch.cuda.synchronize()
            for r in range(P):
                if call == 1:
                    sf.sifar_spin(50_000 + 10_000 * r, ps[r].cuda_stream)       # the reducer polls half-written slots
                assert L.sifar_pack(ctx, r, xd[(r + call) % P].data_ptr(), n, SPECULATIVE, ps[r].cuda_stream) == 0
            assert L.sifar_allreduce(ctx, None, out.data_ptr(), n, SPECULATIVE, rs.cuda_stream) == 0
            torch.cuda.synchronize()
            assert L.sifar_status(ctx) == 0
            got, tail = out_to_numpy(out, n, dtype)
            assert_bits_equal(got, oracle.allreduce([xs[(r + call) % P] for r in range(P)], dtype), dtype, f"call {call}")
            assert canary_ok(tail, dtype)
        stats = (ctypes.c_ulonglong * 8)()
        assert L.sifar_get_stats(ctx, stats) == 0
        assert stats[0] == 3 and stats[1] >= 1 and stats[4] == 0          # calls, calls with retry, time-outs
    finally:
        L.sifar_destroy(ctx)
