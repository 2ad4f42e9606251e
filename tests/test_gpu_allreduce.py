"""GPU parity of single all-reduce calls against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import binding as sf
from paper_2607_08973_b200 import synth

from gpu_util import (BF16, F32, MODES, Ctx, allreduce_via_pack, assert_bits_equal, canary_ok, empty_out,
                      out_to_numpy, to_device)

pytestmark = pytest.mark.gpu


def _run_case(oracle, P, n, dtype, mode, dist="uniform", seed=1, repeats=2, max_elems=None):
    with Ctx(P, max_elems or max(n, 1), dtype) as ctx:
        for rep in range(repeats):                      # two calls: both parities
            xs = synth.rank_inputs(P, n, dtype, seed + rep, dist)
            xd = [to_device(x) for x in xs]
            out = empty_out(n, dtype)
            torch.cuda.synchronize()
            allreduce_via_pack(ctx, xd, n, mode, out)
            torch.cuda.synchronize()
            assert sf.sifar_status(ctx.h) == 0
            got, tail = out_to_numpy(out, n, dtype)
            assert canary_ok(tail, dtype), "wrote past n"
            assert_bits_equal(got, oracle.allreduce(xs, dtype), dtype, f"P={P} n={n} dt={dtype} mode={mode} rep={rep}")
        st = sf.sifar_get_stats(ctx.h)
        assert st["calls"] == repeats and st["epoch"] == repeats and st["timeouts"] == 0


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 7, 8])
def test_small_and_ragged_sizes(oracle, P, dtype, mode):
    for n in (1, 5, 6, 7, 8, 9, 4095, 4096, 4097, 6 * 1000 + 1, 6 * 1000 - 1):
        _run_case(oracle, P, n, dtype, mode, repeats=2)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("P,n", [(2, 1 << 20), (4, (1 << 20) + 3), (8, 1 << 21), (8, 3 * (1 << 20) + 5), (6, 777_777)])
def test_multi_tile_sizes(oracle, P, n, dtype, mode):
    """Several grid-stride iterations of every CTA plus a ragged tail."""
    _run_case(oracle, P, n, dtype, mode, dist="gauss", repeats=3)


@pytest.mark.parametrize("mode", MODES)
def test_zero_elements_advances_the_call_number(mode):
    with Ctx(4, 1024, BF16) as ctx:
        out = empty_out(16, BF16)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), 0, mode, 0)
        sf.sifar_allreduce(ctx.h, None, 0, 0, mode, 0)
        torch.cuda.synchronize()
        st = sf.sifar_get_stats(ctx.h)
        assert st["epoch"] == 2 and st["calls"] == 2
        assert sf.sifar_rank_buffer(ctx.h, 0, mode)[1] == 3


@pytest.mark.parametrize("dtype", [BF16, F32])
def test_special_values(oracle, dtype):
    """Signed zeros, subnormals, infinities, NaN: bit-exact except NaN payloads."""
    P = 3
    if dtype == BF16:
        edge = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x0080, 0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x7FC0,
                         0x3F80, 0xBF80, 0x3F81, 0x3B80, 0x4B80, 0xCB80, 0x4380, 0x3580], dtype=np.uint16)
    else:
        edge = np.array([0, 0x80000000, 1, 0x80000001, 0x007FFFFF, 0x00800000, 0x7F7FFFFF, 0xFF7FFFFF, 0x7F800000,
                         0xFF800000, 0x7FC00000, 0x3F800000, 0xBF800000, 0x3F800001, 0x33800000, 0x4B800000,
                         0xCB800000], dtype=np.uint32).view(np.float32)
    k = edge.size
    idx = np.stack(np.meshgrid(*[np.arange(k)] * P, indexing="ij")).reshape(P, -1)
    xs = [np.ascontiguousarray(edge[idx[r]]) for r in range(P)]
    n = xs[0].size
    want = oracle.allreduce(xs, dtype)
    for mode in MODES:
        with Ctx(P, n, dtype) as ctx:
            out = empty_out(n, dtype)
            allreduce_via_pack(ctx, [to_device(x) for x in xs], n, mode, out)
            torch.cuda.synchronize()
            got, _ = out_to_numpy(out, n, dtype)
            if dtype == BF16:
                nan = (want & 0x7FFF) > 0x7F80
                assert np.array_equal((got & 0x7FFF) > 0x7F80, nan)
                assert np.array_equal(got[~nan], want[~nan])
                assert np.all(got[nan] == 0x7FFF)          # the GPU narrowing canonicalises NaN like the oracle
            else:
                assert_bits_equal(got, want, dtype, f"mode {mode}")


def test_caller_buffers_in_barrier_mode(oracle):
    """Application-agnostic use: arbitrary caller buffers, reused every call, announced with sifar_arrive."""
    P, n = 4, 10_007
    with Ctx(P, n, BF16) as ctx:
        bufs = [torch.zeros(n + 8, dtype=torch.int16, device="cuda") for _ in range(P)]
        streams = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        for call in range(3):
            xs = synth.rank_inputs(P, n, BF16, 100 + call, "gauss")
            done = torch.cuda.Event()
            for r in range(P):
                with torch.cuda.stream(streams[r]):
                    sf.sifar_wait_writable(ctx.h, r, streams[r].cuda_stream)
                    bufs[r][:n].copy_(torch.from_numpy(xs[r].view(np.int16).copy()), non_blocking=False)
                    sf.sifar_arrive(ctx.h, r, sf.BARRIER_ONESHOT, streams[r].cuda_stream)
            out = empty_out(n, BF16)
            sf.sifar_allreduce(ctx.h, [b.data_ptr() for b in bufs], out.data_ptr(), n, sf.BARRIER_ONESHOT,
                               rs.cuda_stream)
            torch.cuda.synchronize()
            got, tail = out_to_numpy(out, n, BF16)
            assert canary_ok(tail, BF16)
            assert_bits_equal(got, oracle.allreduce(xs, BF16), BF16, f"call {call}")


def test_modes_alternate_on_one_context(oracle):
    P, n = 8, 12_345
    with Ctx(P, n, BF16) as ctx:
        order = [0, 1, 2, 2, 1, 0, 0, 2, 1, 1, 2, 0]
        for call, mode in enumerate(order):
            xs = synth.rank_inputs(P, n, BF16, 500 + call, "gauss")
            out = empty_out(n, BF16)
            xd = [to_device(x) for x in xs]
            torch.cuda.synchronize()
            allreduce_via_pack(ctx, xd, n, mode, out)
            torch.cuda.synchronize()
            got, _ = out_to_numpy(out, n, BF16)
            assert_bits_equal(got, oracle.allreduce(xs, BF16), BF16, f"call {call} mode {mode}")
        assert sf.sifar_get_stats(ctx.h)["epoch"] == len(order)


def test_shrinking_then_growing_payload(oracle):
    """Stale tags much older than the previous call of the same parity must not validate."""
    P = 4
    sizes = [6000, 60, 61, 6000, 7, 5999, 6000]
    with Ctx(P, 6000, BF16) as ctx:
        for call, n in enumerate(sizes):
            xs = synth.rank_inputs(P, n, BF16, 900 + call, "uniform")
            out = empty_out(n, BF16)
            xd = [to_device(x) for x in xs]
            torch.cuda.synchronize()
            allreduce_via_pack(ctx, xd, n, sf.SPECULATIVE, out)
            torch.cuda.synchronize()
            got, tail = out_to_numpy(out, n, BF16)
            assert canary_ok(tail, BF16)
            assert_bits_equal(got, oracle.allreduce(xs, BF16), BF16, f"call {call} n {n}")


@pytest.mark.parametrize("pinned", [False, True])
def test_host_buffer_entry_point(oracle, pinned):
    """Pageable buffers take the staging path, pinned ones are read and written in place by the kernels."""
    P = 8
    with Ctx(P, 50_001, BF16) as ctx:
        for n in (50_001, 4096, 7):
            for mode in MODES:
                xs = synth.rank_inputs(P, n, BF16, 77 + mode + n, "gauss")
                if pinned:
                    hx = [torch.from_numpy(x.view(np.int16).copy()).pin_memory() for x in xs]
                    hout = torch.zeros(n, dtype=torch.int16).pin_memory()
                    sf.sifar_allreduce_host(ctx.h, [t.data_ptr() for t in hx], hout.data_ptr(), n, mode)
                    out = hout.numpy().view(np.uint16)
                else:
                    out = np.zeros(n, dtype=np.uint16)
                    sf.sifar_allreduce_host(ctx.h, [x.ctypes.data for x in xs], out.ctypes.data, n, mode)
                assert_bits_equal(out, oracle.allreduce(xs, BF16), BF16, f"host pinned={pinned} n={n} mode {mode}")


def test_argument_validation():
    with pytest.raises(sf.SifarError):
        sf.sifar_create(0, 16, BF16)
    with pytest.raises(sf.SifarError):
        sf.sifar_create(9, 16, BF16)
    with pytest.raises(sf.SifarError):
        sf.sifar_create(2, 16, 7)
    with Ctx(2, 1024, BF16) as ctx:
        out = empty_out(1024, BF16)
        bad = [lambda: sf.sifar_allreduce(ctx.h, None, out.data_ptr(), 2048, 1, 0),        # n > max
               lambda: sf.sifar_allreduce(ctx.h, None, out.data_ptr(), 16, 5, 0),          # mode
               lambda: sf.sifar_allreduce(ctx.h, None, out.data_ptr() + 2, 16, 1, 0),      # alignment
               lambda: sf.sifar_allreduce(ctx.h, None, 0, 16, 1, 0),                       # NULL out
               lambda: sf.sifar_allreduce(ctx.h, [out.data_ptr(), out.data_ptr()], out.data_ptr(), 16, 2, 0),
               lambda: sf.sifar_allreduce(ctx.h, None, sf.sifar_rank_buffer(ctx.h, 1, 1)[0], 16, 1, 0),  # aliasing
               lambda: sf.sifar_pack(ctx.h, 2, out.data_ptr(), 16, 1, 0)]                  # rank
        for f in bad:
            with pytest.raises(sf.SifarError) as ei:
                f()
            assert ei.value.code == sf.ERR_INVALID
        torch.cuda.synchronize()
        assert sf.sifar_get_stats(ctx.h)["epoch"] == 0      # nothing was launched, call number untouched
