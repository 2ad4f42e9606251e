"""The flagged-tile format of the speculative mode (large payloads): plain data, one arrival flag per 16 KiB
block, tiles reduced as they land; and the early start of a large reducer under the kernel before it."""
import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import binding as sf
from paper_2607_08973_b200 import synth

from gpu_util import BF16, F32, Ctx, assert_bits_equal, canary_ok, empty_out, out_to_numpy, to_device

pytestmark = pytest.mark.gpu


def _first_tiles_n(P, dtype, extra):
    """Smallest n in the flagged-tile format, plus `extra` elements."""
    n = (8 << 20) // (P * (2 if dtype == BF16 else 4)) + extra
    assert sf.sifar_spec_format(P, dtype, n) == sf.FORMAT_TILES
    return n


@pytest.mark.parametrize("P,dtype,extra", [(8, BF16, 0), (8, BF16, 5), (8, BF16, 8192 * 3 + 7), (4, BF16, 4099), (2, BF16, 1),
                                           (3, BF16, 12345), (8, F32, 0), (8, F32, 3), (5, F32, 4096 * 2 + 1), (1, BF16, 9)])
def test_flagged_tiles_match_the_oracle(oracle, P, dtype, extra):
    n = _first_tiles_n(P, dtype, extra)
    with Ctx(P, n, dtype) as ctx:
        xs = synth.rank_inputs(P, n, dtype, 77 + extra, "uniform")
        xd = [to_device(x) for x in xs]
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        for call in range(3):                         # both parities, and a parity used for the second time
            out = empty_out(n, dtype)
            torch.cuda.synchronize()
            for r in range(P):
                sf.sifar_pack(ctx.h, r, xd[(r + call) % P].data_ptr(), n, sf.SPECULATIVE, ps[r].cuda_stream)
            sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, sf.SPECULATIVE, rs.cuda_stream)
            torch.cuda.synchronize()
            assert sf.sifar_status(ctx.h) == 0
            got, tail = out_to_numpy(out, n, dtype)
            want = oracle.allreduce([xs[(r + call) % P] for r in range(P)], dtype)
            assert_bits_equal(got, want, dtype, f"call {call}")
            assert canary_ok(tail, dtype)


@pytest.mark.parametrize("P,n,dtype", [(8, 8 << 20, BF16), (8, 4 << 20, F32), (2, (8 << 20) + 11, BF16)])
def test_flagged_tiles_with_producers_up_to_300_us_late(oracle, P, n, dtype):
    """Config-4 sizes; the reducer starts at once, every rank's producer is held back a different time."""
    assert sf.sifar_spec_format(P, dtype, n) == sf.FORMAT_TILES
    delays_us = [(37 * r * r + 300 - 40 * r) % 301 for r in range(P)]
    with Ctx(P, n, dtype) as ctx:
        xs = synth.rank_inputs(P, n, dtype, 5, "uniform")
        xd = [to_device(x) for x in xs]
        out = empty_out(n, dtype)
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        torch.cuda.synchronize()
        for r in range(P):
            sf.sifar_spin(delays_us[r] * 1000 + 100_000, ps[r].cuda_stream)      # held back 100-400 us
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, sf.SPECULATIVE, ps[r].cuda_stream)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, sf.SPECULATIVE, rs.cuda_stream)   # starts at once
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        got, tail = out_to_numpy(out, n, dtype)
        assert_bits_equal(got, oracle.allreduce(xs, dtype), dtype, "late producers")
        assert canary_ok(tail, dtype)
        st = sf.sifar_get_stats(ctx.h)
        assert st["calls_with_retry"] == 1 and st["flag_polls"] > 0 and st["timeouts"] == 0


MODES = [sf.BARRIER_ONESHOT, sf.DUALBUF, sf.SPECULATIVE]


@pytest.mark.parametrize("policy", [sf.SWEEP_NEVER, sf.SWEEP_AUTO, sf.SWEEP_ALWAYS])
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("P,dtype,n", [(8, BF16, (6 << 20) + 5), (3, F32, (4 << 20) + 3)])
def test_queued_tiles_are_swept_by_the_janitors_or_by_the_sweep_kernel(oracle, mode, policy, P, dtype, n):
    """A large call (more than 8 tiles per SM, ragged tail) whose producers are late, then one on ready data,
    then a late one again: the same bits whoever sweeps the queued tiles, and the call numbers stay in step."""
    with Ctx(P, n, dtype, timeout_us=2_000_000) as ctx:
        sf.sifar_debug_sweep_policy(ctx.h, policy)
        xs = synth.rank_inputs(P, n, dtype, 21 + policy, "uniform")
        xd = [to_device(x) for x in xs]
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        for call, late in enumerate((True, False, True)):
            out = empty_out(n, dtype)
            torch.cuda.synchronize()
            for r in range(P):
                if late:
                    sf.sifar_spin(100_000 + 30_000 * ((r * 5 + call) % P), ps[r].cuda_stream)
                sf.sifar_pack(ctx.h, r, xd[(r + call) % P].data_ptr(), n, mode, ps[r].cuda_stream)
            if not late:
                torch.cuda.synchronize()
            sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, rs.cuda_stream)
            torch.cuda.synchronize()
            assert sf.sifar_status(ctx.h) == 0, (call, sf.sifar_last_error())
            got, tail = out_to_numpy(out, n, dtype)
            want = oracle.allreduce([xs[(r + call) % P] for r in range(P)], dtype)
            assert_bits_equal(got, want, dtype, f"call {call}")
            assert canary_ok(tail, dtype)
        st = sf.sifar_get_stats(ctx.h)
        assert st["epoch"] == 3 and st["calls"] == 3 and st["timeouts"] == 0
        if mode == sf.SPECULATIVE:
            assert st["calls_with_retry"] == 2       # the two late calls, not the one on ready data


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("policy", [sf.SWEEP_NEVER, sf.SWEEP_AUTO])
def test_a_rank_that_is_too_late_for_a_large_call_times_out_and_the_context_recovers(oracle, mode, policy):
    """One rank's producer is held back 20 ms against a 2 ms limit: the janitors, or the sweep kernel, give up
    after the limit, the kernels end by themselves, the late producer finds the context dead and leaves, and
    after a reset the same call works."""
    P, dtype, n = 4, BF16, (5 << 20) + 3
    with Ctx(P, n, dtype, timeout_us=2000) as ctx:
        sf.sifar_debug_sweep_policy(ctx.h, policy)
        xs = synth.rank_inputs(P, n, dtype, 31, "uniform")
        xd = [to_device(x) for x in xs]
        out = empty_out(n, dtype)
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        torch.cuda.synchronize()
        sf.sifar_spin(20_000_000, ps[P - 1].cuda_stream)                 # rank P-1: 20 ms late
        for r in range(P):
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, ps[r].cuda_stream)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, rs.cuda_stream)
        torch.cuda.synchronize()                                         # returns: every wait is bounded
        assert sf.sifar_status(ctx.h) == sf.ERR_TIMEOUT
        assert sf.sifar_get_stats(ctx.h)["timeouts"] >= 1
        sf.sifar_reset(ctx.h, 0)
        sf.sifar_set_timeout_us(ctx.h, 2_000_000)
        assert sf.sifar_status(ctx.h) == 0
        for r in range(P):
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, ps[r].cuda_stream)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, rs.cuda_stream)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        got, tail = out_to_numpy(out, n, dtype)
        assert_bits_equal(got, oracle.allreduce(xs, dtype), dtype, "after the reset")
        assert canary_ok(tail, dtype)


def test_sweep_policy_is_checked():
    with Ctx(2, 1024, BF16) as ctx:
        with pytest.raises(sf.SifarError):
            sf.sifar_debug_sweep_policy(ctx.h, 3)


def test_a_fused_producer_that_signals_block_by_block(oracle):
    """The caller's own kernel stores plain data and releases the block flags itself (sifar_tile_flags,
    device helper signal_block): first half of the blocks, a pause, then the rest."""
    P, dtype = 4, BF16
    n = _first_tiles_n(P, dtype, 8192 * 5 + 3)
    with Ctx(P, n, dtype) as ctx:
        xs = synth.rank_inputs(P, n, dtype, 31, "gauss")
        xd = [to_device(x) for x in xs]
        out = empty_out(n, dtype)
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        where = []
        for r in range(P):
            ptr, epoch = sf.sifar_rank_buffer(ctx.h, r, sf.SPECULATIVE)
            flags, per_flag, stride = sf.sifar_tile_flags(ctx.h, r)
            assert per_flag == 8192 and stride >= 1
            where.append((ptr, epoch, flags, stride))
        nblocks = (n * 2 // 16 + 1023) // 1024
        half = nblocks // 2
        torch.cuda.synchronize()
        for r, (ptr, epoch, flags, stride) in enumerate(where):
            s = ps[r].cuda_stream
            sf.sifar_spin(100_000, s)
            sf.sifar_store_blocks(xd[r].data_ptr(), ptr, flags, stride, 0, half, n, dtype, epoch, s)
            sf.sifar_spin(150_000, s)
            sf.sifar_store_blocks(xd[r].data_ptr(), ptr, flags, stride, half, nblocks - half, n, dtype, epoch, s)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, sf.SPECULATIVE, rs.cuda_stream)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        got, tail = out_to_numpy(out, n, dtype)
        assert_bits_equal(got, oracle.allreduce(xs, dtype), dtype, "block by block")
        assert canary_ok(tail, dtype)
        assert sf.sifar_get_stats(ctx.h)["calls_with_retry"] == 1


@pytest.mark.parametrize("mode", [sf.DUALBUF, sf.SPECULATIVE])
def test_early_reducers_keep_the_stream_order_of_their_results(oracle, mode):
    """Large reducers whose producers run on other streams start reading while the kernel before them on their
    stream still runs; what they write must still land in stream order.  Several contexts reduce into the SAME
    result buffer back to back: it must hold the last call's sum, every time."""
    P, n, dtype, nctx = 8, 2 << 20, BF16, 4
    ctxs = [Ctx(P, n, dtype) for _ in range(nctx)]
    try:
        xs = [synth.rank_inputs(P, n, dtype, 900 + i, "gauss") for i in range(nctx)]
        xd = [[to_device(x) for x in xi] for xi in xs]
        want_last = oracle.allreduce(xs[-1], dtype)
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        out = empty_out(n, dtype)
        for rep in range(6):
            torch.cuda.synchronize()
            for i, c in enumerate(ctxs):
                for r in range(P):
                    sf.sifar_pack(c.h, r, xd[i][r].data_ptr(), n, mode, ps[r].cuda_stream)
            if rep % 2 == 0:
                torch.cuda.synchronize()              # data ready; odd repetitions: producers still running
            sf.sifar_spin(200_000, rs.cuda_stream)    # a kernel for the first reducer to start under
            for c in ctxs:
                sf.sifar_allreduce(c.h, None, out.data_ptr(), n, mode, rs.cuda_stream)
            torch.cuda.synchronize()
            assert all(sf.sifar_status(c.h) == 0 for c in ctxs)
            got, tail = out_to_numpy(out, n, dtype)
            assert_bits_equal(got, want_last, dtype, f"repetition {rep}")
            assert canary_ok(tail, dtype)
    finally:
        for c in ctxs:
            c.__exit__()


def test_pack_and_allreduce_must_agree_on_the_format():
    P, dtype = 8, BF16
    n_tiles = _first_tiles_n(P, dtype, 0)
    with Ctx(P, n_tiles, dtype) as ctx:
        x = torch.zeros(n_tiles, dtype=torch.int16, device="cuda")
        out = torch.zeros(n_tiles, dtype=torch.int16, device="cuda")
        for r in range(P):
            sf.sifar_pack(ctx.h, r, x.data_ptr(), 4096, sf.SPECULATIVE, 0)        # slots
        with pytest.raises(sf.SifarError) as ei:
            sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n_tiles, sf.SPECULATIVE, 0)   # tiles
        assert ei.value.code == sf.ERR_INVALID and "format" in str(ei.value)
        torch.cuda.synchronize()
