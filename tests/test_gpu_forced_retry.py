"""Forced retries (the retry-latency experiment of Section 6.3, "Retry Overhead"): results do not
change, the extra loads are counted, and the knob is refused outside its range."""
import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import binding as sf
from paper_2607_08973_b200 import synth

from gpu_util import (BF16, F32, Ctx, allreduce_via_pack, assert_bits_equal, canary_ok, empty_out,
                      out_to_numpy, to_device)
from test_gpu_chains import _oracle_w, _ring, _rows

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("P,n", [(2, 4096), (3, 6 * 257 + 5), (8, 4096), (8, 200_003)])
@pytest.mark.parametrize("rounds", [1, 3])
def test_forced_retries_leave_the_result_unchanged_and_are_counted(oracle, rounds, P, n, dtype):
    xs = synth.rank_inputs(P, n, dtype, seed=0xF0CE + rounds, dist="uniform")
    want = oracle.allreduce(xs, dtype)
    xs_dev = [to_device(x) for x in xs]
    nslots = sf.sifar_slot_count(dtype, n)
    with Ctx(P, n, dtype) as ctx:
        sf.sifar_debug_force_retries(ctx.h, rounds)
        for call in range(3):
            out = empty_out(n, dtype)
            allreduce_via_pack(ctx, xs_dev, n, sf.SPECULATIVE, out)
            torch.cuda.synchronize()
            assert sf.sifar_status(ctx.h) == 0
            got, tail = out_to_numpy(out, n, dtype)
            assert_bits_equal(got, want, dtype, f"forced={rounds} P={P} n={n} call={call}")
            assert canary_ok(tail, dtype)
        st = sf.sifar_get_stats(ctx.h)
        assert st["calls"] == 3 and st["calls_with_retry"] == 3
        assert st["slot_reloads"] >= 3 * rounds * P * nslots
        # back to normal: data that is ready before the reducer starts needs no re-load
        sf.sifar_debug_force_retries(ctx.h, 0)
        s = torch.cuda.Stream()
        out = empty_out(n, dtype)
        allreduce_via_pack(ctx, xs_dev, n, sf.SPECULATIVE, out, producer_streams=[s] * P, reducer_stream=s)
        torch.cuda.synchronize()
        st2 = sf.sifar_get_stats(ctx.h)
        assert st2["calls"] == 4 and st2["calls_with_retry"] == 3 and st2["slot_reloads"] == st["slot_reloads"]
        assert_bits_equal(out_to_numpy(out, n, dtype)[0], want, dtype, "after forced retries were switched off")


def test_forced_retries_do_not_touch_the_barrier_modes(oracle):
    P, n = 4, 10_000
    xs = synth.rank_inputs(P, n, BF16, seed=0xF0CF, dist="uniform")
    want = oracle.allreduce(xs, BF16)
    xs_dev = [to_device(x) for x in xs]
    with Ctx(P, n, BF16) as ctx:
        sf.sifar_debug_force_retries(ctx.h, 5)
        for mode in (sf.BARRIER_ONESHOT, sf.DUALBUF):
            out = empty_out(n, BF16)
            allreduce_via_pack(ctx, xs_dev, n, mode, out)
            torch.cuda.synchronize()
            assert_bits_equal(out_to_numpy(out, n, BF16)[0], want, BF16, f"mode {mode}")
        st = sf.sifar_get_stats(ctx.h)
        assert st["calls_with_retry"] == 0 and st["slot_reloads"] == 0


@pytest.mark.parametrize("impl", [sf.CHAIN_GRAPH, sf.CHAIN_PERSISTENT])
@pytest.mark.parametrize("P,n", [(2, 4096), (8, 4096), (8, 16384 * 2 + 7)])
def test_forced_retries_in_the_decode_chains(oracle, P, n, impl):
    d = synth.chain_workload("llama", P)
    steps = 16
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, 2 * steps)
    with Ctx(P, n, BF16, 5_000_000) as ctx:
        sf.sifar_debug_force_retries(ctx.h, 2)
        ring, stride = _ring(n, BF16, steps)
        ch = sf.sifar_chain_create(ctx.h, sf.make_workload(**d), n, sf.SPECULATIVE, impl, ring.data_ptr(), steps, steps)
        try:
            for run in range(2):
                sf.sifar_chain_run(ch, 0)
                torch.cuda.synchronize()
                assert sf.sifar_status(ctx.h) == 0
                got = _rows(ring, stride, steps, n, BF16)
                for s in range(steps):
                    assert_bits_equal(got[s], want[run * steps + s], BF16, f"run {run} step {s}")
            st = sf.sifar_get_stats(ctx.h)
            assert st["calls"] == 2 * steps and st["calls_with_retry"] == 2 * steps
            assert st["slot_reloads"] >= 2 * steps * 2 * P * sf.sifar_slot_count(BF16, n)
        finally:
            sf.sifar_chain_destroy(ch)


def test_waiting_cleanup_ctas_leave_although_the_arrival_count_was_re_armed(oracle):
    """Grids above the SM count keep their last CTAs waiting for the arrival count; the first of them re-arms
    the counter when nothing was queued, and the others must still get out.  Forced retries spread the CTAs'
    finishing times enough to make a waiter miss the complete count, which once ended in a time-out."""
    P, n, dtype = 8, 200_003, F32
    xs = synth.rank_inputs(P, n, dtype, seed=0xF0D0, dist="uniform")
    want = oracle.allreduce(xs, dtype)
    xs_dev = [to_device(x) for x in xs]
    ps, rs = [torch.cuda.Stream() for _ in range(P)], torch.cuda.Stream()
    for rounds in (0, 1, 2):
        with Ctx(P, n, dtype, timeout_us=200_000) as ctx:
            sf.sifar_debug_force_retries(ctx.h, rounds)
            out = empty_out(n, dtype)
            for it in range(200):
                allreduce_via_pack(ctx, xs_dev, n, sf.SPECULATIVE, out, ps, rs)
                torch.cuda.synchronize()
                assert sf.sifar_status(ctx.h) == 0, f"rounds={rounds} call {it}"
            assert_bits_equal(out_to_numpy(out, n, dtype)[0], want, dtype, f"rounds={rounds}")


def test_forced_retry_knob_range():
    with Ctx(2, 64, BF16) as ctx:
        assert sf.lib().sifar_debug_force_retries(ctx.h, 65) == sf.ERR_INVALID
        assert sf.lib().sifar_debug_force_retries(None, 1) == sf.ERR_INVALID
        assert sf.lib().sifar_debug_force_retries(ctx.h, 64) == 0
