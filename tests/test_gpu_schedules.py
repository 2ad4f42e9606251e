"""Host-scripted producer / reducer orderings, failure detection and call-number limits (all bounded, no GPU fault)."""
import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import binding as sf
from paper_2607_08973_b200 import synth

from gpu_util import BF16, F32, MODES, Ctx, assert_bits_equal, empty_out, out_to_numpy, to_device

pytestmark = pytest.mark.gpu


def _scripted(oracle, P, n, mode, delays_us, reducer_first, dtype=BF16, seed=7):
    """One call; rank r's pack is held back `delays_us[r]` microseconds behind a spin kernel on its stream."""
    with Ctx(P, n, dtype) as ctx:
        xs = synth.rank_inputs(P, n, dtype, seed, "gauss")
        xd = [to_device(x) for x in xs]
        out = empty_out(n, dtype)
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        torch.cuda.synchronize()
        for r in range(P):
            if delays_us[r]:
                sf.sifar_spin(int(delays_us[r] * 1000), ps[r].cuda_stream)
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, ps[r].cuda_stream)
        if not reducer_first:
            torch.cuda.synchronize()
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, rs.cuda_stream)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        got, _ = out_to_numpy(out, n, dtype)
        assert_bits_equal(got, oracle.allreduce(xs, dtype), dtype, f"mode {mode} delays {delays_us}")
        return sf.sifar_get_stats(ctx.h)


@pytest.mark.parametrize("mode", MODES)
def test_producers_done_before_the_reducer_starts(oracle, mode):
    st = _scripted(oracle, 8, 16384, mode, [0] * 8, reducer_first=False)
    assert st["slot_reloads"] == 0 and st["calls_with_retry"] == 0 and st["flag_polls"] == 0


@pytest.mark.parametrize("mode", MODES)
def test_reducer_starts_before_every_producer(oracle, mode):
    st = _scripted(oracle, 8, 16384, mode, [300] * 8, reducer_first=True)
    if mode == sf.SPECULATIVE:
        assert st["calls_with_retry"] == 1 and st["slot_reloads"] >= sf.sifar_slot_count(BF16, 16384)
    else:
        assert st["flag_polls"] > 0


@pytest.mark.parametrize("mode", MODES)
def test_one_late_rank(oracle, mode):
    st = _scripted(oracle, 8, 16384, mode, [0, 0, 0, 20, 0, 0, 0, 0], reducer_first=True)
    assert st["timeouts"] == 0


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("dtype", [BF16, F32])
def test_ranks_arrive_in_reverse_order(oracle, mode, dtype):
    st = _scripted(oracle, 8, 6001, mode, [80 - 10 * r for r in range(8)], reducer_first=True, dtype=dtype)
    assert st["timeouts"] == 0


@pytest.mark.parametrize("mode", MODES)
def test_a_rank_that_never_arrives_times_out_and_the_context_recovers(oracle, mode):
    P, n = 4, 4096
    with Ctx(P, n, BF16, timeout_us=2000) as ctx:
        xs = synth.rank_inputs(P, n, BF16, 11, "gauss")
        xd = [to_device(x) for x in xs]
        out = empty_out(n, BF16)
        for r in range(P - 1):                       # rank P-1 stays silent
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, 0)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, 0)
        torch.cuda.synchronize()                     # returns: the wait is bounded
        assert sf.sifar_status(ctx.h) == sf.ERR_TIMEOUT
        with pytest.raises(sf.SifarError) as ei:
            sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, 0)
        assert ei.value.code == sf.ERR_TIMEOUT
        assert sf.sifar_get_stats(ctx.h)["timeouts"] >= 1
        # the GPU is fine and the context works again after a reset
        sf.sifar_reset(ctx.h, 0)
        assert sf.sifar_status(ctx.h) == 0
        for r in range(P):
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, 0)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, 0)
        torch.cuda.synchronize()
        got, _ = out_to_numpy(out, n, BF16)
        assert_bits_equal(got, oracle.allreduce(xs, BF16), BF16, "after reset")
        assert sf.sifar_get_stats(ctx.h)["epoch"] == 1


@pytest.mark.parametrize("mode", MODES)
def test_call_numbers_near_the_32_bit_limit(oracle, mode):
    P, n = 2, 1000
    with Ctx(P, n, BF16) as ctx:
        sf.sifar_debug_set_epoch(ctx.h, 2 ** 32 - 8)
        xs = synth.rank_inputs(P, n, BF16, 5, "uniform")
        xd = [to_device(x) for x in xs]
        want = oracle.allreduce(xs, BF16)
        ok_calls = 0
        for _ in range(10):
            out = empty_out(n, BF16)
            try:
                for r in range(P):
                    sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, 0)
                sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, 0)
            except sf.SifarError as e:
                assert e.code == sf.ERR_EPOCH
                break
            torch.cuda.synchronize()
            got, _ = out_to_numpy(out, n, BF16)
            assert_bits_equal(got, want, BF16, f"call {ok_calls}")
            ok_calls += 1
        assert ok_calls == 6                          # call numbers 2^32-7 .. 2^32-2 are usable, then refusal
        assert sf.sifar_status(ctx.h) == 0
        sf.sifar_reset(ctx.h, 0)
        assert sf.sifar_rank_buffer(ctx.h, 0, mode)[1] == 1


def test_half_written_partial_then_the_rest(oracle):
    """A fused producer that stores its slots itself (device helper store_slot): first half, a pause, second half."""
    P, n = 4, 6 * 5000
    nslots = sf.sifar_slot_count(BF16, n)
    with Ctx(P, n, BF16) as ctx:
        xs = synth.rank_inputs(P, n, BF16, 21, "gauss")
        xd = [to_device(x) for x in xs]
        out = empty_out(n, BF16)
        where = [sf.sifar_rank_buffer(ctx.h, r, sf.SPECULATIVE) for r in range(P)]
        ps = [torch.cuda.Stream() for _ in range(P)]
        rs = torch.cuda.Stream()
        torch.cuda.synchronize()
        half = nslots // 2
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, sf.SPECULATIVE, rs.cuda_stream)
        for r, (ptr, epoch) in enumerate(where):                # the slot stores take tag and address as arguments
            sf.sifar_spin(20_000, ps[r].cuda_stream)
            sf.sifar_store_slots(xd[r].data_ptr(), ptr, 0, half, n, BF16, epoch, ps[r].cuda_stream)
            sf.sifar_spin(100_000, ps[r].cuda_stream)
            sf.sifar_store_slots(xd[r].data_ptr(), ptr, half, nslots - half, n, BF16, epoch, ps[r].cuda_stream)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        got, _ = out_to_numpy(out, n, BF16)
        assert_bits_equal(got, oracle.allreduce(xs, BF16), BF16, "half-written")
        st = sf.sifar_get_stats(ctx.h)
        assert st["calls_with_retry"] == 1 and st["slot_reloads"] > 0


@pytest.mark.parametrize("mode", MODES)
def test_a_producer_that_is_not_ordered_after_the_previous_call_is_refused(oracle, mode):
    """The producer of call e + 1 must be ordered after the reducer of call e (it takes the call number from
    device memory).  One that runs too early finds the number one short: SIFAR_ERR_EPOCH, in every mode, no hang."""
    P, n = 2, 4096
    with Ctx(P, n, BF16, timeout_us=20_000) as ctx:
        xs = synth.rank_inputs(P, n, BF16, 3, "gauss")
        xd = [to_device(x) for x in xs]
        out = empty_out(n, BF16)
        rs, ps = torch.cuda.Stream(), torch.cuda.Stream()
        for r in range(P):
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, ps.cuda_stream)
        torch.cuda.synchronize()
        sf.sifar_spin(3_000_000, rs.cuda_stream)              # the reducer of call 1 is held back 3 ms ...
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, rs.cuda_stream)
        sf.sifar_pack(ctx.h, 0, xd[0].data_ptr(), n, mode, ps.cuda_stream)   # ... the producer of call 2 is not
        ps.synchronize()
        assert sf.sifar_status(ctx.h) == sf.ERR_EPOCH
        torch.cuda.synchronize()
        sf.sifar_reset(ctx.h, 0)
        for r in range(P):
            sf.sifar_pack(ctx.h, r, xd[r].data_ptr(), n, mode, ps.cuda_stream)
        sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, rs.cuda_stream)
        torch.cuda.synchronize()
        got, _ = out_to_numpy(out, n, BF16)
        assert_bits_equal(got, oracle.allreduce(xs, BF16), BF16, "after reset")
