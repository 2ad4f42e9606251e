"""The allocation-free entry point against the context-based one and against the CPU oracle (collected last on
purpose).

sifar_allreduce_noalloc serves callers that may not allocate device memory after
start-up (an engine with its own arena, a latency-critical decode loop); its
kernel keeps its bookkeeping in a fixed array inside the library.  Here it must
give, bit for bit, what sifar_allreduce gives on the same inputs and what the
oracle computes from them, on two calls in a row (the second call finds the array
as the first one left it), whether this file runs alone in a fresh process or
after every other test.
"""
import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import binding as sf
from paper_2607_08973_b200 import synth

pytestmark = pytest.mark.gpu

BF16, F32 = sf.BF16, sf.F32


def _dev(x):
    return torch.from_numpy(x.view(np.int16).copy() if x.dtype == np.uint16 else x.copy()).cuda()


def _host(t, dtype):
    h = t.cpu().numpy()
    return h.view(np.uint16) if dtype == BF16 else h


def _existing_entry_point(ctx, xd, n, dtype):
    """sifar_allreduce on caller buffers (barrier mode), each rank announced with sifar_arrive."""
    out = torch.zeros(n + 16, dtype=xd[0].dtype, device="cuda")
    for r in range(len(xd)):
        sf.sifar_wait_writable(ctx, r, 0)
        sf.sifar_arrive(ctx, r, sf.BARRIER_ONESHOT, 0)
    sf.sifar_allreduce(ctx, [x.data_ptr() for x in xd], out.data_ptr(), n, sf.BARRIER_ONESHOT, 0)
    torch.cuda.synchronize()
    assert sf.sifar_status(ctx) == 0
    return _host(out, dtype)[:n]


@pytest.mark.parametrize("P,n,dtype", [(8, 4096, BF16), (8, 100_003, BF16), (3, 6 * 4096 + 5, F32), (2, 1 << 20, BF16)])
def test_noalloc_matches_context_entry_point_on_two_calls_in_a_row(oracle, P, n, dtype):
    ctx = sf.sifar_create(P, n, dtype)
    try:
        td = torch.int16 if dtype == BF16 else torch.float32
        for call in range(2):
            xs = synth.rank_inputs(P, n, dtype, 4242 + call, "gauss")
            xd = [_dev(x) for x in xs]
            out = torch.zeros(n + 16, dtype=td, device="cuda")
            torch.cuda.synchronize()
            sf.sifar_allreduce_noalloc([x.data_ptr() for x in xd], out.data_ptr(), n, dtype, 0)
            torch.cuda.synchronize()
            got = _host(out, dtype)
            want = _existing_entry_point(ctx, xd, n, dtype)
            want_cpu = oracle.allreduce(xs, dtype)
            if dtype == F32:
                assert np.array_equal(got[:n].view(np.uint32), want.view(np.uint32)), f"call {call}"
                assert np.array_equal(got[:n].view(np.uint32), want_cpu.view(np.uint32)), f"call {call} vs oracle"
            else:
                assert np.array_equal(got[:n], want), f"call {call}"
                assert np.array_equal(got[:n], want_cpu), f"call {call} vs oracle"
            assert not got[n:].any(), "wrote past n"
    finally:
        sf.sifar_destroy(ctx)


@pytest.mark.parametrize("P,n,dtype", [(P, n, BF16) for P in (1, 8) for n in (1, 7, 8, 9)] +
                         [(P, n, F32) for P in (1, 8) for n in (1, 3, 5)])
def test_noalloc_small_and_tail_only_sizes_against_the_oracle(oracle, P, n, dtype):
    """n below one 16-byte vector takes the tail path alone (one CTA, no vector); P = 1 is the identity.
    The bookkeeping is read back: the CTA count is re-armed, every call is booked with its n."""
    td = torch.int16 if dtype == BF16 else torch.float32
    before = sf.sifar_noalloc_counters()
    assert before["cta_arrive"] == 0
    for call in range(2):
        xs = synth.rank_inputs(P, n, dtype, 900 + 17 * call + n, "gauss")
        xd = [_dev(x) for x in xs]
        out = torch.zeros(n + 16, dtype=td, device="cuda")
        sf.sifar_allreduce_noalloc([x.data_ptr() for x in xd], out.data_ptr(), n, dtype, 0)
        torch.cuda.synchronize()
        got, want = _host(out, dtype), oracle.allreduce(xs, dtype)
        if dtype == F32:
            assert np.array_equal(got[:n].view(np.uint32), want.view(np.uint32))
        else:
            assert np.array_equal(got[:n], want)
        assert not got[n:].any(), "wrote past n"
        now = sf.sifar_noalloc_counters()
        assert now == {"cta_arrive": 0, "calls": before["calls"] + call + 1, "elements": n}


def test_noalloc_rearms_its_cta_count_after_a_many_cta_call():
    n = 1 << 20
    x = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(8)]
    out = torch.zeros(n, dtype=torch.int16, device="cuda")
    calls = sf.sifar_noalloc_counters()["calls"]
    sf.sifar_allreduce_noalloc([t.data_ptr() for t in x], out.data_ptr(), n, BF16, 0)
    assert sf.sifar_noalloc_counters() == {"cta_arrive": 0, "calls": calls + 1, "elements": n}


def test_noalloc_refuses_sizes_beyond_its_fixed_limit():
    limit = sf.sifar_noalloc_max_elems()
    assert limit == 1 << 20
    x = torch.zeros(64, dtype=torch.int16, device="cuda")
    out = torch.zeros(64, dtype=torch.int16, device="cuda")
    with pytest.raises(sf.SifarError) as ei:
        sf.sifar_allreduce_noalloc([x.data_ptr(), x.data_ptr()], out.data_ptr(), limit + 1, BF16, 0)
    assert ei.value.code == sf.ERR_INVALID and "exceeds the fixed limit" in str(ei.value)
    with pytest.raises(sf.SifarError):
        sf.sifar_allreduce_noalloc([x.data_ptr()], x.data_ptr(), 64, BF16, 0)      # out overlaps an input
    sf.sifar_allreduce_noalloc([x.data_ptr()], out.data_ptr(), 0, BF16, 0)         # n = 0: nothing to do
    torch.cuda.synchronize()
