"""GPU parity of the decode-step chain with P readers (every rank reduces for itself)."""
import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import binding as sf
from paper_2607_08973_b200 import synth

from gpu_util import (BF16, F32, MODES, Ctx, allreduce_via_pack, assert_bits_equal, empty_out, out_to_numpy,
                      to_device)
from test_gpu_chains import _oracle_w

pytestmark = pytest.mark.gpu

SYM_MODES = MODES + (sf.SYMCHAIN_TWOSHOT, sf.SYMCHAIN_FLAGVAL, sf.SYMCHAIN_FLAGVAL_ORDERED)
RETRYING = (sf.SPECULATIVE, sf.SYMCHAIN_FLAGVAL, sf.SYMCHAIN_FLAGVAL_ORDERED)     # modes that book re-loads


def _rings(P, n, dtype, rows):
    stride = sf.sifar_chain_ring_stride(dtype, n)
    return torch.zeros(P * rows * stride, dtype=torch.uint8, device="cuda"), stride


def _copies(rings, stride, P, rows, n, dtype):
    """[P, rows, n] results, one copy per rank."""
    h = rings.cpu().numpy().reshape(P, rows, stride)
    nd = np.uint16 if dtype == BF16 else np.float32
    nb = n * nd().itemsize
    return np.stack([np.stack([h[r, i, :nb].view(nd) for i in range(rows)]) for r in range(P)])


def run_sym(P, n, dtype, d, mode, steps, runs=2, timeout_us=5_000_000, forced=0):
    outs, stamps = [], None
    with Ctx(P, n, dtype, timeout_us) as ctx:
        if forced:
            sf.sifar_debug_force_retries(ctx.h, forced)
        rings, stride = _rings(P, n, dtype, steps)
        ch = sf.sifar_symchain_create(ctx.h, sf.make_workload(**d), n, mode, rings.data_ptr(), steps, steps)
        try:
            s = torch.cuda.Stream()
            for _ in range(runs):
                sf.sifar_symchain_run(ch, s.cuda_stream)
                torch.cuda.synchronize()
                assert sf.sifar_status(ctx.h) == 0, sf.sifar_status(ctx.h)
                outs.append(_copies(rings, stride, P, steps, n, dtype))
            stamps = np.array(sf.sifar_symchain_stamps(ch, steps), dtype=np.int64)
            per_rank = [np.array(sf.sifar_symchain_rank_stamps(ch, r, steps), dtype=np.int64) for r in range(P)]
            retries = sf.sifar_symchain_retries(ch, P)
            stats = sf.sifar_get_stats(ctx.h)
        finally:
            sf.sifar_symchain_destroy(ch)
    return np.concatenate(outs, axis=1), stamps, per_rank, retries, stats


def _check_all_copies(got, want, dtype, what):
    P = got.shape[0]
    for r in range(P):
        for t in range(want.shape[0]):
            assert_bits_equal(got[r, t], want[t], dtype, f"{what} rank {r} step {t + 1}")


@pytest.mark.parametrize("mode", SYM_MODES)
@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("P,n", [(1, 100), (2, 4096), (3, 6 * 257 + 5), (5, 7), (8, 4096), (8, 40_003)])
def test_every_rank_gets_the_oracle_chain(oracle, P, n, dtype, mode):
    d = synth.chain_workload("llama", P)
    steps = 8
    want = oracle.chain(_oracle_w(oracle, d), P, n, dtype, 2 * steps)
    got, stamps, per_rank, retries, stats = run_sym(P, n, dtype, d, mode, steps)
    _check_all_copies(got, want, dtype, f"P={P} n={n} dt={dtype} mode={mode}")
    assert stats["calls"] == 2 * steps and stats["epoch"] == 2 * steps
    assert np.all(np.diff(stamps) > 0)
    for r in range(P):
        assert np.all(np.diff(per_rank[r]) > 0)
        assert np.all(per_rank[r][1:] <= stamps[1:])
    if mode not in RETRYING:
        assert sum(retries) == 0 and stats["slot_reloads"] == 0


@pytest.mark.parametrize("mode", SYM_MODES)
def test_token_chain_and_moe_shapes(oracle, mode):
    for name, P, n, steps in (("token", 2, 4096, 64), ("moe", 8, 4096 * 8, 24)):
        d = synth.chain_workload(name, P)
        want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, 2 * steps)
        got, *_ = run_sym(P, n, BF16, d, mode, steps)
        _check_all_copies(got, want, BF16, f"{name} mode={mode}")


@pytest.mark.parametrize("mode", SYM_MODES)
def test_skewed_ranks_integers(oracle, mode):
    """Seeded per-rank delays of up to 20 us before every store: ranks fall behind each other in turn."""
    P, n, steps = 8, 16384, 32
    d = synth.chain_workload("skew", P)
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, 2 * steps)
    got, stamps, per_rank, retries, stats = run_sym(P, n, BF16, d, mode, steps)
    _check_all_copies(got, want, BF16, f"skew mode={mode}")
    if mode == sf.SPECULATIVE:
        # the rank with the longest delay of a step sees everybody else's data at once; the others wait for it
        assert stats["calls_with_retry"] > steps and max(retries) <= 2 * steps
        assert min(retries) < 2 * steps, "some rank is last in some step and need not retry there"
        assert stats["slot_reloads"] > 0


@pytest.mark.parametrize("mode", SYM_MODES)
def test_more_than_one_unit_per_thread(oracle, mode):
    P, n, steps = 8, 1_000_003, 4
    d = synth.chain_workload("llama", P)
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, 2 * steps)
    got, *_ = run_sym(P, n, BF16, d, mode, steps, timeout_us=20_000_000)
    _check_all_copies(got, want, BF16, f"large mode={mode}")


def test_forced_retries_and_floor(oracle):
    P, n, steps = 4, 4096, 8
    d = synth.chain_workload("llama", P)
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, 2 * steps)
    got, _, _, retries, stats = run_sym(P, n, BF16, d, sf.SPECULATIVE, steps, forced=2)
    _check_all_copies(got, want, BF16, "forced")
    assert retries == [2 * steps] * P and stats["calls_with_retry"] == 2 * steps
    # the floor: every rank feeds on its own partial; no call number advances
    with Ctx(P, n, BF16) as ctx:
        rings, _ = _rings(P, n, BF16, steps)
        ch = sf.sifar_symchain_create(ctx.h, sf.make_workload(**d), n, sf.CHAIN_NO_ALLREDUCE, rings.data_ptr(), steps, steps)
        for _ in range(2):
            sf.sifar_symchain_run(ch, 0)
        torch.cuda.synchronize()
        st = np.array(sf.sifar_symchain_stamps(ch, steps), dtype=np.int64)
        assert np.all(np.diff(st) > 0)
        assert sf.sifar_get_stats(ctx.h)["epoch"] == 0
        sf.sifar_symchain_destroy(ch)


def test_bad_arguments_are_refused():
    with Ctx(2, 64, BF16) as ctx:
        rings, _ = _rings(2, 64, BF16, 4)
        w = sf.make_workload(**synth.chain_workload("llama", 2))
        import ctypes
        L = sf._wl()
        for args in ((ctx.h, ctypes.byref(w), 0, 2, rings.data_ptr(), 4, 4),
                     (ctx.h, ctypes.byref(w), 65, 2, rings.data_ptr(), 4, 4),
                     (ctx.h, ctypes.byref(w), 64, 8, rings.data_ptr(), 4, 4),
                     (ctx.h, ctypes.byref(w), 64, 2, None, 4, 4),
                     (ctx.h, ctypes.byref(w), 64, 2, rings.data_ptr(), 1, 4),
                     (ctx.h, ctypes.byref(w), 64, 2, rings.data_ptr(), 4, 6),
                     (ctx.h, ctypes.byref(w), 64, 2, rings.data_ptr(), 3, 3)):
            assert not L.sifar_symchain_create(*args)
        assert L.sifar_symchain_run(None, None) == sf.ERR_INVALID
        assert L.sifar_symchain_destroy(None) == 0


@pytest.mark.parametrize("symmetric", [False, True])
def test_context_is_usable_for_the_barrier_mode_after_a_persistent_chain(oracle, symmetric):
    """The persistent kernels keep done flags of their own: a later pack must not wait for the library's."""
    P, n, steps = 4, 4096, 4
    d = synth.chain_workload("llama", P)
    xs = synth.rank_inputs(P, n, BF16, seed=77, dist="uniform")
    xs_dev = [to_device(x) for x in xs]
    with Ctx(P, n, BF16, timeout_us=300_000) as ctx:
        rings, _ = _rings(P, n, BF16, steps)
        if symmetric:
            ch = sf.sifar_symchain_create(ctx.h, sf.make_workload(**d), n, sf.BARRIER_ONESHOT, rings.data_ptr(), steps, steps)
            sf.sifar_symchain_run(ch, 0)
            sf.sifar_symchain_destroy(ch)
        else:
            ch = sf.sifar_chain_create(ctx.h, sf.make_workload(**d), n, sf.BARRIER_ONESHOT, sf.CHAIN_PERSISTENT,
                                       rings.data_ptr(), steps, steps)
            sf.sifar_chain_run(ch, 0)
            sf.sifar_chain_destroy(ch)
        out = empty_out(n, BF16)
        allreduce_via_pack(ctx, xs_dev, n, sf.BARRIER_ONESHOT, out)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        assert_bits_equal(out_to_numpy(out, n, BF16)[0], oracle.allreduce(xs, BF16), BF16, "after the chain")


@pytest.mark.parametrize("mode", SYM_MODES)
def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(oracle, mode):
    """Ranks that are delayed by up to 1 ms against a 50 us limit: the waiting ranks give up, the kernel ends,
    the status is sticky, and after a reset the context works again."""
    P, n, steps = 4, 4096, 8
    d = dict(synth.chain_workload("llama", P), delay_max_ns=1_000_000)
    xs = synth.rank_inputs(P, n, BF16, seed=78, dist="uniform")
    xs_dev = [to_device(x) for x in xs]
    with Ctx(P, n, BF16, timeout_us=50) as ctx:
        rings, _ = _rings(P, n, BF16, steps)
        ch = sf.sifar_symchain_create(ctx.h, sf.make_workload(**d), n, mode, rings.data_ptr(), steps, steps)
        sf.sifar_symchain_run(ch, 0)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == sf.ERR_TIMEOUT
        assert sf.lib().sifar_get_stats  # the library still answers
        assert sf._wl().sifar_symchain_run(ch, None) == sf.ERR_TIMEOUT      # refused: the status is sticky
        sf.sifar_symchain_destroy(ch)
        sf.sifar_reset(ctx.h, 0)
        sf.sifar_set_timeout_us(ctx.h, 2_000_000)
        assert sf.sifar_status(ctx.h) == 0
        out = empty_out(n, BF16)
        allreduce_via_pack(ctx, xs_dev, n, min(mode, sf.SPECULATIVE), out)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        assert_bits_equal(out_to_numpy(out, n, BF16)[0], oracle.allreduce(xs, BF16), BF16, "after the reset")
