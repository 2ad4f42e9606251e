"""GPU parity of the decode-step chains (stream, graph, persistent) and of the device generator."""
import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import binding as sf
from paper_2607_08973_b200 import synth

from gpu_util import (BF16, F32, MODES, Ctx, allreduce_via_pack, assert_bits_equal, empty_out, out_to_numpy,
                      to_device)

pytestmark = pytest.mark.gpu

IMPLS = (sf.CHAIN_STREAMS, sf.CHAIN_GRAPH, sf.CHAIN_PERSISTENT)


_MOE_WANT = {}


def _workloads(name, P):
    d = synth.chain_workload(name, P)
    return sf.make_workload(**d), d


def _oracle_w(oracle, d):
    return oracle.Workload(d["kind"], d["seed"], d["scale"], d["sigma"], d["outlier_mod"], d["delay_max_ns"])


def _ring(n, dtype, rows):
    stride = sf.sifar_chain_ring_stride(dtype, n)
    return torch.zeros(rows * stride, dtype=torch.uint8, device="cuda"), stride


def _rows(ring, stride, rows, n, dtype):
    h = ring.cpu().numpy().reshape(rows, stride)
    nd = np.uint16 if dtype == BF16 else np.float32
    return np.stack([h[i, : n * nd().itemsize].view(nd) for i in range(rows)])


def run_chain(P, n, dtype, d, mode, impl, steps, runs=1, ring_len=None, timeout_us=5_000_000):
    """Runs `runs` x `steps` steps; returns [runs*steps, n] results when ring_len == steps, and the stats."""
    ring_len = ring_len or steps
    outs = []
    with Ctx(P, n, dtype, timeout_us) as ctx:
        ring, stride = _ring(n, dtype, ring_len)
        ch = sf.sifar_chain_create(ctx.h, sf.make_workload(**d), n, mode, impl, ring.data_ptr(), ring_len, steps)
        try:
            s = torch.cuda.Stream()
            for _ in range(runs):
                sf.sifar_chain_run(ch, s.cuda_stream)
                torch.cuda.synchronize()
                assert sf.sifar_status(ctx.h) == 0, sf.sifar_status(ctx.h)
                outs.append(_rows(ring, stride, ring_len, n, dtype))
            stats = sf.sifar_get_stats(ctx.h)
        finally:
            sf.sifar_chain_destroy(ch)
    return np.concatenate(outs), stats


@pytest.mark.parametrize("dtype", [BF16, F32])
@pytest.mark.parametrize("kind", [0, 1, 2])
def test_device_generator_matches_the_oracle_generator(oracle, kind, dtype):
    w = sf.make_workload(kind, 0xC0FFEE + kind, 0.125, 0.1, 100, 20000)
    ow = oracle.Workload(kind, 0xC0FFEE + kind, 0.125, 0.1, 100, 20000)
    td = torch.int16 if dtype == BF16 else torch.float32
    for n in (1, 7, 8, 9, 4096, 100_003):
        for r in (0, 3, 7):
            dst = torch.zeros(n + 16, dtype=td, device="cuda")
            sf.sifar_workload_first(w, r, dtype, dst.data_ptr(), n)
            first = dst.cpu().numpy()[:n]
            first = first.view(np.uint16) if dtype == BF16 else first
            assert_bits_equal(first, oracle.workload_first(ow, r, n, dtype), dtype, f"first kind={kind} n={n} r={r}")
            prev_h = oracle.workload_first(ow, (r + 1) % 8, n, dtype)         # any tensor serves as "previous result"
            if kind == 1 and dtype == BF16:
                pass                                                          # integers in [-64,64]: valid previous result
            prev = torch.from_numpy(prev_h.view(np.int16).copy() if dtype == BF16 else prev_h.copy()).cuda()
            prev_pad = torch.zeros(n + 16, dtype=td, device="cuda")
            prev_pad[:n] = prev
            for t in (2, 65, 10_000):
                sf.sifar_workload_next(w, r, t, dtype, prev_pad.data_ptr(), dst.data_ptr(), n)
                got = dst.cpu().numpy()[:n]
                got = got.view(np.uint16) if dtype == BF16 else got
                assert_bits_equal(got, oracle.workload_next(ow, r, t, prev_h, dtype), dtype,
                                  f"next kind={kind} n={n} r={r} t={t}")
    L = oracle.lib()
    for t in (1, 2, 999):
        assert sf.sifar_workload_delays(w, 8, t) == [L.oracle_gen_delay_ns(w.seed, r, t, 20000) for r in range(8)]


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("mode", MODES)
def test_config1_token_chain(oracle, mode, impl):
    """P=2, one token of hidden 4096, 64 chained all-reduces, next input = previous output + noise."""
    P, n, steps = 2, 4096, 64
    _, d = _workloads("token", P)
    got, st = run_chain(P, n, BF16, d, mode, impl, steps)
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, steps)
    for t in range(steps):
        assert_bits_equal(got[t], want[t], BF16, f"step {t + 1}")
    assert st["calls"] == steps and st["epoch"] == steps and st["timeouts"] == 0


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("b", [1, 16])
def test_config2_llama_shaped_decode_step(oracle, b, mode, impl):
    P, n, steps = 8, 4096 * b, 64
    _, d = _workloads("llama", P)
    got, _ = run_chain(P, n, BF16, d, mode, impl, steps)
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, steps)
    for t in range(steps):
        assert_bits_equal(got[t], want[t], BF16, f"step {t + 1}")


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("b", [1, 32, 64])
def test_config3_moe_shaped_decode_step(oracle, b, mode, impl):
    P, n, steps = 8, 4096 * b, 120
    _, d = _workloads("moe", P)
    ring_len = 120 if b == 1 else 24
    got, _ = run_chain(P, n, BF16, d, mode, impl, steps, ring_len=ring_len)
    if b not in _MOE_WANT:                            # the oracle's chain is the same for every mode and form
        _MOE_WANT[b] = oracle.chain(_oracle_w(oracle, d), P, n, BF16, steps)
    want = _MOE_WANT[b]
    for j in range(ring_len):
        t = steps - ring_len + j                      # the ring keeps the last ring_len results
        assert_bits_equal(got[j], want[t], BF16, f"step {t + 1}")


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("P,n,dtype", [(2, 12_289, BF16), (4, 50_001, F32), (3, 6_007, BF16), (8, 100_000, F32)])
def test_config4_chained_sweep_shapes(oracle, P, n, dtype, mode, impl):
    """Uniform values, ragged sizes, two runs of one chain (the second run continues the first)."""
    steps = 10
    _, d = _workloads("sweep", P)
    got, st = run_chain(P, n, dtype, d, mode, impl, steps, runs=2)
    want = oracle.chain(_oracle_w(oracle, d), P, n, dtype, 2 * steps)
    for t in range(2 * steps):
        assert_bits_equal(got[t], want[t], dtype, f"step {t + 1}")
    assert st["epoch"] == 2 * steps


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("mode", MODES)
def test_config5_skewed_arrival_short(oracle, mode, impl):
    """Integer inputs, every producer delayed by a seeded 0-20 us spin: 200 chained calls, bit-exact."""
    P, n, steps, runs = 8, 16384, 100, 2
    _, d = _workloads("skew", P)
    got, st = run_chain(P, n, BF16, d, mode, impl, steps, runs=runs)
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, steps * runs)
    for t in range(steps * runs):
        assert_bits_equal(got[t], want[t], BF16, f"step {t + 1}")
    vals = (want.astype(np.uint32) << 16).view(np.float32)
    assert np.all(vals == np.round(vals)) and np.abs(vals).max() <= 512
    if mode == sf.SPECULATIVE:
        # with 0-20 us of skew between ranks the reducer must have met stale slots
        assert st["slot_reloads"] > 0 and 0 < st["calls_with_retry"] <= steps * runs


def test_modes_agree_bitwise_on_every_step(oracle):
    P, n, steps = 8, 8192, 64
    _, d = _workloads("llama", P)
    ref = None
    for impl in IMPLS:
        for mode in MODES:
            got, _ = run_chain(P, n, BF16, d, mode, impl, steps)
            if ref is None:
                ref = got
            assert np.array_equal(got, ref), (impl, mode)


@pytest.mark.parametrize("mode", [sf.DUALBUF, sf.SPECULATIVE])
@pytest.mark.parametrize("n,steps,name,handoff_max", [(4096, 64, "llama", "0"), (16384 * 8 + 5, 24, "moe", "1000000000"),
                                                      (4096 * 3 + 1, 64, "skew", "0")])
def test_both_forms_of_the_result_hand_over_at_both_grid_sizes(oracle, monkeypatch, mode, n, steps, name, handoff_max):
    """Inside the persistent kernel a result reaches the next step's producers in tagged words (small grids) or
    by one ready flag per chunk (large grids); the size decides.  Here each form runs where the other is the
    default: the flag form at a decode payload, the tagged words on a grid whose threads take two units per step."""
    monkeypatch.setenv("SIFAR_CHAIN_HANDOFF_MAX", handoff_max)
    P = 8
    _, d = _workloads(name, P)
    got, st = run_chain(P, n, BF16, d, mode, sf.CHAIN_PERSISTENT, steps, runs=2)
    want = oracle.chain(_oracle_w(oracle, d), P, n, BF16, 2 * steps)
    for t in range(2 * steps):
        assert_bits_equal(got[t], want[t], BF16, f"step {t + 1}")
    assert st["timeouts"] == 0 and st["calls"] == 2 * steps


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("n,clustered,tagged_modes", [(4096, 1, (sf.DUALBUF, sf.SPECULATIVE)), (4096 * 16, 0, (sf.DUALBUF, sf.SPECULATIVE)),
                                                      (4096 * 32, 0, ())])
def test_the_kernel_runs_with_the_layout_the_host_chose(mode, n, clustered, tagged_modes):
    """Small grids: one thread-block cluster per chunk and tagged hand-over words; larger ones spread out; the
    largest by ready flag.  The kernel reports what it really ran with."""
    P, steps = 8, 8
    _, d = _workloads("llama", P)
    with Ctx(P, n, BF16) as ctx:
        ring, _ = _ring(n, BF16, steps)
        ch = sf.sifar_chain_create(ctx.h, sf.make_workload(**d), n, mode, sf.CHAIN_PERSISTENT, ring.data_ptr(), steps, steps)
        try:
            sf.sifar_chain_run(ch, 0)
            g = sf.sifar_chain_geometry(ch)
        finally:
            sf.sifar_chain_destroy(ch)
        assert sf.sifar_status(ctx.h) == 0
    assert g["clustered"] == clustered and g["kernel_clustered"] == clustered
    assert g["kernel_cluster_ctas"] == (P + 1 if clustered else 1)
    assert g["tagged"] == g["kernel_tagged"] == int(mode in tagged_modes)
    assert g["ctas"] == g["chunks"] * (P + 1)


@pytest.mark.parametrize("handoff_max", ["100000", "0"])
@pytest.mark.parametrize("mode", MODES)
def test_a_wait_that_runs_out_ends_the_persistent_chain_and_the_context_recovers(oracle, monkeypatch, mode, handoff_max):
    """Ranks delayed by up to 1 ms against a 50 us limit: whoever waits gives up, the kernel ends by itself, the
    status is sticky, and after a reset the context works again; with either form of the result hand-over."""
    monkeypatch.setenv("SIFAR_CHAIN_HANDOFF_MAX", handoff_max)
    P, n, steps = 4, 4096, 8
    d = dict(synth.chain_workload("llama", P), delay_max_ns=1_000_000)
    xs = synth.rank_inputs(P, n, BF16, seed=79, dist="uniform")
    xs_dev = [to_device(x) for x in xs]
    with Ctx(P, n, BF16, timeout_us=50) as ctx:
        ring, _ = _ring(n, BF16, steps)
        ch = sf.sifar_chain_create(ctx.h, sf.make_workload(**d), n, mode, sf.CHAIN_PERSISTENT, ring.data_ptr(), steps, steps)
        sf.sifar_chain_run(ch, 0)
        torch.cuda.synchronize()                                         # returns: every wait is bounded
        assert sf.sifar_status(ctx.h) == sf.ERR_TIMEOUT
        with pytest.raises(sf.SifarError) as ei:                         # refused: the status is sticky
            sf.sifar_chain_run(ch, 0)
        assert ei.value.code == sf.ERR_TIMEOUT
        sf.sifar_chain_destroy(ch)
        sf.sifar_reset(ctx.h, 0)
        sf.sifar_set_timeout_us(ctx.h, 2_000_000)
        assert sf.sifar_status(ctx.h) == 0
        out = empty_out(n, BF16)
        allreduce_via_pack(ctx, xs_dev, n, mode, out)
        torch.cuda.synchronize()
        assert sf.sifar_status(ctx.h) == 0
        assert_bits_equal(out_to_numpy(out, n, BF16)[0], oracle.allreduce(xs, BF16), BF16, "after the reset")


def test_no_allreduce_floor_runs():
    """The chain without all-reduce runs in every implementation and leaves the call number alone."""
    P, n, steps = 8, 4096, 64
    _, d = _workloads("llama", P)
    for impl in IMPLS:
        _, st = run_chain(P, n, BF16, d, sf.CHAIN_NO_ALLREDUCE, impl, steps)
        assert st["epoch"] == 0 and st["timeouts"] == 0


def test_persistent_chain_timestamps_are_monotonic():
    P, n, steps = 8, 4096, 64
    _, d = _workloads("llama", P)
    with Ctx(P, n, BF16) as ctx:
        ring, _ = _ring(n, BF16, 2)
        for mode in (*MODES, sf.CHAIN_NO_ALLREDUCE):
            ch = sf.sifar_chain_create(ctx.h, sf.make_workload(**d), n, mode, sf.CHAIN_PERSISTENT, ring.data_ptr(), 2, steps)
            sf.sifar_chain_run(ch, 0)
            stamps = np.array(sf.sifar_chain_stamps(ch, steps), dtype=np.int64)
            assert np.all(np.diff(stamps) >= 0) and stamps[-1] - stamps[0] < 50_000_000
            # a result is complete with its last chunk: the run's stamps bound every chunk's own stamps
            C = sf.sifar_chain_chunks(ch)
            assert C == -(-sf.sifar_slot_count(BF16, n) // 128) if mode == sf.SPECULATIVE else C >= 1
            per_chunk = np.array([sf.sifar_chain_chunk_stamps(ch, c, steps) for c in range(C)], dtype=np.int64)
            assert np.array_equal(per_chunk[:, 1:].max(axis=0), stamps[1:]) and per_chunk[:, 0].min() == stamps[0]
            sf.sifar_chain_destroy(ch)
            sf.sifar_reset(ctx.h, 0)


def test_sixteen_byte_accesses_are_not_torn():
    """The speculative slots rest on this: over a thousand million slot reads against concurrent slot stores,
    never a slot whose four words come from two different stores."""
    torn, reads = 0, 0
    for _ in range(4):                                 # four bounded runs of a few hundred milliseconds each
        t, r = sf.sifar_tear_check(1 << 16, 4000)
        torn, reads = torn + t, reads + r
    assert reads >= 1_000_000_000
    assert torn == 0


def test_phase_trace_orders_the_phases_of_a_step():
    """The traced build records the per-step timeline; phases of one step appear in protocol order."""
    P, n, steps = 8, 4096, 64
    _, d = _workloads("llama", P)
    with Ctx(P, n, BF16) as ctx:
        ring, _ = _ring(n, BF16, 2)
        for mode in MODES:
            ch = sf.sifar_chain_create(ctx.h, sf.make_workload(**d), n, mode, sf.CHAIN_PERSISTENT, ring.data_ptr(), 2, steps)
            sf.sifar_chain_trace(ch, True)
            sf.sifar_chain_run(ch, 0)
            T = np.array(sf.sifar_chain_trace(ch, True, steps), dtype=np.int64)[2:]
            assert sf.sifar_status(ctx.h) == 0
            entered, seen, reduced, released = T[:, 0], T[:, 1], T[:, 2], T[:, 3]
            assert np.all(entered <= seen) and np.all(seen <= reduced) and np.all(reduced <= released)
            for r in range(P):
                ready, stored = T[:, 4 + 3 * r], T[:, 5 + 3 * r]
                assert np.all(ready <= stored)
                assert np.all(stored <= reduced)                  # no result before every rank has stored
                # producers wait for the previous result: with both barriers for the whole chunk, otherwise (at
                # this size) each thread takes its unit over as soon as the reducer's thread has validated and
                # stored it, which may be before the whole chunk is out
                handed = released if mode == sf.BARRIER_ONESHOT else seen
                assert np.all(handed[:-1] <= ready[1:])
                if mode != sf.SPECULATIVE:
                    assert np.all(stored <= T[:, 6 + 3 * r]) and np.all(T[:, 6 + 3 * r] <= seen)
            sf.sifar_chain_destroy(ch)
            sf.sifar_reset(ctx.h, 0)
