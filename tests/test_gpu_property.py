"""Property test: random rank counts, sizes, modes and values, always bit-exact with the oracle."""
import numpy as np
import pytest
import torch
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from paper_2607_08973_b200 import binding as sf

from gpu_util import BF16, F32, Ctx, allreduce_via_pack, assert_bits_equal, canary_ok, empty_out, out_to_numpy, to_device

pytestmark = pytest.mark.gpu


@settings(max_examples=60, deadline=None, suppress_health_check=list(HealthCheck))
@given(P=st.integers(1, 8), n=st.integers(0, 5000), dtype=st.sampled_from([BF16, F32]), mode=st.integers(0, 2),
       seed=st.integers(0, 2 ** 31 - 1), calls=st.integers(1, 3))
def test_random_shapes_and_bit_patterns(oracle, P, n, dtype, mode, seed, calls):
    rng = np.random.default_rng(seed)
    with Ctx(P, 5000, dtype) as ctx:
        for _ in range(calls):
            if dtype == BF16:
                xs = [rng.integers(0, 1 << 16, size=n, dtype=np.uint64).astype(np.uint16) for _ in range(P)]
                xs = [np.where((x & 0x7FFF) > 0x7F80, 0x3F80, x).astype(np.uint16) for x in xs]     # no NaN inputs
            else:
                xs = [(rng.standard_normal(n) * np.exp2(rng.integers(-30, 30, size=n))).astype(np.float32)
                      for _ in range(P)]
            out = empty_out(n, dtype)
            xd = [to_device(x) for x in xs]
            torch.cuda.synchronize()
            if n:
                allreduce_via_pack(ctx, xd, n, mode, out)
            else:
                sf.sifar_allreduce(ctx.h, None, out.data_ptr(), 0, mode, 0)
            torch.cuda.synchronize()
            assert sf.sifar_status(ctx.h) == 0
            got, tail = out_to_numpy(out, n, dtype)
            assert canary_ok(tail, dtype)
            if n:
                want = oracle.allreduce(xs, dtype)
                if dtype == BF16:
                    nan = (want & 0x7FFF) > 0x7F80            # inf - inf
                    assert np.array_equal(got[~nan], want[~nan]) and np.all(got[nan] == 0x7FFF)
                else:
                    assert_bits_equal(got, want, dtype, f"P={P} n={n} mode={mode}")


@settings(max_examples=40, deadline=None, suppress_health_check=list(HealthCheck))
@given(P=st.integers(1, 8), n=st.integers(1, 3000), dtype=st.sampled_from([BF16, F32]), mode=st.integers(0, 4),
       kind=st.integers(0, 2), seed=st.integers(0, 2 ** 31 - 1), one_reader=st.booleans(),
       delay=st.sampled_from([0, 0, 3000]))
def test_random_decode_chains(oracle, P, n, dtype, mode, kind, seed, one_reader, delay):
    """Random workloads through the persistent chains (one reader, P readers, twoshot): every step of two runs."""
    if mode == 3 or (one_reader and mode == 4):
        mode = sf.SPECULATIVE                 # 3 is the floor without all-reduce, 4 exists with P readers only
    d = dict(kind=kind, seed=seed, scale=1.0 / P if kind != 1 else 1.0, sigma=0.25, outlier_mod=(0, 7)[seed & 1],
             delay_max_ns=delay)
    steps = 4
    want = oracle.chain(oracle.Workload(d["kind"], d["seed"], d["scale"], d["sigma"], d["outlier_mod"],
                                        d["delay_max_ns"]), P, n, dtype, 2 * steps)
    stride = sf.sifar_chain_ring_stride(dtype, n)
    nd = np.uint16 if dtype == BF16 else np.float32
    copies = 1 if one_reader else P
    with Ctx(P, n, dtype, timeout_us=5_000_000) as ctx:
        rings = torch.zeros(copies * steps * stride, dtype=torch.uint8, device="cuda")
        w = sf.make_workload(**d)
        if one_reader:
            ch = sf.sifar_chain_create(ctx.h, w, n, mode, sf.CHAIN_PERSISTENT, rings.data_ptr(), steps, steps)
            run, destroy = sf.sifar_chain_run, sf.sifar_chain_destroy
        else:
            ch = sf.sifar_symchain_create(ctx.h, w, n, mode, rings.data_ptr(), steps, steps)
            run, destroy = sf.sifar_symchain_run, sf.sifar_symchain_destroy
        try:
            for k in range(2):
                run(ch, 0)
                torch.cuda.synchronize()
                assert sf.sifar_status(ctx.h) == 0
                h = rings.cpu().numpy().reshape(copies, steps, stride)[:, :, : n * nd().itemsize].copy().view(nd)
                for r in range(copies):
                    for s in range(steps):
                        assert_bits_equal(h[r, s], want[k * steps + s], dtype,
                                          f"P={P} n={n} mode={mode} kind={kind} copy {r} step {k * steps + s + 1}")
        finally:
            destroy(ch)
