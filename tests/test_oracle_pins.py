"""Pins of the CPU oracle against facts that do not come from the oracle itself.

Every expected value here is produced by a different route than the oracle's own
code: hand-derived fixtures, exact integer / rational arithmetic, float64
arithmetic (a binary32 add equals the float64 add rounded once to binary32,
because 53 >= 2*24 + 2), torch's CPU casts, and algebraic identities.
"""
import itertools
import math
import os
import struct
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2607_08973_b200 import synth

BF16, F32 = 0, 1
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "bf16_ties.txt")


# ----------------------------------------------------------------------------
# independent helpers (none of them shares code with oracle/)
# ----------------------------------------------------------------------------
def f32_value_to_bits(v: float) -> int:
    return struct.unpack("<I", struct.pack("<f", v))[0]


def bits_to_f32_value(b: int) -> float:
    return struct.unpack("<f", struct.pack("<I", b))[0]


def bf16_bits_to_value(b: int) -> float:
    return bits_to_f32_value((b & 0xFFFF) << 16)


def round_to_bf16_rational(v: float) -> int:
    """Nearest bf16 (8-bit significand, emin -126, ties to even) of a finite float, via Fractions."""
    if v == 0.0:
        return 0x8000 if math.copysign(1.0, v) < 0 else 0x0000
    sign = 0x8000 if v < 0 else 0
    a = Fraction(abs(v))
    _, e = math.frexp(abs(v))            # abs(v) = m * 2^e, m in [0.5, 1)
    q_exp = max(e - 8, -133)             # spacing of bf16 numbers around v (subnormal floor 2^-133)
    quantum = Fraction(2) ** q_exp
    q = round(a / quantum)               # Fraction.__round__ is round-half-even
    val = q * quantum
    if val >= Fraction(2) ** 128:
        return sign | 0x7F80
    bits = f32_value_to_bits(float(val))  # exactly representable, so no second rounding
    assert bits & 0xFFFF == 0
    return sign | (bits >> 16)


def int_to_bf16_bits(s: int) -> int:
    """RNE of an integer to 8 significant bits, in integer arithmetic only."""
    if s == 0:
        return 0
    sign = 0x8000 if s < 0 else 0
    a = abs(s)
    L = a.bit_length()
    if L > 8:
        sh = L - 8
        q, rem, half = a >> sh, a & ((1 << sh) - 1), 1 << (sh - 1)
        if rem > half or (rem == half and (q & 1)):
            q += 1
        a = q << sh
    return sign | (f32_value_to_bits(float(a)) >> 16)


# ----------------------------------------------------------------------------
# golden fixtures
# ----------------------------------------------------------------------------
def _golden_cases():
    cases = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            lhs, rhs = line.split("->")
            tok = lhs.split()
            dtype, P, xs = tok[0], int(tok[1]), [int(t, 16) for t in tok[2:]]
            assert len(xs) == P
            cases.append((dtype, xs, int(rhs.strip(), 16)))
    return cases


@pytest.mark.parametrize("dtype,xs,want", _golden_cases())
def test_golden_fixtures(oracle, dtype, xs, want):
    if dtype == "bf16":
        out = oracle.allreduce([np.array([x], dtype=np.uint16) for x in xs], BF16)
        assert int(out[0]) == want
    else:
        out = oracle.allreduce([np.array([x], dtype=np.uint32).view(np.float32) for x in xs], F32)
        assert int(out.view(np.uint32)[0]) == want


def test_golden_file_is_nontrivial():
    c = _golden_cases()
    assert len(c) >= 20 and {d for d, _, _ in c} == {"bf16", "f32"}


# ----------------------------------------------------------------------------
# bf16 rounding and widening
# ----------------------------------------------------------------------------
def test_widening_is_exact_for_all_bf16(oracle):
    b = np.arange(65536, dtype=np.uint16)
    got = oracle.bf16_to_f32(b).view(np.uint32)
    want = torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).float().numpy().view(np.uint32)
    np.testing.assert_array_equal(got, want)
    # and narrowing a widened bf16 is the identity on every non-NaN pattern
    back = oracle.f32_to_bf16(got.view(np.float32))
    nan = ((b & 0x7FFF) > 0x7F80)
    np.testing.assert_array_equal(back[~nan], b[~nan])
    assert np.all(back[nan] == 0x7FFF)


def test_rounding_against_rational_arithmetic(oracle):
    rng = np.random.default_rng(1234)
    bits = rng.integers(0, 1 << 32, size=20000, dtype=np.uint64).astype(np.uint32)
    # add the neighbourhoods of every tie and of the exponent boundaries
    base = (rng.integers(0, 1 << 16, size=3000, dtype=np.uint64).astype(np.uint32) << 16)
    near = np.concatenate([base | 0x7FFF, base | 0x8000, base | 0x8001, base | 0xFFFF, base])
    edges = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0x00800000, 0x007FFFFF, 0x007F8000, 0x7F7FFFFF,
                      0x7F7F8000, 0x7F7F7FFF, 0x7F800000, 0x80000000, 0xFF7FFFFF, 0xFF800000],
                     dtype=np.uint32)
    bits = np.concatenate([bits, near, edges])
    vals = bits.view(np.float32)
    finite = np.isfinite(vals)
    got = oracle.f32_bits_to_bf16(bits)
    for b, v, g in zip(bits[finite], vals[finite], got[finite]):
        assert int(g) == round_to_bf16_rational(float(v)), hex(int(b))
    inf = np.isinf(vals)
    np.testing.assert_array_equal(got[inf], (bits[inf] >> 16).astype(np.uint16))
    assert np.all(got[np.isnan(vals)] == 0x7FFF)


def test_rounding_against_torch_cast(oracle):
    rng = np.random.default_rng(99)
    bits = rng.integers(0, 1 << 32, size=1 << 22, dtype=np.uint64).astype(np.uint32)
    hi = np.arange(1 << 16, dtype=np.uint32) << 16        # every bf16, with the four critical tails
    bits = np.concatenate([bits, hi | 0x7FFF, hi | 0x8000, hi | 0x8001, hi])
    vals = bits.view(np.float32)
    got = oracle.f32_bits_to_bf16(bits)
    want = torch.from_numpy(vals.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    ok = ~np.isnan(vals)
    np.testing.assert_array_equal(got[ok], want[ok])
    # NaN class is preserved (payload canonicalised)
    assert np.all((got[~ok] & 0x7FFF) > 0x7F80)


# ----------------------------------------------------------------------------
# the reduction
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [BF16, F32])
def test_single_rank_is_identity(oracle, dtype):
    if dtype == BF16:
        x = np.arange(65536, dtype=np.uint16)
        x = x[(x & 0x7FFF) <= 0x7F80]                      # all non-NaN patterns: +-0, subnormals, +-inf
        np.testing.assert_array_equal(oracle.allreduce([x], BF16), x)
    else:
        rng = np.random.default_rng(5)
        bits = rng.integers(0, 1 << 32, size=1 << 18, dtype=np.uint64).astype(np.uint32)
        bits = np.concatenate([bits, np.array([0, 0x80000000, 1, 0x80000001, 0x7F800000, 0xFF800000], np.uint32)])
        bits = bits[~np.isnan(bits.view(np.float32))]
        out = oracle.allreduce([bits.view(np.float32)], F32)
        np.testing.assert_array_equal(out.view(np.uint32), bits)


@pytest.mark.parametrize("P", [2, 4, 8])
def test_equal_copies_scale_exactly(oracle, P):
    x = np.arange(65536, dtype=np.uint16)
    v = (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    keep = np.isfinite(v) & (np.abs(v) * P < 2.0 ** 128 * (1 - 2.0 ** -9))   # P*x stays a finite bf16
    x, v = x[keep], v[keep]
    out = oracle.allreduce([x] * P, BF16)
    got = (out.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    np.testing.assert_array_equal(got, v * P)              # power-of-two scaling is exact
    np.testing.assert_array_equal(np.signbit(got), np.signbit(v))
    # for normal inputs: same mantissa, exponent field + log2(P)
    normal = ((x >> 7) & 0xFF) > 0
    np.testing.assert_array_equal(out[normal], x[normal] + (int(math.log2(P)) << 7))


@pytest.mark.parametrize("P", [2, 3, 4, 5, 8])
def test_integer_inputs_against_integer_arithmetic(oracle, P):
    rng = np.random.default_rng(100 + P)
    n = 4096
    ints = rng.integers(-64, 65, size=(P, n))
    ints[:, :4] = [[64] * 4, ] * P                         # force the extremes +-64*P
    ints[:, 4:8] = [[-64] * 4, ] * P
    xs = [np.array([int_to_bf16_bits(int(v)) for v in row], dtype=np.uint16) for row in ints]
    want = np.array([int_to_bf16_bits(int(s)) for s in ints.sum(axis=0)], dtype=np.uint16)
    orders = itertools.permutations(range(P)) if P <= 4 else \
        [rng.permutation(P) for _ in range(24)]
    for order in orders:
        out = oracle.allreduce([xs[r] for r in order], BF16)
        np.testing.assert_array_equal(out, want)
    # fp32: the integer sum itself
    outf = oracle.allreduce([row.astype(np.float32) for row in ints], F32)
    np.testing.assert_array_equal(outf, ints.sum(axis=0).astype(np.float32))


def test_two_rank_bf16_pairs_against_float64_route(oracle):
    """All 65536 bf16 values against 192 partners: fp32 add == float64 add rounded once."""
    rng = np.random.default_rng(7)
    allb = np.arange(65536, dtype=np.uint16)
    partners = np.concatenate([
        np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x007F, 0x0080, 0x3F80, 0xBF80, 0x3F81, 0x3B80,
                  0x7F7F, 0xFF7F, 0x7F80, 0xFF80, 0x4B80, 0xCB80], dtype=np.uint16),
        rng.integers(0, 1 << 16, size=176, dtype=np.uint64).astype(np.uint16)])
    a = np.repeat(allb, partners.size)
    b = np.tile(partners, allb.size)
    out = oracle.allreduce([a, b], BF16)
    av = (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    bv = (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    with np.errstate(invalid="ignore", over="ignore"):
        s32 = (av + bv).astype(np.float32)                 # exact-ish in float64, one rounding to binary32
    want = torch.from_numpy(s32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = np.isnan(s32)
    np.testing.assert_array_equal(out[~nan], want[~nan])
    assert np.all(out[nan] == 0x7FFF)


def test_all_two_rank_bf16_pairs_exhaustively(tmp_path):
    """All 2^32 pairs of bf16 values through the C oracle, against the binary64 route and a distance-based
    rounding written separately in tests/golden/pairs_bruteforce.c (four processes, a quarter of `a` each); and
    the oracle's binary32 -> bf16 rounding on all 2^32 binary32 bit patterns against the same distance rule."""
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    flags = ["-std=c11", "-ffp-contract=off", "-fno-fast-math"]
    o1, o2, exe = str(tmp_path / "oracle.o"), str(tmp_path / "pairs.o"), str(tmp_path / "pairs_bruteforce")
    subprocess.check_call(["gcc", "-O1", *flags, "-c", os.path.join(root, "oracle", "sifar_oracle.c"), "-o", o1])
    subprocess.check_call(["gcc", "-O2", *flags, "-c", os.path.join(root, "tests", "golden", "pairs_bruteforce.c"), "-o", o2])
    subprocess.check_call(["gcc", o1, o2, "-lm", "-o", exe])
    for mode in ([], ["round"]):          # all pairs of bf16 values; then the rounding alone on all binary32 patterns
        procs = [subprocess.Popen([exe, *mode, str(q * 16384), str(q * 16384 + 16383)], stdout=subprocess.PIPE,
                                  stderr=subprocess.PIPE, text=True) for q in range(4)]
        checked = 0
        for pr in procs:
            out, err = pr.communicate(timeout=600)
            assert pr.returncode == 0, err
            c, bad = (int(v) for v in out.split())
            assert bad == 0
            checked += c
        assert checked == 1 << 32


@pytest.mark.parametrize("P", [3, 5, 8])
@pytest.mark.parametrize("dtype", [BF16, F32])
def test_rank_order_accumulation_against_float64_route(oracle, P, dtype):
    """Left-to-right binary32 accumulation, each add emulated as float64 add + one rounding."""
    rng = np.random.default_rng(31 * P + dtype)
    n = 1 << 16
    if dtype == BF16:
        xs = [rng.integers(0, 1 << 16, size=n, dtype=np.uint64).astype(np.uint16) for _ in range(P)]
        xs = [np.where((x & 0x7FFF) > 0x7F80, 0x3F80, x).astype(np.uint16) for x in xs]   # no NaN inputs
        vals = [(x.astype(np.uint32) << 16).view(np.float32) for x in xs]
    else:
        # wide dynamic range so that rounding happens at every add
        vals = [(rng.standard_normal(n) * np.exp2(rng.integers(-20, 20, size=n))).astype(np.float32)
                for _ in range(P)]
        xs = vals
    acc = vals[0].astype(np.float32)
    with np.errstate(invalid="ignore", over="ignore"):
        for r in range(1, P):
            acc = (acc.astype(np.float64) + vals[r].astype(np.float64)).astype(np.float32)
    out = oracle.allreduce(xs, dtype)
    nan = np.isnan(acc)
    if dtype == BF16:
        want = torch.from_numpy(acc).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        np.testing.assert_array_equal(out[~nan], want[~nan])
        assert np.all(out[nan] == 0x7FFF)
    else:
        np.testing.assert_array_equal(out[~nan].view(np.uint32), acc[~nan].view(np.uint32))
        assert np.all(np.isnan(out[nan]))


def test_torch_cpu_special_case(oracle):
    """The whole definition written with torch CPU ops on N(0,1) data."""
    P, n = 8, 1 << 16
    xs = synth.rank_inputs(P, n, BF16, seed=42, dist="gauss")
    ts = [torch.from_numpy(x.view(np.int16)).view(torch.bfloat16) for x in xs]
    acc = ts[0].float()
    for t in ts[1:]:
        acc = acc + t.float()
    want = acc.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(oracle.allreduce(xs, BF16), want)


def test_empty_input(oracle):
    assert oracle.allreduce([np.zeros(0, np.uint16)] * 3, BF16).size == 0


# ----------------------------------------------------------------------------
# the workload generator: a definition, pinned by range / moments / frequencies,
# and by the independent numpy restatement in the shared input module
# ----------------------------------------------------------------------------
def test_generator_restatements_agree(oracle):
    L = oracle.lib()
    i = np.arange(4096, dtype=np.uint32)
    for seed, r, t in [(0, 0, 1), (0x5EED0002, 7, 64), (0xFFFFFFFF, 3, 10000), (12345, 15, 0xFFFFFFFF)]:
        g, u, k = synth.gauss(seed, r, t, i), synth.uniform(seed, r, t, i), synth.int129(seed, r, t, i)
        for j in range(0, 4096, 7):
            assert L.oracle_gen_gauss(seed, r, t, j) == g[j]
            assert L.oracle_gen_uniform(seed, r, t, j) == u[j]
            assert L.oracle_gen_int129(seed, r, t, j) == k[j]
            assert L.oracle_gen_is_outlier(seed, r, j, 100) == int(synth.is_outlier(seed, r, np.uint32(j), 100))
        assert L.oracle_gen_delay_ns(seed, r, t, 20000) == int(synth.delay_ns(seed, r, np.uint32(t), 20000))


def test_generator_statistics(oracle):
    w = oracle.Workload(oracle.KIND_GAUSS, 0x5EED0002, 1.0, 0.1, 100, 0)
    n = 1 << 20
    g = oracle.workload_first(oracle.Workload(0, 77, 1.0, 0.1, 0, 0), 3, n, F32).astype(np.float64)
    assert abs(g.mean()) < 5e-3 and abs(g.var() - 1.0) < 1e-2 and np.abs(g).max() < 6.0
    kurt = ((g - g.mean()) ** 4).mean() / g.var() ** 2
    assert abs(kurt - 2.9) < 0.05                           # Irwin-Hall(12): excess kurtosis -0.1
    u = oracle.workload_first(oracle.Workload(2, 77, 1.0, 0.1, 0, 0), 3, n, F32).astype(np.float64)
    assert u.min() >= -1.0 and u.max() < 1.0 and abs(u.mean()) < 3e-3 and abs(u.var() - 1 / 3) < 3e-3
    k = oracle.workload_first(oracle.Workload(1, 77, 1.0, 0.1, 0, 0), 3, n, F32)
    assert k.min() == -64 and k.max() == 64 and np.all(k == np.round(k))
    counts = np.bincount((k + 64).astype(np.int64), minlength=129)
    chi2 = ((counts - n / 129) ** 2 / (n / 129)).sum()
    assert chi2 < 200                                       # 128 dof: mean 128, sd 16
    # outliers: about one element in 100 is scaled by exactly 100
    base = oracle.workload_first(oracle.Workload(0, 0x5EED0002, 1.0, 0.1, 0, 0), 1, n, F32)
    outl = oracle.workload_first(w, 1, n, F32)
    changed = outl != base
    assert abs(changed.mean() - 0.01) < 1e-3
    np.testing.assert_array_equal(outl[changed], base[changed] * np.float32(100.0))
    # ranks and steps are decorrelated
    a = oracle.workload_first(oracle.Workload(0, 77, 1.0, 0.1, 0, 0), 0, n, F32)
    assert abs(np.corrcoef(a, g)[0, 1]) < 5e-3


def test_mix_avalanche():
    x = np.arange(1 << 14, dtype=np.uint32) * np.uint32(2654435761)
    base = synth._mix(x)
    for bit in range(32):
        flipped = synth._mix(x ^ np.uint32(1 << bit))
        d = base ^ flipped
        pop = np.unpackbits(d.view(np.uint8)).sum() / x.size
        assert 14.5 < pop < 17.5, (bit, pop)


def test_chain_update_rules(oracle):
    """The gauss update is two separately rounded products and one add; checked through float64."""
    P, n, t = 4, 4096, 5
    w = oracle.Workload(oracle.KIND_GAUSS, 9, 0.25, 0.1, 0, 0)
    prev = synth.rank_inputs(1, n, BF16, seed=3, dist="gauss")[0]
    i = np.arange(n, dtype=np.uint32)
    pv = (prev.astype(np.uint32) << 16).view(np.float32)
    for r in range(P):
        z = synth.gauss(9, r, t, i)
        a = (pv.astype(np.float64) * np.float64(np.float32(0.25))).astype(np.float32)
        b = (z.astype(np.float64) * np.float64(np.float32(0.1))).astype(np.float32)
        s = (a.astype(np.float64) + b.astype(np.float64)).astype(np.float32)
        want = torch.from_numpy(s).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        np.testing.assert_array_equal(oracle.workload_next(w, r, t, prev, BF16), want)
        np.testing.assert_array_equal(oracle.workload_next(w, r, t, pv, F32), s)


def test_integer_chain_stays_integer_and_exact(oracle):
    P, n, steps = 8, 512, 40
    w = oracle.Workload(oracle.KIND_INT, 0x5EED0005, 1.0, 1.0, 0, 20000)
    outs = oracle.chain(w, P, n, BF16, steps)
    i = np.arange(n, dtype=np.uint32)
    prev = None
    for s in range(steps):
        t = s + 1
        k = np.stack([synth.int129(0x5EED0005, r, t, i).astype(np.int64) for r in range(P)])
        x = k - 64 if prev is None else ((prev[None, :] + k) % 129) - 64      # Python-style mod: result in [0,128]
        assert x.min() >= -64 and x.max() <= 64
        tot = x.sum(axis=0)
        want = np.array([int_to_bf16_bits(int(v)) for v in tot], dtype=np.uint16)
        np.testing.assert_array_equal(outs[s], want)
        prev = np.array([int(bf16_bits_to_value(int(b))) for b in want], dtype=np.int64)


def test_chain_is_composition_of_steps(oracle):
    P, n, steps = 2, 300, 6
    w = oracle.Workload(oracle.KIND_GAUSS, 0x5EED0001, 1.0, 0.1, 0, 0)
    outs = oracle.chain(w, P, n, BF16, steps)
    prev = None
    for s in range(steps):
        xs = [oracle.workload_first(w, r, n, BF16) if s == 0 else oracle.workload_next(w, r, s + 1, prev, BF16)
              for r in range(P)]
        prev = oracle.allreduce(xs, BF16)
        np.testing.assert_array_equal(outs[s], prev)
    # resuming in the middle gives the same tail
    tail = oracle.chain(w, P, n, BF16, 3, t0=4, out_prev=outs[2])
    np.testing.assert_array_equal(tail, outs[3:6])


def test_fp32_chain_is_composition_of_steps_and_follows_the_float64_route(oracle):
    """The fp32 branch of the chain: every step equals the all-reduce of the ranks' next partials, a run resumed in
    the middle gives the same tail, and the whole chain is re-derived here through float64 (every product, the
    sum of the update and every rank-order add rounded to binary32 separately), which shares nothing with the C code."""
    P, n, steps = 3, 257, 7
    w = oracle.Workload(oracle.KIND_UNIFORM, 0x5EED0004, 1.0 / 3.0, 0.5, 0, 0)
    outs = oracle.chain(w, P, n, F32, steps)
    assert outs.dtype == np.float32 and outs.shape == (steps, n)
    prev = None
    for s in range(steps):
        xs = [oracle.workload_first(w, r, n, F32) if s == 0 else oracle.workload_next(w, r, s + 1, prev, F32)
              for r in range(P)]
        prev = oracle.allreduce(xs, F32)
        np.testing.assert_array_equal(outs[s].view(np.uint32), prev.view(np.uint32))
    tail = oracle.chain(w, P, n, F32, 3, t0=5, out_prev=outs[3])
    np.testing.assert_array_equal(tail.view(np.uint32), outs[4:7].view(np.uint32))
    # float64 route: binary32 products and sums are exact in binary64, so one rounding each reproduces them
    i = np.arange(n, dtype=np.uint32)
    f32, f64 = np.float32, np.float64
    prev = None
    for s in range(steps):
        t = s + 1
        xs = []
        for r in range(P):
            z = synth.uniform(0x5EED0004, r, t, i)
            if prev is None:
                xs.append(z.astype(f32))
            else:
                a = (prev.astype(f64) * f64(f32(1.0 / 3.0))).astype(f32)
                b = (z.astype(f64) * f64(f32(0.5))).astype(f32)
                xs.append((a.astype(f64) + b.astype(f64)).astype(f32))
        acc = xs[0]
        for r in range(1, P):
            acc = (acc.astype(f64) + xs[r].astype(f64)).astype(f32)
        np.testing.assert_array_equal(outs[s].view(np.uint32), acc.view(np.uint32))
        prev = acc
