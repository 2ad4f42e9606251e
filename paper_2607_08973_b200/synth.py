"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds NO arithmetic of the all-reduce itself: it only produces input
tensors and names the workload recipes.  Both the CPU oracle and the CUDA library
are fed from here; neither of them imports the other.

Two sources of numbers:

* ``word`` / ``uniform`` / ``gauss`` / ``int129``: a numpy restatement of the
  integer counter generator that the decode-step workloads use on both sides
  (six chained 32-bit mixes over seed, stream, rank, step, element, lane).  All
  derived reals are exact in binary32.
* ``CONFIGS``: the five workload recipes (shapes, value distribution, chain
  length) that stand in for the paper's Llama-3.1-8B / Qwen3.5 decode workloads
  (Section 5 "Models"); no weights and no dataset items are involved.

bf16 tensors are returned as ``numpy.uint16`` bit patterns; the float->bf16 cast
of generated inputs uses torch's CPU cast (a library routine).
"""
from __future__ import annotations

import numpy as np

STREAM_VALUE, STREAM_OUTLIER, STREAM_DELAY = 1, 2, 3
KIND_GAUSS, KIND_INT, KIND_UNIFORM = 0, 1, 2
BF16, F32 = 0, 1

_M1, _M2, _GOLD = np.uint32(0x7FEB352D), np.uint32(0x846CA68B), np.uint32(0x9E3779B9)


def _mix(x: np.ndarray) -> np.ndarray:
    x = x.astype(np.uint32, copy=True)
    x ^= x >> np.uint32(16)
    x *= _M1
    x ^= x >> np.uint32(15)
    x *= _M2
    x ^= x >> np.uint32(16)
    return x


def word(seed, stream, r, t, i, k) -> np.ndarray:
    """Counter generator; every argument broadcasts as uint32."""
    with np.errstate(over="ignore"):
        u = lambda v: np.asarray(v, dtype=np.uint64).astype(np.uint32)
        h = _mix(u(seed))
        h = _mix(h ^ u(stream))
        h = _mix(h + u(r))
        h = _mix(h ^ (u(t) * _GOLD))
        h = _mix(h + u(i))
        h = _mix(h ^ u(k))
    return h


def uniform(seed, r, t, i) -> np.ndarray:
    w = word(seed, STREAM_VALUE, r, t, i, 0)
    c = (w >> np.uint32(8)).astype(np.int64) - (1 << 23)
    return (c.astype(np.float32) * np.float32(1.0 / 8388608.0)).astype(np.float32)


def gauss(seed, r, t, i) -> np.ndarray:
    i = np.asarray(i)
    s = np.zeros(i.shape, dtype=np.int64)
    for k in range(6):
        w = word(seed, STREAM_VALUE, r, t, i, k)
        s += (w & np.uint32(0xFFFF)).astype(np.int64) + (w >> np.uint32(16)).astype(np.int64)
    return ((s - 393210).astype(np.float32) * np.float32(1.0 / 65536.0)).astype(np.float32)


def int129(seed, r, t, i) -> np.ndarray:
    return (word(seed, STREAM_VALUE, r, t, i, 0) % np.uint32(129)).astype(np.int32)


def is_outlier(seed, r, i, outlier_mod) -> np.ndarray:
    if outlier_mod == 0:
        return np.zeros(np.shape(i), dtype=bool)
    return word(seed, STREAM_OUTLIER, r, 0, i, 0) % np.uint32(outlier_mod) == 0


def delay_ns(seed, r, t, delay_max_ns) -> np.ndarray:
    if delay_max_ns == 0:
        return np.zeros(np.shape(t), dtype=np.uint32)
    return word(seed, STREAM_DELAY, r, t, 0, 0) % np.uint32(delay_max_ns + 1)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns through torch's CPU cast."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def rank_inputs(P: int, n: int, dtype: int, seed: int, dist: str = "uniform",
                outlier_mod: int = 0) -> list[np.ndarray]:
    """P independent rank buffers for a single all-reduce call.

    ``dist``: "uniform" U(-1,1), "gauss" ~N(0,1), "int" integers in [-64, 64].
    """
    i = np.arange(n, dtype=np.uint32)
    xs = []
    for r in range(P):
        if dist == "uniform":
            v = uniform(seed, r, 1, i)
        elif dist == "gauss":
            v = gauss(seed, r, 1, i)
        elif dist == "int":
            v = (int129(seed, r, 1, i) - 64).astype(np.float32)
        else:
            raise ValueError(dist)
        if outlier_mod:
            v = np.where(is_outlier(seed, r, i, outlier_mod), v * np.float32(100.0), v).astype(np.float32)
        xs.append(to_bf16_bits(v) if dtype == BF16 else v)
    return xs


# ---------------------------------------------------------------------------
# Workload recipes.  kind/seed/scale/sigma/outlier_mod/delay_max_ns are the six
# fields of the workload descriptor that the oracle and the CUDA library each
# declare for themselves.
# ---------------------------------------------------------------------------
def chain_workload(name: str, P: int) -> dict:
    if name == "token":            # config 1: P=2, one token, next = previous + N(0, sigma=0.1)
        return dict(kind=KIND_GAUSS, seed=0x5EED0001, scale=1.0, sigma=0.1, outlier_mod=0, delay_max_ns=0)
    if name == "llama":            # config 2: 64 ARs, update = out/P + noise
        return dict(kind=KIND_GAUSS, seed=0x5EED0002, scale=1.0 / P, sigma=0.1, outlier_mod=0, delay_max_ns=0)
    if name == "moe":              # config 3: 120 ARs, 1% of first partials x100
        return dict(kind=KIND_GAUSS, seed=0x5EED0003, scale=1.0 / P, sigma=0.1, outlier_mod=100, delay_max_ns=0)
    if name == "sweep":            # config 4 chained: U(-1,1), update = out/P + 0.5*U
        return dict(kind=KIND_UNIFORM, seed=0x5EED0004, scale=1.0 / P, sigma=0.5, outlier_mod=0, delay_max_ns=0)
    if name == "skew":             # config 5: integers, 0-20 us producer delays
        return dict(kind=KIND_INT, seed=0x5EED0005, scale=1.0, sigma=1.0, outlier_mod=0, delay_max_ns=20000)
    raise ValueError(name)


CONFIGS = {
    1: dict(name="token", P=2, n=[4096], steps=64, dtype=BF16),
    2: dict(name="llama", P=8, n=[4096 * b for b in (1, 2, 4, 8, 16)], steps=64, dtype=BF16),
    3: dict(name="moe", P=8, n=[4096 * b for b in (1, 8, 32, 64)], steps=120, dtype=BF16),
    4: dict(name="sweep", P=[2, 4, 8], n=[1 << e for e in range(10, 26)], steps=100, dtype=[BF16, F32]),
    5: dict(name="skew", P=8, n=[16384], steps=10000, dtype=BF16),
}
