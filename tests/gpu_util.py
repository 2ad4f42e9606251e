"""Helpers of the GPU parity tests: torch is used for device memory and streams only."""
from __future__ import annotations

import numpy as np
import torch

from paper_2607_08973_b200 import binding as sf

BF16, F32 = sf.BF16, sf.F32
MODES = (sf.BARRIER_ONESHOT, sf.DUALBUF, sf.SPECULATIVE)


def to_device(x: np.ndarray) -> torch.Tensor:
    """uint16 bit patterns travel as int16 tensors, float32 as float32."""
    if x.dtype == np.uint16:
        t = torch.from_numpy(x.view(np.int16).copy())
    else:
        t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32).copy())
    return t.cuda()


def empty_out(n: int, dtype: int) -> torch.Tensor:
    # a little slack, filled with a canary, so that writes past n are caught
    td = torch.int16 if dtype == BF16 else torch.float32
    t = torch.empty(n + 64, dtype=td, device="cuda")
    if dtype == BF16:
        t.fill_(0x5A5A)
    else:
        t.fill_(12345.0)
    return t


def out_to_numpy(t: torch.Tensor, n: int, dtype: int) -> tuple[np.ndarray, np.ndarray]:
    h = t.cpu().numpy()
    if dtype == BF16:
        h = h.view(np.uint16)
    return h[:n].copy(), h[n:].copy()


def canary_ok(tail: np.ndarray, dtype: int) -> bool:
    return bool(np.all(tail == (0x5A5A if dtype == BF16 else np.float32(12345.0))))


class Ctx:
    """Context manager around sifar_create / sifar_destroy."""

    def __init__(self, P: int, max_elems: int, dtype: int, timeout_us: int = 2_000_000):
        self.P, self.max_elems, self.dtype = P, max_elems, dtype
        self.h = sf.sifar_create(P, max_elems, dtype)
        sf.sifar_set_timeout_us(self.h, timeout_us)

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        if self.h:
            sf.lib().sifar_destroy(self.h)
            self.h = 0
        return False


def allreduce_via_pack(ctx: Ctx, xs_dev, n: int, mode: int, out: torch.Tensor,
                       producer_streams=None, reducer_stream=None) -> None:
    """Packs every rank on its own stream, then enqueues the reducer with no event in between."""
    P = ctx.P
    ps = producer_streams or [torch.cuda.Stream() for _ in range(P)]
    rs = reducer_stream or torch.cuda.Stream()
    for r in range(P):
        sf.sifar_pack(ctx.h, r, xs_dev[r].data_ptr(), n, mode, ps[r].cuda_stream)
    sf.sifar_allreduce(ctx.h, None, out.data_ptr(), n, mode, rs.cuda_stream)


def assert_bits_equal(got: np.ndarray, want: np.ndarray, dtype: int, what: str = "") -> None:
    if dtype == F32:
        g, w = got.view(np.uint32), want.view(np.uint32)
        nan = np.isnan(want)
        assert np.array_equal(np.isnan(got), nan), f"{what}: NaN pattern differs"
        bad = np.nonzero((g != w) & ~nan)[0]
    else:
        bad = np.nonzero(got != want)[0]
    assert bad.size == 0, f"{what}: {bad.size} mismatches, first at {bad[:5]}: got {got[bad[:5]]} want {want[bad[:5]]}"
