"""Thin ctypes binding of ``libsifar.so`` (``include/sifar.h``) and of
``libsifar_bench.so`` (``include/sifar_workload.h``): same names as the headers.

Argument marshalling only.  Every step of the all-reduce runs in the CUDA
library; there is no CPU fallback: if the library has not been built, the first
call raises.  Device pointers are plain integers (``tensor.data_ptr()``), streams
are ``torch.cuda.Stream().cuda_stream`` integers (0 = default stream).
"""
from __future__ import annotations

import ctypes
import os

BF16, F32 = 0, 1
BARRIER_ONESHOT, DUALBUF, SPECULATIVE = 0, 1, 2
OK, ERR_INVALID, ERR_NOMEM, ERR_CUDA, ERR_TIMEOUT, ERR_EPOCH = 0, -1, -2, -3, -4, -5
MODE_NAMES = {BARRIER_ONESHOT: "barrier_oneshot", DUALBUF: "dualbuf", SPECULATIVE: "speculative"}
FORMAT_SLOTS, FORMAT_TILES = 0, 1

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsifar.so")
_BENCH_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libsifar_bench.so")
_lib = None
_bench_lib = None


class SifarError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"sifar error {code}: {text}")
        self.code = code


def lib() -> ctypes.CDLL:
    """Load the CUDA library (once).  Raises if it is missing: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} not found: build it with `python -m paper_2607_08973_b200.build`; "
                "there is no CPU fallback")
        L = ctypes.CDLL(_LIB_PATH)
        vp, sz, ci, cu = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint
        sig = {
            "sifar_create": (vp, [ci, sz, ci]),
            "sifar_destroy": (ci, [vp]),
            "sifar_allreduce": (ci, [vp, vp, vp, sz, ci, vp]),
            "sifar_allreduce_host": (ci, [vp, vp, vp, sz, ci]),
            "sifar_rank_buffer": (ci, [vp, ci, ci, ctypes.POINTER(vp), ctypes.POINTER(cu)]),
            "sifar_pack": (ci, [vp, ci, vp, sz, ci, vp]),
            "sifar_arrive": (ci, [vp, ci, ci, vp]),
            "sifar_wait_writable": (ci, [vp, ci, vp]),
            "sifar_status": (ci, [vp]),
            "sifar_get_stats": (ci, [vp, ctypes.POINTER(ctypes.c_ulonglong)]),
            "sifar_set_timeout_us": (ci, [vp, cu]),
            "sifar_reset": (ci, [vp, vp]),
            "sifar_debug_set_epoch": (ci, [vp, cu]),
            "sifar_debug_force_retries": (ci, [vp, cu]),
            "sifar_debug_sweep_policy": (ci, [vp, ci]),
            "sifar_spec_format": (ci, [ci, ci, sz]),
            "sifar_tile_flags": (ci, [vp, ci, ctypes.POINTER(vp), ctypes.POINTER(sz), ctypes.POINTER(sz)]),
            "sifar_slot_count": (sz, [ci, sz]),
            "sifar_algorithmic_bytes": (sz, [ci, ci, sz, ci]),
            "sifar_last_error": (ctypes.c_char_p, []),
            "sifar_allreduce_noalloc": (ci, [vp, ci, vp, sz, ci, vp]),
            "sifar_noalloc_max_elems": (sz, []),
            "sifar_noalloc_counters": (ci, [ctypes.POINTER(ctypes.c_ulonglong)]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def sifar_last_error() -> str:
    return lib().sifar_last_error().decode()


def _check(rc: int) -> int:
    if rc != OK:
        raise SifarError(rc, sifar_last_error())
    return rc


def sifar_create(P: int, max_elems: int, dtype: int) -> int:
    h = lib().sifar_create(P, max_elems, dtype)
    if not h:
        raise SifarError(ERR_INVALID, sifar_last_error())
    return h


def sifar_destroy(ctx: int) -> int:
    return _check(lib().sifar_destroy(ctx))


def _ptr_array(ptrs):
    if ptrs is None:
        return None
    return (ctypes.c_void_p * len(ptrs))(*ptrs)


def sifar_allreduce(ctx: int, rank_ptrs, out: int, n: int, mode: int, stream: int = 0) -> int:
    return _check(lib().sifar_allreduce(ctx, _ptr_array(rank_ptrs), out, n, mode, stream))


def sifar_allreduce_host(ctx: int, host_rank_ptrs, host_out: int, n: int, mode: int) -> int:
    return _check(lib().sifar_allreduce_host(ctx, _ptr_array(host_rank_ptrs), host_out, n, mode))


def sifar_rank_buffer(ctx: int, rank: int, mode: int) -> tuple[int, int]:
    p, e = ctypes.c_void_p(), ctypes.c_uint()
    _check(lib().sifar_rank_buffer(ctx, rank, mode, ctypes.byref(p), ctypes.byref(e)))
    return (p.value or 0), e.value


def sifar_pack(ctx: int, rank: int, src: int, n: int, mode: int, stream: int = 0) -> int:
    return _check(lib().sifar_pack(ctx, rank, src, n, mode, stream))


def sifar_arrive(ctx: int, rank: int, mode: int, stream: int = 0) -> int:
    return _check(lib().sifar_arrive(ctx, rank, mode, stream))


def sifar_wait_writable(ctx: int, rank: int, stream: int = 0) -> int:
    return _check(lib().sifar_wait_writable(ctx, rank, stream))


def sifar_status(ctx: int) -> int:
    return lib().sifar_status(ctx)


def sifar_get_stats(ctx: int) -> dict:
    buf = (ctypes.c_ulonglong * 8)()
    _check(lib().sifar_get_stats(ctx, buf))
    keys = ("calls", "calls_with_retry", "slot_reloads", "flag_polls", "timeouts", "epoch")
    return {k: int(buf[i]) for i, k in enumerate(keys)}


def sifar_set_timeout_us(ctx: int, us: int) -> int:
    return _check(lib().sifar_set_timeout_us(ctx, us))


def sifar_reset(ctx: int, stream: int = 0) -> int:
    return _check(lib().sifar_reset(ctx, stream))


def sifar_debug_set_epoch(ctx: int, calls_so_far: int) -> int:
    return _check(lib().sifar_debug_set_epoch(ctx, calls_so_far))


def sifar_spec_format(P: int, dtype: int, n: int) -> int:
    fmt = lib().sifar_spec_format(P, dtype, n)
    if fmt < 0:
        raise SifarError(fmt, sifar_last_error())
    return fmt


def sifar_tile_flags(ctx: int, rank: int) -> tuple[int, int, int]:
    """(device address of the rank's flag of block 0, elements per flag, words between two blocks' flags)."""
    p, k, st = ctypes.c_void_p(), ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().sifar_tile_flags(ctx, rank, ctypes.byref(p), ctypes.byref(k), ctypes.byref(st)))
    return (p.value or 0), k.value, st.value


def sifar_debug_force_retries(ctx: int, rounds: int) -> int:
    return _check(lib().sifar_debug_force_retries(ctx, rounds))


SWEEP_NEVER, SWEEP_AUTO, SWEEP_ALWAYS = 0, 1, 2


def sifar_debug_sweep_policy(ctx: int, policy: int) -> int:
    return _check(lib().sifar_debug_sweep_policy(ctx, policy))


def sifar_slot_count(dtype: int, n: int) -> int:
    return lib().sifar_slot_count(dtype, n)


def sifar_algorithmic_bytes(P: int, dtype: int, n: int, mode: int) -> int:
    return lib().sifar_algorithmic_bytes(P, dtype, n, mode)


def sifar_allreduce_noalloc(rank_ptrs, out: int, n: int, dtype: int, stream: int = 0) -> int:
    """All-reduce of ready plain partials for callers that must not allocate (see include/sifar.h)."""
    return _check(lib().sifar_allreduce_noalloc(_ptr_array(rank_ptrs), len(rank_ptrs), out, n, dtype, stream))


def sifar_noalloc_max_elems() -> int:
    return lib().sifar_noalloc_max_elems()


def sifar_noalloc_counters() -> dict:
    buf = (ctypes.c_ulonglong * 3)()
    _check(lib().sifar_noalloc_counters(buf))
    return {"cta_arrive": int(buf[0]), "calls": int(buf[1]), "elements": int(buf[2])}


# ---------------------------------------------------------------------------
# include/sifar_workload.h (libsifar_bench.so): synthetic decode-step chains
# ---------------------------------------------------------------------------
CHAIN_STREAMS, CHAIN_GRAPH, CHAIN_PERSISTENT = 0, 1, 2
CHAIN_NO_ALLREDUCE = 3
SYMCHAIN_TWOSHOT = 4
SYMCHAIN_FLAGVAL, SYMCHAIN_FLAGVAL_ORDERED, SYMCHAIN_UNCHECKED = 5, 6, 7
IMPL_NAMES = {CHAIN_STREAMS: "streams", CHAIN_GRAPH: "graph", CHAIN_PERSISTENT: "persistent"}


class sifar_workload(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("seed", ctypes.c_uint), ("scale", ctypes.c_float),
                ("sigma", ctypes.c_float), ("outlier_mod", ctypes.c_uint), ("delay_max_ns", ctypes.c_uint)]


def make_workload(kind: int, seed: int, scale: float, sigma: float, outlier_mod: int = 0,
                  delay_max_ns: int = 0) -> sifar_workload:
    return sifar_workload(kind, seed, scale, sigma, outlier_mod, delay_max_ns)


def _wl() -> ctypes.CDLL:
    """Load the workload library (once); it links against libsifar.so, which is loaded first."""
    global _bench_lib
    if _bench_lib is None:
        lib()
        if not os.path.exists(_BENCH_LIB_PATH):
            raise RuntimeError(
                f"{_BENCH_LIB_PATH} not found: build it with `python -m paper_2607_08973_b200.build`; "
                "there is no CPU fallback")
        L = ctypes.CDLL(_BENCH_LIB_PATH)
        vp, sz, ci, cu = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_uint
        wp = ctypes.POINTER(sifar_workload)
        ullp = ctypes.POINTER(ctypes.c_ulonglong)
        sig = {
            "sifar_chain_ring_stride": (sz, [ci, sz]),
            "sifar_chain_create": (vp, [vp, wp, sz, ci, ci, vp, ci, ci]),
            "sifar_chain_run": (ci, [vp, vp]),
            "sifar_chain_stamps": (ci, [vp, ullp]),
            "sifar_chain_chunk_stamps": (ci, [vp, ci, ullp]),
            "sifar_chain_chunks": (ci, [vp]),
            "sifar_chain_geometry": (ci, [vp, ctypes.POINTER(ctypes.c_uint)]),
            "sifar_chain_launches_per_run": (ci, [vp]),
            "sifar_chain_trace": (ci, [vp, ci, ullp]),
            "sifar_chain_destroy": (ci, [vp]),
            "sifar_symchain_create": (vp, [vp, wp, sz, ci, vp, ci, ci]),
            "sifar_symchain_run": (ci, [vp, vp]),
            "sifar_symchain_stamps": (ci, [vp, ullp]),
            "sifar_symchain_rank_stamps": (ci, [vp, ci, ullp]),
            "sifar_symchain_retries": (ci, [vp, ullp]),
            "sifar_symchain_destroy": (ci, [vp]),
            "sifar_workload_first": (ci, [wp, ci, ci, vp, sz, vp]),
            "sifar_workload_next": (ci, [wp, ci, cu, ci, vp, vp, sz, vp]),
            "sifar_workload_delays": (ci, [wp, ci, cu, ctypes.POINTER(cu)]),
            "sifar_spin": (ci, [cu, vp]),
            "sifar_tear_check": (ci, [cu, cu, ullp, ullp]),
            "sifar_workload_preload": (ci, []),
            "sifar_store_slots": (ci, [vp, vp, sz, sz, sz, ci, cu, vp]),
            "sifar_store_blocks": (ci, [vp, vp, vp, sz, sz, sz, sz, ci, cu, vp]),
        }
        for name, (res, args) in sig.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _bench_lib = L
    return _bench_lib


def sifar_workload_preload() -> int:
    """Loads the helper kernels' code now, so that no later first launch has to wait for an idle device."""
    return _check(_wl().sifar_workload_preload())


def sifar_chain_ring_stride(dtype: int, n: int) -> int:
    return _wl().sifar_chain_ring_stride(dtype, n)


def sifar_chain_create(ctx: int, w: sifar_workload, n: int, mode: int, impl: int, out_ring: int, ring_len: int,
                       steps_per_run: int) -> int:
    h = _wl().sifar_chain_create(ctx, ctypes.byref(w), n, mode, impl, out_ring, ring_len, steps_per_run)
    if not h:
        raise SifarError(ERR_INVALID, sifar_last_error())
    return h


def sifar_chain_run(chain: int, stream: int = 0) -> int:
    return _check(_wl().sifar_chain_run(chain, stream))


def sifar_chain_stamps(chain: int, steps_per_run: int) -> list[int]:
    buf = (ctypes.c_ulonglong * (steps_per_run + 1))()
    _check(_wl().sifar_chain_stamps(chain, buf))
    return list(buf)


def sifar_chain_chunk_stamps(chain: int, chunk: int, steps_per_run: int) -> list[int]:
    buf = (ctypes.c_ulonglong * (steps_per_run + 1))()
    _check(_wl().sifar_chain_chunk_stamps(chain, chunk, buf))
    return list(buf)


def sifar_chain_chunks(chain: int) -> int:
    return _wl().sifar_chain_chunks(chain)


def sifar_chain_geometry(chain: int) -> dict:
    out = (ctypes.c_uint * 8)()
    _check(_wl().sifar_chain_geometry(chain, out))
    keys = ("chunks", "units_per_thread", "ctas", "clustered", "tagged", "kernel_clustered", "kernel_cluster_ctas",
            "kernel_tagged")
    return dict(zip(keys, (int(x) for x in out)))


def sifar_chain_trace(chain: int, enable: bool, steps_per_run: int = 0):
    """Switches the phase trace on/off; with steps_per_run > 0 also returns the last run's [steps][48] stamps."""
    if steps_per_run:
        buf = (ctypes.c_ulonglong * (steps_per_run * 48))()
        _check(_wl().sifar_chain_trace(chain, int(enable), buf))
        return [list(buf[i * 48:(i + 1) * 48]) for i in range(steps_per_run)]
    _check(_wl().sifar_chain_trace(chain, int(enable), None))
    return None


def sifar_chain_launches_per_run(chain: int) -> int:
    return _wl().sifar_chain_launches_per_run(chain)


def sifar_chain_destroy(chain: int) -> int:
    return _check(_wl().sifar_chain_destroy(chain))


def sifar_symchain_create(ctx: int, w: sifar_workload, n: int, mode: int, out_rings: int, ring_len: int,
                          steps_per_run: int) -> int:
    h = _wl().sifar_symchain_create(ctx, ctypes.byref(w), n, mode, out_rings, ring_len, steps_per_run)
    if not h:
        raise SifarError(ERR_INVALID, sifar_last_error())
    return h


def sifar_symchain_run(chain: int, stream: int = 0) -> int:
    return _check(_wl().sifar_symchain_run(chain, stream))


def sifar_symchain_stamps(chain: int, steps_per_run: int) -> list[int]:
    buf = (ctypes.c_ulonglong * (steps_per_run + 1))()
    _check(_wl().sifar_symchain_stamps(chain, buf))
    return list(buf)


def sifar_symchain_rank_stamps(chain: int, rank: int, steps_per_run: int) -> list[int]:
    buf = (ctypes.c_ulonglong * (steps_per_run + 1))()
    _check(_wl().sifar_symchain_rank_stamps(chain, rank, buf))
    return list(buf)


def sifar_symchain_retries(chain: int, P: int) -> list[int]:
    buf = (ctypes.c_ulonglong * P)()
    _check(_wl().sifar_symchain_retries(chain, buf))
    return list(buf)


def sifar_symchain_destroy(chain: int) -> int:
    return _check(_wl().sifar_symchain_destroy(chain))


def sifar_workload_first(w: sifar_workload, rank: int, dtype: int, dst: int, n: int, stream: int = 0) -> int:
    return _check(_wl().sifar_workload_first(ctypes.byref(w), rank, dtype, dst, n, stream))


def sifar_workload_next(w: sifar_workload, rank: int, t: int, dtype: int, prev_out: int, dst: int, n: int,
                        stream: int = 0) -> int:
    return _check(_wl().sifar_workload_next(ctypes.byref(w), rank, t, dtype, prev_out, dst, n, stream))


def sifar_workload_delays(w: sifar_workload, P: int, t: int) -> list[int]:
    buf = (ctypes.c_uint * P)()
    _check(_wl().sifar_workload_delays(ctypes.byref(w), P, t, buf))
    return list(buf)


def sifar_spin(ns: int, stream: int = 0) -> int:
    return _check(_wl().sifar_spin(ns, stream))


def sifar_tear_check(nslots: int, rounds: int) -> tuple[int, int]:
    torn, reads = ctypes.c_ulonglong(), ctypes.c_ulonglong()
    _check(_wl().sifar_tear_check(nslots, rounds, ctypes.byref(torn), ctypes.byref(reads)))
    return torn.value, reads.value


def sifar_store_slots(src: int, slots: int, first_slot: int, nslots: int, n: int, dtype: int, tag: int,
                      stream: int = 0) -> int:
    return _check(_wl().sifar_store_slots(src, slots, first_slot, nslots, n, dtype, tag, stream))


def sifar_store_blocks(src: int, dst: int, flags: int, stride_words: int, first_block: int, nblocks: int, n: int,
                       dtype: int, tag: int, stream: int = 0) -> int:
    return _check(_wl().sifar_store_blocks(src, dst, flags, stride_words, first_block, nblocks, n, dtype, tag, stream))
