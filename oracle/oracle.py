"""ctypes face of `hisparse_oracle.c` (the plain single-threaded CPU oracle).

TEST INFRASTRUCTURE ONLY: see the header of `hisparse_oracle.c` for what it restates from the
paper and how it is pinned.  This module only marshals arguments.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hisparse_oracle.c")
_SO = os.path.join(_HERE, "_hisparse_oracle.so")

STATUS_OUT_OF_RANGE = 1
STATUS_DUPLICATE = 2
FLAG_NO_BYTES = 1
POLICY_LRU, POLICY_FIFO, POLICY_RANDOM = 0, 1, 2


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _SO)
    return _SO


_lib = None


def _L() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, i64, u32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32
        L.oracle_create.argtypes = [i32, i32, i32, i32, i32, i64, vp, vp, vp, u32]
        L.oracle_create.restype = vp
        L.oracle_destroy.argtypes = [vp]
        L.oracle_destroy.restype = None
        L.oracle_append.argtypes = [vp, vp]
        L.oracle_append.restype = i32
        L.oracle_prefetch.argtypes = [vp, i32]
        L.oracle_prefetch.restype = i32
        L.oracle_resolve.argtypes = [vp, i32, vp, vp, vp, vp]
        L.oracle_resolve.restype = i32
        for name in ("oracle_slot_pos", "oracle_last_use", "oracle_pos2slot", "oracle_plan_pos", "oracle_plan_slot"):
            getattr(L, name).argtypes = [vp, i32, i32]
            getattr(L, name).restype = vp
        L.oracle_plan_n.argtypes = [vp, i32, i32]
        L.oracle_plan_n.restype = ctypes.c_int32
        L.oracle_steps.argtypes = [vp, i32, i32]
        L.oracle_steps.restype = u32
        L.oracle_pool.argtypes = [vp, i32]
        L.oracle_pool.restype = vp
        L.oracle_len.argtypes = [vp, i32]
        L.oracle_len.restype = i64
        L.oracle_newest.argtypes = [vp, i32]
        L.oracle_newest.restype = i64
        L.oracle_status.argtypes = [vp]
        L.oracle_status.restype = u32
        L.oracle_clear_status.argtypes = [vp]
        L.oracle_clear_status.restype = None
        L.oracle_set_policy.argtypes = [vp, i32, ctypes.c_uint64]
        L.oracle_set_policy.restype = i32
        L.oracle_mix64_value.argtypes = [ctypes.c_uint64]
        L.oracle_mix64_value.restype = ctypes.c_uint64
        L.oracle_random_key_value.argtypes = [ctypes.c_uint64, i32, i32, u32, i32]
        L.oracle_random_key_value.restype = u32
        L.oracle_kv_footprint_bytes.argtypes = [i64, i64, i64, i64]
        L.oracle_kv_footprint_bytes.restype = i64
        _lib = L
    return _lib


def kv_footprint_bytes(N: int, L: int, slots: int, record_bytes: int) -> int:
    return int(_L().oracle_kv_footprint_bytes(N, L, slots, record_bytes))


def mix64(z: int) -> int:
    """The oracle's 64-bit mixing function (exported so that a test can pin it)."""
    return int(_L().oracle_mix64_value(z & 0xFFFFFFFFFFFFFFFF))


def random_key(seed: int, r: int, g: int, t: int, slot: int) -> int:
    """The oracle's key of the RANDOM replacement policy for one slot."""
    return int(_L().oracle_random_key_value(seed & 0xFFFFFFFFFFFFFFFF, r, g, t, slot))


def _view(ptr: int, n: int, dtype) -> np.ndarray:
    ct = {np.int32: ctypes.c_int32, np.uint32: ctypes.c_uint32, np.uint8: ctypes.c_uint8}[dtype]
    return np.ctypeslib.as_array(ctypes.cast(ptr, ctypes.POINTER(ct)), shape=(n,))


class Oracle:
    """One oracle instance = one set of (request, layer) caches over caller-owned host histories.

    `host_history[r]` is a writable uint8 numpy array `[L][capacity[r]][E]` (the oracle's appends
    write through into it); pass `flags=FLAG_NO_BYTES` to track metadata only, in which case the
    histories may be omitted.
    """

    def __init__(self, num_requests: int, num_layers: int, layers_per_group: int, cache_slots: int,
                 top_k: int, entry_bytes: int, capacity: Sequence[int], init_len: Sequence[int],
                 host_history: Sequence[np.ndarray] | None = None, flags: int = 0, policy: int = POLICY_LRU,
                 policy_seed: int = 0):
        self.N, self.L, self.lpg, self.B, self.k, self.E = (num_requests, num_layers, layers_per_group,
                                                            cache_slots, top_k, entry_bytes)
        self.capacity = np.asarray(capacity, dtype=np.int64)
        self._init_len = np.asarray(init_len, dtype=np.int64)
        self._host: List[np.ndarray] = list(host_history) if host_history is not None else []
        host_ptrs = None
        if self._host:
            for r, h in enumerate(self._host):
                assert h.dtype == np.uint8 and h.flags.c_contiguous
                assert h.size == num_layers * int(self.capacity[r]) * entry_bytes
            host_ptrs = (ctypes.c_void_p * num_requests)(*[h.ctypes.data for h in self._host])
        elif not (flags & FLAG_NO_BYTES):
            raise ValueError("host_history is required unless FLAG_NO_BYTES is set")
        self._h = _L().oracle_create(num_requests, num_layers, layers_per_group, cache_slots, top_k,
                                     entry_bytes, self.capacity.ctypes.data, self._init_len.ctypes.data,
                                     host_ptrs, flags)
        if not self._h:
            raise ValueError("oracle_create rejected the configuration")
        self.flags = flags
        if _L().oracle_set_policy(self._h, policy, policy_seed) != 0:
            raise ValueError("unknown replacement policy")
        self.policy = policy

    def close(self):
        if getattr(self, "_h", None):
            _L().oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def append(self, new_kv: np.ndarray | None = None) -> None:
        if self.flags & FLAG_NO_BYTES:
            rc = _L().oracle_append(self._h, None)
        else:
            a = np.ascontiguousarray(new_kv, dtype=np.uint8)
            assert a.size == self.N * self.L * self.E
            rc = _L().oracle_append(self._h, a.ctypes.data)
        if rc != 0:
            raise RuntimeError("oracle_append: history capacity exhausted")

    def resolve(self, layer: int, sel: np.ndarray):
        sel = np.ascontiguousarray(sel, dtype=np.int32).reshape(self.N, self.k)
        table = np.empty((self.N, self.k), dtype=np.int32)
        hits = np.empty(self.N, dtype=np.int32)
        misses = np.empty(self.N, dtype=np.int32)
        rc = _L().oracle_resolve(self._h, layer, sel.ctypes.data, table.ctypes.data, hits.ctypes.data,
                                 misses.ctypes.data)
        if rc != 0:
            raise ValueError("oracle_resolve: bad layer")
        return table, hits, misses

    def prefetch(self, layer: int) -> None:
        if _L().oracle_prefetch(self._h, layer) != 0:
            raise ValueError("oracle_prefetch: not a shared layer")

    # ---- state ----
    def slot_pos(self, r: int, layer: int) -> np.ndarray:
        return _view(_L().oracle_slot_pos(self._h, r, layer), self.B, np.int32).copy()

    def last_use(self, r: int, layer: int) -> np.ndarray:
        return _view(_L().oracle_last_use(self._h, r, layer), self.B, np.uint32).copy()

    def pos2slot(self, r: int, layer: int) -> np.ndarray:
        return _view(_L().oracle_pos2slot(self._h, r, layer), int(self.capacity[r]), np.int32).copy()

    def plan(self, r: int, layer: int):
        n = int(_L().oracle_plan_n(self._h, r, layer))
        pos = _view(_L().oracle_plan_pos(self._h, r, layer), self.k, np.int32)[:n].copy()
        slot = _view(_L().oracle_plan_slot(self._h, r, layer), self.k, np.int32)[:n].copy()
        return pos, slot

    def pool(self, layer: int) -> np.ndarray:
        """Cache pool of one layer, `[N][B+1][E]` bytes (slot B is the reserved newest-token slot)."""
        p = _L().oracle_pool(self._h, layer)
        return _view(p, self.N * (self.B + 1) * self.E, np.uint8).reshape(self.N, self.B + 1, self.E)

    def length(self, r: int) -> int:
        return int(_L().oracle_len(self._h, r))

    def newest(self, r: int) -> int:
        return int(_L().oracle_newest(self._h, r))

    def steps(self, r: int, layer: int) -> int:
        return int(_L().oracle_steps(self._h, r, layer))

    @property
    def status(self) -> int:
        return int(_L().oracle_status(self._h))

    def clear_status(self) -> None:
        _L().oracle_clear_status(self._h)
