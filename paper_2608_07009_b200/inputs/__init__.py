"""Seeded synthetic inputs: host KV-history bytes and DSA/NSA/Quest-shaped selection traces.

This module only draws inputs (no cache arithmetic lives here).  The CPU oracle's tests and the
CUDA path's tests and benchmark both take their inputs from it, so that neither side ever feeds
the other.  The generator itself is `tracegen.c` (plain C, counter-based splitmix64 streams),
built into `_tracegen.so` next to this file and called through ctypes.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess
from typing import List, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tracegen.c")
_SO = os.path.join(_HERE, "_tracegen.so")

KIND_DSA_ZIPF, KIND_DSA_MIX, KIND_NSA_BLOCKS, KIND_QUEST_PAGES = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile tracegen.c with gcc (a few hundred ms); returns the shared library's path."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm", "-lpthread"])
        os.replace(tmp, _SO)
    return _SO


class _TraceParams(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_int32), ("num_requests", ctypes.c_int32), ("num_streams", ctypes.c_int32),
        ("top_k", ctypes.c_int32), ("append_every", ctypes.c_int32), ("recent_window", ctypes.c_int32),
        ("zipf_support", ctypes.c_int32), ("keep", ctypes.c_int32), ("zipf_s", ctypes.c_double),
        ("ar_rho", ctypes.c_double), ("seed", ctypes.c_uint64), ("config_id", ctypes.c_int32),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.hs_record_fill.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                     ctypes.c_int64, ctypes.c_uint64]
        L.hs_record_fill.restype = None
        L.hs_history_fill.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                      ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_uint64,
                                      ctypes.c_int]
        L.hs_history_fill.restype = None
        L.hs_new_kv_fill.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                     ctypes.c_int64, ctypes.c_uint64]
        L.hs_new_kv_fill.restype = None
        L.hs_trace_create.argtypes = [ctypes.POINTER(_TraceParams), ctypes.c_void_p, ctypes.c_void_p]
        L.hs_trace_create.restype = ctypes.c_void_p
        L.hs_trace_destroy.argtypes = [ctypes.c_void_p]
        L.hs_trace_destroy.restype = None
        L.hs_trace_step.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.hs_trace_step.restype = None
        _lib = L
    return _lib


# ----------------------------------------------------------------------------- workloads


@dataclasses.dataclass
class Workload:
    """One synthetic workload: cache geometry plus the recipe of its selection trace."""
    name: str
    kind: int
    num_requests: int          # N
    num_layers: int            # L
    layers_per_group: int      # layers sharing one selection stream (1 = every layer selects)
    top_k: int                 # k
    cache_slots: int           # B
    entry_bytes: int           # E
    init_len: List[int]        # records already in host history per request
    steps: int
    append_every: int = 1
    keep: int = 0              # row entries kept from the previous step
    recent_window: int = 1024
    zipf_support: int = 0
    zipf_s: float = 1.0
    ar_rho: float = 0.0
    seed: int = 0
    config_id: int = 0

    @property
    def num_groups(self) -> int:
        return self.num_layers // self.layers_per_group

    @property
    def capacity(self) -> List[int]:
        extra = self.steps // self.append_every + 1
        return [n + extra for n in self.init_len]

    def host_bytes(self) -> int:
        return sum(self.num_layers * c * self.entry_bytes for c in self.capacity)

    def device_pool_bytes(self) -> int:
        return self.num_requests * self.num_layers * (self.cache_slots + 1) * self.entry_bytes


def c1_tiny_dsa(seed: int = 0) -> Workload:
    """1 request, 1 layer, 8192 tokens, 1152-B records, k=256, B=1024, 64 steps; 80 % of each row
    kept, the rest redrawn from Zipf(1.1) over recency rank; one token appended per step."""
    return Workload("c1_tiny_dsa", KIND_DSA_ZIPF, 1, 1, 1, 256, 1024, 1152, [8192], 64,
                    keep=round(0.8 * 256), zipf_support=8192, zipf_s=1.1, seed=seed, config_id=1)


def c2_dsa_decode(seed: int = 0, num_requests: int = 32, num_layers: int = 16, steps: int = 256,
                  context: int = 32768) -> Workload:
    """32 requests x 16 layers, 32768 tokens, k=2048, B=4096; 90 % kept, of the 205 redrawn 102 come
    from the last 1024 tokens and 103 are uniform over the history."""
    return Workload("c2_dsa_decode", KIND_DSA_MIX, num_requests, num_layers, 1, 2048, 4096, 1152,
                    [context] * num_requests, steps, keep=round(0.9 * 2048), recent_window=1024,
                    seed=seed, config_id=2)


def c3_dsa_long(overlap: float = 0.9, seed: int = 0, steps: int = 128, short_ctx: int = 131072,
                long_ctx: int = 1048576, num_short: int = 8) -> Workload:
    """8 requests at 131072 tokens plus one at 1048576; 8 layers in 2 groups of 4 that share their
    selections (anchor layers 0 and 4); k=2048, B=4096; overlap is swept over 0.5/0.75/0.9/0.98."""
    return Workload("c3_dsa_long_ov%02d" % round(overlap * 100), KIND_DSA_MIX, num_short + 1, 8, 4,
                    2048, 4096, 1152, [short_ctx] * num_short + [long_ctx], steps,
                    keep=round(overlap * 2048), recent_window=1024, seed=seed, config_id=3)


def c4_nsa_blocks(seed: int = 0, num_requests: int = 16, num_layers: int = 16, steps: int = 256) -> Workload:
    """16 requests x 16 layers, 1024 blocks of 128 KiB (64 tokens x 4 KV heads x 128 dim x K,V bf16),
    16 selected + 2 local blocks, B=64 blocks; 14 of 16 kept, 2 redrawn by Zipf(1.0) over a fixed
    seeded popularity order of the 1022 non-local blocks; a block completes every 64 steps."""
    return Workload("c4_nsa_blocks", KIND_NSA_BLOCKS, num_requests, num_layers, 1, 18, 64, 131072,
                    [1024] * num_requests, steps, append_every=64, keep=14, zipf_support=1022,
                    zipf_s=1.0, seed=seed, config_id=4)


def c5_quest_pages(seed: int = 0, num_requests: int = 16, num_layers: int = 32, steps: int = 64) -> Workload:
    """16 requests x 32 layers, 2048 pages of 64 KiB (16 tokens x 8 KV heads x 128 dim x K,V bf16),
    top-256 pages of Gaussian scores with AR(1) drift 0.95, B=512 pages; a page every 16 steps."""
    return Workload("c5_quest_pages", KIND_QUEST_PAGES, num_requests, num_layers, 1, 256, 512, 65536,
                    [2048] * num_requests, steps, append_every=16, ar_rho=0.95, seed=seed, config_id=5)


def scaled_all_hit(num_requests: int = 2048, seed: int = 0) -> Workload:
    """Supplementary point for the all-hit metadata path: many requests, one layer, k=2048, B=4096,
    tiny records, rows repeated unchanged (keep = k) so that every selection hits after step 1."""
    return Workload("scaled_all_hit", KIND_DSA_MIX, num_requests, 1, 1, 2048, 4096, 16,
                    [8192] * num_requests, 8, append_every=1 << 30, keep=2048, seed=seed, config_id=6)


class Trace:
    """Iterator over decode steps of a workload's selection trace.

    `step()` returns `(sel, appended, lens)`: `sel` is int32 `[G][N][k]` (row g feeds the resolve of
    anchor layer g*layers_per_group), `appended` says whether every request appends one record
    BEFORE this step's resolves, `lens` is the history length the rows were drawn against.
    """

    def __init__(self, w: Workload):
        self.w = w
        p = _TraceParams(w.kind, w.num_requests, w.num_groups, w.top_k, w.append_every, w.recent_window,
                         w.zipf_support, w.keep, w.zipf_s, w.ar_rho, w.seed, w.config_id)
        init_len = np.asarray(w.init_len, dtype=np.int64)
        cap = np.asarray(w.capacity, dtype=np.int64)
        self._h = lib().hs_trace_create(ctypes.byref(p), init_len.ctypes.data, cap.ctypes.data)
        self.lens = init_len.copy()

    def step(self):
        w = self.w
        sel = np.empty((w.num_groups, w.num_requests, w.top_k), dtype=np.int32)
        appended = ctypes.c_int32(0)
        lens = np.empty(w.num_requests, dtype=np.int64)
        lib().hs_trace_step(self._h, sel.ctypes.data, ctypes.byref(appended), lens.ctypes.data)
        self.lens = lens
        return sel, bool(appended.value), lens

    def close(self):
        if self._h:
            lib().hs_trace_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ----------------------------------------------------------------------------- history bytes


def record_bytes(r: int, layer: int, pos: int, entry_bytes: int, seed: int = 0) -> np.ndarray:
    out = np.empty(entry_bytes, dtype=np.uint8)
    lib().hs_record_fill(out.ctypes.data, r, layer, pos, entry_bytes, seed)
    return out


def fill_history(base_ptr: int, r: int, num_layers: int, capacity: int, pos0: int, pos1: int,
                 entry_bytes: int, seed: int = 0, threads: Optional[int] = None) -> None:
    """Fill request r's history buffer (layout [L][capacity][E]) for pos0 <= pos < pos1."""
    if threads is None:
        threads = min(32, os.cpu_count() or 1)
    lib().hs_history_fill(base_ptr, r, num_layers, capacity, pos0, pos1, entry_bytes, seed, threads)


def new_history(w: Workload, r: int) -> np.ndarray:
    """A pageable numpy history buffer for request r, filled up to its initial length."""
    cap = w.capacity[r]
    buf = np.zeros((w.num_layers, cap, w.entry_bytes), dtype=np.uint8)
    fill_history(buf.ctypes.data, r, w.num_layers, cap, 0, w.init_len[r], w.entry_bytes, w.seed)
    return buf


def new_kv(w: Workload, positions: np.ndarray) -> np.ndarray:
    """Records `[N][L][E]` appended at this step: request r appends position positions[r]."""
    out = np.empty((w.num_requests, w.num_layers, w.entry_bytes), dtype=np.uint8)
    pos = np.ascontiguousarray(positions, dtype=np.int64)
    lib().hs_new_kv_fill(out.ctypes.data, w.num_requests, w.num_layers, pos.ctypes.data, w.entry_bytes, w.seed)
    return out


# ----------------------------------------------------------------------------- tiny random cases


def random_rows(rng: np.random.Generator, steps: int, k: int, universe: int, pad_prob: float = 0.0) -> np.ndarray:
    """`[steps][k]` rows of distinct positions drawn uniformly from [0, universe); each entry is
    replaced by the pad value -1 with probability pad_prob."""
    rows = np.empty((steps, k), dtype=np.int32)
    for s in range(steps):
        rows[s] = rng.permutation(universe)[:k] if universe >= k else -1
        if pad_prob > 0:
            rows[s][rng.random(k) < pad_prob] = -1
    return rows
