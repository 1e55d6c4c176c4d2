"""Thin Python binding of the C-ABI in include/hisparse.h (argument marshalling only).

Every step of the path runs in the CUDA library `_hisparse.so`; this module passes pointers of
torch tensors and stream handles to it.  There is no fallback: if the library is missing, import
of the binding fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

OK, EINVAL, ENOTPINNED, ENOMEM, ECUDA, ESTATE, ETOOBIG = 0, -1, -2, -3, -4, -5, -6
NOALLOC_MAX_REQUESTS, NOALLOC_MAX_SELECTIONS = 1024, 65536
FLAG_SKIP_IO, FLAG_DEBUG_VALIDATE, FLAG_INLINE_WRITE_THROUGH, FLAG_PHASE_TIMERS, FLAG_NO_PDL = 1, 2, 4, 8, 16
FLAG_EAGER_ORDER, FLAG_WIDE_BLOCKS, FLAG_NARROW_BLOCKS = 32, 64, 128
STATUS_OUT_OF_RANGE, STATUS_DUPLICATE, STATUS_CAPACITY, STATUS_INCONSISTENT, STATUS_TIMEOUT = 1, 2, 4, 8, 16
MAX_CACHE_SLOTS, MAX_TOP_K = 16384, 4096
POLICY_LRU, POLICY_FIFO, POLICY_RANDOM = 0, 1, 2

EXPORTS = [
    "hisparse_create", "hisparse_destroy", "hisparse_append", "hisparse_resolve", "hisparse_prefetch", "hisparse_prefetch_hint",
    "hisparse_join", "hisparse_layer_pool", "hisparse_gather", "hisparse_gather_check", "hisparse_status",
    "hisparse_clear_status", "hisparse_dump_state", "hisparse_order_lag", "hisparse_load_state", "hisparse_load_appends", "hisparse_dump_plan", "hisparse_device_bytes",
    "hisparse_launch_geometry", "hisparse_phase_times", "hisparse_layer_times", "hisparse_selftest_wait_timeout", "hisparse_host_alloc", "hisparse_host_free", "hisparse_host_link_probe",
    "hisparse_scatter_read_probe", "hisparse_resolve_noalloc", "hisparse_strerror", "hisparse_last_cuda_error",
    "hisparse_attention_workspace_bytes", "hisparse_sparse_attention",
]


class HiSparseError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        msg = lib().hisparse_strerror(code).decode()
        if code == ECUDA:
            msg += " (cudaError %d)" % lib().hisparse_last_cuda_error()
        super().__init__("%s: %s" % (what, msg))


class Config(ctypes.Structure):
    _fields_ = [
        ("num_requests", ctypes.c_int32), ("num_layers", ctypes.c_int32), ("layers_per_group", ctypes.c_int32),
        ("cache_slots", ctypes.c_int32), ("top_k", ctypes.c_int32), ("entry_bytes", ctypes.c_int64),
        ("capacity", ctypes.c_void_p), ("init_len", ctypes.c_void_p), ("host_history", ctypes.c_void_p),
        ("device", ctypes.c_int32), ("flags", ctypes.c_uint32), ("ctas_per_request", ctypes.c_int32),
        ("policy", ctypes.c_int32), ("policy_seed", ctypes.c_uint64),
    ]


class ExternalState(ctypes.Structure):
    """hisparse_external_state_t: caller-owned state of one layer's caches (see hisparse_resolve_noalloc)."""
    _fields_ = [
        ("num_requests", ctypes.c_int32), ("cache_slots", ctypes.c_int32), ("top_k", ctypes.c_int32),
        ("entry_bytes", ctypes.c_int64), ("device", ctypes.c_int32), ("pool_dev", ctypes.c_void_p),
        ("slot_pos_dev", ctypes.c_void_p), ("last_use_dev", ctypes.c_void_p), ("lru_order_dev", ctypes.c_void_p),
        ("pos2slot_dev", ctypes.c_void_p), ("capacity_dev", ctypes.c_void_p), ("init_len_dev", ctypes.c_void_p),
        ("p2s_offset_dev", ctypes.c_void_p), ("host_layer_dev", ctypes.c_void_p), ("resolves_dev", ctypes.c_void_p),
        ("num_appends_dev", ctypes.c_void_p),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """The CUDA library; raises if it has not been built (see build.build_cuda / __graft_entry__.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_build.SO):
            raise RuntimeError("CUDA library %s is missing: run `python -m paper_2608_07009_b200.build` "
                               "(there is no CPU fallback)" % _build.SO)
        L = ctypes.CDLL(_build.SO)
        vp, i32, i64, u32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32, ctypes.c_size_t
        P = ctypes.POINTER
        sig = {
            "hisparse_create": ([P(Config), P(vp)], i32),
            "hisparse_destroy": ([vp], i32),
            "hisparse_append": ([vp, vp, vp], i32),
            "hisparse_resolve": ([vp, i32, vp, vp, vp, vp, vp], i32),
            "hisparse_prefetch": ([vp, i32, vp], i32),
            "hisparse_prefetch_hint": ([vp, i32, vp, vp, vp], i32),
            "hisparse_join": ([vp, vp], i32),
            "hisparse_layer_pool": ([vp, i32], vp),
            "hisparse_gather": ([vp, i32, vp, vp, vp], i32),
            "hisparse_gather_check": ([vp, i32, vp, vp, vp, vp], i32),
            "hisparse_status": ([vp, P(u32)], i32),
            "hisparse_clear_status": ([vp], i32),
            "hisparse_dump_state": ([vp, i32, i32, vp, vp, vp, vp, P(i64), P(i64), P(u32)], i32),
            "hisparse_load_state": ([vp, i32, i32, vp, vp, u32], i32),
            "hisparse_order_lag": ([vp, i32, i32, P(u32)], i32),
            "hisparse_load_appends": ([vp, ctypes.c_int32], i32),
            "hisparse_dump_plan": ([vp, i32, i32, vp, vp, P(ctypes.c_int32)], i32),
            "hisparse_device_bytes": ([P(Config), P(sz), P(sz)], i32),
            "hisparse_launch_geometry": ([vp, P(ctypes.c_int32), P(ctypes.c_int32), P(ctypes.c_int32)], i32),
            "hisparse_phase_times": ([vp, vp], i32),
            "hisparse_layer_times": ([vp, vp], i32),
            "hisparse_selftest_wait_timeout": ([vp, ctypes.c_uint64, P(ctypes.c_uint64)], i32),
            "hisparse_host_alloc": ([sz, P(vp)], i32),
            "hisparse_host_free": ([vp], i32),
            "hisparse_host_link_probe": ([i32, sz, i32, P(ctypes.c_double)], i32),
            "hisparse_scatter_read_probe": ([i32, vp, sz, i64, ctypes.c_int32, ctypes.c_int32, i32, P(ctypes.c_double)], i32),
            "hisparse_resolve_noalloc": ([P(ExternalState), vp, vp, vp, vp, vp, vp], i32),
            "hisparse_attention_workspace_bytes": ([vp, i32, i32, P(sz)], i32),
            "hisparse_sparse_attention": ([vp, i32, vp, i32, i32, vp, ctypes.c_float, vp, vp, vp, sz, vp], i32),
            "hisparse_strerror": ([i32], ctypes.c_char_p),
            "hisparse_last_cuda_error": ([], i32),
        }
        for name, (args, res) in sig.items():
            fn = getattr(L, name)
            fn.argtypes, fn.restype = args, res
        _lib = L
    return _lib


def _check(code: int, what: str) -> None:
    if code != OK:
        raise HiSparseError(code, what)


def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _dev_ptr(t, dtype_name: str, numel: Optional[int] = None) -> int:
    import torch
    want = getattr(torch, dtype_name)
    if not (t.is_cuda and t.dtype == want and t.is_contiguous()):
        raise ValueError("expected a contiguous CUDA %s tensor" % dtype_name)
    if numel is not None and t.numel() != numel:
        raise ValueError("expected %d elements, got %d" % (numel, t.numel()))
    return t.data_ptr()


class HostHistory:
    """Pinned, device-mapped host memory for one request's KV history, laid out [L][capacity][E]."""

    def __init__(self, num_layers: int, capacity: int, entry_bytes: int):
        self.shape = (num_layers, capacity, entry_bytes)
        self.nbytes = num_layers * capacity * entry_bytes
        p = ctypes.c_void_p()
        _check(lib().hisparse_host_alloc(self.nbytes, ctypes.byref(p)), "hisparse_host_alloc")
        self.ptr = p.value

    def numpy(self) -> np.ndarray:
        buf = (ctypes.c_uint8 * self.nbytes).from_address(self.ptr)
        return np.frombuffer(buf, dtype=np.uint8).reshape(self.shape)

    def free(self) -> None:
        if self.ptr:
            _check(lib().hisparse_host_free(self.ptr), "hisparse_host_free")
            self.ptr = None


def device_bytes(num_requests, num_layers, layers_per_group, cache_slots, top_k, entry_bytes, capacity):
    cap = np.asarray(capacity, dtype=np.int64)
    il = np.zeros_like(cap)
    cfg = Config(num_requests, num_layers, layers_per_group, cache_slots, top_k, entry_bytes,
                 cap.ctypes.data, il.ctypes.data, None, 0, 0, 0, 0, 0)
    kv, meta = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().hisparse_device_bytes(ctypes.byref(cfg), ctypes.byref(kv), ctypes.byref(meta)), "hisparse_device_bytes")
    return kv.value, meta.value


def host_link_probe(device: int = 0, nbytes: int = 1 << 30, reps: int = 10) -> float:
    """Best-of-reps bulk pinned H2D memcpy bandwidth in GB/s (the host-link peak)."""
    out = ctypes.c_double()
    _check(lib().hisparse_host_link_probe(device, nbytes, reps, ctypes.byref(out)), "hisparse_host_link_probe")
    return out.value


def scatter_read_probe(host_ptr: int, host_bytes: int, entry_bytes: int, num_records: int, num_ctas: int,
                       reps: int = 5, device: int = 0) -> float:
    out = ctypes.c_double()
    _check(lib().hisparse_scatter_read_probe(device, host_ptr, host_bytes, entry_bytes, num_records, num_ctas, reps,
                                             ctypes.byref(out)), "hisparse_scatter_read_probe")
    return out.value


def resolve_noalloc(state: ExternalState, sel, slot_table, hits, misses, status=None, stream=None) -> None:
    """Resolve on caller-owned state without any device allocation (hisparse_resolve_noalloc).

    For callers that may not call cudaMalloc (all of HBM handed to their own allocator, or a stream capture in
    progress): every tensor is the caller's; the kernel's scratch is a fixed array inside the library.  Calls
    on one device share that array, so do not let two of them overlap on the GPU.
    """
    n, k = state.num_requests, state.top_k
    _check(lib().hisparse_resolve_noalloc(ctypes.byref(state), _dev_ptr(sel, "int32", n * k),
                                          _dev_ptr(slot_table, "int32", n * k), _dev_ptr(hits, "int32", n),
                                          _dev_ptr(misses, "int32", n),
                                          status.data_ptr() if status is not None else None, _stream_ptr(stream)),
           "hisparse_resolve_noalloc")


class HiSparse:
    """One handle = the caches and metadata of N requests on one GPU (see include/hisparse.h)."""

    def __init__(self, num_requests: int, num_layers: int, layers_per_group: int, cache_slots: int, top_k: int,
                 entry_bytes: int, capacity: Sequence[int], init_len: Sequence[int], host_history: Sequence,
                 device: int = 0, flags: int = 0, ctas_per_request: int = 0, policy: int = 0, policy_seed: int = 0):
        self.N, self.L, self.lpg, self.B, self.k, self.E = (num_requests, num_layers, layers_per_group, cache_slots,
                                                            top_k, entry_bytes)
        self.device = device
        self.capacity = np.ascontiguousarray(capacity, dtype=np.int64)
        self.init_len = np.ascontiguousarray(init_len, dtype=np.int64)
        if len(self.capacity) != num_requests or len(self.init_len) != num_requests or len(host_history) != num_requests:
            raise ValueError("capacity, init_len and host_history need one entry per request")
        self._hist = list(host_history)          # keep the pinned buffers alive
        ptrs = (ctypes.c_void_p * num_requests)(*[h.ptr if isinstance(h, HostHistory) else int(h) for h in host_history])
        cfg = Config(num_requests, num_layers, layers_per_group, cache_slots, top_k, entry_bytes,
                     self.capacity.ctypes.data, self.init_len.ctypes.data, ctypes.addressof(ptrs), device, flags,
                     ctas_per_request, policy, policy_seed)
        h = ctypes.c_void_p()
        _check(lib().hisparse_create(ctypes.byref(cfg), ctypes.byref(h)), "hisparse_create")
        self._h = h

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().hisparse_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the path ----
    def append(self, new_kv, stream=None) -> None:
        _check(lib().hisparse_append(self._h, _dev_ptr(new_kv, "uint8", self.N * self.L * self.E), _stream_ptr(stream)),
               "hisparse_append")

    def resolve(self, layer: int, sel, slot_table=None, hits=None, misses=None, stream=None):
        import torch
        dev = "cuda:%d" % self.device
        if slot_table is None:
            slot_table = torch.empty((self.N, self.k), dtype=torch.int32, device=dev)
        if hits is None:
            hits = torch.empty(self.N, dtype=torch.int32, device=dev)
        if misses is None:
            misses = torch.empty(self.N, dtype=torch.int32, device=dev)
        sel_ptr = _dev_ptr(sel, "int32", self.N * self.k) if sel is not None else None
        _check(lib().hisparse_resolve(self._h, layer, sel_ptr, _dev_ptr(slot_table, "int32", self.N * self.k),
                                      _dev_ptr(hits, "int32", self.N), _dev_ptr(misses, "int32", self.N),
                                      _stream_ptr(stream)), "hisparse_resolve")
        return slot_table, hits, misses

    def prefetch(self, layer: int, side_stream) -> None:
        _check(lib().hisparse_prefetch(self._h, layer, _stream_ptr(side_stream)), "hisparse_prefetch")

    def prefetch_hint(self, layer: int, hint_sel, side_stream, stream=None) -> None:
        _check(lib().hisparse_prefetch_hint(self._h, layer, _dev_ptr(hint_sel, "int32", self.N * self.k),
                                            _stream_ptr(stream), _stream_ptr(side_stream)), "hisparse_prefetch_hint")

    def join(self, stream=None) -> None:
        _check(lib().hisparse_join(self._h, _stream_ptr(stream)), "hisparse_join")

    # ---- the sparse-attention consumer ----
    def attention_workspace_bytes(self, num_heads: int, value_dims: int) -> int:
        n = ctypes.c_size_t()
        _check(lib().hisparse_attention_workspace_bytes(self._h, num_heads, value_dims, ctypes.byref(n)),
               "hisparse_attention_workspace_bytes")
        return n.value

    def sparse_attention(self, layer: int, q, slot_table, value_dims: int, scale: float, out=None, lse=None,
                         workspace=None, stream=None):
        """q: bf16 CUDA tensor [N][H][E/2]; returns (out float32 [N][H][value_dims], lse float32 [N][H])."""
        import torch
        dev = "cuda:%d" % self.device
        H = q.shape[1]
        if not (q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous() and q.shape == (self.N, H, self.E // 2)):
            raise ValueError("expected a contiguous CUDA bfloat16 tensor [N][H][E/2]")
        if out is None:
            out = torch.empty((self.N, H, value_dims), dtype=torch.float32, device=dev)
        if lse is None:
            lse = torch.empty((self.N, H), dtype=torch.float32, device=dev)
        need = self.attention_workspace_bytes(H, value_dims)
        if workspace is None:
            workspace = torch.empty(need, dtype=torch.uint8, device=dev)
        _check(lib().hisparse_sparse_attention(self._h, layer, q.data_ptr(), H, value_dims,
                                               _dev_ptr(slot_table, "int32", self.N * self.k), scale,
                                               _dev_ptr(out, "float32", self.N * H * value_dims),
                                               _dev_ptr(lse, "float32", self.N * H), workspace.data_ptr(),
                                               workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
               "hisparse_sparse_attention")
        return out, lse

    # ---- consumer stand-ins ----
    def layer_pool(self, layer: int) -> int:
        p = lib().hisparse_layer_pool(self._h, layer)
        if not p:
            raise ValueError("bad layer")
        return p

    def gather(self, layer: int, slot_table, out=None, stream=None):
        import torch
        if out is None:
            out = torch.empty((self.N, self.k, self.E), dtype=torch.uint8, device="cuda:%d" % self.device)
        _check(lib().hisparse_gather(self._h, layer, _dev_ptr(slot_table, "int32", self.N * self.k),
                                     _dev_ptr(out, "uint8", self.N * self.k * self.E), _stream_ptr(stream)),
               "hisparse_gather")
        return out

    def gather_check(self, layer: int, sel, slot_table, mismatches, stream=None) -> None:
        _check(lib().hisparse_gather_check(self._h, layer, _dev_ptr(sel, "int32", self.N * self.k),
                                           _dev_ptr(slot_table, "int32", self.N * self.k),
                                           _dev_ptr(mismatches, "int32", 1), _stream_ptr(stream)),
               "hisparse_gather_check")

    # ---- inspection (synchronising) ----
    def status(self) -> int:
        bits = ctypes.c_uint32()
        _check(lib().hisparse_status(self._h, ctypes.byref(bits)), "hisparse_status")
        return bits.value

    def clear_status(self) -> None:
        _check(lib().hisparse_clear_status(self._h), "hisparse_clear_status")

    def dump_state(self, req: int, layer: int, with_pos2slot: bool = True) -> dict:
        B = self.B
        slot_pos = np.empty(B, dtype=np.int32)
        last_use = np.empty(B, dtype=np.uint32)
        order = np.empty(B, dtype=np.int32)
        p2s = np.empty(int(self.capacity[req]), dtype=np.int32) if with_pos2slot else None
        ln, newest, t = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_uint32()
        _check(lib().hisparse_dump_state(self._h, req, layer, slot_pos.ctypes.data, last_use.ctypes.data,
                                         order.ctypes.data, p2s.ctypes.data if with_pos2slot else None,
                                         ctypes.byref(ln), ctypes.byref(newest), ctypes.byref(t)),
               "hisparse_dump_state")
        return dict(slot_pos=slot_pos, last_use=last_use, lru_order=order, pos2slot=p2s, len=ln.value,
                    newest=newest.value, resolves=t.value)

    def load_appends(self, appends: int) -> None:
        _check(lib().hisparse_load_appends(self._h, appends), "hisparse_load_appends")

    def load_state(self, req: int, layer: int, slot_pos: np.ndarray, last_use: np.ndarray, resolves: int) -> None:
        sp = np.ascontiguousarray(slot_pos, dtype=np.int32)
        lu = np.ascontiguousarray(last_use, dtype=np.uint32)
        assert sp.size == self.B and lu.size == self.B
        _check(lib().hisparse_load_state(self._h, req, layer, sp.ctypes.data, lu.ctypes.data, resolves),
               "hisparse_load_state")

    def order_lag(self, req: int, layer: int) -> int:
        """Resolves of (req, layer's group) the recency list has not absorbed yet (0 = dump_state's lru_order is the
        slots sorted by (last_use, slot))."""
        lag = ctypes.c_uint32()
        _check(lib().hisparse_order_lag(self._h, req, layer, ctypes.byref(lag)), "hisparse_order_lag")
        return int(lag.value)

    def dump_plan(self, req: int, layer: int):
        pos = np.empty(self.k, dtype=np.int32)
        slot = np.empty(self.k, dtype=np.int32)
        n = ctypes.c_int32()
        _check(lib().hisparse_dump_plan(self._h, req, layer, pos.ctypes.data, slot.ctypes.data, ctypes.byref(n)),
               "hisparse_dump_plan")
        return pos[: n.value].copy(), slot[: n.value].copy()

    def phase_times(self) -> np.ndarray:
        """uint64 [N][16] stamps of the last anchor resolve (needs FLAG_PHASE_TIMERS): 8 in ns, 8 in SM cycles."""
        out = np.zeros((self.N, 16), dtype=np.uint64)
        _check(lib().hisparse_phase_times(self._h, out.ctypes.data), "hisparse_phase_times")
        return out

    def layer_times(self) -> np.ndarray:
        """uint64 [L][2]: start and end (ns) of each layer's last resolve kernel since the previous call (needs
        FLAG_PHASE_TIMERS); a layer without one reads (2**64 - 1, 0).  Synchronises and clears the stamps."""
        out = np.zeros((2, self.L), dtype=np.uint64)
        _check(lib().hisparse_layer_times(self._h, out.ctypes.data), "hisparse_layer_times")
        return np.ascontiguousarray(out.T)

    def selftest_wait_timeout(self, limit_ns: int) -> int:
        """Runs the library's bounded wait on a barrier that never completes; returns the nanoseconds waited."""
        out = ctypes.c_uint64()
        _check(lib().hisparse_selftest_wait_timeout(self._h, limit_ns, ctypes.byref(out)), "hisparse_selftest_wait_timeout")
        return out.value

    def launch_geometry(self):
        s, t, m = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        _check(lib().hisparse_launch_geometry(self._h, ctypes.byref(s), ctypes.byref(t), ctypes.byref(m)),
               "hisparse_launch_geometry")
        return dict(ctas_per_request=s.value, threads=t.value, smem_bytes=m.value)
