"""Drives the CUDA path (through the C-ABI binding) and the CPU oracle side by side on the same
seeded inputs and compares them element by element.  Shared by the `-m gpu` parity tests."""
from __future__ import annotations

import numpy as np
import torch

from oracle import Oracle, FLAG_NO_BYTES
from paper_2608_07009_b200 import HiSparse, HostHistory, inputs


def check_recency_list(order, last_use, lag, resolves):
    """The recency list the kernels keep is the slots sorted by (stamp, slot) whenever it is current (lag 0).  After
    `lag` resolves without misses it is still a permutation, and the slots not stamped since (stamp below the first
    stamp of those resolves) still stand in it in (stamp, slot) order."""
    B = len(last_use)
    want = np.lexsort((np.arange(B), last_use))
    if lag == 0:
        assert np.array_equal(order, want)
        return
    assert lag <= resolves
    assert np.array_equal(np.sort(order), np.arange(B))
    thr = 2 * (resolves - lag) + 2
    assert np.array_equal(order[last_use[order] < thr], want[last_use[want] < thr])


class Pair:
    """One CUDA handle and one oracle over separate copies of the same host histories."""

    def __init__(self, w: inputs.Workload, flags: int = 0, ctas_per_request: int = 0, oracle_bytes: bool = True,
                 device: int = 0, policy: int = 0, policy_seed: int = 0):
        self.w = w
        self.dev = torch.device("cuda:%d" % device)
        cap, il = w.capacity, w.init_len
        self.hist_gpu = [HostHistory(w.num_layers, cap[r], w.entry_bytes) for r in range(w.num_requests)]
        for r, h in enumerate(self.hist_gpu):
            inputs.fill_history(h.ptr, r, w.num_layers, cap[r], 0, il[r], w.entry_bytes, w.seed)
        try:
            self.gpu = HiSparse(w.num_requests, w.num_layers, w.layers_per_group, w.cache_slots, w.top_k, w.entry_bytes,
                                cap, il, self.hist_gpu, device=device, flags=flags, ctas_per_request=ctas_per_request,
                                policy=policy, policy_seed=policy_seed)
        except Exception:
            for h in self.hist_gpu:
                h.free()
            raise
        self.oracle_bytes = oracle_bytes
        if oracle_bytes:
            self.hist_cpu = [inputs.new_history(w, r) for r in range(w.num_requests)]
            self.oracle = Oracle(w.num_requests, w.num_layers, w.layers_per_group, w.cache_slots, w.top_k,
                                 w.entry_bytes, cap, il, self.hist_cpu, policy=policy, policy_seed=policy_seed)
        else:
            self.hist_cpu = None
            self.oracle = Oracle(w.num_requests, w.num_layers, w.layers_per_group, w.cache_slots, w.top_k,
                                 w.entry_bytes, cap, il, None, FLAG_NO_BYTES, policy=policy, policy_seed=policy_seed)
        self.mism = torch.zeros(1, dtype=torch.int32, device=self.dev)

    def close(self):
        self.gpu.close()
        self.oracle.close()
        for h in self.hist_gpu:
            h.free()

    # ---- one decode step ----
    def append(self):
        w = self.w
        pos = np.array([self.oracle.length(r) for r in range(w.num_requests)], dtype=np.int64)
        kv = inputs.new_kv(w, pos)
        self.oracle.append(kv if self.oracle_bytes else None)
        self.gpu.append(torch.from_numpy(kv).to(self.dev))

    def resolve_and_compare(self, layer: int, sel: np.ndarray, check_bytes: bool = True, side_stream=None):
        w = self.w
        sel = np.ascontiguousarray(sel, dtype=np.int32).reshape(w.num_requests, w.top_k)
        sel_d = torch.from_numpy(sel).to(self.dev)
        tab_o, h_o, m_o = self.oracle.resolve(layer, sel)
        tab_d, h_d, m_d = self.gpu.resolve(layer, sel_d)
        if side_stream is not None and layer % w.layers_per_group == 0:
            for l in range(layer + 1, layer + w.layers_per_group):
                self.gpu.prefetch(l, side_stream)
                self.oracle.prefetch(l)
        tab_g = tab_d.cpu().numpy()
        assert np.array_equal(tab_g, tab_o), "slot table differs at layer %d" % layer
        assert np.array_equal(h_d.cpu().numpy(), h_o) and np.array_equal(m_d.cpu().numpy(), m_o)
        if check_bytes:
            self.gpu.gather_check(layer, sel_d, tab_d, self.mism)
            if self.oracle_bytes:
                got = self.gpu.gather(layer, tab_d).cpu().numpy()
                pool = self.oracle.pool(layer).reshape(-1, w.entry_bytes)
                valid = tab_o >= 0
                want = pool[np.where(valid, tab_o, 0)]
                want[~valid] = 0
                assert np.array_equal(got, want), "gathered bytes differ at layer %d" % layer
        return tab_g, h_o, m_o

    def compare_state(self, layer: int, requests=None):
        w = self.w
        for r in (range(w.num_requests) if requests is None else requests):
            st = self.gpu.dump_state(r, layer)
            assert np.array_equal(st["slot_pos"], self.oracle.slot_pos(r, layer)), (r, layer)
            lu = self.oracle.last_use(r, layer)
            assert np.array_equal(st["last_use"], lu), (r, layer)
            assert np.array_equal(st["pos2slot"], self.oracle.pos2slot(r, layer)), (r, layer)
            assert st["len"] == self.oracle.length(r) and st["newest"] == self.oracle.newest(r)
            assert st["resolves"] == self.oracle.steps(r, layer)
            check_recency_list(st["lru_order"], lu, self.gpu.order_lag(r, layer), st["resolves"])
            pp, ps = self.gpu.dump_plan(r, layer)
            op, os_ = self.oracle.plan(r, layer)
            assert np.array_equal(pp, op) and np.array_equal(ps, os_)

    def compare_whole_pool(self, layer: int):
        """Every slot of every request's cache of this layer, reserved slot included."""
        w = self.w
        total = w.num_requests * (w.cache_slots + 1)
        want = self.oracle.pool(layer).reshape(total, w.entry_bytes)
        per = w.num_requests * w.top_k
        for start in range(0, total, per):
            idx = np.arange(start, start + per, dtype=np.int32)
            idx[idx >= total] = -1
            tab = torch.from_numpy(idx.reshape(w.num_requests, w.top_k)).to(self.dev)
            got = self.gpu.gather(layer, tab).cpu().numpy().reshape(per, w.entry_bytes)
            n = min(per, total - start)
            assert np.array_equal(got[:n], want[start:start + n]), "pool bytes differ at layer %d" % layer

    def finish(self, expect_status: int = 0):
        assert int(self.mism.item()) == 0, "gathered bytes differ from the host history"
        assert self.gpu.status() == expect_status      # synchronises: the write-through has landed
        assert self.oracle.status == expect_status
        if self.oracle_bytes:                          # write-through parity: appended records, every layer
            for r, (hg, hc) in enumerate(zip(self.hist_gpu, self.hist_cpu)):
                lo, hi = self.w.init_len[r], self.oracle.length(r)
                assert np.array_equal(hg.numpy()[:, lo:hi], hc[:, lo:hi]), "host history differs for request %d" % r


def run_trace(w: inputs.Workload, steps: int, flags: int = 0, ctas_per_request: int = 0, oracle_bytes: bool = True,
              state_every: int = 1, pool_every: int = 0, use_prefetch: bool = False, state_requests=None,
              policy: int = 0, policy_seed: int = 0):
    """Replays `steps` steps of the workload's trace through both sides, comparing as it goes."""
    pair = Pair(w, flags, ctas_per_request, oracle_bytes, policy=policy, policy_seed=policy_seed)
    side = torch.cuda.Stream() if use_prefetch else None
    tr = inputs.Trace(w)
    total_h = total_m = 0
    try:
        for step in range(steps):
            sel, appended, _ = tr.step()
            if appended:
                pair.append()
            for layer in range(w.num_layers):
                g = layer // w.layers_per_group
                _, h, m = pair.resolve_and_compare(layer, sel[g], side_stream=side)
                if layer % w.layers_per_group == 0:
                    total_h += int(h.sum())
                    total_m += int(m.sum())
                if state_every and step % state_every == 0:
                    pair.compare_state(layer, state_requests)
                if pool_every and step % pool_every == 0 and oracle_bytes:
                    pair.compare_whole_pool(layer)
        pair.finish()
    finally:
        tr.close()
        pair.close()
    return total_h, total_m
