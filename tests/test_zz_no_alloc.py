"""hisparse_resolve_noalloc against hisparse_resolve.

Some callers cannot allocate device memory when they need a resolve: an engine whose own allocator holds all
of HBM, or code running while a stream capture is open.  For them the library has one entry point that takes
every persistent array from the caller and keeps its scratch (the miss plan shared by a request's two thread
blocks) in a fixed array inside the library.  This test drives that entry point through the C-ABI on state
held in torch tensors and checks two calls in a row, bit for bit, against the ordinary handle-based resolve on
the same selections: slot tables, hit/miss counts, every state array and the bytes that were fetched.
The file sorts last on purpose, so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from paper_2608_07009_b200 import inputs, hisparse as hs
from paper_2608_07009_b200 import HiSparse, HostHistory, ExternalState, HiSparseError, resolve_noalloc

pytestmark = pytest.mark.gpu


def test_noalloc_matches_handle_on_two_calls():
    dev = torch.device("cuda:0")
    N, B, k, E = 3, 300, 130, 1152
    lens = [900, 1500, 700]
    w = inputs.Workload("noalloc", inputs.KIND_DSA_MIX, N, 1, 1, k, B, E, lens, 4, append_every=1 << 30, keep=100,
                        recent_window=64, seed=11, config_id=12)      # no appends: the trace never selects past the history
    cap = w.capacity
    hist = [HostHistory(1, cap[r], E) for r in range(N)]
    for r, h in enumerate(hist):
        inputs.fill_history(h.ptr, r, 1, cap[r], 0, lens[r], E, w.seed)
    ref = HiSparse(N, 1, 1, B, k, E, cap, lens, hist)

    # caller-owned state, cold
    pool = torch.zeros((N, B + 1, E), dtype=torch.uint8, device=dev)
    slot_pos = torch.full((N, B), -1, dtype=torch.int32, device=dev)
    last_use = torch.zeros((N, B), dtype=torch.int32, device=dev)          # uint32 bit patterns
    order = torch.arange(B, dtype=torch.int16, device=dev).repeat(N, 1).contiguous()   # uint16 bit patterns
    offs = np.concatenate([[0], np.cumsum(cap)[:-1]]).astype(np.int64)
    pos2slot = torch.full((int(sum(cap)),), -1, dtype=torch.int16, device=dev)
    cap_d = torch.tensor(cap, dtype=torch.int64, device=dev)
    len_d = torch.tensor(lens, dtype=torch.int64, device=dev)
    off_d = torch.from_numpy(offs).to(dev)
    # pinned, mapped host memory has the same address on the device under unified addressing
    host_d = torch.tensor([h.ptr for h in hist], dtype=torch.int64, device=dev)
    resolves = torch.zeros(N, dtype=torch.int32, device=dev)
    appends = torch.zeros(1, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    st = ExternalState(N, B, k, E, 0, pool.data_ptr(), slot_pos.data_ptr(), last_use.data_ptr(), order.data_ptr(),
                       pos2slot.data_ptr(), cap_d.data_ptr(), len_d.data_ptr(), off_d.data_ptr(), host_d.data_ptr(),
                       resolves.data_ptr(), appends.data_ptr())
    tab = torch.empty((N, k), dtype=torch.int32, device=dev)
    hits = torch.empty(N, dtype=torch.int32, device=dev)
    misses = torch.empty(N, dtype=torch.int32, device=dev)

    tr = inputs.Trace(w)
    try:
        for call in range(2):
            sel, _, _ = tr.step()
            sel_d = torch.from_numpy(np.ascontiguousarray(sel[0])).to(dev)
            tab_ref, h_ref, m_ref = ref.resolve(0, sel_d)
            resolve_noalloc(st, sel_d, tab, hits, misses, status)
            torch.cuda.synchronize()
            assert torch.equal(tab, tab_ref), "slot table differs on call %d" % call
            assert torch.equal(hits, h_ref) and torch.equal(misses, m_ref)
            if call == 0:
                assert int(misses.sum()) == N * k          # cold caches
            else:
                assert 0 < int(misses.sum()) < N * k and int(hits.sum()) > 0
            got = pool.view(N * (B + 1), E)[tab.long().clamp(min=0)]
            want = ref.gather(0, tab_ref)
            assert torch.equal(got, want), "fetched bytes differ on call %d" % call
            for r in range(N):
                s = ref.dump_state(r, 0)
                assert np.array_equal(slot_pos[r].cpu().numpy(), s["slot_pos"])
                assert np.array_equal(last_use[r].cpu().numpy().view(np.uint32), s["last_use"])
                assert np.array_equal(order[r].cpu().numpy().view(np.uint16).astype(np.int32), s["lru_order"])
                assert np.array_equal(pos2slot[offs[r]:offs[r] + cap[r]].cpu().numpy().astype(np.int32), s["pos2slot"])
                assert int(resolves[r]) == s["resolves"] == call + 1
        assert int(status.item()) == 0 and ref.status() == 0
        # sizes beyond the fixed scratch are refused with their own error code, before anything is enqueued
        big = ExternalState.from_buffer_copy(bytes(st))
        big.num_requests = hs.NOALLOC_MAX_REQUESTS + 1
        with pytest.raises(HiSparseError) as e:
            hs._check(hs.lib().hisparse_resolve_noalloc(big, sel_d.data_ptr(), tab.data_ptr(), hits.data_ptr(),
                                                        misses.data_ptr(), None, None), "hisparse_resolve_noalloc")
        assert e.value.code == hs.ETOOBIG
    finally:
        tr.close()
        ref.close()
        for h in hist:
            h.free()
