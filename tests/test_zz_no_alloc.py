"""hisparse_resolve_noalloc against the CPU oracle (and against hisparse_resolve).

Some callers cannot allocate device memory when they need a resolve: an engine whose own allocator holds all
of HBM, or code running while a stream capture is open.  For them the library has one entry point that takes
every persistent array from the caller and keeps its scratch (the miss plan shared by a request's two thread
blocks) in a fixed array inside the library.  This test drives that entry point through the C-ABI on state
held in torch tensors and checks four calls in a row (a cold one, two with hits and misses, one in which every
selection hits), bit for bit, against the CPU oracle on the same selections: slot tables, hit/miss counts, every
state array and the bytes that were fetched; the ordinary handle-based resolve must agree as well.
The file sorts last on purpose, so that a failure here cannot hide another test's result.
"""
import numpy as np
import pytest
import torch

from oracle import Oracle
from paper_2608_07009_b200 import inputs, hisparse as hs
from paper_2608_07009_b200 import HiSparse, HostHistory, ExternalState, HiSparseError, resolve_noalloc

pytestmark = pytest.mark.gpu


def test_noalloc_matches_oracle_and_handle_call_after_call():
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
    orc = Oracle(N, 1, 1, B, k, E, cap, lens, [inputs.new_history(w, r) for r in range(N)])

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
        sel = None
        for call in range(4):
            if call < 3:
                sel, _, _ = tr.step()              # the last call repeats the previous row: every selection hits
            row = np.ascontiguousarray(sel[0])
            sel_d = torch.from_numpy(row).to(dev)
            tab_o, h_o, m_o = orc.resolve(0, row)
            tab_ref, h_ref, m_ref = ref.resolve(0, sel_d)
            resolve_noalloc(st, sel_d, tab, hits, misses, status)
            torch.cuda.synchronize()
            assert np.array_equal(tab.cpu().numpy(), tab_o), "slot table differs from the oracle's on call %d" % call
            assert np.array_equal(hits.cpu().numpy(), h_o) and np.array_equal(misses.cpu().numpy(), m_o)
            assert torch.equal(tab, tab_ref) and torch.equal(hits, h_ref) and torch.equal(misses, m_ref)
            if call == 0:
                assert int(misses.sum()) == N * k          # cold caches
            elif call < 3:
                assert 0 < int(misses.sum()) < N * k and int(hits.sum()) > 0
            else:
                assert int(misses.sum()) == 0 and int(hits.sum()) == N * k
            # the whole pool (reserved slots excepted: nothing was appended), not only the selected records
            assert np.array_equal(pool[:, :B].cpu().numpy(), orc.pool(0)[:, :B]), "cache bytes differ on call %d" % call
            for r in range(N):
                lu = orc.last_use(r, 0)
                assert np.array_equal(slot_pos[r].cpu().numpy(), orc.slot_pos(r, 0))
                assert np.array_equal(last_use[r].cpu().numpy().view(np.uint32), lu)
                assert np.array_equal(pos2slot[offs[r]:offs[r] + cap[r]].cpu().numpy().astype(np.int32), orc.pos2slot(r, 0))
                assert int(resolves[r]) == orc.steps(r, 0) == call + 1
                # this entry point keeps the caller's recency list current in every call
                assert np.array_equal(order[r].cpu().numpy().view(np.uint16).astype(np.int64),
                                      np.lexsort((np.arange(B), lu)))
                s = ref.dump_state(r, 0)
                assert np.array_equal(s["slot_pos"], orc.slot_pos(r, 0)) and np.array_equal(s["last_use"], lu)
        assert int(status.item()) == 0 and ref.status() == 0 and orc.status == 0
        # sizes beyond the fixed scratch are refused with their own error code, before anything is enqueued
        big = ExternalState.from_buffer_copy(bytes(st))
        big.num_requests = hs.NOALLOC_MAX_REQUESTS + 1
        with pytest.raises(HiSparseError) as e:
            hs._check(hs.lib().hisparse_resolve_noalloc(big, sel_d.data_ptr(), tab.data_ptr(), hits.data_ptr(),
                                                        misses.data_ptr(), None, None), "hisparse_resolve_noalloc")
        assert e.value.code == hs.ETOOBIG
        # a pool that bulk copies could not write to (not 16-byte aligned) is refused the same way
        odd = ExternalState.from_buffer_copy(bytes(st))
        odd.pool_dev = pool.data_ptr() + 4
        with pytest.raises(HiSparseError) as e:
            hs._check(hs.lib().hisparse_resolve_noalloc(odd, sel_d.data_ptr(), tab.data_ptr(), hits.data_ptr(),
                                                        misses.data_ptr(), None, None), "hisparse_resolve_noalloc")
        assert e.value.code == hs.EINVAL
    finally:
        tr.close()
        ref.close()
        orc.close()
        for h in hist:
            h.free()
