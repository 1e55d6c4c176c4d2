"""Parity at the configurations' full sizes, in the launch configuration bench.py times (one CUDA-graph replay
per step: append + one Resolve per layer, prefetch on a side stream for shared-selection groups).

The oracle tracks metadata only here (no second copy of tens of GB of history): slot tables and hit/miss counts
are compared for every request and layer, the full LRU state for sampled (request, layer) pairs, and the bytes by
property — every table entry must address bytes equal to the host history (device-side compare of ALL selections)
and, for sampled entries, equal to the generator's record computed one by one.
C4 / C5 need 34 GB / 69 GB of pinned history at their full 16 / 32 layers.  They run at full size; if the host
cannot pin that much (or HISPARSE_REDUCED_LAYERS=1 is set) the full-size test is skipped with that reason and a
separate `_reduced_layers` test runs the 4-layer variant (every other dimension being the configuration's own), so
that a pass always means the stated size was run.
"""
import os

import numpy as np
import pytest
import torch

from oracle import Oracle, FLAG_NO_BYTES
from paper_2608_07009_b200 import HiSparse, HostHistory, HiSparseError, inputs, hisparse as hs
from gpu_harness import check_recency_list

pytestmark = pytest.mark.gpu
REDUCED = os.environ.get("HISPARSE_REDUCED_LAYERS", "0") == "1"


def run_full(w, steps, sample_pairs, use_prefetch=False):
    dev = torch.device("cuda:0")
    N, L, lpg, G, k, B, E = (w.num_requests, w.num_layers, w.layers_per_group, w.num_groups, w.top_k,
                             w.cache_slots, w.entry_bytes)
    cap = w.capacity
    hist = []
    try:
        for r in range(N):
            hist.append(HostHistory(L, cap[r], E))
    except HiSparseError:
        for h in hist:
            h.free()
        raise
    for r, h in enumerate(hist):
        inputs.fill_history(h.ptr, r, L, cap[r], 0, w.init_len[r], E, w.seed)
    gpu = HiSparse(N, L, lpg, B, k, E, cap, w.init_len, hist)
    orc = Oracle(N, L, lpg, B, k, E, cap, w.init_len, None, FLAG_NO_BYTES)
    tr = inputs.Trace(w)
    sel_st = torch.empty((G, N, k), dtype=torch.int32, device=dev)
    kv_st = torch.zeros((N, L, E), dtype=torch.uint8, device=dev)
    tabs = torch.empty((L, N, k), dtype=torch.int32, device=dev)
    hits = torch.empty((L, N), dtype=torch.int32, device=dev)
    misses = torch.empty((L, N), dtype=torch.int32, device=dev)
    mism = torch.zeros(1, dtype=torch.int32, device=dev)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    graphs = {}
    rng = np.random.default_rng(0)

    def enqueue(with_append):
        if with_append:
            gpu.append(kv_st, stream=main)
        for layer in range(L):
            gpu.resolve(layer, sel_st[layer // lpg], tabs[layer], hits[layer], misses[layer], stream=main)
            if use_prefetch and layer % lpg == 0:
                for l2 in range(layer + 1, layer + lpg):
                    gpu.prefetch(l2, side)

    try:
        torch.cuda.synchronize()
        with torch.cuda.stream(main):
            for step in range(steps):
                sel, appended, lens = tr.step()
                if appended:
                    kv_st.copy_(torch.from_numpy(inputs.new_kv(w, lens - 1)))
                    orc.append()
                sel_st.copy_(torch.from_numpy(sel))
                if appended not in graphs:
                    torch.cuda.synchronize()
                    g = torch.cuda.CUDAGraph()
                    g.capture_begin()
                    enqueue(appended)
                    g.capture_end()
                    graphs[appended] = g
                graphs[appended].replay()
                torch.cuda.synchronize()
                tabs_h, hits_h, miss_h = tabs.cpu().numpy(), hits.cpu().numpy(), misses.cpu().numpy()
                for layer in range(L):
                    s = sel[layer // lpg]
                    tab_o, h_o, m_o = orc.resolve(layer, s)
                    assert np.array_equal(tabs_h[layer], tab_o), "slot table differs: step %d layer %d" % (step, layer)
                    assert np.array_equal(hits_h[layer], h_o) and np.array_equal(miss_h[layer], m_o)
                    gpu.gather_check(layer, sel_st[layer // lpg], tabs[layer], mism, stream=main)
                for (r, layer) in sample_pairs:
                    st = gpu.dump_state(r, layer)
                    assert np.array_equal(st["slot_pos"], orc.slot_pos(r, layer))
                    lu = orc.last_use(r, layer)
                    assert np.array_equal(st["last_use"], lu)
                    assert np.array_equal(st["pos2slot"], orc.pos2slot(r, layer))
                    check_recency_list(st["lru_order"], lu, gpu.order_lag(r, layer), st["resolves"])
                    assert st["len"] == orc.length(r) and st["newest"] == orc.newest(r)
                    pp, ps = gpu.dump_plan(r, layer)
                    op, os_ = orc.plan(r, layer)
                    assert np.array_equal(pp, op) and np.array_equal(ps, os_)
                # sampled records, recomputed one by one from the generator
                layer = int(rng.integers(L))
                got = gpu.gather(layer, tabs[layer], stream=main)
                for _ in range(8):
                    r, j = int(rng.integers(N)), int(rng.integers(k))
                    p = int(sel[layer // lpg][r, j])
                    if p >= 0:
                        assert np.array_equal(got[r, j].cpu().numpy(), inputs.record_bytes(r, layer, p, E, w.seed))
                del got
        assert int(mism.item()) == 0, "cache bytes differ from the host history"
        assert gpu.status() == 0 and orc.status == 0
    finally:
        tr.close()
        graphs.clear()
        gpu.close()
        orc.close()
        for h in hist:
            h.free()


def test_c2_dsa_decode_full_size():
    w = inputs.c2_dsa_decode(steps=4)
    run_full(w, 4, [(0, 0), (13, 7), (31, 15)])


def test_c3_dsa_long_full_size_with_prefetch():
    w = inputs.c3_dsa_long(0.5, steps=3)
    run_full(w, 3, [(0, 0), (8, 1), (8, 4), (3, 7)], use_prefetch=True)


# Which of the large configurations ran at their full number of layers in this session: a green result always
# means "ran at the stated size".  When the host cannot pin a configuration's history the full-size test is SKIPPED
# with that reason (never passed on a smaller shape), and only then does its `_reduced_layers` companion run.
FULL_SIZE_RAN = {}


def full_size(name, make, steps, full_layers):
    if REDUCED:
        FULL_SIZE_RAN[name] = False
        pytest.skip("HISPARSE_REDUCED_LAYERS=1: %s not run at its full %d layers" % (name, full_layers))
    try:
        w = make(full_layers)
        run_full(w, steps, [(0, 0), (15, w.num_layers - 1)])
    except HiSparseError as e:
        if e.code != hs.ENOMEM:
            raise
        FULL_SIZE_RAN[name] = False
        pytest.skip("%s NOT TESTED AT FULL SIZE: the host could not pin %d layers of history" % (name, full_layers))
    FULL_SIZE_RAN[name] = True


def reduced_layers(name, make, steps):
    if FULL_SIZE_RAN.get(name, False):
        pytest.skip("%s ran at its full size; the 4-layer variant is not needed" % name)
    w = make(4)
    run_full(w, steps, [(0, 0), (15, w.num_layers - 1)])


def test_c4_nsa_blocks_full_size():
    full_size("c4", lambda layers: inputs.c4_nsa_blocks(steps=66, num_layers=layers), 66, 16)


def test_c4_nsa_blocks_reduced_layers():
    reduced_layers("c4", lambda layers: inputs.c4_nsa_blocks(steps=66, num_layers=layers), 66)


def test_c5_quest_pages_full_size():
    full_size("c5", lambda layers: inputs.c5_quest_pages(steps=17, num_layers=layers), 17, 32)


def test_c5_quest_pages_reduced_layers():
    reduced_layers("c5", lambda layers: inputs.c5_quest_pages(steps=17, num_layers=layers), 17)
