"""Pins for the CPU oracle: it is checked against things other than itself — a hand-derived worked
example, an independently written ordered-list simulator, textbook LRU for k = 1, the B = k closed
form, and the invariants the paper fixes (Sec. 3.1: exact outputs, bounded footprint)."""
import collections
import os

import numpy as np
import pytest

from oracle import Oracle, STATUS_DUPLICATE, STATUS_OUT_OF_RANGE, FLAG_NO_BYTES, kv_footprint_bytes
from paper_2608_07009_b200 import inputs
from lru_list_sim import ListLRUSim

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def meta_oracle(B, k, length, cap=None, N=1, L=1, lpg=1):
    cap = cap if cap is not None else length + 64
    return Oracle(N, L, lpg, B, k, 16, [cap] * N, [length] * N, None, FLAG_NO_BYTES)


def order_from_stamps(last_use):
    return [int(s) for s in np.lexsort((np.arange(len(last_use)), last_use))]


# ---------------------------------------------------------------- worked example (hand-derived)

def test_worked_example_golden():
    rows = []
    with open(os.path.join(GOLDEN, "worked_example_b4_k2.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append([[int(x) for x in part.split()] for part in line.split(";")])
    assert len(rows) == 5
    o = meta_oracle(4, 2, 64)
    for (t,), sel, table, (h, m), slot_pos, last_use in rows:
        tab, hits, misses = o.resolve(0, np.array([sel], dtype=np.int32))
        assert tab[0].tolist() == table, "step %d" % t
        assert (int(hits[0]), int(misses[0])) == (h, m)
        assert o.slot_pos(0, 0).tolist() == slot_pos
        assert o.last_use(0, 0).tolist() == last_use
        assert o.steps(0, 0) == t


# ---------------------------------------------------------------- brute force on tiny inputs

@pytest.mark.parametrize("B", [1, 2, 3, 4, 7, 8, 12])
def test_against_list_simulator(B):
    rng = np.random.default_rng(1000 + B)
    for k in range(1, B + 1):
        for universe in sorted({k, k + 1, B, B + 1, 2 * B, 3 * B}):
            if universe < k:
                continue
            for pad_prob, with_append in ((0.0, False), (0.25, False), (0.0, True), (0.2, True)):
                length = universe
                o = meta_oracle(B, k, length, cap=length + 64)
                sim = ListLRUSim(B, k, length)
                prev_newest = -1
                for step in range(40):
                    if with_append and step % 2 == 1:
                        o.append()
                        sim.append()
                    cur_len = sim.len
                    row = inputs.random_rows(rng, 1, k, cur_len, pad_prob)[0]
                    if with_append and sim.newest >= 0 and step % 3 == 0:
                        # make sure the newest record, and the one that was newest before it, get selected
                        forced = [p for p in dict.fromkeys((sim.newest, prev_newest)) if p >= 0][:k]
                        keep = [p for p in row.tolist() if p not in forced][: k - len(forced)]
                        row = np.array(forced + keep + [-1] * (k - len(forced) - len(keep)), dtype=np.int32)
                    prev_newest = sim.newest
                    tab, hits, misses = o.resolve(0, row[None])
                    out, h, m, plan, _ = sim.resolve(row)
                    assert tab[0].tolist() == out
                    assert (int(hits[0]), int(misses[0])) == (h, m)
                    assert o.slot_pos(0, 0).tolist() == sim.slot_pos
                    assert order_from_stamps(o.last_use(0, 0)) == sim.order
                    ppos, pslot = o.plan(0, 0)
                    assert list(zip(ppos.tolist(), pslot.tolist())) == plan
                    assert h + m == int((row >= 0).sum())
                assert o.status == 0
                o.close()


# ---------------------------------------------------------------- k = 1 is textbook LRU

def textbook_lru_misses(accesses, capacity):
    cache = collections.OrderedDict()
    out = []
    for p in accesses:
        if p in cache:
            cache.move_to_end(p)
            out.append(0)
        else:
            if len(cache) == capacity:
                cache.popitem(last=False)
            cache[p] = True
            out.append(1)
    return out, list(cache.keys())


@pytest.mark.parametrize("B", [1, 2, 5, 16])
def test_k1_is_textbook_lru(B):
    rng = np.random.default_rng(7 * B)
    accesses = rng.integers(0, 3 * B + 1, size=400).tolist()
    o = meta_oracle(B, 1, 4 * B + 8)
    got = [int(o.resolve(0, np.array([[p]], dtype=np.int32))[2][0]) for p in accesses]
    want, resident = textbook_lru_misses(accesses, B)
    assert got == want
    assert sorted(p for p in o.slot_pos(0, 0).tolist() if p >= 0) == sorted(resident)
    # recency order of the resident records is the textbook one as well
    sp, lu = o.slot_pos(0, 0), o.last_use(0, 0)
    by_recency = [int(sp[s]) for s in order_from_stamps(lu) if sp[s] >= 0]
    assert by_recency == resident


def test_k1_cyclic_scan_always_misses():
    B = 6
    o = meta_oracle(B, 1, 64)
    misses = [int(o.resolve(0, np.array([[i % (B + 1)]], dtype=np.int32))[2][0]) for i in range(50)]
    assert misses == [1] * 50


# ---------------------------------------------------------------- B = k keeps only the current top-k

@pytest.mark.parametrize("k", [1, 3, 8, 32])
def test_b_equals_k_misses_are_set_difference(k):
    rng = np.random.default_rng(k)
    o = meta_oracle(k, k, 4 * k + 4)
    prev = set()
    for _ in range(60):
        row = inputs.random_rows(rng, 1, k, 4 * k + 4)[0]
        _, hits, misses = o.resolve(0, row[None])
        cur = set(row.tolist())
        assert int(misses[0]) == len(cur - prev)
        assert int(hits[0]) == len(cur & prev)
        assert set(o.slot_pos(0, 0).tolist()) == cur
        prev = cur


# ---------------------------------------------------------------- repeated selection

def test_repeated_selection_hits_after_first_step():
    B, k = 16, 8
    o = meta_oracle(B, k, 100)
    row = np.array([[3, 50, 7, 99, 0, 21, 22, 23]], dtype=np.int32)
    tab0, h, m = o.resolve(0, row)
    assert (int(h[0]), int(m[0])) == (0, k)
    assert tab0[0].tolist() == list(range(k))          # cold cache fills slots 0,1,2.. in selection order
    sp = o.slot_pos(0, 0)
    for _ in range(5):
        tab, h, m = o.resolve(0, row)
        assert (int(h[0]), int(m[0])) == (k, 0)
        assert (tab == tab0).all() and (o.slot_pos(0, 0) == sp).all()


# ---------------------------------------------------------------- invariants on a DSA-shaped trace with bytes

def check_invariants(o, w, layer, sel, tab, hits, misses, prev_table_by_pos, step_t):
    N, B, k, E = w.num_requests, w.cache_slots, w.top_k, w.entry_bytes
    pool = o.pool(layer)
    for r in range(N):
        sp, lu, p2s = o.slot_pos(r, layer), o.last_use(r, layer), o.pos2slot(r, layer)
        valid = sel[r] >= 0
        assert int(hits[r]) + int(misses[r]) == int(valid.sum())
        # exact outputs: every selected record's bytes are where the table says
        for j in np.nonzero(valid)[0]:
            local = int(tab[r, j]) - r * (B + 1)
            assert 0 <= local <= B
            want = inputs.record_bytes(r, layer, int(sel[r, j]), E, w.seed)
            assert (pool[r, local] == want).all()
        # bounded footprint and inverse maps
        occ = sp >= 0
        assert occ.sum() <= B and len(set(sp[occ].tolist())) == int(occ.sum())
        for s in np.nonzero(occ)[0]:
            assert p2s[sp[s]] == s
        assert (p2s >= 0).sum() == occ.sum()
        # hits stay in place
        for j in np.nonzero(valid)[0]:
            p = int(sel[r, j])
            if (r, p) in prev_table_by_pos and prev_table_by_pos[(r, p)] == int(p2s[p]) and p2s[p] >= 0:
                assert int(tab[r, j]) - r * (B + 1) == prev_table_by_pos[(r, p)]
        # stamp order: hit > fetched > untouched
        hit_stamp, miss_stamp = 2 * step_t + 1, 2 * step_t
        assert ((lu == hit_stamp) | (lu == miss_stamp) | (lu < miss_stamp)).all()
        assert int((lu == miss_stamp).sum()) == int(misses[r])


def test_invariants_on_tiny_dsa_trace():
    w = inputs.c1_tiny_dsa()
    w.steps = 12
    hist = [inputs.new_history(w, 0)]
    o = Oracle(1, 1, 1, w.cache_slots, w.top_k, w.entry_bytes, w.capacity, w.init_len, hist)
    tr = inputs.Trace(w)
    resident_before = {}
    total_m = 0
    for step in range(w.steps):
        sel, appended, lens = tr.step()
        if appended:
            o.append(inputs.new_kv(w, lens - 1))
        p2s_before = o.pos2slot(0, 0)
        tab, hits, misses = o.resolve(0, sel[0])
        for j in range(w.top_k):     # a hit's slot is the slot it already had
            p = int(sel[0, 0, j])
            if p >= 0 and p != o.newest(0) and p2s_before[p] >= 0:
                assert int(tab[0, j]) == int(p2s_before[p])
        check_invariants(o, w, 0, sel[0], tab, hits, misses, resident_before, step + 1)
        if step == 0:
            assert int(misses[0]) + int((sel[0, 0] == o.newest(0)).sum()) == w.top_k
        else:
            total_m += int(misses[0])
    assert 0 < total_m < (w.steps - 1) * (w.top_k - w.keep + 1)
    # write-through reached the host history
    for p in range(w.init_len[0], o.length(0)):
        assert (hist[0][0, p] == inputs.record_bytes(0, 0, p, w.entry_bytes, w.seed)).all()


def test_newest_slot_and_write_through():
    w = inputs.Workload("t", inputs.KIND_DSA_MIX, 2, 2, 1, 4, 8, 48, [10, 20], 8)
    hist = [inputs.new_history(w, r) for r in range(2)]
    o = Oracle(2, 2, 1, 8, 4, 48, w.capacity, w.init_len, hist)
    o.append(inputs.new_kv(w, np.array([10, 20])))
    assert o.newest(0) == 10 and o.newest(1) == 20 and o.length(1) == 21
    sel = np.array([[10, 1, 2, -1], [20, 19, 0, 5]], dtype=np.int32)
    tab, h, m = o.resolve(1, sel)
    assert tab[0, 0] == 8 and tab[1, 0] == 9 + 8      # reserved slot B of each request
    assert h.tolist() == [1, 1] and m.tolist() == [2, 3]
    assert o.pos2slot(0, 1)[10] == -1                  # the reserved slot is outside the page table
    o.append(inputs.new_kv(w, np.array([11, 21])))
    tab, h, m = o.resolve(1, sel)                       # 10 / 20 are host-only now: fetched back
    assert h.tolist() == [2, 3] and m.tolist() == [1, 1]
    for r in range(2):
        local = int(tab[r, 0]) - r * 9
        assert local < 8
        assert (o.pool(1)[r, local] == inputs.record_bytes(r, 1, int(sel[r, 0]), 48, w.seed)).all()
        assert (o.pool(1)[r, 8] == inputs.record_bytes(r, 1, 11 + 10 * r, 48, w.seed)).all()


# ---------------------------------------------------------------- padding, range, duplicates

def test_all_padding_row_changes_nothing():
    o = meta_oracle(4, 4, 32)
    o.resolve(0, np.array([[1, 2, 3, 4]], dtype=np.int32))
    sp, lu = o.slot_pos(0, 0), o.last_use(0, 0)
    tab, h, m = o.resolve(0, np.full((1, 4), -1, dtype=np.int32))
    assert tab.tolist() == [[-1] * 4] and h[0] == 0 and m[0] == 0
    assert (o.slot_pos(0, 0) == sp).all() and (o.last_use(0, 0) == lu).all()
    assert o.status == 0


def test_out_of_range_sets_status_only():
    o = meta_oracle(4, 3, 32)
    tab, h, m = o.resolve(0, np.array([[5, 32, -7]], dtype=np.int32))
    assert tab[0].tolist() == [0, -1, -1] and (int(h[0]), int(m[0])) == (0, 1)
    assert o.status == STATUS_OUT_OF_RANGE
    assert o.slot_pos(0, 0).tolist() == [5, -1, -1, -1]


def test_duplicate_follows_first_occurrence():
    o = meta_oracle(4, 4, 32)
    tab, h, m = o.resolve(0, np.array([[9, 4, 9, 4]], dtype=np.int32))
    assert tab[0].tolist() == [0, 1, 0, 1] and (int(h[0]), int(m[0])) == (0, 2)
    assert o.status == STATUS_DUPLICATE
    tab, h, m = o.resolve(0, np.array([[4, 4, 9, 7]], dtype=np.int32))
    assert tab[0].tolist() == [1, 1, 0, 2] and (int(h[0]), int(m[0])) == (2, 1)


# ---------------------------------------------------------------- shared-selection groups (plan then copy)

@pytest.mark.parametrize("lpg,use_prefetch", [(2, True), (2, False), (4, True), (4, False)])
def test_shared_layers_follow_anchor(lpg, use_prefetch):
    L = 2 * lpg
    w = inputs.Workload("g", inputs.KIND_DSA_MIX, 3, L, lpg, 6, 10, 32, [40, 50, 60], 12)
    hist = [inputs.new_history(w, r) for r in range(3)]
    o = Oracle(3, L, lpg, 10, 6, 32, w.capacity, w.init_len, hist)
    rng = np.random.default_rng(5)
    for step in range(12):
        pos = np.array([o.length(r) for r in range(3)])
        o.append(inputs.new_kv(w, pos))
        for a in range(0, L, lpg):
            sel = np.stack([inputs.random_rows(rng, 1, 6, int(pos[r]) + 1)[0] for r in range(3)])
            tab_a, h_a, m_a = o.resolve(a, sel)
            if use_prefetch:
                for l in range(a + 1, a + lpg):
                    o.prefetch(l)
            for l in range(a + 1, a + lpg):
                tab, h, m = o.resolve(l, sel)
                assert (tab == tab_a).all() and (h == h_a).all() and (m == m_a).all()
            for l in range(a, a + lpg):
                for r in range(3):
                    for j in range(6):
                        local = int(tab_a[r, j]) - r * 11
                        assert (o.pool(l)[r, local] == inputs.record_bytes(r, l, int(sel[r, j]), 32, w.seed)).all()


# ---------------------------------------------------------------- footprint closed form

def test_footprint_formula():
    # Sec. 3.3 "(2) Admission": 78 layers x 4096 slots vs 78 layers x 128K tokens, at the per-token
    # size implied by the quoted 13.09 GB (1280 B per token and layer).
    per_token = 1280
    assert kv_footprint_bytes(1, 78, 131072, per_token) == 78 * 131072 * 1280
    assert abs(kv_footprint_bytes(1, 78, 131072, per_token) / 1e9 - 13.09) < 0.01
    assert abs(kv_footprint_bytes(1, 78, 4096, per_token) / 1e9 - 0.41) < 0.01
    ratio = kv_footprint_bytes(1, 78, 131072, per_token) / kv_footprint_bytes(1, 78, 4096, per_token)
    assert ratio == 32      # "about 30x"


def test_rejects_bad_geometry():
    with pytest.raises(ValueError):
        meta_oracle(4, 5, 32)          # k > B
    with pytest.raises(ValueError):
        Oracle(1, 3, 2, 4, 2, 16, [8], [4], None, FLAG_NO_BYTES)   # L not a multiple of the group size
