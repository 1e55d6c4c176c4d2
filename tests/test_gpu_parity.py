"""Parity of the CUDA path (called through the C-ABI binding) with the CPU oracle: bit-exact slot
tables, hit/miss counts, LRU state after every step, miss plans and cache bytes."""
import numpy as np
import pytest
import torch

from paper_2608_07009_b200 import inputs, hisparse as hs
from paper_2608_07009_b200 import HiSparse, HostHistory, HiSparseError
from gpu_harness import Pair, run_trace

pytestmark = pytest.mark.gpu


def tiny_workload(N, L, lpg, k, B, E, lens, steps=40):
    return inputs.Workload("tiny", inputs.KIND_DSA_MIX, N, L, lpg, k, B, E, list(lens), steps)


# ------------------------------------------------------------------ tiny-case matrix

@pytest.mark.parametrize("B", [1, 2, 3, 4, 7, 8, 12])
def test_tiny_matrix(B):
    rng = np.random.default_rng(100 + B)
    ks = sorted({1, max(1, B // 2), B})
    for k in ks:
        for universe, pad, with_append, E in ((k, 0.0, False, 16), (B + 1, 0.25, True, 48),
                                              (3 * B, 0.0, True, 1152), (2 * B, 0.2, False, 16)):
            N = 3
            lens = [universe, universe + 1, universe + 5]
            w = tiny_workload(N, 1, 1, k, B, E, lens)
            pair = Pair(w)
            prev_newest = [-1] * N
            try:
                for step in range(40):
                    if with_append and step % 2 == 1:
                        pair.append()
                    rows = []
                    for r in range(N):
                        cur = pair.oracle.length(r)
                        row = inputs.random_rows(rng, 1, k, cur, pad)[0]
                        newest = pair.oracle.newest(r)
                        if with_append and newest >= 0 and step % 3 == 0:
                            forced = [p for p in dict.fromkeys((newest, prev_newest[r])) if p >= 0][:k]
                            keep = [p for p in row.tolist() if p not in forced][: k - len(forced)]
                            row = np.array(forced + keep + [-1] * (k - len(forced) - len(keep)), dtype=np.int32)
                        prev_newest[r] = newest
                        rows.append(row)
                    pair.resolve_and_compare(0, np.stack(rows))
                    pair.compare_state(0)
                    if step % 8 == 0:
                        pair.compare_whole_pool(0)
                pair.finish()
            finally:
                pair.close()


@pytest.mark.parametrize("lpg,use_prefetch", [(2, True), (2, False), (4, True), (4, False)])
def test_shared_groups_tiny(lpg, use_prefetch):
    rng = np.random.default_rng(lpg)
    L = 2 * lpg
    w = tiny_workload(3, L, lpg, 6, 10, 48, [40, 50, 60], steps=16)
    pair = Pair(w)
    side = torch.cuda.Stream() if use_prefetch else None
    try:
        for step in range(16):
            pair.append()
            for a in range(0, L, lpg):
                sel = np.stack([inputs.random_rows(rng, 1, 6, pair.oracle.length(r))[0] for r in range(3)])
                for l in range(a, a + lpg):
                    pair.resolve_and_compare(l, sel, side_stream=side)
                    pair.compare_state(l)
                    pair.compare_whole_pool(l)
        pair.finish()
    finally:
        pair.close()


# ------------------------------------------------------------------ degenerate rows

def test_all_padding_out_of_range_and_duplicates():
    w = tiny_workload(2, 1, 1, 4, 6, 32, [20, 30])
    pair = Pair(w)
    try:
        pair.resolve_and_compare(0, np.array([[1, 2, 3, 4], [5, 6, 7, 8]]))
        pair.resolve_and_compare(0, np.full((2, 4), -1))
        pair.compare_state(0)
        pair.finish(0)
        pair.resolve_and_compare(0, np.array([[1, 20, -9, 2], [29, 30, 5, 1000000]]))
        pair.compare_state(0)
        pair.finish(hs.STATUS_OUT_OF_RANGE)
        pair.gpu.clear_status()
        pair.oracle.clear_status()
        pair.resolve_and_compare(0, np.array([[9, 4, 9, 4], [7, 7, 7, 7]]))
        pair.resolve_and_compare(0, np.array([[4, 4, 9, 10], [-1, 7, 11, 7]]))
        pair.compare_state(0)
        pair.finish(hs.STATUS_DUPLICATE)
    finally:
        pair.close()


def test_k_equals_b_all_miss_every_step():
    k = B = 64
    w = tiny_workload(2, 1, 1, k, B, 64, [1000, 1000])
    pair = Pair(w)
    try:
        for step in range(6):
            base = (step % 2) * 500
            sel = np.stack([np.arange(base + 7 * r, base + 7 * r + k) for r in range(2)])
            _, h, m = pair.resolve_and_compare(0, sel)
            assert m.tolist() == [k, k] and h.tolist() == [0, 0]
            pair.compare_state(0)
        pair.finish()
    finally:
        pair.close()


def test_inline_write_through_and_flag_combinations():
    w = inputs.c1_tiny_dsa()
    w.steps = 10
    for flags in (hs.FLAG_INLINE_WRITE_THROUGH, hs.FLAG_INLINE_WRITE_THROUGH | hs.FLAG_NO_PDL | hs.FLAG_PHASE_TIMERS,
                  hs.FLAG_NO_PDL | hs.FLAG_DEBUG_VALIDATE):
        run_trace(w, w.steps, flags=flags, pool_every=5)


def test_history_capacity_status():
    w = tiny_workload(2, 1, 1, 2, 4, 16, [5, 6], steps=1)     # capacity = len + 2
    pair = Pair(w)
    try:
        kv = torch.zeros((2, 1, 16), dtype=torch.uint8, device="cuda")
        for _ in range(2):
            pair.gpu.append(kv)
        assert pair.gpu.status() == 0
        pair.gpu.append(kv)
        assert pair.gpu.status() == hs.STATUS_CAPACITY
        st = pair.gpu.dump_state(0, 0)
        assert st["len"] == 7 and st["newest"] == -1
    finally:
        pair.close()


# ------------------------------------------------------------------ DSA / NSA / Quest shaped traces

def test_c1_tiny_dsa_full():
    w = inputs.c1_tiny_dsa()
    h, m = run_trace(w, w.steps, flags=hs.FLAG_DEBUG_VALIDATE, pool_every=16)
    assert h + m == w.steps * w.top_k


@pytest.mark.parametrize("S", [1, 2, 4, 8])
def test_c2_shape_reduced_all_cluster_sizes(S):
    # real k and B (several 1024-thread tiles), fewer requests / layers / tokens
    w = inputs.c2_dsa_decode(num_requests=5, num_layers=2, steps=6, context=6000)
    run_trace(w, w.steps, ctas_per_request=S, flags=hs.FLAG_DEBUG_VALIDATE)


def test_ragged_sizes():
    # k and B that are no multiples of the block size or of 32
    w = inputs.Workload("ragged", inputs.KIND_DSA_MIX, 3, 2, 1, 1000, 3001, 80, [5000, 7000, 2500], 8,
                        keep=800, recent_window=300, seed=3, config_id=9)
    run_trace(w, w.steps, flags=hs.FLAG_DEBUG_VALIDATE, pool_every=4)


def test_maximum_sizes():
    w = inputs.Workload("max", inputs.KIND_DSA_MIX, 2, 1, 1, hs.MAX_TOP_K, hs.MAX_CACHE_SLOTS, 16,
                        [40000, 20000], 4, keep=3000, recent_window=2048, seed=4, config_id=10)
    run_trace(w, w.steps, flags=hs.FLAG_DEBUG_VALIDATE)


@pytest.mark.parametrize("overlap", [0.5, 0.98])
def test_c3_shape_reduced_with_prefetch(overlap):
    w = inputs.c3_dsa_long(overlap, steps=5, short_ctx=8192, long_ctx=65536, num_short=3)
    run_trace(w, w.steps, use_prefetch=True, flags=hs.FLAG_DEBUG_VALIDATE)


@pytest.mark.parametrize("S", [1, 2, 8])
def test_long_context_page_table_not_staged(S):
    # page-table slices of 180 KB and 400 KB do not fit the staging ring: the blocks of a cluster share the lookups
    w = inputs.c3_dsa_long(0.5, steps=4, short_ctx=90000, long_ctx=200000, num_short=2)
    w.entry_bytes = 64
    run_trace(w, w.steps, use_prefetch=True, ctas_per_request=S, flags=hs.FLAG_DEBUG_VALIDATE)


def test_c4_nsa_blocks_reduced():
    w = inputs.c4_nsa_blocks(num_requests=4, num_layers=2, steps=70)
    w.entry_bytes = 16384            # same block-granular selection, smaller blocks
    run_trace(w, w.steps, pool_every=32)


def test_c5_quest_pages_reduced():
    w = inputs.c5_quest_pages(num_requests=3, num_layers=2, steps=20)
    w.entry_bytes = 4096
    run_trace(w, w.steps, pool_every=10)


def test_skip_io_keeps_metadata_exact():
    w = inputs.c2_dsa_decode(num_requests=2, num_layers=1, steps=4, context=5000)
    pair = Pair(w, flags=hs.FLAG_SKIP_IO, oracle_bytes=False)
    tr = inputs.Trace(w)
    try:
        for _ in range(4):
            sel, app, _ = tr.step()
            if app:
                pair.append()
            tab, _, _ = pair.resolve_and_compare(0, sel[0], check_bytes=False)
            pair.compare_state(0)
        # no record was fetched: every LRU slot still holds the zeros it was created with
        tab_d = torch.from_numpy(tab).cuda()
        got = pair.gpu.gather(0, tab_d).cpu().numpy()
        lru = (tab % (w.cache_slots + 1)) != w.cache_slots
        assert not got[lru].any()
    finally:
        tr.close()
        pair.close()


# ------------------------------------------------------------------ replacement policies of the ablation

@pytest.mark.parametrize("policy", [hs.POLICY_FIFO, hs.POLICY_RANDOM])
def test_policies_tiny(policy):
    rng = np.random.default_rng(policy)
    for B, k in ((1, 1), (3, 2), (8, 8), (12, 5), (40, 17)):
        w = tiny_workload(2, 1, 1, k, B, 48, [3 * B + 2, 2 * B + 1])
        pair = Pair(w, policy=policy, policy_seed=99, flags=hs.FLAG_DEBUG_VALIDATE)
        try:
            for step in range(40):
                if step % 5 == 4:
                    pair.append()
                rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0] for r in range(2)])
                pair.resolve_and_compare(0, rows)
                pair.compare_state(0)
            pair.finish()
        finally:
            pair.close()


@pytest.mark.parametrize("policy", [hs.POLICY_FIFO, hs.POLICY_RANDOM])
def test_policies_c2_shape_and_groups(policy):
    w = inputs.c2_dsa_decode(num_requests=3, num_layers=2, steps=6, context=6000)
    run_trace(w, w.steps, flags=hs.FLAG_DEBUG_VALIDATE, policy=policy, policy_seed=7)
    w = inputs.c3_dsa_long(0.5, steps=4, short_ctx=5000, long_ctx=40000, num_short=2)
    run_trace(w, w.steps, flags=hs.FLAG_DEBUG_VALIDATE, policy=policy, policy_seed=7, use_prefetch=True)
    w = inputs.Workload("ragged", inputs.KIND_DSA_MIX, 2, 1, 1, 1000, 9001, 32, [12000, 9500], 5,
                        keep=700, recent_window=300, seed=3, config_id=9)
    run_trace(w, w.steps, flags=hs.FLAG_DEBUG_VALIDATE, policy=policy, policy_seed=7)


# ------------------------------------------------------------------ 512-thread blocks (two per SM)

NARROW = hs.FLAG_NARROW_BLOCKS | hs.FLAG_DEBUG_VALIDATE


@pytest.mark.parametrize("B", [1, 3, 8, 12])
def test_narrow_blocks_tiny_matrix(B):
    rng = np.random.default_rng(40 + B)
    for k in range(1, B + 1):
        w = tiny_workload(2, 1, 1, k, B, 32, [2 * B + 3, 3 * B + 1])
        pair = Pair(w, flags=NARROW)
        try:
            assert pair.gpu.launch_geometry()["threads"] == 512
            for step in range(12):
                if step % 3 == 2:
                    pair.append()
                rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.15)[0] for r in range(2)])
                pair.resolve_and_compare(0, rows)
                pair.compare_state(0)
            pair.finish()
        finally:
            pair.close()


@pytest.mark.parametrize("S", [1, 2, 4, 8])
def test_narrow_blocks_c2_shape(S):
    w = inputs.c2_dsa_decode(num_requests=5, num_layers=2, steps=6, context=6000)
    run_trace(w, w.steps, ctas_per_request=S, flags=NARROW)


@pytest.mark.parametrize("policy", [hs.POLICY_LRU, hs.POLICY_FIFO, hs.POLICY_RANDOM])
def test_narrow_blocks_shapes_groups_and_policies(policy):
    # ragged k and B; B = 8192 (16 list entries per thread); groups with prefetch; page table not staged (shared lookups)
    w = inputs.Workload("ragged", inputs.KIND_DSA_MIX, 3, 2, 1, 1000, 3001, 80, [5000, 7000, 2500], 6,
                        keep=800, recent_window=300, seed=3, config_id=9)
    run_trace(w, w.steps, flags=NARROW, policy=policy, policy_seed=3, pool_every=3)
    w = inputs.Workload("wide", inputs.KIND_DSA_MIX, 2, 1, 1, 2048, 8192, 16, [30000, 20000], 4,
                        keep=1500, recent_window=2048, seed=4, config_id=10)
    run_trace(w, w.steps, flags=NARROW, policy=policy, policy_seed=3)
    w = inputs.c3_dsa_long(0.5, steps=4, short_ctx=8192, long_ctx=65536, num_short=2)
    run_trace(w, w.steps, use_prefetch=True, flags=NARROW, policy=policy, policy_seed=3)
    w = inputs.c3_dsa_long(0.5, steps=3, short_ctx=90000, long_ctx=200000, num_short=2)
    w.entry_bytes = 64
    run_trace(w, w.steps, use_prefetch=True, ctas_per_request=2, flags=NARROW, policy=policy, policy_seed=3)


@pytest.mark.parametrize("init_len,policy,k,B", [(250, hs.POLICY_LRU, 64, 128), (250, hs.POLICY_FIFO, 64, 128),
                                                 (1500, hs.POLICY_LRU, 64, 128), (700, hs.POLICY_RANDOM, 64, 128),
                                                 (3000, hs.POLICY_LRU, 512, 1100), (40000, hs.POLICY_LRU, 100, 300)])
def test_resident_wave_of_looping_blocks(init_len, policy, k, B):
    """More requests than blocks fit the GPU at once: the launch is one resident wave whose blocks take the requests
    b, b + blocks, b + 2 blocks, .. one after the other, with the next request's row and page-table slice staged
    ahead.  Requests in which nothing misses and requests with misses alternate at random, so that a block meets
    every order of the two: it runs the short loop until its first request with a miss and the general loop from
    there on."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    N = (6 if k <= 64 else 3) * sms + 37            # at most 3 blocks per SM are resident: every block loops
    # (init_len 40000: a page-table slice too long to stage, so the blocks never enter the short loop)
    rng = np.random.default_rng(init_len + policy)
    w = tiny_workload(N, 1, 1, k, B, 16 if init_len > 10000 else 32, [init_len] * N, steps=8)
    pair = Pair(w, flags=hs.FLAG_DEBUG_VALIDATE, policy=policy, policy_seed=11)
    try:
        assert pair.gpu.launch_geometry()["threads"] == 512
        for step in range(7):
            if step % 2 == 1:
                pair.append()
            rows = []
            for r in range(N):
                res = pair.oracle.slot_pos(r, 0)
                res = res[res >= 0]
                if step > 0 and rng.random() < 0.5 and len(res) >= k // 2:     # nothing misses
                    n = int(rng.integers(k // 2, min(k, len(res)) + 1))
                    row = rng.choice(res, size=n, replace=False).astype(np.int32)
                    if pair.oracle.newest(r) >= 0 and n < k and rng.random() < 0.5:
                        row = np.append(row, np.int32(pair.oracle.newest(r)))
                    row = rng.permutation(np.concatenate([row, np.full(k - len(row), -1, dtype=np.int32)]))
                else:
                    row = inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0]
                rows.append(row)
            _, _, m = pair.resolve_and_compare(0, np.stack(rows))
            assert 0 < int((m == 0).sum()) < N or step == 0
            pair.compare_state(0)
        pair.finish()
    finally:
        pair.close()


def test_block_size_is_chosen_by_the_grid_and_refused_when_it_cannot_fit():
    w = tiny_workload(2, 1, 1, 4, 8, 32, [20, 30])
    pair = Pair(w)
    assert pair.gpu.launch_geometry()["threads"] == 1024          # one wave: one block per SM
    pair.close()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    w = tiny_workload(sms + 1, 1, 1, 4, 8, 32, [20] * (sms + 1), steps=4)
    for flags, threads in ((0, 512), (hs.FLAG_WIDE_BLOCKS, 1024)):  # more blocks than SMs: two per SM unless told not to
        pair = Pair(w, flags=flags | hs.FLAG_DEBUG_VALIDATE)
        try:
            assert pair.gpu.launch_geometry()["threads"] == threads
            rng = np.random.default_rng(9)
            for step in range(3):
                pair.append()
                rows = np.stack([inputs.random_rows(rng, 1, 4, pair.oracle.length(r), 0.1)[0] for r in range(sms + 1)])
                pair.resolve_and_compare(0, rows)
            pair.compare_state(0, requests=[0, sms])
            pair.finish()
        finally:
            pair.close()
    hist = [HostHistory(1, 40000, 16) for _ in range(2)]
    try:
        for flags in (hs.FLAG_NARROW_BLOCKS | hs.FLAG_WIDE_BLOCKS, hs.FLAG_NARROW_BLOCKS):
            with pytest.raises(HiSparseError):                     # both at once; B beyond 16 list entries per thread
                HiSparse(2, 1, 1, 8193 if flags == hs.FLAG_NARROW_BLOCKS else 64, 8, 16, [40000, 40000], [100, 100], hist,
                         flags=flags)
        with pytest.raises(HiSparseError):
            HiSparse(2, 1, 1, 4096, 2049, 16, [40000, 40000], [5000, 5000], hist, flags=hs.FLAG_NARROW_BLOCKS)
    finally:
        for h in hist:
            h.free()


# ------------------------------------------------------------------ recency list left behind by hit-only resolves

def _hit_only_rows(rng, pair, k, newest_too, layer=0):
    """A row per request drawn from what is resident (so that nothing misses), padded with -1."""
    rows = []
    for r in range(pair.w.num_requests):
        res = pair.oracle.slot_pos(r, layer)
        res = res[res >= 0]
        n = int(rng.integers(0, min(k, len(res)) + 1))
        row = rng.choice(res, size=n, replace=False).astype(np.int32)
        if newest_too and pair.oracle.newest(r) >= 0 and n < k:
            row = np.append(row, np.int32(pair.oracle.newest(r)))
        row = np.concatenate([row, np.full(k - len(row), -1, dtype=np.int32)])
        rows.append(rng.permutation(row))
    return np.stack(rows)


@pytest.mark.parametrize("policy", [hs.POLICY_LRU, hs.POLICY_FIFO, hs.POLICY_RANDOM])
@pytest.mark.parametrize("B,k,S", [(4, 2, 1), (12, 5, 2), (40, 17, 1), (300, 130, 4), (5000, 2100, 1), (16384, 257, 2)])
def test_list_catches_up_after_hit_only_runs(policy, B, k, S):
    """Runs of 1..9 resolves in which nothing misses (the list is left behind and only stamps are written), each
    followed by resolves with misses (the list is re-sorted before victims are taken): everything still equals the
    oracle, and the list's lag is what the schedule says."""
    rng = np.random.default_rng(1000 * policy + B)
    w = tiny_workload(2, 1, 1, k, B, 32, [3 * B + 7, 2 * B + 3])
    pair = Pair(w, policy=policy, policy_seed=5, flags=hs.FLAG_DEBUG_VALIDATE, ctas_per_request=S)
    try:
        for run in (1, 2, 3, 1, 5, 9, 2):
            for _ in range(2):   # resolves with misses
                pair.append()
                rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0] for r in range(2)])
                _, _, m = pair.resolve_and_compare(0, rows)
                pair.compare_state(0)
                for r in range(2):
                    assert pair.gpu.order_lag(r, 0) == 0 or m[r] == 0
            for i in range(run):
                _, _, m = pair.resolve_and_compare(0, _hit_only_rows(rng, pair, k, newest_too=i % 2 == 1))
                assert int(m.sum()) == 0
                pair.compare_state(0)
                if policy != hs.POLICY_FIFO:
                    assert all(pair.gpu.order_lag(r, 0) >= i + 1 for r in range(2))
                else:
                    assert all(pair.gpu.order_lag(r, 0) == 0 for r in range(2))
        pair.finish()
    finally:
        pair.close()


@pytest.mark.parametrize("flags", [0, hs.FLAG_NARROW_BLOCKS])
def test_list_catches_up_after_long_hit_only_runs(flags):
    """70 and 300 skipped resolves: 7 and 9 stable splits when the list is rebuilt."""
    rng = np.random.default_rng(3)
    B, k = 37, 9
    w = tiny_workload(2, 1, 1, k, B, 32, [150, 90], steps=8)
    pair = Pair(w, flags=flags | hs.FLAG_DEBUG_VALIDATE)
    try:
        for run in (70, 300):
            for _ in range(3):
                rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0] for r in range(2)])
                pair.resolve_and_compare(0, rows, check_bytes=False)
                pair.compare_state(0)
            for i in range(run):
                pair.resolve_and_compare(0, _hit_only_rows(rng, pair, k, newest_too=False), check_bytes=False)
            pair.compare_state(0)
            assert pair.gpu.order_lag(0, 0) >= run
        rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.0)[0] for r in range(2)])
        pair.resolve_and_compare(0, rows)
        pair.compare_state(0)
        assert pair.gpu.order_lag(0, 0) == 0
        pair.finish()
    finally:
        pair.close()


def test_eager_list_flag_gives_the_same_results_and_never_lags():
    rng = np.random.default_rng(77)
    B, k = 300, 130
    w = tiny_workload(2, 1, 1, k, B, 32, [3 * B + 7, 2 * B + 3])
    pair = Pair(w, flags=hs.FLAG_DEBUG_VALIDATE | hs.FLAG_EAGER_ORDER)
    try:
        for step in range(12):
            if step % 3 == 0:
                rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0] for r in range(2)])
            else:
                rows = _hit_only_rows(rng, pair, k, newest_too=False)
            pair.resolve_and_compare(0, rows)
            pair.compare_state(0)
            assert all(pair.gpu.order_lag(r, 0) == 0 for r in range(2))
        pair.finish()
    finally:
        pair.close()


def test_hit_only_resolves_in_shared_groups_and_after_resume():
    """Groups of layers: a hit-only anchor resolve still hands its table to the shared layers and an empty plan to
    the prefetch.  A state dumped while the list lags resumes exactly (load_state rebuilds the list)."""
    rng = np.random.default_rng(5)
    B, k = 64, 20
    w = tiny_workload(2, 4, 2, k, B, 48, [200, 150])
    pair = Pair(w, flags=hs.FLAG_DEBUG_VALIDATE)
    side = torch.cuda.Stream()
    try:
        for step in range(10):
            pair.append()
            for g in range(2):
                if step % 4 == 0:
                    rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0] for r in range(2)])
                else:
                    rows = _hit_only_rows(rng, pair, k, newest_too=step % 2 == 1, layer=2 * g)
                for layer in (2 * g, 2 * g + 1):
                    pair.resolve_and_compare(layer, rows, side_stream=side)
                    pair.compare_state(layer)
        assert pair.gpu.order_lag(0, 0) > 0
        # resume into a second handle from the dumped stamps while the list lags
        st = [[pair.gpu.dump_state(r, 2 * g) for g in range(2)] for r in range(2)]
        appends = st[0][0]["len"] - w.init_len[0]
        other = HiSparse(2, 4, 2, B, k, 48, w.capacity, w.init_len, pair.hist_gpu, flags=hs.FLAG_DEBUG_VALIDATE)
        try:
            other.load_appends(appends)
            for r in range(2):
                for g in range(2):
                    other.load_state(r, 2 * g, st[r][g]["slot_pos"], st[r][g]["last_use"], st[r][g]["resolves"])
                    assert other.order_lag(r, 2 * g) == 0
            rows = np.stack([inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0] for r in range(2)])
            rows_d = torch.from_numpy(rows).to(pair.dev)
            tab_a, h_a, m_a = pair.gpu.resolve(0, rows_d)
            tab_b, h_b, m_b = other.resolve(0, rows_d)
            assert torch.equal(tab_a, tab_b) and torch.equal(h_a, h_b) and torch.equal(m_a, m_b)
            for r in range(2):
                a, b = pair.gpu.dump_state(r, 0), other.dump_state(r, 0)
                for key in ("slot_pos", "last_use", "lru_order", "pos2slot"):
                    assert np.array_equal(a[key], b[key]), key
            assert other.status() == 0
        finally:
            other.close()
    finally:
        pair.close()


# ------------------------------------------------------------------ speculative hints

def test_speculative_hint_is_a_discarded_resolve():
    # layer l's selection as a hint for layer l+1 (Sec. 3.5): on the oracle side a hint is one more resolve
    w = inputs.c2_dsa_decode(num_requests=3, num_layers=3, steps=5, context=5000)
    pair = Pair(w)
    tr = inputs.Trace(w)
    side = torch.cuda.Stream()
    try:
        for step in range(w.steps):
            sel, app, _ = tr.step()
            if app:
                pair.append()
            for layer in range(w.num_layers):
                pair.resolve_and_compare(layer, sel[layer])
                if layer + 1 < w.num_layers:
                    hint = torch.from_numpy(np.ascontiguousarray(sel[layer])).to(pair.dev)
                    pair.gpu.prefetch_hint(layer + 1, hint, side)
                    pair.oracle.resolve(layer + 1, sel[layer])
                pair.compare_state(layer)
        pair.finish()
    finally:
        tr.close()
        pair.close()
    grouped = Pair(tiny_workload(3, 2, 2, 6, 10, 48, [40, 50, 60]))
    try:
        with pytest.raises(HiSparseError) as e:      # shared-selection groups use the exact prefetch instead
            grouped.gpu.prefetch_hint(0, torch.zeros((3, 6), dtype=torch.int32, device="cuda"), side)
        assert e.value.code == hs.EINVAL
    finally:
        grouped.close()


# ------------------------------------------------------------------ CUDA graph replay of whole steps

def test_graph_replay_matches_oracle():
    w = inputs.c3_dsa_long(0.75, steps=6, short_ctx=4096, long_ctx=16384, num_short=2)
    pair = Pair(w)
    tr = inputs.Trace(w)
    dev = pair.dev
    N, k, L, G, lpg = w.num_requests, w.top_k, w.num_layers, w.num_groups, w.layers_per_group
    sel_d = torch.empty((G, N, k), dtype=torch.int32, device=dev)
    kv_d = torch.empty((N, L, w.entry_bytes), dtype=torch.uint8, device=dev)
    tabs = torch.empty((L, N, k), dtype=torch.int32, device=dev)
    hits = torch.empty((L, N), dtype=torch.int32, device=dev)
    misses = torch.empty((L, N), dtype=torch.int32, device=dev)
    main, side = torch.cuda.Stream(), torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    try:
        torch.cuda.synchronize()
        with torch.cuda.stream(main):
            graph.capture_begin()
            pair.gpu.append(kv_d, stream=main)
            for layer in range(L):
                pair.gpu.resolve(layer, sel_d[layer // lpg], tabs[layer], hits[layer], misses[layer], stream=main)
                if layer % lpg == 0:
                    for l in range(layer + 1, layer + lpg):
                        pair.gpu.prefetch(l, side)
            graph.capture_end()
        for step in range(w.steps):
            sel, app, lens = tr.step()
            assert app
            kv = inputs.new_kv(w, lens - 1)
            pair.oracle.append(kv)
            kv_d.copy_(torch.from_numpy(kv))
            sel_d.copy_(torch.from_numpy(sel))
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            for layer in range(L):
                tab_o, h_o, m_o = pair.oracle.resolve(layer, sel[layer // lpg])
                assert np.array_equal(tabs[layer].cpu().numpy(), tab_o)
                assert np.array_equal(hits[layer].cpu().numpy(), h_o)
                assert np.array_equal(misses[layer].cpu().numpy(), m_o)
                pair.gpu.gather_check(layer, sel_d[layer // lpg], tabs[layer], pair.mism)
                pair.compare_state(layer)
            if step % 3 == 0:
                for layer in range(L):
                    pair.compare_whole_pool(layer)
        pair.finish()
    finally:
        tr.close()
        pair.close()


# ------------------------------------------------------------------ checkpoint / resume

def test_dump_then_load_state_resumes_exactly():
    w = inputs.c3_dsa_long(0.75, steps=8, short_ctx=3000, long_ctx=9000, num_short=2)     # 2 groups of 4 layers
    w.entry_bytes = 64
    pair = Pair(w)
    tr = inputs.Trace(w)
    N, L, lpg = w.num_requests, w.num_layers, w.layers_per_group
    try:
        for step in range(8):
            sel, app, _ = tr.step()
            if step == 4:
                # checkpoint every (request, group), then bring up a fresh handle over the same host histories
                pair.gpu.join()
                snap = {(r, a): pair.gpu.dump_state(r, a) for r in range(N) for a in range(0, L, lpg)}
                appends = snap[(0, 0)]["len"] - w.init_len[0]
                old = pair.gpu
                pair.gpu = HiSparse(N, L, lpg, w.cache_slots, w.top_k, w.entry_bytes, w.capacity, w.init_len,
                                    pair.hist_gpu)
                old.close()
                pair.gpu.load_appends(appends)
                for (r, a), st in snap.items():
                    pair.gpu.load_state(r, a, st["slot_pos"], st["last_use"], st["resolves"])
                for layer in range(L):
                    pair.compare_whole_pool(layer)
            if app:
                pair.append()
            for layer in range(L):
                pair.resolve_and_compare(layer, sel[layer // lpg])
                pair.compare_state(layer)
        pair.finish()
        bad = snap[(0, 0)]["slot_pos"].copy()
        bad[1] = bad[0]
        with pytest.raises(HiSparseError) as e:
            pair.gpu.load_state(0, 0, bad, snap[(0, 0)]["last_use"], 1)
        assert e.value.code == hs.EINVAL
    finally:
        tr.close()
        pair.close()


# ------------------------------------------------------------------ failure detection without a fault

def test_bounded_wait_expires_and_the_handle_stays_usable():
    w = tiny_workload(2, 1, 1, 4, 8, 32, [20, 30])
    pair = Pair(w)
    try:
        pair.resolve_and_compare(0, np.array([[1, 2, 3, 4], [5, 6, 7, 8]]))
        waited = pair.gpu.selftest_wait_timeout(2_000_000)              # a barrier nothing completes, 2 ms limit
        assert 2_000_000 <= waited < 200_000_000
        assert pair.gpu.status() == hs.STATUS_TIMEOUT                    # reported, not hung, no fault
        pair.gpu.clear_status()
        pair.resolve_and_compare(0, np.array([[4, 9, 1, -1], [8, 7, 0, 29]]))   # the context is intact
        pair.compare_state(0)
        pair.finish()
    finally:
        pair.close()


# ------------------------------------------------------------------ boundary errors

def test_layer_times_bracket_every_resolve():
    """With PHASE_TIMERS every anchor resolve leaves its start and end stamps per layer; layers resolved one after the
    other on a stream are ordered in time; reading clears the stamps."""
    w = inputs.c2_dsa_decode(num_requests=3, num_layers=4, steps=3, context=3000)
    pair = Pair(w, flags=hs.FLAG_PHASE_TIMERS)
    tr = inputs.Trace(w)
    try:
        sel, appended, _ = tr.step()
        if appended:
            pair.append()
        for layer in range(4):
            pair.resolve_and_compare(layer, sel[layer])
        lt = pair.gpu.layer_times().astype(np.int64)
        assert lt.shape == (4, 2)
        assert np.all(lt[:, 1] > lt[:, 0]) and np.all(lt[:, 1] - lt[:, 0] < 10_000_000)
        assert np.all(lt[1:, 0] >= lt[:-1, 1])
        cleared = pair.gpu.layer_times()
        assert np.all(cleared[:, 0] == np.uint64(2**64 - 1)) and np.all(cleared[:, 1] == 0)
        pair.finish()
    finally:
        tr.close()
        pair.close()


def test_create_rejects_bad_arguments():
    hist = HostHistory(1, 64, 32)
    try:
        def make(**kw):
            a = dict(num_requests=1, num_layers=1, layers_per_group=1, cache_slots=8, top_k=4, entry_bytes=32,
                     capacity=[64], init_len=[10], host_history=[hist])
            a.update(kw)
            return HiSparse(**a)
        for bad in (dict(top_k=9), dict(entry_bytes=40), dict(cache_slots=hs.MAX_CACHE_SLOTS + 1),
                    dict(num_layers=3, layers_per_group=2), dict(init_len=[65]), dict(ctas_per_request=3)):
            with pytest.raises(HiSparseError) as e:
                make(**bad)
            assert e.value.code == hs.EINVAL
        pageable = np.zeros(64 * 32, dtype=np.uint8)
        with pytest.raises(HiSparseError) as e:
            make(host_history=[pageable.ctypes.data])
        assert e.value.code == hs.ENOTPINNED
        h = make()
        sel = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
        with pytest.raises(HiSparseError) as e:
            h.resolve(1, sel)
        assert e.value.code == hs.EINVAL
        with pytest.raises(HiSparseError):
            h.prefetch(0, torch.cuda.Stream())
        h.close()
        kv, meta = hs.device_bytes(1, 1, 1, 8, 4, 32, [64])
        assert kv == 1 * 1 * 9 * 32 and meta > 0
    finally:
        hist.free()


# ------------------------------------------------------------------ the boundary from plain C

def test_c_program_uses_the_library(tmp_path):
    import os
    import subprocess
    from paper_2608_07009_b200 import build
    root = build.ROOT
    exe = str(tmp_path / "c_abi_smoke")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    subprocess.check_call(["gcc", "-std=c99", os.path.join(root, "tests", "c_abi_smoke.c"), "-I", os.path.join(root, "include"),
                           "-I", os.path.join(cuda, "include"), "-o", exe, build.SO, "-L", os.path.join(cuda, "lib64"),
                           "-lcudart", "-Wl,-rpath," + os.path.dirname(build.SO), "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    out = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and "C-ABI OK" in out.stdout, out.stdout + out.stderr
