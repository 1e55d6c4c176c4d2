"""Randomised parity soak: seeded random geometries (B, k, N, layer groups, record sizes, context lengths on both
sides of the page-table staging limit), cluster sizes, block sizes, eager or lazy recency list, replacement policies,
padding, repeated positions and repeated rows (resolves without misses) — every step compared bit for bit with the
oracle (tables, counts, LRU state, plans, bytes)."""
import numpy as np
import pytest
import torch

from paper_2608_07009_b200 import inputs, hisparse as hs
from gpu_harness import Pair

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_random_configurations(seed):
    rng = np.random.default_rng(seed)
    rng2 = np.random.default_rng(1000 + seed)     # geometry of the launch, repeated rows
    for _ in range(12):
        B = int(rng.choice([5, 33, 100, 257, 1000, 4096, 6000]))
        k = int(rng.integers(1, min(B, hs.MAX_TOP_K) + 1))
        N = int(rng.integers(1, 6))
        lpg = int(rng.choice([1, 1, 2, 4]))
        L = lpg * int(rng.integers(1, 3))
        E = int(rng.choice([16, 48, 1152, 4096]))
        lens = [int(rng.integers(k + 2, 40 * B + 100)) for _ in range(N)]
        if rng.random() < 0.3:
            lens[0] = int(rng.integers(80000, 200000))       # page table too large to stage in shared memory
        S = int(rng.choice([0, 1, 2, 4, 8]))
        policy = int(rng.choice([hs.POLICY_LRU, hs.POLICY_LRU, hs.POLICY_FIFO, hs.POLICY_RANDOM]))
        steps = 8
        w = inputs.Workload("soak", inputs.KIND_DSA_MIX, N, L, lpg, k, B, E, lens, steps, keep=int(k * rng.random()),
                            recent_window=int(rng.integers(1, 2000)), seed=int(rng.integers(1 << 30)), config_id=77)
        flags = hs.FLAG_DEBUG_VALIDATE | (hs.FLAG_EAGER_ORDER if rng2.random() < 0.2 else 0)
        narrow = rng2.random() < 0.5
        try:
            pair = Pair(w, flags=flags | (hs.FLAG_NARROW_BLOCKS if narrow else 0), ctas_per_request=S, policy=policy,
                        policy_seed=5, oracle_bytes=E <= 1152)
            assert pair.gpu.launch_geometry()["threads"] == (512 if narrow else 1024)
        except hs.HiSparseError:                    # the shape does not allow 512-thread blocks
            assert narrow
            pair = Pair(w, flags=flags, ctas_per_request=S, policy=policy, policy_seed=5, oracle_bytes=E <= 1152)
        hit_only_steps = rng2.random() < 0.5
        prev = None
        tr = inputs.Trace(w)
        side = torch.cuda.Stream() if lpg > 1 and rng.random() < 0.7 else None
        repeat = rng.random() < 0.3
        try:
            for _step in range(steps):
                if hit_only_steps and prev is not None and rng2.random() < 0.4:
                    sel, appended = prev, False     # the same rows again: nothing misses, the list is left behind
                else:
                    sel, appended, _ = tr.step()
                    sel = [x.copy() for x in sel]
                prev = sel
                if appended:
                    pair.append()
                for layer in range(L):
                    if layer % lpg == 0:
                        s = sel[layer // lpg]
                        if rng.random() < 0.3:
                            s[rng.random(s.shape) < 0.1] = -1
                        if repeat and k > 1:
                            for r in range(N):
                                s[r, int(rng.integers(k))] = s[r, int(rng.integers(k))]
                    pair.resolve_and_compare(layer, sel[layer // lpg], side_stream=side)
                    pair.compare_state(layer)
            status = pair.gpu.status()
            assert status == pair.oracle.status and (status & ~hs.STATUS_DUPLICATE) == 0
            assert int(pair.mism.item()) == 0
        finally:
            tr.close()
            pair.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_random_looping_waves(seed):
    """More requests than the GPU holds blocks (one resident wave of looping blocks): random row lengths (multiples of
    four and not, so both the short loop and the general loop are taken), cache sizes, contexts on both sides of the
    page-table staging limit, layer groups with a side-stream prefetch, policies; requests without and with misses
    mixed at random in every launch."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    rng = np.random.default_rng(seed)
    for _ in range(5):
        k = int(rng.choice([4, 7, 16, 33, 64, 100, 128, 256]))
        B = int(k * rng.choice([1, 2, 3]) + rng.integers(0, 9))
        init_len = int(rng.choice([B + 5, 3 * B, 1000, 5000, 40000]))
        lpg = int(rng.choice([1, 1, 2]))
        policy = int(rng.choice([hs.POLICY_LRU, hs.POLICY_LRU, hs.POLICY_FIFO, hs.POLICY_RANDOM]))
        N = 3 * sms + int(rng.integers(1, 400))
        w = inputs.Workload("loop", inputs.KIND_DSA_MIX, N, lpg, lpg, k, B, 16, [init_len] * N, 8)
        pair = Pair(w, flags=hs.FLAG_DEBUG_VALIDATE, policy=policy, policy_seed=3)
        side = torch.cuda.Stream() if lpg > 1 else None
        try:
            assert pair.gpu.launch_geometry()["threads"] == 512
            for step in range(6):
                if step % 2 == 1:
                    pair.append()
                rows = []
                for r in range(N):
                    res = pair.oracle.slot_pos(r, 0)
                    res = res[res >= 0]
                    if step > 0 and rng.random() < 0.6 and len(res) >= max(1, k // 2):     # nothing misses
                        n = int(rng.integers(max(1, k // 2), min(k, len(res)) + 1))
                        row = rng.choice(res, size=n, replace=False).astype(np.int32)
                        if pair.oracle.newest(r) >= 0 and n < k and rng.random() < 0.5:
                            row = np.append(row, np.int32(pair.oracle.newest(r)))
                        row = rng.permutation(np.concatenate([row, np.full(k - len(row), -1, dtype=np.int32)]))
                    else:
                        row = inputs.random_rows(rng, 1, k, pair.oracle.length(r), 0.1)[0]
                    rows.append(row)
                rows = np.stack(rows)
                for layer in range(lpg):
                    pair.resolve_and_compare(layer, rows, side_stream=side)
                    pair.compare_state(layer, requests=range(0, N, 7))
            pair.finish()
        finally:
            pair.close()
