"""The catch-up rule of the lazily kept recency list, as a host model checked against the oracle's stamps.

The CUDA path keeps, next to the stamps of Sec. 3.2, a list of the slots from least to most recent.  Resolves in
which nothing misses only write stamps and leave the list behind; the next resolve that needs victims brings it up
to date with this rule: slots not stamped since keep their relative order; the slots stamped since follow, laid out
by slot and then split stably, once per bit of the index of the resolve that stamped them.  This file restates the
rule in numpy and checks, on stamps produced by the oracle, that it yields exactly the slots sorted by
(stamp, slot) - for any number of skipped resolves, and for the one-resolve-at-a-time update as a special case.
(The kernel's own implementation of the rule is checked on the GPU, tests/test_gpu_parity.py.)
"""
import numpy as np
import pytest

from oracle import Oracle, FLAG_NO_BYTES
from paper_2608_07009_b200 import inputs


def catch_up(order_old: np.ndarray, last_use: np.ndarray, order_t: int, t: int) -> np.ndarray:
    """order_old is current for resolve count order_t; last_use are the stamps after resolve t (resolves
    order_t+1 .. t had no misses, so they stamped 2u+1 only)."""
    B = len(last_use)
    thr = 2 * order_t + 2
    touched = last_use >= thr
    untouched_part = [s for s in order_old if not touched[s]]
    seg = [s for s in range(B) if touched[s]]                      # by slot
    nsteps = t - order_t
    b = 0
    while b < 32 and ((nsteps - 1) >> b) != 0:                     # one stable split per bit of the step index
        key = [((int(last_use[s]) - thr) >> 1 >> b) & 1 for s in seg]
        seg = [s for s, bit in zip(seg, key) if bit == 0] + [s for s, bit in zip(seg, key) if bit == 1]
        b += 1
    return np.array(untouched_part + seg, dtype=np.int64)


def sorted_by_stamp(last_use: np.ndarray) -> np.ndarray:
    return np.lexsort((np.arange(len(last_use)), last_use))


@pytest.mark.parametrize("B,k", [(1, 1), (4, 2), (12, 5), (37, 9), (300, 130)])
def test_catch_up_equals_sorting_by_stamp(B, k):
    rng = np.random.default_rng(B)
    length = 3 * B + 5
    o = Oracle(1, 1, 1, B, k, 16, [length + 8], [length], None, FLAG_NO_BYTES)
    try:
        t = 0
        for run in (1, 2, 3, 5, 8, 17, 40, 1, 130):
            for _ in range(2):                                     # resolves with misses: the list is kept current
                row = inputs.random_rows(rng, 1, k, length, 0.1)
                o.resolve(0, row)
                t += 1
            order_t, order_old = t, sorted_by_stamp(o.last_use(0, 0).astype(np.int64))
            for i in range(run):                                   # nothing misses: stamps only
                res = o.slot_pos(0, 0)
                res = res[res >= 0]
                n = int(rng.integers(0, min(k, len(res)) + 1))
                row = np.full((1, k), -1, dtype=np.int32)
                row[0, :n] = rng.choice(res, size=n, replace=False)
                _, _, m = o.resolve(0, row)
                assert int(m[0]) == 0
                t += 1
                lu = o.last_use(0, 0).astype(np.int64)
                assert np.array_equal(catch_up(order_old, lu, order_t, t), sorted_by_stamp(lu)), (run, i)
            assert o.steps(0, 0) == t
    finally:
        o.close()


def test_one_resolve_behind_is_the_ordinary_update():
    """With a single outstanding resolve the rule has no split pass: untouched slots in their old order, then the
    hit slots by slot - the list update every resolve with misses performs (victims aside)."""
    lu_before = np.array([2, 5, 4, 0, 6, 6], dtype=np.int64)      # current for t = 3
    order_old = sorted_by_stamp(lu_before)                         # [3, 0, 2, 1, 4, 5]
    lu_after = lu_before.copy()
    lu_after[[4, 1]] = 2 * 4 + 1                                   # resolve 4 hits slots 4 and 1
    got = catch_up(order_old, lu_after, 3, 4)
    assert got.tolist() == [3, 0, 2, 5, 1, 4]
    assert np.array_equal(got, sorted_by_stamp(lu_after))
