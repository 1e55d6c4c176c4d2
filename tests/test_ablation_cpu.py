"""The offline farthest-next-use simulator of the policy ablation (host only): it must be optimal on tiny inputs
(exhaustive search over every eviction choice) and never miss more than the online policies of the oracle."""
import functools

import numpy as np
import pytest

from oracle import Oracle, FLAG_NO_BYTES, POLICY_FIFO, POLICY_LRU, POLICY_RANDOM
from paper_2608_07009_b200 import inputs
from paper_2608_07009_b200.ablation import belady_misses


def optimal_misses(rows, B):
    rows = [tuple(int(p) for p in r if p >= 0) for r in rows]

    @functools.lru_cache(maxsize=None)
    def best(t, resident):
        if t == len(rows):
            return 0
        cur = set(rows[t])
        res = set(resident)
        miss = cur - res
        keep_pool = sorted(res - cur)
        room = B - len(cur)
        if len(keep_pool) <= room:
            return len(miss) + best(t + 1, tuple(sorted(cur | set(keep_pool))))
        import itertools
        return len(miss) + min(best(t + 1, tuple(sorted(cur | set(c)))) for c in itertools.combinations(keep_pool, room))
    return best(0, ())


@pytest.mark.parametrize("B,k,U", [(2, 1, 4), (3, 1, 5), (3, 2, 5), (4, 2, 6)])
def test_belady_is_optimal_on_tiny_inputs(B, k, U):
    rng = np.random.default_rng(B * 10 + k)
    for _ in range(5):
        rows = inputs.random_rows(rng, 9, k, U)
        assert int(belady_misses(rows, B).sum()) == optimal_misses(rows, B)


def test_belady_bounds_the_online_policies():
    rng = np.random.default_rng(3)
    B, k, U = 24, 8, 60
    rows = inputs.random_rows(rng, 80, k, U)
    bel = int(belady_misses(rows, B).sum())
    for pol in (POLICY_LRU, POLICY_FIFO, POLICY_RANDOM):
        o = Oracle(1, 1, 1, B, k, 16, [U + 8], [U], None, FLAG_NO_BYTES, policy=pol, policy_seed=4)
        online = sum(int(o.resolve(0, r[None])[2][0]) for r in rows)
        assert bel <= online
    assert int(belady_misses(rows, B)[0]) == k          # cold cache
