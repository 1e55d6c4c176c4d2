"""Pins for the oracle's alternative replacement policies (the paper's cache-locality study, Sec. 4.3 / Fig. 6,
replays FIFO and random replacement against the same selection stream as LRU)."""
import collections

import numpy as np
import pytest

import os

from oracle import Oracle, FLAG_NO_BYTES, POLICY_FIFO, POLICY_LRU, POLICY_RANDOM
from oracle import oracle as oracle_mod
from paper_2608_07009_b200 import inputs
from lru_list_sim import ListLRUSim

POLICIES = {"lru": POLICY_LRU, "fifo": POLICY_FIFO, "random": POLICY_RANDOM}


def make(B, k, length, policy, seed=0):
    return Oracle(1, 1, 1, B, k, 16, [length + 64], [length], None, FLAG_NO_BYTES, policy=POLICIES[policy],
                  policy_seed=seed)


GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
GAMMA = 0x9E3779B97F4A7C15      # splitmix64's increment
M64 = (1 << 64) - 1


def test_mix64_is_the_published_splitmix64_output_function():
    """splitmix64 seeded with 0 returns mix(0 + gamma), mix(0 + 2 gamma), ...; the oracle's mix64 adds gamma itself, so
    mix64(0), mix64(gamma), mix64(2 gamma) must be the generator's published first three outputs for seed 0."""
    published = [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    assert [oracle_mod.mix64((i * GAMMA) & M64) for i in range(3)] == published


def test_random_key_worked_example_and_argument_placement():
    with open(os.path.join(GOLDEN, "random_key_worked.txt")) as f:
        rows = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    vals = {ln.split("=")[0].strip(): int(ln.rsplit("=", 1)[1], 16) for ln in rows}
    assert oracle_mod.mix64(vals["a0"]) == vals["a6"] and oracle_mod.mix64(vals["b0"]) == vals["b6"]
    assert oracle_mod.random_key(0x1234, 3, 2, 5, 7) == vals["key"] == 0xC66719FE
    # where each argument enters: request and group are folded into the seed word (high / low half), the resolve
    # count and the slot are added to the mixed seed (high / low half); the key is the LOW half of the last mix
    seed = 0x0123456789ABCDEF
    key = oracle_mod.random_key
    assert key(seed, 5, 9, 11, 13) == key(seed ^ (5 << 32) ^ 9, 0, 0, 11, 13)
    base = oracle_mod.mix64(seed ^ (5 << 32 | 9))
    assert key(seed, 5, 9, 11, 13) == oracle_mod.mix64((base + (11 << 32) + 13) & M64) & 0xFFFFFFFF
    assert len({key(seed, r, g, t, s) for r in range(3) for g in range(3) for t in range(3) for s in range(3)}) == 81


@pytest.mark.parametrize("policy", ["fifo", "random"])
@pytest.mark.parametrize("B", [1, 2, 3, 5, 8, 12])
def test_policy_against_list_simulator(policy, B):
    rng = np.random.default_rng(B * 31 + len(policy))
    for k in range(1, B + 1):
        for universe in sorted({k, B + 1, 3 * B}):
            if universe < k:
                continue
            o = make(B, k, universe, policy, seed=77)
            sim = ListLRUSim(B, k, universe, policy=policy, seed=77)
            for step in range(40):
                row = inputs.random_rows(rng, 1, k, universe, 0.1 if step % 4 == 0 else 0.0)[0]
                tab, hits, misses = o.resolve(0, row[None])
                out, h, m, plan, _ = sim.resolve(row)
                assert tab[0].tolist() == out
                assert (int(hits[0]), int(misses[0])) == (h, m)
                assert o.slot_pos(0, 0).tolist() == sim.slot_pos
                ppos, pslot = o.plan(0, 0)
                assert list(zip(ppos.tolist(), pslot.tolist())) == plan
                if policy == "fifo":      # the stamps are fetch times only: their order is the insertion order
                    lu = o.last_use(0, 0)
                    assert [int(s) for s in np.lexsort((np.arange(B), lu))] == sim.order
            o.close()


@pytest.mark.parametrize("B", [1, 3, 8])
def test_fifo_k1_is_a_textbook_queue(B):
    rng = np.random.default_rng(B)
    accesses = rng.integers(0, 2 * B + 2, size=300).tolist()
    o = make(B, 1, 4 * B + 8, "fifo")
    got = [int(o.resolve(0, np.array([[p]], dtype=np.int32))[2][0]) for p in accesses]
    queue, want = collections.deque(), []
    for p in accesses:
        if p in queue:
            want.append(0)
        else:
            if len(queue) == B:
                queue.popleft()
            queue.append(p)
            want.append(1)
    assert got == want
    assert sorted(x for x in o.slot_pos(0, 0).tolist() if x >= 0) == sorted(queue)


def test_random_victims_are_valid_and_seed_dependent():
    B, k = 32, 8
    rng = np.random.default_rng(1)
    rows = inputs.random_rows(rng, 60, k, 200)
    tables = []
    for seed in (1, 2):
        o = make(B, k, 200, "random", seed)
        tabs = []
        for row in rows:
            prev = o.slot_pos(0, 0)
            tab, h, m = o.resolve(0, row[None])
            sp = o.slot_pos(0, 0)
            assert len(set(tab[0].tolist())) == k and int(h[0]) + int(m[0]) == k
            for j, p in enumerate(row.tolist()):          # hits stay where they were
                if p in prev.tolist():
                    assert tab[0, j] == prev.tolist().index(p)
            assert set(row.tolist()) <= set(sp.tolist())
            tabs.append(tab.copy())
        tables.append(np.concatenate(tabs))
    assert not np.array_equal(tables[0], tables[1])


def test_miss_rate_trend_on_dsa_trace():
    """Same selection stream under each policy (the method of Sec. 4.3): B = k misses the most, LRU at 2k misses no
    more than FIFO at 2k, and doubling the LRU cache lowers the miss count further."""
    w = inputs.c2_dsa_decode(num_requests=1, num_layers=1, steps=60, context=8192)
    def misses(B, policy):
        o = Oracle(1, 1, 1, B, w.top_k, 16, w.capacity, w.init_len, None, FLAG_NO_BYTES, policy=policy, policy_seed=5)
        tr = inputs.Trace(w)
        tot = 0
        for s in range(60):
            sel, app, _ = tr.step()
            if app:
                o.append()
            _, h, m = o.resolve(0, sel[0])
            if s >= 10:
                tot += int(m[0])
        tr.close()
        return tot
    k = w.top_k
    m_k, m_lru2, m_fifo2, m_rand2, m_lru4 = (misses(k, POLICY_LRU), misses(2 * k, POLICY_LRU), misses(2 * k, POLICY_FIFO),
                                             misses(2 * k, POLICY_RANDOM), misses(4 * k, POLICY_LRU))
    assert m_k > m_fifo2 >= m_lru2 > m_lru4
    assert m_k > m_rand2 >= m_lru4
