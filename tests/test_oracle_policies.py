"""Pins of the oracle's other cache policies (Sec. 5.1): LFU against an independent replay,
Belady against its optimality and a hand-worked trace."""
import numpy as np
import pytest

import oracle


class DictLFU:
    """Textbook LFU: a use counter per column (kept for the whole session, resident or not); the
    resident column with the smallest counter is evicted, the lower index on a tie.  A step's
    columns are processed one by one in ascending index; columns of the current step are never
    chosen as victims; a miss that finds no victim is used without being cached."""

    def __init__(self, capacity):
        self.cap = capacity
        self.count = {}
        self.res = set()
        self.hits = self.misses = self.evictions = self.bypassed = 0

    def step(self, cols):
        cols = sorted(cols)
        pinned = set(cols)
        before = set(self.res)
        for c in cols:
            if c in before:
                self.hits += 1
            else:
                self.misses += 1
                if len(self.res) < self.cap:
                    self.res.add(c)
                else:
                    cand = [v for v in self.res if v not in pinned]
                    if cand:
                        victim = min(cand, key=lambda v: (self.count.get(v, 0), v))
                        self.res.remove(victim)
                        self.evictions += 1
                        self.res.add(c)
                    else:
                        self.bypassed += 1
        for c in cols:
            self.count[c] = self.count.get(c, 0) + 1


@pytest.mark.parametrize("d,cap", [(6, 0), (6, 2), (6, 6), (9, 4), (12, 5), (16, 8), (16, 3), (16, 16)])
def test_lfu_matches_independent_replay(d, cap):
    rng = np.random.default_rng(7 * d + cap)
    for trace in range(40):
        cache = oracle.Cache(d, cap, "lfu")
        ref = DictLFU(cap)
        # skewed popularity so that counters differ
        p = rng.random(d) ** 3 + 0.02
        p /= p.sum()
        for t in range(30):
            k = int(rng.integers(0, d + 1)) if trace % 2 else int(rng.integers(1, max(2, d // 2)))
            cols = rng.choice(d, size=k, replace=False, p=p)
            m = np.zeros(d, dtype=np.uint8)
            m[cols] = 1
            oracle.cache_update(cache, m)
            ref.step(cols.tolist())
            assert sorted(np.nonzero(cache.resident())[0].tolist()) == sorted(ref.res)
            assert cache.counters.tolist() == [ref.hits, ref.misses, ref.evictions, ref.bypassed]
            assert cache.count.tolist() == [ref.count.get(i, 0) for i in range(d)]
            assert int(cache.n_resident[0]) == len(ref.res) <= cap


def test_lfu_keeps_the_frequent_column_where_lru_drops_it():
    # column 0 is used three times early, then 1 and 2 fill the cache of two slots one after
    # another: LRU drops 0 (oldest use), LFU drops the column used once
    seq = [[0], [0], [0], [1], [2]]
    lru, lfu = oracle.Cache(4, 2, "lru"), oracle.Cache(4, 2, "lfu")
    for cols in seq:
        m = np.zeros(4, np.uint8)
        m[cols] = 1
        oracle.cache_update(lru, m)
        oracle.cache_update(lfu, m)
    assert lru.resident().tolist() == [0, 1, 1, 0]
    assert lfu.resident().tolist() == [1, 0, 1, 0]
    assert lfu.count.tolist() == [3, 1, 1, 0]


def _masks(rng, T, d, k, corr):
    """A trace whose consecutive masks share about `corr` of their columns."""
    cur = rng.choice(d, size=k, replace=False)
    out = np.zeros((T, d), dtype=np.uint8)
    for t in range(T):
        keep = cur[rng.random(k) < corr]
        rest = np.setdiff1d(np.arange(d), keep)
        cur = np.concatenate([keep, rng.choice(rest, size=k - len(keep), replace=False)])
        out[t, cur] = 1
    return out


def test_belady_hand_trace_and_optimality():
    # capacity 2, columns one at a time: 0 1 2 0 1 -> Belady evicts 1 (next use farther than 0's)
    # when 2 arrives?  next uses at that point: 0 -> t=3, 1 -> t=4: 1 is farther, so 1 goes; then
    # 0 hits, 1 misses: 1 hit in total.  LRU evicts 0 and gets no hit at all.
    seq = [0, 1, 2, 0, 1]
    m = np.zeros((5, 3), np.uint8)
    for t, c in enumerate(seq):
        m[t, c] = 1
    assert oracle.belady_hits(m, 2) == (1, 4)
    lru = oracle.Cache(3, 2)
    for t in range(5):
        oracle.cache_update(lru, m[t])
    assert lru.counters[0] == 0
    # on random correlated traces no online policy beats the offline one
    rng = np.random.default_rng(0)
    for trial in range(12):
        d, k, cap = 48, 8, int(rng.integers(8, 30))
        masks = _masks(rng, 40, d, k, corr=float(rng.choice([0.3, 0.6, 0.9])))
        hb, mb = oracle.belady_hits(masks, cap)
        assert hb + mb == 40 * k
        for pol in ("lru", "lfu"):
            c = oracle.Cache(d, cap, pol)
            for t in range(40):
                oracle.cache_update(c, masks[t])
            assert c.counters[0] <= hb
        # everything fits: only cold misses
        assert oracle.belady_hits(masks, d)[1] == int(masks.any(axis=0).sum())
