"""Pins of the oracle's unit-cache policy (usage scores with decay): with a decay below one half the victim is the
least recently used unit, with decay 1 the least frequently used one -- both checked against textbook
implementations written here -- plus the invariants of a batch access."""
import collections

import numpy as np
import pytest

from oracle.ltri_oracle import UnitCachePolicy


@pytest.mark.parametrize("decay", [0.1, 0.3, 0.45])
def test_small_decay_is_least_recently_used(decay):
    r = np.random.default_rng(1)
    cap = 6
    pol = UnitCachePolicy(cap, decay)
    lru = collections.OrderedDict()
    for step in range(400):
        u = int(r.integers(0, 14))
        fetched = pol.access([u])
        if u in lru:
            lru.move_to_end(u)
            assert fetched == []
        else:
            if len(lru) == cap:
                lru.popitem(last=False)
            lru[u] = True
            assert fetched == [u]
        assert sorted(int(t) for t in pol.tags if t >= 0) == sorted(lru)
    assert pol.hits + pol.misses == 400 and pol.hits > 50


def test_decay_one_is_least_frequently_used():
    r = np.random.default_rng(2)
    cap = 5
    pol = UnitCachePolicy(cap, 1.0)
    slots = [None] * cap          # textbook: (unit, count) per slot, victim = lowest count, lowest slot among equals
    for step in range(300):
        u = int(r.integers(0, 11))
        pol.access([u])
        held = [s[0] if s else None for s in slots]
        if u in held:
            i = held.index(u)
            slots[i] = (u, slots[i][1] + 1)
        else:
            counts = [s[1] if s else 0 for s in slots]
            i = counts.index(min(counts))
            slots[i] = (u, 1)
        assert [s[0] if s else -1 for s in slots] == pol.tags.tolist()
        assert [float(s[1]) if s else 0.0 for s in slots] == pol.scores.tolist()


def test_batch_access_invariants():
    r = np.random.default_rng(3)
    cap = 8
    pol = UnitCachePolicy(cap, 0.1)
    named_total = 0
    for step in range(200):
        k = int(r.integers(1, cap + 1))
        units = sorted(r.choice(30, size=k, replace=False).tolist())
        before = set(int(t) for t in pol.tags if t >= 0)
        fetched = pol.access(units)
        after = [int(t) for t in pol.tags if t >= 0]
        named_total += k
        assert len(set(after)) == len(after) <= cap                  # no unit twice
        assert set(units) <= set(after)                              # every named unit is held afterwards
        assert set(fetched) == set(units) - before                   # exactly the absent ones were fetched
        assert all(pol.scores[np.nonzero(pol.tags == u)[0][0]] >= 1 for u in units)
    assert pol.hits + pol.misses == named_total
    with pytest.raises(ValueError):
        UnitCachePolicy(2, 0.1).access([1, 2, 3])
