"""Pins for the oracle's slot cache, waves and grouping (Sections 3.3, 3.4; no GPU)."""
import itertools
from collections import OrderedDict

import numpy as np
import pytest

from oracle import cache


def random_calls(rng, E, k, T, n_calls, skew=1.0):
    w = 1.0 / np.arange(1, E + 1) ** skew
    w /= w.sum()
    for _ in range(n_calls):
        yield np.stack([rng.choice(E, size=k, replace=False, p=w) for _ in range(T)]).astype(np.int32)


@pytest.mark.parametrize("E,C,Cw,k,T", [(64, 16, 0, 8, 16), (64, 16, 8, 8, 16), (64, 32, 0, 8, 4),
                                         (8, 2, 0, 2, 5), (16, 5, 3, 4, 7), (64, 8, 0, 8, 1)])
def test_invariants_on_random_streams(E, C, Cw, k, T):
    rng = np.random.default_rng(E * 1000 + C)
    sc = cache.SlotCache(E, C, Cw, bytes_per_expert=3244032)
    cw = Cw or C
    total_active = 0
    for ids in random_calls(rng, E, k, T, 40):
        before = sc.expert_slot.copy()
        plan = sc.resolve(ids)
        active = sorted(set(ids.reshape(-1).tolist()))
        total_active += len(active)
        assert plan.n_active == len(active) and plan.n_waves == -(-len(active) // cw)
        # every active expert is in exactly one wave, nobody else is
        in_maps = np.zeros(E, dtype=int)
        for w, m in enumerate(plan.expert_maps):
            members = np.nonzero(m >= 0)[0]
            assert 0 < len(members) <= cw
            assert len(set(m[members].tolist())) == len(members)          # map injective in a wave
            assert (plan.wave_of[members] == w).all()
            in_maps[members] += 1
        assert (in_maps[active] == 1).all() and in_maps.sum() == len(active)
        # hits first: no resident-at-entry expert sits in a later wave than a missing one
        res = [e for e in active if before[e] >= 0]
        mis = [e for e in active if before[e] < 0]
        if res and mis:
            assert plan.wave_of[res].max() <= plan.wave_of[mis].min()
        assert [m[0] for m in plan.misses] == mis
        for e in res:                                                      # a hit keeps its slot
            assert plan.slot_of[e] == before[e]
        # victims are never slots the same wave uses
        for (e, s, w) in plan.misses:
            others = [x for x in np.nonzero(plan.wave_of == w)[0] if x != e]
            assert all(plan.slot_of[x] != s for x in others)
        # state is a consistent partial bijection
        for s in range(C):
            e = sc.slot_expert[s]
            if e >= 0:
                assert sc.expert_slot[e] == s
        assert (sc.expert_slot >= 0).sum() == (sc.slot_expert >= 0).sum()
    st = sc.stats
    assert st.hits + st.misses == st.lookups == total_active
    assert st.h2d_bytes == st.misses * 3244032 and st.forwards == 40


def test_full_residency_bypass():
    sc = cache.SlotCache(64, 64)
    rng = np.random.default_rng(1)
    for ids in random_calls(rng, 64, 8, 16, 5):
        plan = sc.resolve(ids)
        active = sorted(set(ids.reshape(-1).tolist()))
        assert plan.n_waves == 1 and not plan.misses
        assert (plan.slot_of[active] == active).all()
    assert sc.stats == cache.Stats() and sc.tick == 0 and not sc.slot_stamp.any()


def test_one_reference_per_call_is_textbook_lru():
    """T=1, k=1: one reference per call, so recency is a total order and the cache must
    behave exactly like an OrderedDict-based LRU of capacity C."""
    E, C = 20, 6
    rng = np.random.default_rng(7)
    od = OrderedDict()
    sc = cache.SlotCache(E, C)
    hits = misses = 0
    for e in rng.integers(0, E, size=2000).tolist():
        plan = sc.resolve(np.array([[e]], dtype=np.int32))
        if e in od:
            od.move_to_end(e)
            hits += 1
            assert not plan.misses
        else:
            if len(od) >= C:
                od.popitem(last=False)
            od[e] = True
            misses += 1
            assert len(plan.misses) == 1
        assert set(np.nonzero(sc.expert_slot >= 0)[0].tolist()) == set(od)
    assert (sc.stats.hits, sc.stats.misses) == (hits, misses) and misses > C


def batched_lru(E, C, calls):
    """LRU over batched references (single-wave case), written around a dict: all experts
    of a call share one timestamp; an absentee takes a free slot (lowest index) or evicts the
    entry with the oldest timestamp that the call does not use, ties to the lower slot."""
    where = {}                                    # expert -> [stamp, slot]
    hits = misses = 0
    for now, ids in enumerate(calls, start=1):
        active = sorted(set(ids.reshape(-1).tolist()))
        for e in [e for e in active if e in where]:
            where[e][0] = now
            hits += 1
        for e in [e for e in active if e not in where]:
            used = {v[1] for v in where.values()}
            free = [s for s in range(C) if s not in used]
            if free:
                slot = free[0]
            else:
                victim = min((v[0], v[1], x) for x, v in where.items() if x not in active)[2]
                slot = where.pop(victim)[1]
            where[e] = [now, slot]
            misses += 1
    return hits, misses, {e: v[1] for e, v in where.items()}


def test_single_wave_equals_batched_lru():
    E, C, k = 32, 12, 4
    rng = np.random.default_rng(7)
    calls = list(random_calls(rng, E, k, 3, 200))            # at most 12 distinct ids per call
    sc = cache.SlotCache(E, C)
    for ids in calls:
        assert sc.resolve(ids).n_waves == 1
    h, m, where = batched_lru(E, C, calls)
    assert (sc.stats.hits, sc.stats.misses) == (h, m)
    assert {e: int(sc.expert_slot[e]) for e in np.nonzero(sc.expert_slot >= 0)[0].tolist()} == where


def test_brute_force_tiny_streams():
    """E=4, C=2, k=1: every stream of length 4; with one reference per call the cache is
    textbook LRU, empty slots fill lowest index first, and the victim is the older slot."""
    for stream in itertools.product(range(4), repeat=4):
        sc = cache.SlotCache(4, 2)
        slots = [None, None]
        age = [0, 0]
        clock = 0
        for e in stream:
            clock += 1
            plan = sc.resolve(np.array([[e]], dtype=np.int32))
            if e in slots:
                s = slots.index(e)
                assert not plan.misses
            else:
                s = 0 if (age[0], 0) <= (age[1], 1) else 1
                slots[s] = e
                assert plan.misses == [(e, s, 0)]
            age[s] = clock
            assert plan.slot_of[e] == s
            assert [(-1 if x is None else x) for x in slots] == sc.slot_expert.tolist()


def test_multi_wave_worked_example():
    """C=2, six experts: worked by hand from the rules in the module header."""
    sc = cache.SlotCache(6, 2)
    p1 = sc.resolve(np.array([[4, 1]], dtype=np.int32))
    assert p1.misses == [(1, 0, 0), (4, 1, 0)] and sc.tick == 1
    # active {0,1,3,5}; resident {1}; order [1,0,3,5]; waves [1,0], [3,5]
    p2 = sc.resolve(np.array([[5, 0], [3, 1]], dtype=np.int32))
    assert p2.n_waves == 2
    assert p2.wave_of.tolist() == [0, 0, -1, 1, -1, 1]
    # wave 0 (tick 2): 1 hits slot 0 (protected); 0 misses -> only slot 1 is free to evict
    # wave 1 (tick 3): both slots stamped 2 -> 3 takes slot 0 (lower index), 5 takes slot 1
    assert p2.misses == [(0, 1, 0), (3, 0, 1), (5, 1, 1)]
    assert p2.slot_of.tolist() == [1, 0, -1, 0, -1, 1]
    assert p2.expert_maps[0].tolist() == [1, 0, -1, -1, -1, -1]
    assert p2.expert_maps[1].tolist() == [-1, -1, -1, 0, -1, 1]
    assert sc.slot_expert.tolist() == [3, 5] and sc.slot_stamp.tolist() == [3, 3]
    assert (sc.stats.lookups, sc.stats.hits, sc.stats.misses, sc.stats.waves) == (6, 1, 5, 3)


def test_invalid_ids_are_dropped_and_flagged():
    sc = cache.SlotCache(8, 4)
    ids = np.array([[1, 9], [-2, 3]], dtype=np.int32)
    plan = sc.resolve(ids)
    assert plan.bad_id and plan.n_active == 2
    counts, offsets, perm = cache.group_pairs(ids, plan, 4, sc.max_waves)
    assert counts.sum() == 2 and sorted(perm.tolist()) == [0, 3]


@pytest.mark.parametrize("E,C,Cw,k,T", [(64, 16, 0, 8, 16), (64, 64, 0, 8, 33), (16, 5, 3, 4, 9)])
def test_grouping_is_a_stable_sort(E, C, Cw, k, T):
    rng = np.random.default_rng(3)
    sc = cache.SlotCache(E, C, Cw)
    for ids in random_calls(rng, E, k, T, 6):
        plan = sc.resolve(ids)
        counts, offsets, perm = cache.group_pairs(ids, plan, C, sc.max_waves)
        flat = ids.reshape(-1)
        keys = plan.wave_of[flat].astype(np.int64) * C + plan.slot_of[flat]
        assert np.array_equal(perm, np.argsort(keys, kind="stable").astype(np.int32))
        assert counts.sum() == flat.size and sorted(perm.tolist()) == list(range(flat.size))
        assert np.array_equal(counts, np.bincount(keys, minlength=sc.max_waves * C))
        assert offsets[0] == 0 and (np.diff(offsets) == counts).all()
        # groups of one wave are contiguous, so a wave's kernel sees one range of rows
        waves = keys[perm] // C
        assert (np.diff(waves) >= 0).all()


def test_wave_capacity_changes_the_schedule_not_the_coverage():
    rng = np.random.default_rng(11)
    ids = next(random_calls(rng, 64, 8, 16, 1, skew=0.3))
    active = sorted(set(ids.reshape(-1).tolist()))
    for C, Cw in [(8, 0), (16, 0), (16, 8), (32, 0), (64, 0)]:
        sc = cache.SlotCache(64, C, Cw)
        plan = sc.resolve(ids)
        covered = sorted(e for m in plan.expert_maps for e in np.nonzero(m >= 0)[0].tolist())
        assert covered == active                          # each selected expert exactly once
