"""Slot cache, waves and token grouping (oracle; test infrastructure; integers only).

Section 3.3 of the paper: each sparse layer owns C expert slots (k <= C <= E), a
global-expert -> slot map and a recency timestamp; resident active experts are
hits, missing ones replace the least-recently-used slots that the current wave
does not protect; with C = E everything is preloaded and lookups and
replacement are switched off.  Section 3.4: the active expert set is cut into
waves of at most C experts; each wave gets an expert map that sends its members
to their slots and every other expert to an inactive sentinel; tokens are
grouped by selected expert for the fused kernel (Figure 1 caption).

The paper gives the rules, not a procedure.  The procedure below is this
build's reading (each choice is listed in the design notes):
  * active list = distinct valid ids, ascending; ids outside [0, E) select nothing.
  * execution order = experts resident at call entry (ascending id), then the rest
    (ascending id); wave w = the w-th run of `wave_cap` experts of that order.
  * one clock tick per wave; a hit or an install stamps the slot with the tick.
  * victim = the unprotected slot with the smallest (stamp, slot index); empty
    slots carry stamp 0, so they fill first, lowest index first.
  * protected = slots of the current wave's members (hits, and misses already installed).
  * sentinel = -1.
  * grouping key of pair p = t*k + j is (wave, slot) of its expert; pairs are
    ordered by key, ties by ascending p (a stable sort).
"""
from dataclasses import dataclass, field

import numpy as np

SENTINEL = -1


@dataclass
class Plan:
    n_active: int
    n_waves: int
    wave_of: np.ndarray            # [E] wave index of each active expert, else -1
    slot_of: np.ndarray            # [E] slot of each active expert at its wave, else -1
    misses: list                   # [(expert, slot, wave)] in the order they are installed
    bad_id: bool                   # some id was outside [0, E)
    expert_maps: list = field(default_factory=list)   # per wave: [E] slot or -1


@dataclass
class Stats:
    lookups: int = 0
    hits: int = 0
    misses: int = 0
    waves: int = 0
    h2d_bytes: int = 0
    forwards: int = 0


class SlotCache:
    """State of one layer's cache.  `bytes_per_expert` only feeds the H2D counter."""

    def __init__(self, num_experts, num_slots, wave_cap=0, bytes_per_expert=0):
        E, C = int(num_experts), int(num_slots)
        Cw = int(wave_cap) if wave_cap else C
        if not (1 <= C <= E and 1 <= Cw <= C):
            raise ValueError("need 1 <= wave_cap <= C <= E")
        self.E, self.C, self.Cw = E, C, Cw
        self.bytes_per_expert = int(bytes_per_expert)
        self.reset()

    def reset(self):
        E, C = self.E, self.C
        self.stats = Stats()
        self.tick = 0
        if C == E:                                   # fully resident: identity, preloaded
            self.expert_slot = np.arange(E, dtype=np.int32)
            self.slot_expert = np.arange(C, dtype=np.int32)
        else:
            self.expert_slot = np.full(E, SENTINEL, dtype=np.int32)
            self.slot_expert = np.full(C, SENTINEL, dtype=np.int32)
        self.slot_stamp = np.zeros(C, dtype=np.uint64)

    @property
    def max_waves(self):
        return -(-self.E // self.Cw)

    def resolve(self, topk_ids):
        """One layer call: active ids -> waves, slots, misses.  Updates the state."""
        E, C, Cw = self.E, self.C, self.Cw
        ids = np.asarray(topk_ids).reshape(-1)
        valid = (ids >= 0) & (ids < E)
        bad = bool((~valid).any())
        active = sorted(set(int(e) for e in ids[valid]))
        n = len(active)
        wave_of = np.full(E, SENTINEL, dtype=np.int32)
        slot_of = np.full(E, SENTINEL, dtype=np.int32)
        if C == E:
            # full residency: no lookups, no replacement, no counters (Section 3.3)
            for e in active:
                wave_of[e] = 0
                slot_of[e] = e
            plan = Plan(n, 1 if n else 0, wave_of, slot_of, [], bad)
            if n:
                plan.expert_maps.append(slot_of.copy())
            return plan

        resident = [e for e in active if self.expert_slot[e] >= 0]
        absent = [e for e in active if self.expert_slot[e] < 0]
        order = resident + absent
        n_waves = -(-n // Cw)
        misses = []
        expert_maps = []
        for w in range(n_waves):
            members = order[w * Cw:(w + 1) * Cw]
            self.tick += 1
            protected = set(int(self.expert_slot[e]) for e in members if self.expert_slot[e] >= 0)
            for e in members:
                s = int(self.expert_slot[e])
                if s >= 0:
                    self.stats.hits += 1
                else:
                    cands = [(int(self.slot_stamp[v]), v) for v in range(C) if v not in protected]
                    _, s = min(cands)
                    old = int(self.slot_expert[s])
                    if old >= 0:
                        self.expert_slot[old] = SENTINEL
                    self.slot_expert[s] = e
                    self.expert_slot[e] = s
                    protected.add(s)
                    misses.append((e, s, w))
                    self.stats.misses += 1
                    self.stats.h2d_bytes += self.bytes_per_expert
                self.slot_stamp[s] = self.tick
                wave_of[e] = w
                slot_of[e] = s
            self.stats.lookups += len(members)
            self.stats.waves += 1
            m = np.full(E, SENTINEL, dtype=np.int32)
            for e in members:
                m[e] = slot_of[e]
            expert_maps.append(m)
        self.stats.forwards += 1
        return Plan(n, n_waves, wave_of, slot_of, misses, bad, expert_maps)


def group_pairs(topk_ids, plan, num_slots, max_waves):
    """Token grouping: histogram, exclusive prefix sum, stable permutation.

    Key of pair p = t*k + j is wave_of[e]*C + slot_of[e]; pairs with an invalid id
    are left out.  Returns (counts [max_waves*C], offsets [max_waves*C + 1], perm).
    """
    ids = np.asarray(topk_ids).reshape(-1)
    C = int(num_slots)
    n_keys = int(max_waves) * C
    E = len(plan.wave_of)
    keys = []
    pairs = []
    for p, e in enumerate(ids):
        e = int(e)
        if 0 <= e < E and plan.wave_of[e] >= 0:
            keys.append(int(plan.wave_of[e]) * C + int(plan.slot_of[e]))
            pairs.append(p)
    counts = np.zeros(n_keys, dtype=np.int32)
    for kk in keys:
        counts[kk] += 1
    offsets = np.zeros(n_keys + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    order = sorted(range(len(pairs)), key=lambda i: keys[i])      # Python's sort is stable
    perm = np.array([pairs[i] for i in order], dtype=np.int32)
    return counts, offsets, perm
