"""The expert pool's replacement policy (Section 3.4: an X-slot LRU pool, waves when the routed union does not
fit) as pure host logic, through the C ABI's acm_pool_plan: hand-worked cases, invariants on random block
sequences, and agreement with the policy restated in Python."""
import numpy as np

from paper_2608_02989_b200 import acm
from tests.helpers import LruModel


def test_hand_worked_blocks():
    # 4 slots holding experts 0..3, all never used; block 1 activates {1, 5}: a hit on 1 (slot 1), 5 goes into the
    # least recently used slot the block does not use, lowest index first: slot 0
    se, lu, tick, loads, hits = acm.pool_plan(8, [0, 1, 2, 3], [0, 0, 0, 0], 0, {1, 5})
    assert (hits, loads, tick) == (1, [(5, 0, 0)], 1)
    assert se == [5, 1, 2, 3] and lu == [1, 1, 0, 0]
    # block 2 activates {2, 6, 7}: hit on 2 (slot 2); 6 and 7 take the two oldest free-to-take slots: 3 (never
    # used), then 0 or 1 (both used at tick 1: the lower index, 0)
    se, lu, tick, loads, hits = acm.pool_plan(8, se, lu, tick, {2, 6, 7})
    assert (hits, loads) == (1, [(6, 3, 0), (7, 0, 0)])
    assert se == [7, 1, 2, 6] and lu == [2, 1, 2, 2]
    # block 3 activates six experts, two of them resident (1, 2): wave 0 may only take slots 0 and 3 (1 and 2 are in
    # use), wave 1 may take anything it has not just filled -- least recently used first, and all four slots carry
    # the same tick by then, so in slot order
    se, lu, tick, loads, hits = acm.pool_plan(8, se, lu, tick, {0, 1, 2, 3, 4, 5})
    assert hits == 2
    assert loads == [(0, 0, 0), (3, 3, 0), (4, 0, 1), (5, 1, 1)]
    assert se == [4, 5, 2, 3]


def test_empty_slots_are_filled_first_and_nothing_loads_on_hits_only():
    se, lu, tick, loads, hits = acm.pool_plan(16, [3, -1, 9, -1], [5, 0, 7, 0], 7, {3, 9})
    assert (hits, loads, se, tick) == (2, [], [3, -1, 9, -1], 8)
    se, lu, tick, loads, hits = acm.pool_plan(16, se, lu, tick, {3, 4, 5})
    assert hits == 1 and loads == [(4, 1, 0), (5, 3, 0)]


def test_random_block_sequences_against_the_restated_policy_and_invariants():
    rng = np.random.default_rng(7)
    for case in range(60):
        E = int(rng.choice([8, 33, 64, 128]))
        n_slots = int(rng.integers(1, E + 1))
        initial = rng.permutation(E)[: int(rng.integers(0, n_slots + 1))].tolist()
        model = LruModel(n_slots, initial)
        se, lu, tick = list(model.slot_expert), list(model.last_use), 0
        for block in range(12):
            n_act = int(rng.integers(0, min(E, 3 * n_slots) + 1))
            activated = set(rng.permutation(E)[:n_act].tolist())
            before = list(se)
            want_hits, want_misses = model.block(set(activated))
            se, lu, tick, loads, hits = acm.pool_plan(E, se, lu, tick, activated)
            assert (hits, len(loads)) == (want_hits, want_misses)
            assert se == model.slot_expert and lu == model.last_use and tick == model.tick
            # invariants: every activated expert is a hit or loaded exactly once, in ascending id and wave order
            resident_before = {e for e in before if e >= 0}
            assert [e for e, _, _ in loads] == sorted(activated - resident_before)
            assert [w for _, _, w in loads] == sorted(w for _, _, w in loads)
            hit_slots = {s for s, e in enumerate(before) if e in activated}
            for w in set(w for _, _, w in loads):
                slots = [s for _, s, ww in loads if ww == w]
                assert len(slots) == len(set(slots))                      # a wave fills a slot once
                if w == 0:
                    assert not (set(slots) & hit_slots)                   # never a slot the running FFN reads
            if len(activated) <= n_slots:
                assert all(w == 0 for _, _, w in loads)                    # fits: one wave
                assert activated <= {e for e in se if e >= 0}              # and everything is resident afterwards


def test_bad_pool_descriptions_are_rejected():
    import pytest
    with pytest.raises(acm.AcmError):
        acm.pool_plan(8, [1, 1], [0, 0], 0, {2})          # an expert in two slots
    with pytest.raises(acm.AcmError):
        acm.pool_plan(8, [9, -1], [0, 0], 0, {2})         # expert id out of range
