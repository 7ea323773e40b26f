"""Host logic: the semi-unified-memory manager model (unit states, mode switches, restore)."""
import numpy as np
import pytest

from paper_2609_34380_b200 import sum_manager as sm


def test_free_units_are_used_before_backed_ones_and_taking_a_backed_unit_switches_to_fast():
    events = []
    m = sm.SumManager(units=6, blocks_per_unit=4, residual_tensors=3, on_evict=lambda t, u: events.append(("evict", t, u)))
    m.check()
    assert m.mode == sm.MODE_FULL and list(m.free) == [3, 4, 5] and m.backed == [0, 1, 2]
    got = m.alloc_kv_blocks(12)                      # exactly the three free units
    assert got is not None and {u for u, _ in got} == {3, 4, 5}
    assert m.mode == sm.MODE_FULL and not events
    m.check()
    one = m.alloc_kv_blocks(1)                       # nothing free, nothing available: a residual unit goes
    assert one is not None and one[0][0] == 2
    assert m.mode == sm.MODE_FAST and events == [("evict", 2, 2)]
    assert m.stale == {2} and list(m.evicted) == [2] and m.backed == [0, 1]
    m.check()


def test_a_request_that_cannot_be_met_changes_nothing():
    m = sm.SumManager(units=4, blocks_per_unit=2, residual_tensors=2)
    held = m.alloc_kv_blocks(3)
    before = (list(m.free), list(m.backed), sorted(m.avail), sorted(m.full), m.mode, {u: set(b) for u, b in m.used.items()})
    assert m.alloc_kv_blocks(6) is None              # 8 blocks exist, 3 are taken
    after = (list(m.free), list(m.backed), sorted(m.avail), sorted(m.full), m.mode, {u: set(b) for u, b in m.used.items()})
    assert before == after
    m.check()
    assert m.alloc_kv_blocks(5) is not None          # exactly what is left, residual units included
    assert m.mode == sm.MODE_FAST and len(m.evicted) == 2
    m.check()
    assert held is not None


def test_freeing_returns_units_wakes_the_restore_worker_and_full_mode_waits_for_every_tensor():
    restored = []
    m = sm.SumManager(units=4, blocks_per_unit=2, residual_tensors=3, on_restore=lambda t, u: restored.append((t, u)))
    blocks = m.alloc_kv_blocks(8)                    # one free unit + all three residual units
    assert m.mode == sm.MODE_FAST and len(m.evicted) == 3 and m.restore_wakeups == 0
    by_unit = {}
    for u, b in blocks:
        by_unit.setdefault(u, []).append((u, b))
    units = sorted(by_unit)
    m.free_kv_blocks(by_unit[units[0]][:1])          # a FULL unit with one block freed becomes AVAIL
    assert units[0] in m.avail and m.restore_wakeups == 0
    m.free_kv_blocks(by_unit[units[0]][1:])          # now empty: FREE, and the worker is woken
    assert units[0] in m.free and m.restore_wakeups == 1
    m.check()
    assert m.restore_weights() == 1 and m.mode == sm.MODE_FAST      # two tensors still evicted
    m.free_kv_blocks(by_unit[units[1]] + by_unit[units[2]])
    assert m.restore_weights(max_tensors=1) == 1 and m.mode == sm.MODE_FAST
    assert m.restore_weights() == 1 and m.mode == sm.MODE_FULL
    assert sorted(t for t, _ in restored) == [0, 1, 2] and not m.stale and not m.evicted
    m.check()
    with pytest.raises(ValueError):
        m.free_kv_blocks([by_unit[units[0]][0]])     # freed twice


def test_invariants_hold_under_random_traffic():
    rng = np.random.default_rng(7)
    m = sm.SumManager(units=24, blocks_per_unit=8, residual_tensors=10)
    held = []
    for step in range(3000):
        r = rng.random()
        if r < 0.5:
            got = m.alloc_kv_blocks(int(rng.integers(0, 20)))
            if got is not None:
                assert len(set(got)) == len(got) and not set(got) & set(held)
                held.extend(got)
        elif r < 0.9 and held:
            k = int(rng.integers(1, min(len(held), 25) + 1))
            idx = rng.choice(len(held), k, replace=False)
            drop = [held[i] for i in idx]
            held = [b for i, b in enumerate(held) if i not in set(idx.tolist())]
            m.free_kv_blocks(drop)
        else:
            m.restore_weights(int(rng.integers(1, 4)))
        m.check()
        assert m.kv_blocks_in_use == len(held)
    m.free_kv_blocks(held)
    m.restore_weights()
    m.check()
    assert m.mode == sm.MODE_FULL and len(m.backed) == 10 and len(m.free) == 14


def test_schedule_from_a_bursty_trace():
    units, bpu, resid = 80, 16, 40                   # 40 residual units, as in the paper's evaluation set-up
    demand = sm.kv_demand_trace(2000, units * bpu, seed=5556)
    modes, mgr = sm.mode_schedule_from_trace(demand, units, bpu, resid)
    again, _ = sm.mode_schedule_from_trace(sm.kv_demand_trace(2000, units * bpu, seed=5556), units, bpu, resid)
    assert modes == again and len(modes) == 2000 and set(modes) <= {sm.MODE_FAST, sm.MODE_FULL}
    mgr.check()
    fast_share = modes.count(sm.MODE_FAST) / len(modes)
    switches = sum(1 for i in range(1, len(modes)) if modes[i] != modes[i - 1])
    assert 0.2 <= fast_share <= 0.9 and 2 <= switches <= 200
    # below half the capacity nothing is ever evicted: a quiet trace stays in full mode
    quiet, _ = sm.mode_schedule_from_trace(np.full(500, units * bpu // 3), units, bpu, resid)
    assert set(quiet) == {sm.MODE_FULL}
