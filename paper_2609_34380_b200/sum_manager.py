"""Host-side model of the semi-unified-memory manager that decides the precision mode.

Paper: "KV-Cache-Pressure-aware DPS", Algorithm "KV block allocation and deallocation in SUM".  The
shared region of GPU memory is a pool of equally sized physical units.  A unit is in exactly one
state:

    FREE    no KV blocks and no residual mapping;
    BACKED  bound to a residual weight tensor (full mode needs every residual tensor BACKED);
    AVAIL   holds KV blocks and has at least one free block;
    FULL    holds KV blocks and has no free block.

Two further sets describe residual weight tensors, not units:

    STALE    residual mappings that were invalidated when their unit was handed to the KV cache;
    EVICTED  weights whose residual bytes live in the host copy only, awaiting restoration.

Allocation takes units from AVAIL, then FREE, then BACKED; taking a BACKED unit switches the system
to the lower-precision (fast) mode at once, because fast mode never reads residual bytes.  Freeing
the last block of a unit returns it to FREE and wakes the restore worker, which rebinds evicted
residual tensors to free units and copies their bytes back; the mode returns to full only when all
of them are back ("Overall concept" paragraph: the mode is reset when the restore worker has
populated all residual tensors).

This is a model for schedules and tests: it moves no memory itself.  The `on_evict` / `on_restore`
callbacks are where a serving engine would unmap / remap the unit and start the copy
(`dps_restore_residual`).  Readings taken where the algorithm is silent: a request that cannot be
satisfied allocates nothing (the partial allocation is rolled back); units are taken in FIFO order
from FREE and in LIFO order from BACKED and AVAIL; an evicted tensor is restored into any free unit.
"""
from __future__ import annotations

from collections import deque
from dataclasses import dataclass, field
from typing import Callable, Deque, Dict, List, Optional, Sequence, Set, Tuple

import numpy as np

MODE_FAST, MODE_FULL = 0, 1
Block = Tuple[int, int]          # (unit, block index inside the unit)


@dataclass
class SumManager:
    units: int                                   # physical units in the shared region
    blocks_per_unit: int                         # KV blocks one unit holds
    residual_tensors: int                        # residual weight tensors, one unit each, BACKED at start
    on_evict: Optional[Callable[[int, int], None]] = None      # (tensor, unit): mapping invalidated
    on_restore: Optional[Callable[[int, int], None]] = None    # (tensor, unit): rebound, copy its bytes back
    free: Deque[int] = field(default_factory=deque)
    backed: List[int] = field(default_factory=list)
    avail: List[int] = field(default_factory=list)
    full: Set[int] = field(default_factory=set)
    stale: Set[int] = field(default_factory=set)
    evicted: Deque[int] = field(default_factory=deque)
    mode: int = MODE_FULL
    restore_wakeups: int = 0

    def __post_init__(self) -> None:
        if not 0 <= self.residual_tensors <= self.units or self.blocks_per_unit < 1:
            raise ValueError("need 0 <= residual_tensors <= units and blocks_per_unit >= 1")
        self.tensor_of_unit: Dict[int, int] = {u: u for u in range(self.residual_tensors)}
        self.backed = list(range(self.residual_tensors))
        self.free = deque(range(self.residual_tensors, self.units))
        self.used: Dict[int, Set[int]] = {}       # unit -> allocated block indices (KV units only)

    # ---- Algorithm: AllocKVBlock ---------------------------------------------------------------
    def alloc_kv_blocks(self, n: int) -> Optional[List[Block]]:
        """n KV blocks, or None (and no change) if the shared region cannot supply them."""
        if n < 0:
            raise ValueError("n must be non-negative")
        result: List[Block] = []
        claimed: List[Tuple[int, Optional[int]]] = []         # units newly turned into KV units (for the roll-back)
        while len(result) < n:
            if not self.avail:
                if self.free:
                    u = self.free.popleft()
                    claimed.append((u, None))
                elif self.backed:
                    u = self.backed.pop()
                    claimed.append((u, self.tensor_of_unit[u]))
                else:
                    self._roll_back(result, claimed)
                    return None
                self.used[u] = set()
                self.avail.append(u)
            u = self.avail.pop()
            taken = self.used[u]
            for b in range(self.blocks_per_unit):
                if len(result) == n:
                    break
                if b not in taken:
                    taken.add(b)
                    result.append((u, b))
            if len(taken) == self.blocks_per_unit:
                self.full.add(u)
            else:
                self.avail.append(u)
        # the request is granted: units drawn from BACKED lose their residual mapping now
        for u, tensor in claimed:
            if tensor is not None:
                del self.tensor_of_unit[u]
                self.mode = MODE_FAST                         # "activate lower-precision mode"
                self.stale.add(tensor)                        # "mark u's residual mapping as stale"
                self.evicted.append(tensor)
                if self.on_evict:
                    self.on_evict(tensor, u)
        return result

    def _roll_back(self, result: List[Block], claimed: List[Tuple[int, Optional[int]]]) -> None:
        for u, b in result:
            self.used[u].discard(b)
            if u in self.full:
                self.full.discard(u)
                self.avail.append(u)
        for u, tensor in reversed(claimed):
            if u in self.avail:
                self.avail.remove(u)
            self.full.discard(u)
            del self.used[u]
            if tensor is None:
                self.free.appendleft(u)
            else:
                self.backed.append(u)

    # ---- Algorithm: FreeKVBlock ----------------------------------------------------------------
    def free_kv_blocks(self, blocks: Sequence[Block]) -> None:
        wake = False
        for u, b in blocks:
            taken = self.used.get(u)
            if taken is None or b not in taken:
                raise ValueError(f"block {(u, b)} is not allocated")
            taken.remove(b)
            if u in self.full:
                self.full.discard(u)
                self.avail.append(u)
            if not taken:
                self.avail.remove(u)
                del self.used[u]
                self.free.append(u)
                if self.evicted:
                    wake = True
        if wake:
            self.restore_wakeups += 1                         # "wake RestoreWeights"

    # ---- the restore worker --------------------------------------------------------------------
    def restore_weights(self, max_tensors: Optional[int] = None) -> int:
        """Rebind up to max_tensors evicted residual tensors to free units (all that fit by default).
        Returns how many were restored; the mode returns to full when none is left evicted."""
        done = 0
        while self.evicted and self.free and (max_tensors is None or done < max_tensors):
            tensor = self.evicted.popleft()
            u = self.free.popleft()
            self.tensor_of_unit[u] = tensor
            self.backed.append(u)
            self.stale.discard(tensor)
            if self.on_restore:
                self.on_restore(tensor, u)
            done += 1
        if not self.evicted and not self.stale:
            self.mode = MODE_FULL
        return done

    # ---- invariants (used by the tests) ----------------------------------------------------------
    def check(self) -> None:
        states = [set(self.free), set(self.backed), set(self.avail), set(self.full)]
        assert sum(len(s) for s in states) == self.units == len(set().union(*states)), "a unit is in exactly one state"
        assert len(self.free) == len(states[0]) and len(self.backed) == len(states[1]) and len(self.avail) == len(states[2])
        assert set(self.used) == states[2] | states[3]
        for u in states[2]:
            assert 0 <= len(self.used[u]) < self.blocks_per_unit
        for u in states[3]:
            assert len(self.used[u]) == self.blocks_per_unit
        assert set(self.tensor_of_unit) == states[1]
        bound = set(self.tensor_of_unit.values())
        assert bound.isdisjoint(self.evicted) and len(bound) + len(self.evicted) == self.residual_tensors
        assert self.stale == set(self.evicted)
        assert (self.mode == MODE_FULL) == (not self.evicted)

    @property
    def kv_blocks_in_use(self) -> int:
        return sum(len(t) for t in self.used.values())


def kv_demand_trace(steps: int, capacity_blocks: int, seed: int) -> np.ndarray:
    """Seeded synthetic KV-cache occupancy (blocks in use after each step): a base load around a third
    of the capacity plus bursts that arrive at random, rise quickly and drain slowly -- a stand-in
    for the bursty request traces the paper evaluates on (its time in fast mode is 47-79 %)."""
    rng = np.random.default_rng(seed)
    base = 0.33 * capacity_blocks
    level = 0.0
    out = np.empty(steps, np.int64)
    for t in range(steps):
        if rng.random() < 0.012:                                 # a burst of long requests arrives
            level += rng.uniform(0.25, 0.6) * capacity_blocks
        level *= 0.97                                            # requests finish, blocks drain
        noise = rng.normal(0.0, 0.02 * capacity_blocks)
        out[t] = int(min(capacity_blocks, max(0.0, base + level + noise)))
    return out


def mode_schedule_from_trace(demand: Sequence[int], units: int, blocks_per_unit: int, residual_tensors: int,
                             steps_per_restore: int = 2) -> Tuple[List[int], SumManager]:
    """Drive a SumManager with a KV occupancy trace; returns the mode of every step (taken at the
    step boundary, before the step's allocations, as the paper's dispatcher does) and the manager.
    The restore worker rebinds one evicted tensor every `steps_per_restore` steps while units are
    free (the copy of one unit's residual bytes takes a few decode steps)."""
    mgr = SumManager(units, blocks_per_unit, residual_tensors)
    held: List[Block] = []
    modes: List[int] = []
    for t, want in enumerate(demand):
        modes.append(mgr.mode)
        want = int(want)
        if want > len(held):
            got = mgr.alloc_kv_blocks(want - len(held))
            if got is not None:                                   # on failure the engine would preempt; the model just skips
                held.extend(got)
        elif want < len(held):
            drop = held[want:]
            del held[want:]
            mgr.free_kv_blocks(drop)
        if mgr.evicted and t % steps_per_restore == 0:
            # keep one unit of head-room so that a restore is not undone by the next allocation
            if len(mgr.free) > 1:
                mgr.restore_weights(1)
    return modes, mgr
