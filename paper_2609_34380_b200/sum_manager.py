"""Host-side model of the shared-region manager that decides the precision mode.

Paper: Algorithm 1 (AllocKVBlock / FreeKVBlock), section "KV-Cache-Pressure-aware DPS".

The shared region is a pool of equally sized physical units.  This model keeps ONE record per unit --
what the unit currently serves (nothing, a residual weight tensor, or KV blocks), which of its KV
blocks are handed out, and when it last changed role -- and derives everything else from those
records:

  * a unit that serves nothing is *free*; one that carries a residual tensor is *backed*; a KV unit
    is *available* while it has a block left and *full* otherwise;
  * a residual tensor without a unit is *evicted*: its bytes exist in the host copy only.

A request for n blocks is planned before anything changes: the blocks still open in partly used KV
units are counted, the number of additional units follows from the shortfall, and those units come
from the free ones first (oldest first) and only then from the backed ones (most recently bound
first).  If the pool cannot cover the request, nothing changes.  Granting a request that consumes a
backed unit evicts that unit's residual tensor and puts the system into fast mode immediately (fast
mode never reads residual bytes, so no data has to move).  Returning the last block of a unit makes
it free again and, if a tensor is evicted, calls for the restore worker.  The restore worker binds
evicted tensors to free units; the mode goes back to full only when no tensor is evicted any more.

The model moves no memory.  `on_evict(tensor, unit)` and `on_restore(tensor, unit)` are the places
where a serving engine would drop / re-create the mapping and start the copy of the residual bytes
(`dps_restore_residual`); `ResidualPlanes` below does exactly that for a list of device planes.
Readings taken where the paper is silent: the order in which units are picked (above), and that an
evicted tensor may be restored into any free unit.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Set, Tuple

import numpy as np

MODE_FAST, MODE_FULL = 0, 1
Block = Tuple[int, int]          # (unit, block index inside the unit)

_IDLE, _RESIDUAL, _KV = 0, 1, 2  # what a unit serves


@dataclass
class _Unit:
    role: int = _IDLE
    tensor: Optional[int] = None                 # residual tensor bound to it (role _RESIDUAL)
    taken: Set[int] = field(default_factory=set)  # KV blocks handed out (role _KV)
    since: int = 0                               # value of the manager's clock when the role last changed


class SumManager:
    def __init__(self, units: int, blocks_per_unit: int, residual_tensors: int,
                 on_evict: Optional[Callable[[int, int], None]] = None,
                 on_restore: Optional[Callable[[int, int], None]] = None) -> None:
        if not 0 <= residual_tensors <= units or blocks_per_unit < 1:
            raise ValueError("need 0 <= residual_tensors <= units and blocks_per_unit >= 1")
        self.units, self.blocks_per_unit, self.residual_tensors = units, blocks_per_unit, residual_tensors
        self.on_evict, self.on_restore = on_evict, on_restore
        self.mode = MODE_FULL
        self.restore_wakeups = 0                  # how often freed units called for the restore worker
        self.evicted: List[int] = []              # residual tensors without a unit, oldest eviction first
        self._clock = 0
        self._unit = [_Unit() for _ in range(units)]
        for u in range(units):                    # tensor t starts on unit t; the rest of the pool is free
            if u < residual_tensors:
                self._set_role(u, _RESIDUAL, tensor=u)
            else:
                self._set_role(u, _IDLE)

    # ---- views derived from the unit records ---------------------------------------------------
    def _set_role(self, u: int, role: int, tensor: Optional[int] = None) -> None:
        self._clock += 1
        rec = self._unit[u]
        rec.role, rec.tensor, rec.since = role, tensor, self._clock
        rec.taken = set()

    def _by_age(self, pick) -> List[int]:
        return sorted((u for u in range(self.units) if pick(self._unit[u])), key=lambda u: self._unit[u].since)

    @property
    def free(self) -> List[int]:
        return self._by_age(lambda r: r.role == _IDLE)

    @property
    def backed(self) -> List[int]:
        return self._by_age(lambda r: r.role == _RESIDUAL)

    @property
    def avail(self) -> List[int]:
        return self._by_age(lambda r: r.role == _KV and len(r.taken) < self.blocks_per_unit)

    @property
    def full(self) -> Set[int]:
        return {u for u in range(self.units) if self._unit[u].role == _KV and len(self._unit[u].taken) == self.blocks_per_unit}

    @property
    def used(self) -> Dict[int, Set[int]]:
        return {u: set(r.taken) for u, r in enumerate(self._unit) if r.role == _KV}

    @property
    def stale(self) -> Set[int]:
        """Residual tensors whose mapping was invalidated and not yet re-created (= the evicted ones)."""
        return set(self.evicted)

    @property
    def tensor_of_unit(self) -> Dict[int, int]:
        return {u: r.tensor for u, r in enumerate(self._unit) if r.role == _RESIDUAL}

    @property
    def kv_blocks_in_use(self) -> int:
        return sum(len(r.taken) for r in self._unit if r.role == _KV)

    # ---- KV block allocation -------------------------------------------------------------------
    def alloc_kv_blocks(self, n: int) -> Optional[List[Block]]:
        """n KV blocks, or None (and no change) if the shared region cannot supply them."""
        if n < 0:
            raise ValueError("n must be non-negative")
        bpu = self.blocks_per_unit
        partly_used = list(reversed(self.avail))                      # most recently touched first
        open_blocks = sum(bpu - len(self._unit[u].taken) for u in partly_used)
        extra_units = -(-max(0, n - open_blocks) // bpu)
        idle, residual = self.free, list(reversed(self.backed))       # oldest free first; newest binding first
        if extra_units > len(idle) + len(residual):
            return None
        from_idle = idle[:extra_units]
        from_residual = residual[:extra_units - len(from_idle)]
        # the plan holds: carry it out
        evictions = [(self._unit[u].tensor, u) for u in from_residual]
        for u in from_idle + from_residual:
            self._set_role(u, _KV)
        blocks: List[Block] = []
        for u in partly_used + from_idle + from_residual:
            rec = self._unit[u]
            for b in range(bpu):
                if len(blocks) == n:
                    break
                if b not in rec.taken:
                    rec.taken.add(b)
                    blocks.append((u, b))
        for tensor, u in evictions:                                   # fast mode from here on: no data moves
            self.mode = MODE_FAST
            self.evicted.append(tensor)
            if self.on_evict:
                self.on_evict(tensor, u)
        return blocks

    # ---- KV block release ----------------------------------------------------------------------
    def free_kv_blocks(self, blocks: Sequence[Block]) -> None:
        emptied = 0
        for u, b in blocks:
            rec = self._unit[u] if 0 <= u < self.units else None
            if rec is None or rec.role != _KV or b not in rec.taken:
                raise ValueError(f"block {(u, b)} is not allocated")
            rec.taken.remove(b)
            if not rec.taken:
                self._set_role(u, _IDLE)
                emptied += 1
        if emptied and self.evicted:
            self.restore_wakeups += 1

    # ---- the restore worker --------------------------------------------------------------------
    def restore_weights(self, max_tensors: Optional[int] = None) -> int:
        """Bind up to max_tensors evicted residual tensors to free units (all that fit by default).
        Returns how many were restored; the mode returns to full when none is left evicted."""
        room = self.free
        count = min(len(self.evicted), len(room), len(room) if max_tensors is None else max_tensors)
        for u in room[:count]:
            tensor = self.evicted.pop(0)
            self._set_role(u, _RESIDUAL, tensor=tensor)
            if self.on_restore:
                self.on_restore(tensor, u)
        if not self.evicted:
            self.mode = MODE_FULL
        return count

    # ---- invariants (used by the tests) ----------------------------------------------------------
    def check(self) -> None:
        free, backed, avail, full = set(self.free), set(self.backed), set(self.avail), self.full
        assert len(free) + len(backed) + len(avail) + len(full) == self.units, "a unit is in exactly one state"
        assert set(self.used) == avail | full
        for u, rec in enumerate(self._unit):
            assert (rec.tensor is not None) == (rec.role == _RESIDUAL)
            assert not rec.taken or rec.role == _KV
            assert rec.role != _KV or rec.taken, "a KV unit without blocks must have been returned to the pool"
            assert all(0 <= b < self.blocks_per_unit for b in rec.taken)
        bound = set(self.tensor_of_unit.values())
        assert len(bound) == len(backed), "one tensor per backed unit"
        assert bound.isdisjoint(self.evicted) and len(set(self.evicted)) == len(self.evicted)
        assert len(bound) + len(self.evicted) == self.residual_tensors
        assert (self.mode == MODE_FULL) == (not self.evicted)


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


class TraceDriver:
    """Feeds a KV occupancy trace to a SumManager one step at a time.  `mode()` is what the dispatcher
    reads at a step boundary; `advance()` applies the step's allocations / releases and lets the
    restore worker bind one evicted tensor every `steps_per_restore` steps while more than one unit
    is free (one unit of head-room, so that a restore is not undone by the very next allocation).
    `ready`, if given, is asked before full mode is reported: a serving engine passes a function that
    says whether every restore copy it started has landed (the manager's own bookkeeping flips to
    full as soon as the last tensor is bound, the bytes arrive later)."""

    def __init__(self, manager: SumManager, demand: Sequence[int], steps_per_restore: int = 2,
                 ready: Optional[Callable[[], bool]] = None) -> None:
        self.manager, self.demand, self.steps_per_restore, self.ready = manager, demand, steps_per_restore, ready
        self.held: List[Block] = []
        self.step = 0

    def mode(self) -> int:
        if self.manager.mode == MODE_FULL and (self.ready is None or self.ready()):
            return MODE_FULL
        return MODE_FAST

    def advance(self) -> None:
        mgr, want = self.manager, int(self.demand[self.step])
        if want > len(self.held):
            got = mgr.alloc_kv_blocks(want - len(self.held))
            if got is not None:                                   # on failure an engine would preempt; the model skips
                self.held.extend(got)
        elif want < len(self.held):
            drop = self.held[want:]
            del self.held[want:]
            mgr.free_kv_blocks(drop)
        if mgr.evicted and self.step % self.steps_per_restore == 0 and len(mgr.free) > 1:
            mgr.restore_weights(1)
        self.step += 1


def mode_schedule_from_trace(demand: Sequence[int], units: int, blocks_per_unit: int, residual_tensors: int,
                             steps_per_restore: int = 2) -> Tuple[List[int], SumManager]:
    """The mode of every step of a trace (read at the step boundary, before the step's allocations, as
    the paper's dispatcher does), and the manager after the last step."""
    mgr = SumManager(units, blocks_per_unit, residual_tensors)
    driver = TraceDriver(mgr, demand, steps_per_restore)
    modes: List[int] = []
    for _ in range(len(demand)):
        modes.append(driver.mode())
        driver.advance()
    return modes, mgr


class ResidualPlanes:
    """Connects a SumManager to real residual planes: tensor t of the manager is the list of device
    planes `planes[t]` (for example the residual planes of the linears of decoder layer t).

    At construction every plane is copied to pinned host memory (the residual backup).  `on_evict`
    only notes that the tensor's bytes may now be overwritten (`poison=True` overwrites them, which is
    what the KV cache would do -- used by the tests).  `on_restore` enqueues the chunked host-to-device
    copies of that tensor on the copy stream and records an event; `landed()` is true when every
    restore started so far has completed, which is the condition for running a full-mode step.
    """

    def __init__(self, planes: Sequence[Sequence["object"]], copy_stream, poison: bool = False, chunk_bytes: int = 0) -> None:
        import torch

        from . import binding
        self._torch, self._binding = torch, binding
        self.planes, self.copy_stream, self.poison, self.chunk_bytes = planes, copy_stream, poison, chunk_bytes
        self.backups = [[binding.dps_backup_residual(r, stream=copy_stream) for r in group] for group in planes]
        copy_stream.synchronize()
        self.pending: List["object"] = []
        self.restored_bytes = 0
        self.evictions = 0

    def on_evict(self, tensor: int, unit: int) -> None:
        self.evictions += 1
        if self.poison:
            for r in self.planes[tensor]:
                r.fill_(0xFF)

    def on_restore(self, tensor: int, unit: int) -> None:
        torch = self._torch
        # the copy must not overtake work already enqueued on the compute stream that may still write the plane
        self.copy_stream.wait_stream(torch.cuda.current_stream())
        for r, host in zip(self.planes[tensor], self.backups[tensor]):
            self._binding.dps_restore_residual(r, host, chunk_bytes=self.chunk_bytes, stream=self.copy_stream)
            self.restored_bytes += r.numel()
        ev = torch.cuda.Event()
        ev.record(self.copy_stream)
        self.pending.append(ev)

    def landed(self) -> bool:
        self.pending = [ev for ev in self.pending if not ev.query()]
        return not self.pending
