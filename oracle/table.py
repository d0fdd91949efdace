"""Oracle of the mapping table (Section 3.2) in block-granular, stream-ordered form.

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA library.

The paper's table maps a logical unit to its CPU pointer, its GPU pointer and a timestamp, and is
updated in two phases: (1) the destination is allocated and recorded and the copy starts in the
background; (2) only once the copy is confirmed complete is the unit marked present at the
destination (Section 3.2).  Units have no fixed home: the source region is given up after the move.

Here the unit is one (layer, 16-token logical block).  Its state is one of
    FREE, GPU, TO_HOST, HOST, TO_GPU
and copies are *stream ordered*: every swap call gets a ticket on its direction's queue ("in" or
"out"); tickets of one queue complete in order; a call may depend on a ticket of the other queue
(the copy that last touched one of its units, or the copy that must finish before a recycled slot
may be overwritten) or on a compute ticket (an attention call that may still read a recycled slot).
A source slot is released when its copy is *issued*, tagged with that copy's ticket: it may be
handed out again at once, but whoever receives it must wait for that ticket.  So a slot is never
overwritten before the copy reading it has finished, and a unit's bytes are never read at the
destination before the copy writing them has finished.

Slot hand-out order (shared rule, so that two implementations can be compared slot by slot; the paper
leaves open which free region a block receives, Section 3.2 only asks that the table name it):
``ready`` holds the slots that are free for certain; ``pending`` is a queue of released slots still
waiting for their ticket.  At the start of every call pending slots whose ticket is confirmed move to
``ready``.  A request for n >= 2 slots goes through the runs of consecutive ready slots in ascending
order and takes the first n of the first run that has n slots at or after the cursor; failing that -
and for a request for a single slot, which does not move the cursor - the first n of the lowest run
that has at least n; failing that, whole runs, longest first (lowest first among equals), until it is
served.  The cursor then stands behind the slots taken last.  What ``ready`` cannot give comes from the
front of ``pending``, and the tickets to wait for are reported.  (Swap lists release their slots in
about the order they took them, so the hand-out walks round the spare part of a pool like a ring and
lists land in consecutive slots whatever sizes the lists before them had; single slots - allocations -
fill the lowest holes.)
"""
from __future__ import annotations

import bisect

FREE, GPU, TO_HOST, HOST, TO_GPU = 0, 1, 2, 3, 4
STATE_NAMES = {FREE: "FREE", GPU: "GPU", TO_HOST: "TO_HOST", HOST: "HOST", TO_GPU: "TO_GPU"}

OK = 0
ERR_INVALID = -1
ERR_RANGE = -2
ERR_NOMEM = -3
ERR_BUSY = -4
ERR_NOT_RESIDENT = -5

Q_NONE, Q_IN, Q_OUT, Q_COMPUTE = 0, 1, 2, 3


class _SlotPool:
    def __init__(self, n):
        self.ready = list(range(n))   # kept in ascending order
        self.cursor = 0               # behind the slots the last request for two or more took from ready
        self.pending = []  # (slot, queue, ticket)

    def _add_ready(self, slot):
        bisect.insort(self.ready, slot)

    def settle(self, done):
        keep = []
        for slot, qu, tk in self.pending:
            if tk <= done[qu]:
                self._add_ready(slot)
            else:
                keep.append((slot, qu, tk))
        self.pending = keep

    def available(self):
        return len(self.ready) + len(self.pending)

    def _runs(self):
        """maximal runs of consecutive ready slots -> [(start, length)] in ascending order"""
        runs = []
        for s in self.ready:
            if runs and runs[-1][0] + runs[-1][1] == s:
                runs[-1][1] += 1
            else:
                runs.append([s, 1])
        return runs

    def take(self, n):
        """-> (slots, {queue: max ticket to wait for}, per-slot (queue, ticket) tags)"""
        slots, waits, tags = [], {}, []
        rove = n >= 2
        while len(slots) < n and self.ready:
            want = n - len(slots)
            runs = self._runs()
            first = None
            if rove:                                         # the first run with `want` slots at or after the cursor
                for start, length in runs:
                    a = max(start, self.cursor)
                    if start + length - a >= want:
                        first, count = a, want
                        break
            if first is None:
                fit = [r for r in runs if r[1] >= want]
                if fit:
                    first, count = fit[0][0], want           # the lowest run that serves the rest of the request
                else:                                        # else whole runs, longest first, lowest among equals
                    first, count = max(runs, key=lambda r: (r[1], -r[0]))
            got = list(range(first, first + count))
            for s in got:
                self.ready.remove(s)
            slots += got
            tags += [(Q_NONE, 0)] * len(got)
            if rove:
                self.cursor = first + count
        while len(slots) < n:
            slot, qu, tk = self.pending.pop(0)
            slots.append(slot)
            tags.append((qu, tk))
            waits[qu] = max(waits.get(qu, 0), tk)
        return slots, waits, tags

    def release(self, slot, queue, ticket):
        if queue == Q_NONE:
            self._add_ready(slot)
        else:
            self.pending.append((slot, queue, ticket))


class MappingTable:
    def __init__(self, n_layers, n_logical, n_gpu_slots, n_host_slots, capacity=None, retain=False):
        self.L, self.NB = n_layers, n_logical
        # Variant beyond the paper (which gives the CPU region up after a swap-in, Section 3.2): with `retain` a unit
        # that is brought in keeps its host slot, and pushing it out again copies nothing unless it was written
        # meanwhile (`mark_dirty`: the append of the new token goes into one block per sequence).
        self.retain = retain
        if capacity is not None and not 0 < capacity <= n_logical:
            raise ValueError("capacity")
        self.gpu = _SlotPool(n_gpu_slots)
        self.host = _SlotPool(n_host_slots)
        n = n_layers * n_logical
        self.side = [FREE] * n          # FREE / GPU / HOST : where the unit is or is heading
        self.gpu_slot = [-1] * n
        self.host_slot = [-1] * n
        self.last_q = [Q_NONE] * n      # queue and ticket of the last copy issued on the unit
        self.last_t = [0] * n
        self.allocated = [False] * n_logical
        self.dirty = [False] * n        # written on the GPU since the host copy was taken (meaningful with a kept host slot)
        self.last_elided = []           # per pair of the last swap(): True where no bytes need to move
        self.issued = {Q_IN: 0, Q_OUT: 0, Q_COMPUTE: 0}
        self.done = {Q_NONE: 0, Q_IN: 0, Q_OUT: 0, Q_COMPUTE: 0}
        self.clock = 0
        self.t_last = [0] * n           # the table's timestamp column
        self.last_compute = [0] * n_layers  # ticket of the newest attention call on each layer
        # run-time resize (Section 4.1): ids below `capacity` are visible to the block manager; `target` is the
        # size a resize in progress is heading to; `moved` holds the layers that have gone through a swap pass
        # since the resize was triggered
        self.capacity = n_logical if capacity is None else capacity
        self.target = None
        self.moved = set()

    # ---- helpers -------------------------------------------------------------------
    def _u(self, layer, block):
        return layer * self.NB + block

    def _settle(self):
        self.gpu.settle(self.done)
        self.host.settle(self.done)

    def _in_flight(self, u):
        return self.last_q[u] != Q_NONE and self.last_t[u] > self.done[self.last_q[u]]

    def state(self, layer, block):
        u = self._u(layer, block)
        if self.side[u] == FREE:
            return FREE
        if self._in_flight(u):
            return TO_GPU if self.side[u] == GPU else TO_HOST
        return self.side[u]

    def confirm(self, queue, ticket):
        """Phase 2: the copies (or attention calls) of `queue` up to `ticket` are known complete."""
        if ticket > self.issued[queue]:
            return ERR_RANGE
        self.done[queue] = max(self.done[queue], ticket)
        self._settle()
        return OK

    # ---- run-time resize of the per-layer cache (Section 4.1) ---------------------------
    def alloc_limit(self):
        """Ids below this may be handed out now.  Growing: the old size until every layer has moved (the new
        space is prepared first, made visible afterwards).  Shrinking: the new size from the trigger on (nothing
        is scheduled onto blocks that are about to go)."""
        return self.capacity if self.target is None else min(self.capacity, self.target)

    def resize_begin(self, new_size):
        """Trigger a change of the per-layer size, in blocks.  NB (the table's physical width) bounds it."""
        if not 0 < new_size <= self.NB:
            return ERR_RANGE
        if self.target is not None:
            return ERR_BUSY
        if new_size != self.capacity:
            self.target = new_size
            self.moved = set()
        return OK

    def layer_pass(self, layer):
        """The layer goes through a swap pass (its space is re-established at the new size).  Once every layer
        has done so the new size takes effect: grown ids become allocatable; shrunk ids leave the free list
        for good (blocks still in use beyond the new size stay accessible until they are freed).
        -> True when this call completed a resize."""
        if not 0 <= layer < self.L or self.target is None:
            return False
        self.moved.add(layer)
        if len(self.moved) < self.L:
            return False
        self.capacity, self.target, self.moved = self.target, None, set()
        return True

    # ---- logical block allocation ----------------------------------------------------
    def alloc(self, block, on_host=False):
        """One unit per layer: a GPU slot while any is available (never, if on_host), else a host slot.  A recycled slot
        whose ticket is still open makes the new unit "in flight" on that ticket, so that whatever
        touches the unit next waits for it."""
        if not 0 <= block < self.NB:
            return ERR_RANGE
        if block >= self.alloc_limit():
            return ERR_NOMEM    # beyond the size visible now
        if self.allocated[block]:
            return ERR_INVALID
        self._settle()
        n_gpu = 0 if on_host else min(self.L, self.gpu.available())
        if self.L - n_gpu > self.host.available():
            return ERR_NOMEM
        for layer in range(self.L):
            u = self._u(layer, block)
            pool, side = (self.gpu, GPU) if layer < n_gpu else (self.host, HOST)
            (slot,), _, (tag,) = pool.take(1)
            self.side[u] = side
            self.gpu_slot[u] = slot if side == GPU else -1
            self.host_slot[u] = slot if side == HOST else -1
            self.last_q[u], self.last_t[u] = tag
            self.dirty[u] = False
        self.allocated[block] = True
        return OK

    def free(self, block):
        """Units must be settled (no copy in flight).  GPU slots carry the last compute ticket:
        an attention call issued earlier may still be reading them."""
        if not 0 <= block < self.NB:
            return ERR_RANGE
        if not self.allocated[block]:
            return ERR_INVALID
        self._settle()
        for layer in range(self.L):
            if self._in_flight(self._u(layer, block)):
                return ERR_BUSY
        for layer in range(self.L):
            u = self._u(layer, block)
            if self.side[u] == GPU:
                ct = self.issued[Q_COMPUTE]
                self.gpu.release(self.gpu_slot[u], Q_COMPUTE if ct > self.done[Q_COMPUTE] else Q_NONE, ct)
                if self.host_slot[u] >= 0:          # a kept host copy goes with the unit
                    self.host.release(self.host_slot[u], Q_NONE, 0)
            else:
                self.host.release(self.host_slot[u], Q_NONE, 0)
            self.side[u], self.gpu_slot[u], self.host_slot[u] = FREE, -1, -1
            self.last_q[u], self.last_t[u] = Q_NONE, 0
        self.allocated[block] = False
        return OK

    # ---- swaps -----------------------------------------------------------------------
    def _check_ids(self, layer, ids):
        if not 0 <= layer < self.L:
            return ERR_RANGE
        seen = set()
        for b in ids:
            if not 0 <= b < self.NB:
                return ERR_RANGE
            if b in seen or not self.allocated[b]:
                return ERR_INVALID
            seen.add(b)
        return OK

    def swap(self, direction, layer, ids):
        """direction Q_OUT: make the units host resident; Q_IN: GPU resident.

        Returns (status, ticket, pairs, waits): pairs = [(block, src_slot, dst_slot)] of the units
        that actually move (units already on, or heading to, the requested side are skipped);
        waits = {queue: ticket} the copy must wait for besides its own queue's order.
        A failed call changes nothing.  ticket is 0 when nothing moves.
        """
        st = self._check_ids(layer, ids)
        if st != OK:
            return st, 0, [], {}
        self._settle()
        want = HOST if direction == Q_OUT else GPU
        movers = [b for b in ids if self.side[self._u(layer, b)] != want]
        dst_pool = self.host if direction == Q_OUT else self.gpu
        src_pool = self.gpu if direction == Q_OUT else self.host
        # a unit that kept its host slot goes back into it: only the others need a new one
        need = [b for b in movers if direction == Q_IN or self.host_slot[self._u(layer, b)] < 0]
        if len(need) > dst_pool.available():
            return ERR_NOMEM, 0, [], {}
        self.layer_pass(layer)
        self.last_elided = []
        if not movers:
            return OK, 0, [], {}
        slots, waits, _ = dst_pool.take(len(need))
        slots = iter(slots)
        self.issued[direction] += 1
        ticket = self.issued[direction]
        self.clock += 1
        pairs = []
        for b in movers:
            u = self._u(layer, b)
            if self._in_flight(u):  # the copy that is still bringing the unit to where it is now
                waits[self.last_q[u]] = max(waits.get(self.last_q[u], 0), self.last_t[u])
            if direction == Q_OUT:
                src = self.gpu_slot[u]
                if self.host_slot[u] >= 0:
                    dst, elide = self.host_slot[u], not self.dirty[u]   # the kept copy is still good unless written
                else:
                    dst, elide = next(slots), False
                self.host_slot[u], self.gpu_slot[u] = dst, -1
                self.dirty[u] = False
                src_pool.release(src, direction, ticket)
            else:
                src, dst, elide = self.host_slot[u], next(slots), False
                self.gpu_slot[u] = dst
                if not self.retain:
                    self.host_slot[u] = -1
                    src_pool.release(src, direction, ticket)
                # with `retain` the host slot stays the unit's; `dirty` keeps whatever it was: a mark made before the
                # unit came in (the step's append is declared up front) must survive until the next copy out
            self.side[u] = want
            self.last_q[u], self.last_t[u] = direction, ticket
            self.t_last[u] = self.clock
            pairs.append((b, src, dst))
            self.last_elided.append(elide)
        if direction == Q_OUT and self.last_compute[layer] > self.done[Q_COMPUTE]:
            # the layer's attention call also appends the new token: copy out only after it
            waits[Q_COMPUTE] = max(waits.get(Q_COMPUTE, 0), self.last_compute[layer])
        waits.pop(direction, None)  # same queue: ordered anyway
        return OK, ticket, pairs, waits

    def drop_host_copy(self, layer, block):
        """A unit that lives on the GPU gives its kept host slot up (it left the host-resident set).  The slot may
        still be read by the copy that is bringing the unit in: whoever gets it next waits for that copy."""
        if not 0 <= layer < self.L or not 0 <= block < self.NB:
            return ERR_RANGE
        if not self.allocated[block]:
            return ERR_INVALID
        self._settle()
        u = self._u(layer, block)
        if self.side[u] == GPU and self.host_slot[u] >= 0:
            tag = (self.last_q[u], self.last_t[u]) if self._in_flight(u) else (Q_NONE, 0)
            self.host.release(self.host_slot[u], *tag)
            self.host_slot[u] = -1
        return OK

    def kept_copies(self):
        """GPU-resident units that hold a kept host copy.  While there are any, a writer has to mark what it writes even
        after `retain` went off: switching off takes effect unit by unit at the next swap-in."""
        return sum(1 for u in range(self.L * self.NB)
                   if self.allocated[u % self.NB] and self.side[u] == GPU and self.host_slot[u] >= 0)

    def mark_dirty(self, layer, ids):
        """The layer's next attention call appends into these blocks: their host copies, where kept, go stale."""
        st = self._check_ids(layer, ids)
        if st != OK:
            return st
        for b in ids:
            self.dirty[self._u(layer, b)] = True
        return OK

    # ---- presence check (Section 3.2: computation may start only on units present on the GPU) ----
    def attention(self, layer, ids):
        """-> (status, compute ticket, waits).  Every unit must be on the GPU or arriving; the call
        then waits for the newest arriving copy among them."""
        st = self._check_ids(layer, ids)
        if st != OK:
            return st, 0, {}
        self._settle()
        waits = {}
        for b in ids:
            u = self._u(layer, b)
            if self.side[u] != GPU:
                return ERR_NOT_RESIDENT, 0, {}
            if self._in_flight(u):
                waits[self.last_q[u]] = max(waits.get(self.last_q[u], 0), self.last_t[u])
        self.issued[Q_COMPUTE] += 1
        self.last_compute[layer] = self.issued[Q_COMPUTE]
        return OK, self.issued[Q_COMPUTE], waits

    # ---- invariants ------------------------------------------------------------------
    def check_invariants(self):
        for pool, slots, n in ((self.gpu, self.gpu_slot, "gpu"), (self.host, self.host_slot, "host")):
            held = [s for s in slots if s >= 0]
            free = list(pool.ready) + [p[0] for p in pool.pending]
            assert len(set(held)) == len(held), f"{n}: a slot is mapped twice"
            assert not (set(held) & set(free)), f"{n}: a mapped slot is on the free list"
            assert len(set(free)) == len(free), f"{n}: a slot is free twice"
        for u, side in enumerate(self.side):
            if side == GPU:
                assert self.gpu_slot[u] >= 0   # a host slot may be kept beside it (retain)
            elif side == HOST:
                assert self.host_slot[u] >= 0 and self.gpu_slot[u] < 0
            else:
                assert self.gpu_slot[u] < 0 and self.host_slot[u] < 0
