"""Definition-level model of Section 3.2's residency rules, for checking any mapping-table implementation.

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA library and none with ``oracle/table.py``.

Section 3.2 states what must hold, whatever the mechanism: a unit (here one layer's K/V of one 16-token block) lives on
the GPU or on the CPU; to move it the destination is allocated and *recorded first*, the copy runs in the background,
the unit counts as *present at the destination only once the copy is confirmed complete*, and the source region is
*given up after the move*.  This module states those rules over a dictionary

    unit -> (where it is, how many times it has been written)

and over the contents of the two memories, slot by slot.  It knows nothing of tickets, queues or the order in which an
implementation hands slots out.  All it asks of an implementation under test is, for every operation it issues on the
device (a copy of a list of units, an attention call that reads units and may append to some), *which earlier
operations it made it wait for*.  The model then runs the operations in an arbitrary order consistent with those waits
(a device is free to) and checks:

  R1  destination recorded before the copy: when a copy runs, its destination slot belongs to no other unit's current
      or in-flight placement (no two live placements share a slot), and the table already names it for the unit;
  R2  present only after completion: whatever reads a unit (an attention call, the next copy of it) finds the unit's
      newest bytes in the slot the table gave for it - so nothing may be ordered before the copy that brings them;
  R3  source given up after the move: a slot is overwritten only by an operation ordered after every operation that
      still reads it - checked by R2 on the reader's side: a reader that finds foreign bytes fails;
  R4  a copy that the implementation elides (kept host copies, a variant beyond the paper) must leave the destination
      exactly as the copy would have: the slot already holds the unit's newest bytes;
  R5  a call that fails changes nothing observable.

Bytes are modelled as tags ``(layer, block, version)``; an append bumps the version where the unit lives.
"""
from __future__ import annotations

OK = 0
GPU_SIDE, HOST_SIDE = "gpu", "host"
# states as the C ABI and the table oracle number them
ST_FREE, ST_GPU, ST_TO_HOST, ST_HOST, ST_TO_GPU = 0, 1, 2, 3, 4
Q_IN, Q_OUT, Q_COMPUTE = 1, 2, 3


class RuleViolation(AssertionError):
    pass


class ResidencyModel:
    """The memories, the units' write counts and the operations issued but not yet run."""

    def __init__(self, n_layers, n_blocks, rng):
        self.L, self.NB, self.rng = n_layers, n_blocks, rng
        self.mem = {GPU_SIDE: {}, HOST_SIDE: {}}       # slot -> (layer, block, version)
        self.version = {}                               # (layer, block) -> writes so far (device order)
        self.queues = {Q_IN: [], Q_OUT: [], Q_COMPUTE: []}   # per stream: [(waits, body)], run in order
        self.ran = {Q_IN: 0, Q_OUT: 0, Q_COMPUTE: 0}
        self.elided = 0

    # ---- what the harness does itself (synchronously, like a test's set-up) ------------------------------------
    def fill_unit(self, layer, block, side, slot):
        self.version[(layer, block)] = 0
        self.mem[side][slot] = (layer, block, 0)

    def forget_block(self, block):
        """A freed block: operations issued earlier may still read its units (their bytes stay where they are until
        a later owner of the slot writes it, which R3 orders behind those readers)."""

    # ---- operations issued by the implementation under test ---------------------------------------------------
    def issue(self, stream, position, waits, body):
        """An operation on `stream` (its `position`-th, counting from 1) that may run once the operations named in
        `waits` ({stream: position}) and everything before it on its own stream have run."""
        if position != len(self.queues[stream]) + 1:
            raise RuleViolation(f"stream {stream}: operation {position} issued out of order")
        self.queues[stream].append((dict(waits), body))

    def copy(self, direction, layer, pairs, elided):
        """-> the body of a copy: pairs = [(block, src slot, dst slot)], direction 'out' (GPU -> host) or 'in'."""
        src, dst = (self.mem[GPU_SIDE], self.mem[HOST_SIDE]) if direction == "out" else (self.mem[HOST_SIDE], self.mem[GPU_SIDE])

        def body():
            for (b, s, d), skip in zip(pairs, elided):
                want = (layer, b, self.version[(layer, b)])
                if src.get(s) != want:
                    raise RuleViolation(f"R2/R3: copy {direction} of {(layer, b)} read slot {s}: found {src.get(s)}, newest is {want}")
                if skip:
                    if dst.get(d) != want:
                        raise RuleViolation(f"R4: elided copy of {(layer, b)}, but slot {d} holds {dst.get(d)}, not {want}")
                    self.elided += 1
                else:
                    dst[d] = want
        return body

    def attention(self, layer, blocks, slots, appended):
        def body():
            g = self.mem[GPU_SIDE]
            for b, s in zip(blocks, slots):
                want = (layer, b, self.version[(layer, b)])
                if g.get(s) != want:
                    raise RuleViolation(f"R2: attention on {(layer, b)} read slot {s}: found {g.get(s)}, newest is {want}")
                if b in appended:   # the new token's rows land in this block
                    self.version[(layer, b)] += 1
                    g[s] = (layer, b, self.version[(layer, b)])
        return body

    # ---- the device ----------------------------------------------------------------------------------------------
    def _runnable(self, stream):
        i = self.ran[stream]
        if i >= len(self.queues[stream]):
            return False
        return all(self.ran[q] >= t for q, t in self.queues[stream][i][0].items())

    def step(self):
        ready = [q for q in self.queues if self._runnable(q)]
        if not ready:
            return False
        q = self.rng.choice(ready)
        self.queues[q][self.ran[q]][1]()
        self.ran[q] += 1
        return True

    def drain(self):
        while self.step():
            pass
        for q in self.queues:
            if self.ran[q] != len(self.queues[q]):
                raise RuleViolation("operations wait for one another in a cycle")

    # ---- checks against what the table says -----------------------------------------------------------------------
    def check_placements(self, view):
        """No two live placements share a slot (R1), and - with the device drained - every unit's newest bytes are
        where the table says the unit is."""
        owners = {GPU_SIDE: {}, HOST_SIDE: {}}
        for l in range(self.L):
            for b in range(self.NB):
                state, gs, hs = view.state(l, b)
                if state == ST_FREE:
                    continue
                for side, slot in ((GPU_SIDE, gs), (HOST_SIDE, hs)):
                    if slot >= 0:
                        if slot in owners[side]:
                            raise RuleViolation(f"R1: {side} slot {slot} belongs to {owners[side][slot]} and to {(l, b)}")
                        owners[side][slot] = (l, b)

    def check_final(self, view):
        self.drain()
        self.check_placements(view)
        for l in range(self.L):
            for b in range(self.NB):
                state, gs, hs = view.state(l, b)
                if state == ST_FREE:
                    continue
                want = (l, b, self.version[(l, b)])
                side, slot = (GPU_SIDE, gs) if state in (ST_GPU, ST_TO_GPU) else (HOST_SIDE, hs)
                if self.mem[side].get(slot) != want:
                    raise RuleViolation(f"{(l, b)} is said to be in {side} slot {slot}, which holds {self.mem[side].get(slot)}, not {want}")


def snapshot(view, L, NB):
    return tuple(view.state(l, b) for l in range(L) for b in range(NB)) + (view.kept_copies(),)


def apply(view, model, op):
    """One call of a test sequence on the implementation under test (`view`: alloc / free / swap / attention /
    mark_dirty / drop_host_copy / confirm / state / kept_copies / set_retention, numbered like the C ABI), mirrored
    into the model.  The caller's duties are the documented ones: a writer marks what it writes while kept copies
    are on or any kept copy exists.  -> the call's status."""
    kind = op[0]
    before = snapshot(view, model.L, model.NB)
    st = OK
    if kind == "alloc":
        st = view.alloc(op[1], bool(op[2]) if len(op) > 2 else False)
        if st == OK:
            model.drain()    # the harness writes a fresh unit only once whatever still used its slot has run
            for l in range(model.L):
                state, gs, hs = view.state(l, op[1])
                side, slot = (GPU_SIDE, gs) if state in (ST_GPU, ST_TO_GPU) else (HOST_SIDE, hs)
                model.fill_unit(l, op[1], side, slot)
    elif kind == "free":
        st = view.free(op[1])
        if st == OK:
            model.forget_block(op[1])
    elif kind in ("out", "in"):
        q = Q_OUT if kind == "out" else Q_IN
        st, ticket, pairs, waits = view.swap(q, op[1], list(op[2]))
        if st == OK and ticket:
            elided = list(view.last_elided)
            if len(elided) != len(pairs):
                raise RuleViolation("elision flags do not match the list")
            if kind == "in" and any(elided):
                raise RuleViolation("a copy in was elided")
            # R1: the table names the destination before the copy has run
            for b, s, d in pairs:
                state, gs, hs = view.state(op[1], b)
                if (kind == "out" and hs != d) or (kind == "in" and gs != d):
                    raise RuleViolation(f"R1: destination slot {d} of {(op[1], b)} is not recorded")
                if state != (ST_TO_HOST if kind == "out" else ST_TO_GPU):
                    raise RuleViolation(f"{(op[1], b)} counts as present before its copy is confirmed (state {state})")
            model.issue(q, ticket, waits, model.copy(kind, op[1], pairs, elided))
    elif kind in ("attn", "attn_append"):
        ids = list(op[2])
        appended = [b for b in ids if b in op[3]] if kind == "attn_append" else []
        if appended and (view.retain_on or view.kept_copies() > 0):
            if view.mark_dirty(op[1], appended) != OK:
                appended = []    # the attention call below fails on the same ids
        st, ticket, waits = view.attention(op[1], ids)
        if st == OK:
            slots = [view.state(op[1], b)[1] for b in ids]
            model.issue(Q_COMPUTE, ticket, waits, model.attention(op[1], ids, slots, appended))
    elif kind == "drop":
        st = view.drop_host_copy(op[1], op[2])
    elif kind == "retain":
        view.set_retention(bool(op[1]))
    elif kind == "confirm":       # the host learns how far the device got (after letting it finish, if asked)
        if op[1]:
            model.drain()
        for q in model.ran:
            view.confirm(q, model.ran[q])
    elif kind == "run":           # the device makes some progress
        for _ in range(op[1]):
            model.step()
    else:
        raise ValueError(kind)
    if st != OK and kind not in ("attn_append",) and snapshot(view, model.L, model.NB) != before:
        raise RuleViolation(f"R5: failed call {op} changed the table")
    model.check_placements(view)
    return st
