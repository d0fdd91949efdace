"""Pins of the oracle's swap semantics, mapping-table state machine, swap protocol and controller."""
import itertools
import os
import random

import numpy as np
import pytest

import oracle
from oracle import policy, table
from paper_2411_09317_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------- swap = block memcpy
def test_swap_raw_definition_and_untouched_bytes():
    BB = 256
    G = synth.random_bytes(1, 8 * BB).copy()
    H = synth.random_bytes(2, 6 * BB).copy()
    G0, H0 = G.copy(), H.copy()
    assert oracle.swap_raw(H, G, BB, [7, 0, 3], [5, 1, 2]) == 0
    assert np.array_equal(G, G0)                                  # the source is left as it was
    for s, d in [(7, 5), (0, 1), (3, 2)]:
        assert np.array_equal(H[d * BB:(d + 1) * BB], G0[s * BB:(s + 1) * BB])
    for d in (0, 3, 4):
        assert np.array_equal(H[d * BB:(d + 1) * BB], H0[d * BB:(d + 1) * BB])
    # round trip into other slots returns the bytes
    assert oracle.swap_raw(G, H, BB, [5, 1, 2], [4, 6, 2]) == 0
    for s, d in [(7, 4), (0, 6), (3, 2)]:
        assert np.array_equal(G[d * BB:(d + 1) * BB], G0[s * BB:(s + 1) * BB])


def test_swap_raw_rejects_bad_lists_without_copying():
    BB = 64
    G = synth.random_bytes(3, 4 * BB).copy()
    H = synth.random_bytes(4, 4 * BB).copy()
    H0 = H.copy()
    assert oracle.swap_raw(H, G, BB, [0, 1], [2, 2]) == -1       # duplicate destination
    assert oracle.swap_raw(H, G, BB, [0, 4], [1, 2]) == -1       # source out of range
    assert oracle.swap_raw(H, G, BB, [0, 1], [-1, 2]) == -1
    assert np.array_equal(H, H0)
    assert oracle.swap_raw(H, G, BB, [], []) == 0


# --------------------------------------------------------- mapping table: device-order executor
class Executor:
    """Runs the copies a MappingTable issued in a random order that respects tickets and waits, with a
    content tag per slot, and checks that every read finds the unit it expects."""

    def __init__(self, tbl, rng):
        self.t, self.rng = tbl, rng
        self.g = {}   # gpu slot -> tag = (layer, block, version); an append bumps the version where the unit then lives
        self.h = {}
        self.version = {}   # (layer, block) -> number of appends the device has run on it
        self.ops = {table.Q_IN: [], table.Q_OUT: [], table.Q_COMPUTE: []}
        self.ran = {table.Q_IN: 0, table.Q_OUT: 0, table.Q_COMPUTE: 0}

    def write_unit(self, layer, block):  # host-side initial fill at alloc time (synchronous)
        u = self.t._u(layer, block)
        self.version[(layer, block)] = 0
        if self.t.side[u] == table.GPU:
            self.g[self.t.gpu_slot[u]] = (layer, block, 0)
        else:
            self.h[self.t.host_slot[u]] = (layer, block, 0)

    def issue(self, queue, ticket, waits, body):
        assert ticket == len(self.ops[queue]) + 1
        self.ops[queue].append((dict(waits), body))

    def runnable(self, queue):
        i = self.ran[queue]
        if i >= len(self.ops[queue]):
            return False
        return all(self.ran[q] >= t for q, t in self.ops[queue][i][0].items())

    def step(self):
        qs = [q for q in self.ops if self.runnable(q)]
        if not qs:
            return False
        q = self.rng.choice(qs)
        self.ops[q][self.ran[q]][1]()
        self.ran[q] += 1
        return True

    def drain(self):
        while self.step():
            pass
        assert all(self.ran[q] == len(self.ops[q]) for q in self.ops), "dependency cycle"


def apply_op(tbl, ex, op):
    kind = op[0]
    if kind == "alloc":
        st = tbl.alloc(op[1])
        if st == table.OK:
            # the harness writes a fresh unit only after the slot's open ticket: model by draining
            ex.drain()
            for l in range(tbl.L):
                ex.write_unit(l, op[1])
        return st
    if kind == "free":
        return tbl.free(op[1])
    if kind in ("out", "in"):
        q = table.Q_OUT if kind == "out" else table.Q_IN
        st, ticket, pairs, waits = tbl.swap(q, op[1], list(op[2]))
        if st == table.OK and ticket:
            layer, elided = op[1], list(tbl.last_elided)
            # (copies kept before the switch went off may still be used: what matters is that kept copies ever existed)
            ex.kept_ever = getattr(ex, "kept_ever", False) or tbl.retain
            assert len(elided) == len(pairs) and (ex.kept_ever or not any(elided))

            def body(pairs=pairs, layer=layer, q=q, elided=elided):
                src, dst = (ex.g, ex.h) if q == table.Q_OUT else (ex.h, ex.g)
                for (b, s, d), skip in zip(pairs, elided):
                    want = (layer, b, ex.version[(layer, b)])
                    assert src.get(s) == want, f"copy read slot {s}: {src.get(s)} != {want}"
                    if skip:    # no bytes move: the destination must already hold exactly what the copy would bring
                        assert dst.get(d) == want, f"elided copy, but slot {d} holds {dst.get(d)} != {want}"
                    else:
                        dst[d] = src[s]
            ex.issue(q, ticket, waits, body)
        return st
    if kind in ("attn", "attn_append"):
        ids = list(op[2])
        appended = [b for b in ids if b in op[3]] if kind == "attn_append" else []
        if appended and tbl.mark_dirty(op[1], appended) != table.OK:
            appended = []   # the attention call below fails on the same ids
        st, ticket, waits = tbl.attention(op[1], ids)
        if st == table.OK:
            layer = op[1]
            slots = [tbl.gpu_slot[tbl._u(layer, b)] for b in ids]

            def body():
                for b, s in zip(ids, slots):
                    want = (layer, b, ex.version[(layer, b)])
                    assert ex.g.get(s) == want, f"attention read slot {s}: {ex.g.get(s)} != {want}"
                    if b in appended:   # the new token's K/V rows land in this block
                        ex.version[(layer, b)] += 1
                        ex.g[s] = (layer, b, ex.version[(layer, b)])
            ex.issue(table.Q_COMPUTE, ticket, waits, body)
        return st
    if kind == "drop":
        return tbl.drop_host_copy(op[1], op[2])
    if kind == "confirm":  # the host learns how far the device got
        ex.drain() if op[1] else None
        for q in ex.ran:
            tbl.confirm(q, ex.ran[q])
        return table.OK
    if kind == "run":       # let the device make some progress
        for _ in range(op[1]):
            ex.step()
        return table.OK
    raise ValueError(kind)


def final_check(tbl, ex):
    ex.drain()
    for l in range(tbl.L):
        for b in range(tbl.NB):
            u = tbl._u(l, b)
            if tbl.side[u] == table.GPU:
                assert ex.g.get(tbl.gpu_slot[u]) == (l, b, ex.version[(l, b)])
            elif tbl.side[u] == table.HOST:
                assert ex.h.get(tbl.host_slot[u]) == (l, b, ex.version[(l, b)])   # the newest bytes, also after elided copies
    tbl.check_invariants()


def test_table_exhaustive_tiny():
    """Every call sequence of length <= 5 over a small alphabet on a 2-layer, 2-block table with 3 + 3
    slots: invariants hold, failed calls change nothing, and data survives in device order."""
    alphabet = [("alloc", 0), ("alloc", 1), ("free", 0), ("out", 0, (0,)), ("out", 1, (0, 1)), ("in", 0, (0,)),
                ("in", 1, (1, 0)), ("attn", 0, (0,)), ("attn", 1, (0, 1)), ("confirm", True), ("run", 1)]
    n_seq = 0
    for length in range(1, 6):
        for seq in itertools.product(alphabet, repeat=length):
            if seq[0][0] not in ("alloc",):
                continue  # everything else fails on an empty table; covered by the length-1 cases below
            tbl = table.MappingTable(2, 2, 3, 3)
            ex = Executor(tbl, random.Random(n_seq))
            for op in seq:
                snap = (list(tbl.side), list(tbl.gpu_slot), list(tbl.host_slot), list(tbl.gpu.ready), list(tbl.host.ready))
                st = apply_op(tbl, ex, op)
                if st != table.OK:
                    assert snap == (list(tbl.side), list(tbl.gpu_slot), list(tbl.host_slot), list(tbl.gpu.ready),
                                    list(tbl.host.ready)), f"failed call {op} changed the table"
                tbl.check_invariants()
            final_check(tbl, ex)
            n_seq += 1
    assert n_seq > 10000


def test_table_exhaustive_tiny_with_kept_host_copies():
    """The same enumeration with host copies kept after a swap-in and appends that write into blocks: an elided copy
    out never leaves stale bytes on the host, whatever the order the device runs things in."""
    alphabet = [("alloc", 0), ("alloc", 1), ("free", 0), ("out", 0, (0,)), ("out", 1, (0, 1)), ("in", 0, (0,)),
                ("in", 1, (1, 0)), ("attn", 0, (0,)), ("attn_append", 0, (0,), (0,)), ("attn_append", 1, (0, 1), (1,)),
                ("drop", 0, 0), ("confirm", True), ("run", 1)]
    n_seq = n_elided = 0
    # from a warm state: both blocks allocated and every unit once out and back in, so that host copies are kept
    warm = [("alloc", 0), ("alloc", 1), ("out", 0, (0, 1)), ("out", 1, (0, 1)), ("in", 0, (0, 1)), ("in", 1, (0, 1)), ("confirm", True)]
    for length in range(1, 5):
        for seq in itertools.product(alphabet, repeat=length):
            tbl = table.MappingTable(2, 2, 4, 4, retain=True)
            ex = Executor(tbl, random.Random(n_seq))
            for op in warm:
                assert apply_op(tbl, ex, op) == table.OK
            for op in seq:
                snap = (list(tbl.side), list(tbl.gpu_slot), list(tbl.host_slot), list(tbl.gpu.ready), list(tbl.host.ready))
                st = apply_op(tbl, ex, op)
                if st != table.OK and op[0] != "attn_append":   # (a failed attention call may have left its dirty marks)
                    assert snap == (list(tbl.side), list(tbl.gpu_slot), list(tbl.host_slot), list(tbl.gpu.ready),
                                    list(tbl.host.ready)), f"failed call {op} changed the table"
                if st == table.OK and op[0] == "out":
                    n_elided += sum(tbl.last_elided)
                tbl.check_invariants()
            final_check(tbl, ex)
            n_seq += 1
    assert n_seq > 10000 and n_elided > 500


def test_kept_host_copy_is_reused_and_written_blocks_are_copied():
    t = table.MappingTable(1, 3, 3, 3, retain=True)
    assert [t.alloc(b, on_host=True) for b in range(3)] == [table.OK] * 3
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [0, 1, 2])
    assert st == table.OK and t.last_elided == [False] * 3
    home = [p[1] for p in pairs]
    assert [t.host_slot[u] for u in range(3)] == home and t.host.available() == 0     # the host slots stay the units'
    t.confirm(table.Q_IN, tk)
    assert t.mark_dirty(0, [2]) == table.OK                                            # the step's append goes into block 2
    assert t.attention(0, [0, 1, 2])[0] == table.OK
    st, tk, pairs, waits = t.swap(table.Q_OUT, 0, [0, 1, 2])
    assert st == table.OK and t.last_elided == [True, True, False]                     # only the written block is copied
    assert [p[2] for p in pairs] == home                                               # ... and everyone returns to its slot
    assert waits == {table.Q_COMPUTE: 1}                                               # after the attention call, as ever
    assert t.gpu.available() == 3                                                      # the GPU slots are given up (pending)
    t.confirm(table.Q_COMPUTE, 1); t.confirm(table.Q_OUT, tk)
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [2])
    t.confirm(table.Q_IN, tk)
    st, tk, pairs, waits = t.swap(table.Q_OUT, 0, [2])                                 # not written since: nothing to copy
    assert t.last_elided == [True]
    # a mark made while the unit is still on the host (the step's appends are declared up front) survives the swap-in
    t.confirm(table.Q_OUT, tk)
    assert t.mark_dirty(0, [2]) == table.OK
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [2]); t.confirm(table.Q_IN, tk)
    st, tk, pairs, waits = t.swap(table.Q_OUT, 0, [2])
    assert t.last_elided == [False]
    # without the option every copy out moves bytes and takes a fresh host slot
    t2 = table.MappingTable(1, 1, 1, 2)
    t2.alloc(0, on_host=True)
    st, tk, pairs, _ = t2.swap(table.Q_IN, 0, [0]); t2.confirm(table.Q_IN, tk)
    assert t2.host_slot[0] == -1
    st, tk, pairs, _ = t2.swap(table.Q_OUT, 0, [0])
    assert t2.last_elided == [False] and pairs[0][2] == 0 and t2.host_slot[0] == 0     # a slot from the pool (the lowest free run)


def test_slot_hand_out_prefers_runs_of_consecutive_slots():
    """The shared hand-out rule by hand: the first run with n slots at or after the cursor; else the lowest run that serves
    the request; else whole runs, longest first; pending slots (with their tickets) only when nothing else is left."""
    p = table._SlotPool(10)
    assert p.take(3)[0] == [0, 1, 2]
    assert p.take(1)[0] == [3]
    p.release(1, table.Q_NONE, 0)                      # ready: {1} and {4..9}
    assert p.take(2)[0] == [4, 5]                      # the single slot cannot serve two: the next run does, and 1 stays
    assert p.take(1)[0] == [1]
    for s in (0, 2):                                   # ready: {0}, {2}, {6..9}
        p.release(s, table.Q_NONE, 0)
    p.release(3, table.Q_OUT, 7)                       # pending behind out-ticket 7
    slots, waits, tags = p.take(7)                     # no run of 7: the longest first, then the lowest, then pending
    assert slots == [6, 7, 8, 9, 0, 2, 3] and waits == {table.Q_OUT: 7} and tags[-1] == (table.Q_OUT, 7)
    assert p.available() == 0
    # a pool whose free set was scrambled one slot at a time still serves a list from one run if it has one
    q = table._SlotPool(64)
    q.take(64)
    for s in (5, 40, 41, 42, 43, 9, 44, 45, 13, 46, 47):
        q.release(s, table.Q_NONE, 0)
    assert q.take(6)[0] == [40, 41, 42, 43, 44, 45]


def test_slot_hand_out_walks_round_the_pool():
    """The cursor by hand: lists that grow and shrink while their slots come back in the order they went keep landing in
    consecutive slots, one list beside the other; a single slot fills the lowest hole and leaves the cursor alone."""
    p = table._SlotPool(24)
    assert p.take(4)[0] == [0, 1, 2, 3]                # a long-lived allocation; the cursor stands at 4
    a = p.take(3)[0]
    b = p.take(3)[0]
    assert (a, b) == ([4, 5, 6], [7, 8, 9])
    for s in a:
        p.release(s, table.Q_NONE, 0)                  # ready: {4..6}, {10..23}
    assert p.take(4)[0] == [10, 11, 12, 13]            # the freed run of three lies behind the cursor, and is too short anyway
    assert p.take(2)[0] == [14, 15]                    # ... and a list that WOULD fit there still goes on from the cursor
    assert p.take(1)[0] == [4]                         # one slot: the lowest hole
    assert p.take(3)[0] == [16, 17, 18]                # ... which did not move the cursor
    for s in b + [10, 11, 12, 13]:
        p.release(s, table.Q_NONE, 0)                  # ready: {5..13}, {19..23}
    assert p.take(5)[0] == [19, 20, 21, 22, 23]        # up to the end of the pool
    assert p.take(5)[0] == [5, 6, 7, 8, 9]             # nothing at or after the cursor: round again, from the lowest run that fits
    assert p.take(3)[0] == [10, 11, 12]                # on from the cursor, inside that run
    p.release(14, table.Q_NONE, 0); p.release(15, table.Q_NONE, 0)   # ready: {13..15}
    assert p.take(2)[0] == [13, 14]
    # the cursor inside a run: slots that came back just below it are passed over while the part above serves the request
    q = table._SlotPool(16)
    assert q.take(6)[0] == [0, 1, 2, 3, 4, 5]
    for s in (3, 4, 5):
        q.release(s, table.Q_NONE, 0)                  # ready: {3..15} as one run, cursor at 6
    assert q.take(4)[0] == [6, 7, 8, 9]
    assert q.take(7)[0] == [10, 11, 12, 13, 14, 15, 3]   # no run of seven: the longest whole, the rest from the lowest


def test_table_error_codes_and_two_phase_states():
    t = table.MappingTable(2, 3, 4, 4)
    assert t.swap(table.Q_OUT, 0, [0])[0] == table.ERR_INVALID      # not allocated
    assert t.alloc(0) == table.OK and t.alloc(0) == table.ERR_INVALID
    assert t.alloc(7) == table.ERR_RANGE
    assert t.swap(table.Q_OUT, 5, [0])[0] == table.ERR_RANGE
    assert t.swap(table.Q_OUT, 0, [0, 0])[0] == table.ERR_INVALID   # duplicate id
    assert t.state(0, 0) == table.GPU
    st, tk, pairs, waits = t.swap(table.Q_OUT, 0, [0])
    assert (st, tk) == (table.OK, 1) and pairs == [(0, 0, 0)]
    assert t.state(0, 0) == table.TO_HOST                            # phase 1: in transit
    assert t.attention(0, [0])[0] == table.ERR_NOT_RESIDENT          # presence check fails
    assert t.free(0) == table.ERR_BUSY
    assert t.swap(table.Q_OUT, 0, [0]) == (table.OK, 0, [], {})      # already heading there: no-op
    t.confirm(table.Q_OUT, 1)
    assert t.state(0, 0) == table.HOST                               # phase 2
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [0])
    assert st == table.OK and t.state(0, 0) == table.TO_GPU
    st, ctk, waits = t.attention(0, [0])                             # arriving: allowed, waits for it
    assert st == table.OK and waits == {table.Q_IN: 1}
    # an out-copy issued before the in-copy is confirmed must wait for it and for the attention call
    st, tk2, pairs, waits = t.swap(table.Q_OUT, 0, [0])
    assert st == table.OK and waits == {table.Q_IN: 1, table.Q_COMPUTE: 1}


def test_table_nomem_and_slot_recycling_waits():
    t = table.MappingTable(1, 4, 2, 2)
    assert [t.alloc(b) for b in range(4)] == [table.OK] * 4           # 2 on the GPU, 2 on the host
    assert [t.state(0, b) for b in range(4)] == [table.GPU, table.GPU, table.HOST, table.HOST]
    assert t.swap(table.Q_IN, 0, [2])[0] == table.ERR_NOMEM           # no GPU slot
    assert t.swap(table.Q_OUT, 0, [0])[0] == table.ERR_NOMEM          # no host slot
    t.free(3)
    st, tk, pairs, waits = t.swap(table.Q_OUT, 0, [0])                 # into the freed host slot
    assert st == table.OK and waits == {}
    # block 2 may now come in, into block 0's old GPU slot - but only after the out-copy has read it
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [2])
    assert st == table.OK and pairs[0][2] == 0 and waits == {table.Q_OUT: 1}


@pytest.mark.parametrize("retain", [False, True])
def test_table_random_long_runs(retain):
    rng = random.Random(5)
    for trial in range(60):
        L, NB = rng.choice([(1, 6), (3, 4), (2, 8)])
        tbl = table.MappingTable(L, NB, rng.randint(NB, L * NB), rng.randint(NB, L * NB) + (L * NB if retain else 0),
                                 retain=retain)
        ex = Executor(tbl, rng)
        for _ in range(120):
            k = rng.random()
            ids = tuple(rng.sample(range(NB), rng.randint(1, NB)))
            layer = rng.randrange(L)
            op = (("alloc", rng.randrange(NB)) if k < 0.15 else ("free", rng.randrange(NB)) if k < 0.2 else
                  ("out", layer, ids) if k < 0.45 else ("in", layer, ids) if k < 0.7 else
                  ("attn", layer, ids) if k < 0.76 else ("drop", layer, ids[0]) if k < 0.78 else
                  ("attn_append", layer, ids, set(rng.sample(ids, 1))) if k < 0.85 else
                  ("confirm", rng.random() < 0.3) if k < 0.93 else ("run", 2))
            if retain and rng.random() < 0.04:
                # the switch itself, while copies are kept: writers go on marking what they write (the executor always
                # does), so a unit that still holds a copy from before is written back when it next goes out
                tbl.retain = rng.random() < 0.5
            apply_op(tbl, ex, op)
            tbl.check_invariants()
        final_check(tbl, ex)


def test_switching_kept_copies_off_does_not_orphan_a_stale_copy():
    """A unit comes in with its copy kept, the switch goes off, the unit is written, goes out, comes back: the write-back
    must have happened (the copy from before the switch is stale), and the table still reports the copy as kept until then."""
    t = table.MappingTable(1, 2, 2, 4, retain=True)
    assert t.alloc(0, True) == table.OK
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [0])
    t.confirm(table.Q_IN, tk)
    assert t.kept_copies() == 1
    t.retain = False                                   # off: takes effect at the unit's next swap-in
    assert t.kept_copies() == 1
    assert t.mark_dirty(0, [0]) == table.OK            # the writer still marks: there is a kept copy
    st, tk, pairs, waits = t.swap(table.Q_OUT, 0, [0])
    assert list(t.last_elided) == [False]              # copied, not skipped
    t.confirm(table.Q_OUT, tk)
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [0])
    t.confirm(table.Q_IN, tk)
    assert t.kept_copies() == 0                        # now the host slot is gone
    t.check_invariants()


# ------------------------------------------------------------------------- protocol golden trace
# ---- run-time resize of the per-layer size (Section 4.1) --------------------------------------------------
def test_resize_grow_is_prepared_first_and_visible_only_after_every_layer_moved():
    L = 3
    t = table.MappingTable(L, 6, 12, 12, capacity=4)
    for b in range(3):
        assert t.alloc(b) == table.OK
    assert t.alloc(4) == table.ERR_NOMEM               # beyond the size: not there yet
    assert t.resize_begin(6) == table.OK
    assert t.alloc(3) == table.OK                      # blocks within the previous size stay usable meanwhile
    assert t.alloc(4) == table.ERR_NOMEM
    assert not t.layer_pass(0) and not t.layer_pass(1)
    assert not t.layer_pass(0)                         # the same layer again is not another layer
    assert t.alloc(4) == table.ERR_NOMEM and t.capacity == 4
    assert t.layer_pass(2)                             # the last layer: the new size takes effect
    assert t.capacity == 6 and t.target is None
    assert t.alloc(4) == table.OK and t.alloc(5) == table.OK
    t.check_invariants()


def test_resize_shrink_stops_handing_out_doomed_blocks_at_once_and_keeps_them_accessible():
    L = 2
    t = table.MappingTable(L, 6, 12, 12)
    for b in range(6):
        assert t.alloc(b) == table.OK
    assert t.free(4) == table.OK
    assert t.resize_begin(3) == table.OK
    assert t.alloc(4) == table.ERR_NOMEM               # from the trigger on, before any layer has passed
    assert t.capacity == 6                             # ... although the size itself has not changed yet
    # a block in use beyond the new size is still swapped and attended to
    st, tk, pairs, waits = t.swap(table.Q_OUT, 0, [5, 1])
    assert st == table.OK and [p[0] for p in pairs] == [5, 1]
    assert t.confirm(table.Q_OUT, tk) == table.OK
    assert t.state(0, 5) == table.HOST
    assert t.target == 3 and t.moved == {0}            # the swap call was layer 0's pass
    st, tk, pairs, waits = t.swap(table.Q_IN, 0, [5])
    assert st == table.OK and t.attention(0, [5, 1])[0] == table.ERR_NOT_RESIDENT
    assert t.swap(table.Q_IN, 0, [1])[0] == table.OK and t.attention(0, [5, 1])[0] == table.OK
    assert t.target == 3
    assert t.layer_pass(1) and t.capacity == 3 and t.target is None
    for q in (table.Q_IN, table.Q_OUT, table.Q_COMPUTE):
        t.confirm(q, t.issued[q])
    assert t.attention(1, [5])[0] == table.OK          # still accessible after the size took effect
    t.confirm(table.Q_COMPUTE, t.issued[table.Q_COMPUTE])
    assert t.free(5) == table.OK and t.alloc(5) == table.ERR_NOMEM and t.alloc(3) == table.ERR_NOMEM
    assert t.free(2) == table.OK and t.alloc(2) == table.OK
    t.check_invariants()


def test_resize_argument_checks_and_one_at_a_time():
    t = table.MappingTable(2, 5, 10, 10, capacity=3)
    assert t.resize_begin(0) == table.ERR_RANGE and t.resize_begin(6) == table.ERR_RANGE
    assert t.resize_begin(3) == table.OK and t.target is None      # same size: nothing to do
    assert t.resize_begin(5) == table.OK and t.resize_begin(4) == table.ERR_BUSY
    assert not t.layer_pass(7) and not t.layer_pass(-1)            # no such layer: no mark
    assert not t.layer_pass(1) and t.layer_pass(0)
    assert t.resize_begin(4) == table.OK
    with pytest.raises(ValueError):
        table.MappingTable(2, 5, 10, 10, capacity=6)


def test_resize_never_exposes_an_id_outside_both_sizes_under_random_traffic():
    """Whatever the interleaving: an id handed out is below the old size and, when shrinking, below the new one too; the
    size changes exactly when the last of the L layers has passed since the trigger."""
    rng = random.Random(5)
    for trial in range(200):
        L, NB = rng.randint(1, 4), rng.randint(2, 8)
        t = table.MappingTable(L, NB, L * NB, L * NB, capacity=rng.randint(1, NB))
        passed, old = set(), t.capacity
        for _ in range(60):
            k = rng.random()
            if k < 0.15:
                new = rng.randint(1, NB)
                busy = t.target is not None
                assert t.resize_begin(new) == (table.ERR_BUSY if busy else table.OK)
                if not busy and new != t.capacity:
                    passed, old = set(), t.capacity
            elif k < 0.45:
                layer = rng.randrange(L)
                in_progress, target = t.target is not None, t.target
                if rng.random() < 0.5:
                    done = t.layer_pass(layer)
                else:
                    ids = [b for b in range(NB) if t.allocated[b]][:2]
                    before = t.capacity
                    assert t.swap(rng.choice([table.Q_IN, table.Q_OUT]), layer, ids)[0] == table.OK
                    done = in_progress and t.target is None
                    for q in (table.Q_IN, table.Q_OUT):
                        t.confirm(q, t.issued[q])
                if in_progress:
                    passed.add(layer)
                    assert done == (len(passed) == L)
                    assert t.capacity == (target if done else old)
                else:
                    assert not done
            elif k < 0.8:
                b = rng.randrange(NB)
                limit = t.capacity if t.target is None else min(t.capacity, t.target)
                st = t.alloc(b, rng.random() < 0.5)
                assert (st == table.ERR_NOMEM) == (b >= limit)
                assert st in (table.OK, table.ERR_INVALID, table.ERR_NOMEM)
            else:
                b = rng.randrange(NB)
                t.free(b)
        t.check_invariants()


def read_golden():
    rows, totals = [], {}
    for line in open(os.path.join(GOLD, "fifo_9layer.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = line.split()
        if f[0] in ("P", "D"):
            rows.append((f[0], int(f[1]), int(f[2]), int(f[3]), int(f[4])))
        else:
            totals[f[0]] = int(f[1])
    return rows, totals


def test_protocol_reproduces_the_nine_layer_example():
    rows, totals = read_golden()
    res = policy.simulate_protocol(9, 2.0, 7, 4, {8, 9}, n_tokens=6)
    started = {}
    for t, kind, layer in res.events:
        started.setdefault(int(t), {})[kind] = layer
    for tag, t, layer_starting, out, inn in rows:
        assert (t % 9) + 1 == layer_starting
        assert started.get(t, {}).get("out", 0) == out, (tag, t)
        assert started.get(t, {}).get("in", 0) == inn, (tag, t)
    assert res.stall == totals["stall"]
    assert res.max_off_gpu == totals["fifo_length"]
    steady = [tr for tr in res.trips if tr[1] is not None and tr[1] >= 3]
    assert steady and all(fin - start == totals["trip_time"] for _, start, fin in steady)
    # Section 3.1: t_swap * m <= t_compute * n with t_swap = 2, n = 9 allows m <= 4.5 swaps per token
    late = [e for e in res.events if e[1] == "out" and 18 <= e[0] < 54]
    assert len(late) / 4 == pytest.approx(4.5)


def test_next_token_prefetches_become_rare_as_more_layers_live_on_the_cpu():
    """Section 3.4.2: fetching a layer that only the NEXT token needs is the rule violation the paper allows to prevent
    waiting, says is rare, and takes - once its share reaches a preset ratio - as the sign that the expansion is too
    small.  In the nine-layer example (swap = 2 compute): with one CPU layer nearly half of the swap-ins are such
    prefetches, with two (the paper's choice) under a quarter, and the link is exactly as busy in both - link slack could
    not tell them apart; with three the computation waits."""
    n, res = 9, {}
    for m in (1, 2, 3):
        res[m] = policy.simulate_protocol(n, 2.0, n - m, m + 2, set(range(n - m + 1, n + 1)), 12)
    share = {m: r.violations / r.in_starts for m, r in res.items()}
    assert res[1].stall == res[2].stall == 0 and res[3].stall > 0
    assert share[1] > 0.4 and 0.15 < share[2] < 0.3 and share[1] > share[2] > share[3]
    assert res[1].swaps_per_token == res[2].swaps_per_token == 4.5
    # by hand, token 2 of the paper's trace (two CPU layers): swap-ins of layers 1 (started while layer 8 computes: a
    # violation), 3, 5, 7, 9 -> one in four and a half
    ins = [(t, l) for t, kind, l in res[2].events if kind == "in" and 7 <= t < 16]
    assert ins == [(7.0, 1), (9.0, 3), (11.0, 5), (13.0, 7), (15.0, 9)]


@pytest.mark.parametrize("t_swap,want_m", [(2.0, 2), (1.5, 2), (1.0, 5), (3.0, 0)])
def test_layer_controller_finds_the_papers_two_cpu_layers(t_swap, want_m):
    """The whole-layer adaptive rule on the protocol simulator, window after window from everything on the GPU: it climbs
    while the share of next-token prefetches is at or above its trigger, steps back when the computation waits, and comes
    to rest at two CPU layers for the paper's nine-layer example (expansion 9 / 7 = 1.28, Section 3.3)."""
    n = 9
    c = policy.LayerController(m_max=n - 2)
    traj = []
    for _ in range(40):
        m = c.m
        r = policy.simulate_protocol(n, t_swap, n - m, m + 2, set(range(n - m + 1, n + 1)), 6)
        c.update(r.stall, 6.0 * n, r.in_starts, r.violations)
        traj.append(m)
    assert traj[0] == 0 and traj[-1] == want_m and traj[-20:].count(want_m) >= 18, traj
    assert max(traj) <= want_m + 1        # at most one probe beyond


def test_protocol_sensitivity():
    # one GPU region fewer, or slower swaps: the computation has to wait (Section 3.4.1)
    assert policy.simulate_protocol(9, 2.0, 6, 4, {7, 8, 9}, 6).stall > 0
    assert policy.simulate_protocol(9, 3.0, 7, 4, {8, 9}, 6).stall > 0
    # a smaller expansion under "swap whenever the link is free" moves as much data for shorter stays
    small = policy.simulate_protocol(9, 2.0, 8, 3, {9}, 8)
    best = policy.simulate_protocol(9, 2.0, 7, 4, {8, 9}, 8)
    assert small.stall == 0
    trip = lambda r: max(fin - st for _, st, fin in r.trips if st is not None and st > 9)
    assert trip(small) < trip(best)
    assert small.swaps_per_token == pytest.approx(best.swaps_per_token, abs=0.6)
    # everything on the GPU: nothing ever moves
    none = policy.simulate_protocol(9, 2.0, 9, 2, set(), 3)
    assert none.events == [] and none.stall == 0


# ------------------------------------------------------------------------------------ controller
@pytest.mark.parametrize("bw,tc,bytes_layer,L", [(50e9, 200e-6, 400e6, 32), (400e9, 300e-6, 400e6, 32),
                                                  (50e9, 2e-3, 100e6, 10), (1e12, 1e-3, 100e6, 8)])
def test_controller_settles_at_the_transparent_ratio(bw, tc, bytes_layer, L):
    r_star = min(1.0, bw * tc / bytes_layer)      # t_swap * m = t_compute * n, per layer (Section 3.1)
    c = policy.Controller(step=1.0 / L)
    trace = []
    for _ in range(200):
        trace.append(c.tick(*policy.fake_clock_step(c.r, bytes_layer, bw, tc, L)))
    tail = trace[-40:]
    tol = c.step + 0.1 * r_star + 1e-9
    assert all(abs(r - r_star) <= tol for r in tail), (r_star, tail[-5:])
    # bandwidth halves (prolonged interference, Section 3.4.2): it follows
    for _ in range(200):
        trace.append(c.tick(*policy.fake_clock_step(c.r, bytes_layer, bw / 2, tc, L)))
    r2 = min(1.0, bw / 2 * tc / bytes_layer)
    assert all(abs(r - r2) <= c.step + 0.1 * r2 + 1e-9 for r in trace[-40:])


def test_controller_probes_a_ratio_that_keeps_stalling_less_and_less_often():
    """Performance record (Section 3.4.2): at the transparent ratio the next step up always stalls.  Without a record
    the rule would try it again every few steps; with it the probes thin out (the wait doubles after every failed one),
    so that in steady state the computation rarely waits - and when conditions improve the record is dropped."""
    bw, tc, bytes_layer, L = 50e9, 200e-6, 400e6, 32
    c = policy.Controller(step=1.0 / L)
    stalled = []
    for _ in range(600):
        m = policy.fake_clock_step(c.r, bytes_layer, bw, tc, L)
        stalled.append(m[0] > c.eps * m[1])
        c.tick(*m)
    # stalled steps come in pairs (two of four trigger the back-off); their spacing grows up to the cap
    first, last = sum(stalled[:100]), sum(stalled[-200:])
    assert first >= 6 and last <= 6, (first, last)
    assert c.hold == c.hold_max and c.r_bad > 0
    # twice the bandwidth: the old bad ratio is fine now; the record must not hold the ratio down for long
    r_star2 = min(1.0, 2 * bw * tc / bytes_layer)
    for _ in range(c.hold_max + 8 * int(r_star2 * L + 2)):
        c.tick(*policy.fake_clock_step(c.r, bytes_layer, 2 * bw, tc, L))
    assert abs(c.r - r_star2) <= c.step + 0.1 * r_star2


def test_controller_tolerates_one_disturbed_step():
    c = policy.Controller(step=0.1)
    for _ in range(3):
        c.tick(0.0, 1.0, 0.5)
    r = c.r
    assert c.tick(0.5, 1.0, 0.5) == r           # a single stall: no change
    assert c.tick(0.0, 1.0, 0.95) == r          # quiet again, link nearly full: hold
    assert c.tick(0.5, 1.0, 0.5) == pytest.approx(r - 0.1)  # second stall within the window: back off


# ------------------------------------------------------------------- throughput records (Section 3.4.2, last paragraph)
def _drive_governor(T, n, step=0.01, stuck_at=None, g=None, k=0):
    """Reports of a synthetic throughput curve T(ratio, i) to a governor; between reports the ratio moves one step
    toward the cap, as a stall-free controller would (or stays at `stuck_at` steps where stalls hold it)."""
    from oracle.policy import Governor
    g = g or Governor(step)
    trace = []
    for i in range(n):
        g.report(k * step, T(k * step, i))
        target = g.cap if stuck_at is None else min(g.cap, stuck_at)
        if k < min(target, 100):
            k += 1
        elif k > target:
            k = target
        trace.append((k, g.state, g.cap))
    return g, k, trace


def test_governor_stops_where_the_workload_stops_scaling():
    from oracle.policy import HOLD
    # throughput grows with the ratio up to 0.05, flat beyond: the paragraph's "stops scaling"
    g, k, trace = _drive_governor(lambda r, i: 100 + 1000 * min(r, 0.05), 12)
    # climbed to 6 steps, saw no gain over 5, tested 5 (no adverse effect), tested 4 (worse), back to 5
    assert [t[0] for t in trace[:9]] == [1, 2, 3, 4, 5, 6, 5, 4, 5]
    assert (k, g.state, g.cap) == (5, HOLD, 5)


def test_governor_walks_down_when_expansion_buys_nothing_and_probes_periodically():
    from oracle.policy import HOLD, PROBE_UP
    g, k, trace = _drive_governor(lambda r, i: 100.0, 40)
    assert (k, g.cap) == (0, 0) and g.state in (HOLD, PROBE_UP)
    probes = [i for i, t in enumerate(trace) if t[1] == PROBE_UP]
    assert len(probes) >= 3 and all(b - a == g.period + 1 for a, b in zip(probes, probes[1:]))   # one probe per period
    assert max(t[0] for t in trace[3:]) == 1                                                     # never more than one step up


def test_governor_follows_demand_that_comes_back():
    from oracle.policy import HOLD
    g, k, trace = _drive_governor(lambda r, i: 100.0 if i < 30 else 100 + 1000 * min(r, 0.08), 90)
    assert all(t[0] <= 1 for t in trace[3:30])
    assert (k, g.cap) == (8, 8) or (k, g.cap) == (9, 9)        # at the new saturation point (or on a probe one above it)
    assert max(t[0] for t in trace) == 9


def test_governor_ignores_noise_within_its_tolerance():
    import numpy as np
    rng = np.random.default_rng(3)
    noise = rng.uniform(-0.004, 0.004, 400)
    # 10 % more throughput per step up to 0.05: far above the tolerance; +-0.4 % noise: far below
    g, k, trace = _drive_governor(lambda r, i: (100 + 1000 * min(r, 0.05)) * (1 + noise[i]), 400)
    assert all(4 <= t[0] <= 6 for t in trace[10:])


def test_governor_ends_a_test_the_controller_cannot_follow():
    from oracle.policy import Governor, HOLD, PROBE_UP, NORMAL
    # a ratio that stalls hold at 2 steps while throughput still grows with it: nothing to compare above 2, no cap
    g, k, _ = _drive_governor(lambda r, i: 100.0 + 1000 * r, 60, stuck_at=2)
    assert k == 2 and g.state == NORMAL and g.cap_ratio() == 1.0
    # flat throughput: down to 0 and HOLD; then the probe one step up cannot be followed (the ratio stays at 0):
    # after `patience` reports away from the cap the test ends where the ratio is
    g = Governor(0.01)
    g, k, _ = _drive_governor(lambda r, i: 100.0, 4, g=g)
    assert (k, g.state, g.cap) == (0, HOLD, 0)
    seen = []
    for i in range(g.period + g.patience):
        g.report(0.0, 100.0)
        seen.append((g.state, g.cap))
    first = seen.index((PROBE_UP, 1))
    assert first in (g.period - 2, g.period - 1)                      # one probe per period of reports in HOLD
    assert seen[first + g.patience - 1] == (PROBE_UP, 1) and seen[first + g.patience] == (HOLD, 0)
