"""The mapping table of Section 3.2, in both its implementations (the oracle's `oracle/table.py` and the library's
`pie_table_*` through the C ABI), driven against the definition-level residency model of `oracle/residency.py`: the
model knows the section's rules and nothing of tickets or slot hand-out, so this is not one port checked against its
twin.  The last tests re-introduce known mistakes into each implementation separately (by patching its source text)
and require that the model catches them."""
import ctypes
import itertools
import os
import random
import subprocess
import types

import numpy as np
import pytest

from oracle import residency as rm
from oracle import table as otable

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
LIB_PATH = os.path.join(ROOT, "paper_2411_09317_b200", "libpie.so")
TABLE_CPP = os.path.join(ROOT, "paper_2411_09317_b200", "csrc", "pie_table.cpp")
TABLE_PY = os.path.join(ROOT, "oracle", "table.py")


# ---------------------------------------------------------------------------------------- views
class OracleView:
    """oracle/table.py behind the interface the model's driver uses"""

    def __init__(self, L, NB, n_gpu, n_host, retain=False, module=otable):
        self.t = module.MappingTable(L, NB, n_gpu, n_host, retain=retain)
        self.L, self.NB = L, NB

    retain_on = property(lambda self: self.t.retain)
    last_elided = property(lambda self: self.t.last_elided)

    def state(self, l, b):
        u = l * self.NB + b
        return self.t.state(l, b), self.t.gpu_slot[u], self.t.host_slot[u]

    def alloc(self, b, on_host=False): return self.t.alloc(b, on_host)
    def free(self, b): return self.t.free(b)
    def swap(self, q, l, ids): return self.t.swap(q, l, ids)
    def attention(self, l, ids):
        st, tk, waits = self.t.attention(l, ids)
        return st, tk, {q: t for q, t in waits.items() if q != otable.Q_COMPUTE}
    def mark_dirty(self, l, ids): return self.t.mark_dirty(l, ids)
    def drop_host_copy(self, l, b): return self.t.drop_host_copy(l, b)
    def confirm(self, q, tk): return self.t.confirm(q, tk)
    def kept_copies(self): return self.t.kept_copies()
    def set_retention(self, on): self.t.retain = bool(on)


class LibView:
    """pie_table_* of a shared library, called through ctypes with marshalling of this file's own"""

    def __init__(self, L, NB, n_gpu, n_host, retain=False, cdll=None):
        self.lib = cdll or ctypes.CDLL(LIB_PATH)
        self.lib.pie_table_create.restype = ctypes.c_void_p
        self.lib.pie_table_create.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64]
        self.lib.pie_table_kept_copies.restype = ctypes.c_int64
        self.h = ctypes.c_void_p(self.lib.pie_table_create(L, NB, n_gpu, n_host))
        assert self.h
        self.L, self.NB, self.retain_on, self.last_elided = L, NB, False, []
        self.set_retention(retain)

    def __del__(self):
        if getattr(self, "h", None):
            self.lib.pie_table_destroy.argtypes = [ctypes.c_void_p]
            self.lib.pie_table_destroy(self.h)
            self.h = None

    @staticmethod
    def _ids(ids):
        a = np.ascontiguousarray(ids, dtype=np.int32)
        return a, a.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(len(a))

    def state(self, l, b):
        s, g, h = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
        assert self.lib.pie_table_state(self.h, ctypes.c_int32(l), ctypes.c_int32(b), ctypes.byref(s), ctypes.byref(g), ctypes.byref(h)) == 0
        return s.value, g.value, h.value

    def alloc(self, b, on_host=False): return self.lib.pie_table_alloc(self.h, ctypes.c_int32(b), ctypes.c_int32(int(on_host)))
    def free(self, b): return self.lib.pie_table_free(self.h, ctypes.c_int32(b))

    def swap(self, q, l, ids):
        a, p, n = self._ids(ids)
        cap = max(len(a), 1)
        moved, src, dst = (np.zeros(cap, np.int32) for _ in range(3))
        elided, waits = np.zeros(cap, np.uint8), np.zeros(4, np.int64)
        tk, nm = ctypes.c_int64(), ctypes.c_int64()
        ptr = lambda x: x.ctypes.data_as(ctypes.c_void_p)
        st = self.lib.pie_table_swap_ex(self.h, ctypes.c_int32(q), ctypes.c_int32(l), p, n, ctypes.byref(tk), ptr(moved), ptr(src),
                                        ptr(dst), ptr(elided), ctypes.byref(nm), ptr(waits))
        k = nm.value if st == 0 else 0
        self.last_elided = [bool(elided[i]) for i in range(k)]
        return st, (tk.value if st == 0 else 0), [(int(moved[i]), int(src[i]), int(dst[i])) for i in range(k)], \
            {q2: int(waits[q2]) for q2 in range(1, 4) if waits[q2]}

    def attention(self, l, ids):
        a, p, n = self._ids(ids)
        waits, tk = np.zeros(4, np.int64), ctypes.c_int64()
        st = self.lib.pie_table_attention(self.h, ctypes.c_int32(l), p, n, ctypes.byref(tk), waits.ctypes.data_as(ctypes.c_void_p))
        return st, (tk.value if st == 0 else 0), {q: int(waits[q]) for q in (1, 2) if waits[q]}

    def mark_dirty(self, l, ids):
        a, p, n = self._ids(ids)
        return self.lib.pie_table_mark_dirty(self.h, ctypes.c_int32(l), p, n)

    def drop_host_copy(self, l, b): return self.lib.pie_table_drop_host_copy(self.h, ctypes.c_int32(l), ctypes.c_int32(b))
    def confirm(self, q, tk): return self.lib.pie_table_confirm(self.h, ctypes.c_int32(q), ctypes.c_int64(tk))
    def kept_copies(self): return int(self.lib.pie_table_kept_copies(self.h))

    def set_retention(self, on):
        self.retain_on = bool(on)
        return self.lib.pie_table_set_retention(self.h, ctypes.c_int32(int(on)))


VIEWS = {"oracle": OracleView, "library": LibView}


# --------------------------------------------------------------------------------------- drivers
PLAIN = [("alloc", 0), ("alloc", 1), ("free", 0), ("out", 0, (0,)), ("out", 1, (0, 1)), ("in", 0, (0,)), ("in", 1, (1, 0)),
         ("attn", 0, (0,)), ("attn", 1, (0, 1)), ("confirm", True), ("run", 1)]
KEPT = [("alloc", 0), ("alloc", 1), ("free", 0), ("out", 0, (0,)), ("out", 1, (0, 1)), ("in", 0, (0,)), ("in", 1, (1, 0)),
        ("attn", 0, (0,)), ("attn_append", 0, (0,), (0,)), ("attn_append", 1, (0, 1), (1,)), ("drop", 0, 0), ("retain", False),
        ("retain", True), ("confirm", True), ("run", 1)]
WARM = [("alloc", 0), ("alloc", 1), ("out", 0, (0, 1)), ("out", 1, (0, 1)), ("in", 0, (0, 1)), ("in", 1, (0, 1)), ("confirm", True)]


def run_sequence(make_view, seq, seed, warm=(), retain=False, slots=(3, 3)):
    view = make_view(2, 2, slots[0], slots[1], retain=retain)
    model = rm.ResidencyModel(2, 2, random.Random(seed))
    for op in warm:
        assert rm.apply(view, model, op) == rm.OK
    for op in seq:
        rm.apply(view, model, op)
    model.check_final(view)
    return model


def exhaustive(make_view, alphabet, max_len, **kw):
    n = elided = 0
    for length in range(1, max_len + 1):
        for seq in itertools.product(alphabet, repeat=length):
            if not kw.get("warm") and seq[0][0] != "alloc":
                continue   # everything else fails on an empty table
            elided += run_sequence(make_view, seq, n, **kw).elided
            n += 1
    return n, elided


def random_runs(make_view, trials, n_ops, retain, seed=5):
    rng = random.Random(seed)
    total_elided = 0
    for _ in range(trials):
        L, NB = rng.choice([(1, 6), (3, 4), (2, 8)])
        view = make_view(L, NB, rng.randint(NB, L * NB), rng.randint(NB, L * NB) + (L * NB if retain else 0), retain=retain)
        model = rm.ResidencyModel(L, NB, rng)
        for _ in range(n_ops):
            k = rng.random()
            ids = tuple(rng.sample(range(NB), rng.randint(1, NB)))
            layer = rng.randrange(L)
            if retain and rng.random() < 0.06:
                rm.apply(view, model, ("retain", rng.random() < 0.5))     # the switch itself, while copies are kept
            if retain and rng.random() < 0.05:
                rm.apply(view, model, ("drop", layer, rng.randrange(NB)))
            if k < 0.15: op = ("alloc", rng.randrange(NB), rng.random() < 0.3)
            elif k < 0.20: op = ("free", rng.randrange(NB))
            elif k < 0.42: op = ("out", layer, ids)
            elif k < 0.64: op = ("in", layer, ids)
            elif k < 0.74: op = ("attn", layer, ids)
            elif k < 0.84: op = ("attn_append", layer, ids, tuple(rng.sample(ids, rng.randint(1, len(ids)))))
            elif k < 0.92: op = ("confirm", rng.random() < 0.5)
            else: op = ("run", rng.randint(1, 4))
            rm.apply(view, model, op)
        model.check_final(view)
        total_elided += model.elided
    return total_elided


# ----------------------------------------------------------------------------------------- tests
@pytest.mark.parametrize("impl", ["oracle", "library"])
def test_every_short_call_sequence_keeps_the_rules(impl):
    n, _ = exhaustive(VIEWS[impl], PLAIN, 4)
    assert n > 2500


@pytest.mark.parametrize("impl", ["oracle", "library"])
def test_every_short_call_sequence_keeps_the_rules_with_kept_host_copies(impl):
    """From a warm state (every unit once out and back in, so that host copies are kept), with appends and with the switch
    going off and on inside the sequence: an elided copy never leaves stale bytes on the host."""
    n, elided = exhaustive(VIEWS[impl], KEPT, 3, warm=WARM, retain=True, slots=(4, 4))
    assert n > 3500 and elided > 300


def _decode_loop_with_changing_shares(view, L, shares, lag):
    """The decode loop's calls on the bare table: per step and layer, bring in the layer's units that are on the host or
    on their way there, attend, and push the first m units (ascending ids) out again; copies are confirmed `lag` tickets
    late, in order.  -> per list (step, direction, (id, source slot, destination slot) triples)."""
    lists, open_tickets = [], []
    for step, m in enumerate(shares):
        for l in range(L):
            away = [b for b in range(view.NB) if view.state(l, b)[0] in (otable.HOST, otable.TO_HOST)]
            if away:
                st, tk, pairs, _ = view.swap(otable.Q_IN, l, away)
                assert st == 0
                lists.append((step, "in", pairs))
                open_tickets.append((otable.Q_IN, tk))
            st, ctk, _ = view.attention(l, list(range(view.NB)))
            assert st == 0
            open_tickets.append((otable.Q_COMPUTE, ctk))
            if m:
                st, tk, pairs, _ = view.swap(otable.Q_OUT, l, list(range(m)))
                assert st == 0
                lists.append((step, "out", pairs))
                open_tickets.append((otable.Q_OUT, tk))
            while len(open_tickets) > lag:
                q, tk = open_tickets.pop(0)
                assert view.confirm(q, tk) == 0
    return lists


def _runs(pairs):
    return 1 + sum(1 for a, b in zip(pairs, pairs[1:]) if b[1] != a[1] + 1 or b[2] != a[2] + 1)


@pytest.mark.parametrize("impl", ["oracle", "library"])
def test_lists_stay_whole_while_the_host_resident_share_grows_and_shrinks(impl):
    """The hand-out rule's purpose, on both implementations: with the spare part of the pools a few lists larger than what
    is in flight, a layer's swap list lands in ONE run of consecutive slots on both sides however the share changed before -
    except in the step of a change itself, where the units that join come from the scattered slots they lived in.  (Sizes
    chosen so that "the lowest run that fits", without the cursor, leaves two of these lists in two runs.)"""
    L, NB = 4, 40
    shares = [3, 3, 4, 4, 6, 6, 9, 9, 7, 7, 4, 4, 5, 5, 8, 8, 8, 8]
    view = VIEWS[impl](L, NB, L * NB + 30, 80)
    for b in range(NB):
        assert view.alloc(b) == 0
    lists = _decode_loop_with_changing_shares(view, L, shares, lag=10)
    steady = [pairs for step, _, pairs in lists if step > 0 and shares[step] == shares[step - 1]]
    assert len(steady) == 10 * 2 * L
    assert all(len(pairs) == shares[step] for step, _, pairs in lists if step > 0 and shares[step] == shares[step - 1])
    assert [_runs(pairs) for pairs in steady] == [1] * len(steady)


def test_both_implementations_hand_out_the_same_slots_through_a_ramp():
    L, NB = 3, 32
    shares = [2, 2, 5, 5, 3, 3, 3, 7, 7, 1, 1, 6]
    out = []
    for impl in ("oracle", "library"):
        view = VIEWS[impl](L, NB, L * NB + 24, 40)      # tight: requests also reach the pending queue
        for b in range(NB):
            assert view.alloc(b) == 0
        out.append(_decode_loop_with_changing_shares(view, L, shares, lag=9))
    assert out[0] == out[1] and len(out[0]) > 60


@pytest.mark.parametrize("impl", ["oracle", "library"])
@pytest.mark.parametrize("retain", [False, True])
def test_long_random_runs_keep_the_rules(impl, retain):
    elided = random_runs(VIEWS[impl], 50, 140, retain)
    assert (elided > 50) if retain else (elided == 0)


def elision_scenario(make_view):
    view = make_view(1, 3, 3, 6, retain=True)
    model = rm.ResidencyModel(1, 3, random.Random(0))
    for op in [("alloc", 0, True), ("alloc", 1, True), ("alloc", 2, True), ("in", 0, (0, 1, 2)), ("confirm", True),
               ("attn_append", 0, (0, 1, 2), (2,)), ("out", 0, (0, 1, 2))]:
        assert rm.apply(view, model, op) == rm.OK
    assert list(view.last_elided) == [True, True, False]
    for op in [("confirm", True), ("in", 0, (2,)), ("confirm", True), ("out", 0, (2,))]:     # copied once: clean again
        assert rm.apply(view, model, op) == rm.OK
    assert list(view.last_elided) == [True]
    model.check_final(view)


@pytest.mark.parametrize("impl", ["oracle", "library"])
def test_unwritten_units_go_back_without_a_copy_and_written_ones_with(impl):
    """The point of keeping host copies: the elision must actually happen (an implementation that never elides keeps
    every rule above)."""
    elision_scenario(VIEWS[impl])


# ------------------------------------------------------------------------ mistakes must be caught
def patched_oracle(old, new):
    src = open(TABLE_PY).read()
    assert src.count(old) >= 1, old
    mod = types.ModuleType("table_mutant")
    exec(compile(src.replace(old, new, 1), TABLE_PY + " (mutant)", "exec"), mod.__dict__)
    return lambda *a, **k: OracleView(*a, module=mod, **k)


def patched_library(tmp_path, name, old, new):
    src = open(TABLE_CPP).read()
    assert src.count(old) >= 1, old
    cpp, so = tmp_path / f"{name}.cpp", tmp_path / f"{name}.so"
    cpp.write_text(src.replace(old, new, 1))
    csrc = os.path.dirname(TABLE_CPP)
    subprocess.check_call(["g++", "-O1", "-std=c++17", "-shared", "-fPIC", f"-I{csrc}", f"-I{os.path.join(ROOT, 'include')}",
                           "-include", os.path.join(csrc, "pie_table.h"), str(cpp), "-o", str(so)])
    cdll = ctypes.CDLL(str(so))
    return lambda *a, **k: LibView(*a, cdll=cdll, **k)


def caught(make_view):
    """Does any of the CPU drivers above object?"""
    try:
        exhaustive(make_view, KEPT, 3, warm=WARM, retain=True, slots=(4, 4))
        random_runs(make_view, 30, 140, True)
        elision_scenario(make_view)
    except AssertionError:
        return True
    return False


ORACLE_MISTAKES = {
    # the four ways to get the kept-copies rule wrong, and the write tracking that stopped with the switch
    "ignores the written mark": ("dst, elide = self.host_slot[u], not self.dirty[u]", "dst, elide = self.host_slot[u], True"),
    "keeps the mark after a copy": ("self.host_slot[u], self.gpu_slot[u] = dst, -1\n                self.dirty[u] = False",
                                    "self.host_slot[u], self.gpu_slot[u] = dst, -1"),
    "releases the kept slot at swap-in": ("if not self.retain:\n                    self.host_slot[u] = -1\n                    src_pool.release(src, direction, ticket)",
                                          "if not self.retain:\n                    self.host_slot[u] = -1\n                src_pool.release(src, direction, ticket)"),
    "gives the kept slot up at swap-in": ("if not self.retain:\n                    self.host_slot[u] = -1", "if True:\n                    self.host_slot[u] = -1"),
    "stops tracking writes when the switch goes off": ("def kept_copies(self):", "def kept_copies(self):\n        if not self.retain:\n            return 0"),
    # and two of the plain rules
    "hands a released slot out without its tag": ("self.pending.append((slot, queue, ticket))", "self._add_ready(slot)"),
    "forgets the copy still bringing the unit": ("if self._in_flight(u):  # the copy that is still bringing the unit to where it is now",
                                                 "if False:"),
}

LIBRARY_MISTAKES = {
    "ignores the written mark": ("skip = kept && !u.dirty;", "skip = kept;"),
    "keeps the mark after a copy": ("u.gpu_slot = -1;\n            u.dirty = 0;", "u.gpu_slot = -1;"),
    "releases the kept slot at swap-in": ("if (!retain_) {\n                u.host_slot = -1;\n                src_pool.release(s, queue, tk);\n            } else {",
                                          "src_pool.release(s, queue, tk);\n            if (!retain_) {\n                u.host_slot = -1;\n            } else {"),
    "gives the kept slot up at swap-in": ("if (!retain_) {\n                u.host_slot = -1;", "if (true) {\n                u.host_slot = -1;"),
    "stops tracking writes when the switch goes off": ("reinterpret_cast<const Table *>(t)->kept_copies() : 0; }",
                                                       "(reinterpret_cast<const Table *>(t)->retain() ? reinterpret_cast<const Table *>(t)->kept_copies() : 0) : 0; }"),
    "hands a released slot out without its tag": ("else pending_.push_back({slot, queue, ticket});", "else add_ready(slot);"),
    "forgets the copy still bringing the unit": ("if (in_flight(u)) waits[u.last_q] = std::max(waits[u.last_q], u.last_t);\n        int32_t s;",
                                                 "int32_t s;"),
}


def test_unpatched_implementations_pass_the_mistake_drivers(tmp_path):
    assert not caught(OracleView) and not caught(LibView)
    assert not caught(patched_library(tmp_path, "same", "skip = kept && !u.dirty;", "skip = kept && !u.dirty;"))   # the rebuild itself is sound


@pytest.mark.parametrize("mistake", sorted(ORACLE_MISTAKES))
def test_a_mistake_in_the_table_oracle_alone_is_caught(mistake):
    assert caught(patched_oracle(*ORACLE_MISTAKES[mistake])), mistake


@pytest.mark.parametrize("mistake", sorted(LIBRARY_MISTAKES))
def test_a_mistake_in_the_library_alone_is_caught(mistake, tmp_path):
    assert caught(patched_library(tmp_path, "mutant", *LIBRARY_MISTAKES[mistake])), mistake
