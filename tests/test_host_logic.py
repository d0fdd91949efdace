"""CPU tests of the library's host side through the C ABI: exported symbols, loud failure without a GPU,
mapping table / protocol scheduler / controller rule against the oracle and the paper's worked example."""
import itertools
import os
import random
import re

import numpy as np
import pytest

from oracle import policy, table as otable
from paper_2411_09317_b200 import binding as pie
from tests.test_oracle_swap_policy import read_golden

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "pie.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(pie_[a-z_0-9]+)\s*\(", header))
    assert len(declared) >= 35
    for name in declared:
        assert hasattr(pie.lib, name), f"{name} declared in pie.h but not exported by libpie.so"
    assert declared == set(pie.EXPORTS)


def test_pool_create_fails_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(pie.PieError) as e:
        pie.pie_pool_create(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, dtype=pie.PIE_F16,
                            n_logical_blocks=8, n_gpu_slots=16, n_host_slots=16)
    assert e.value.status == pie.PIE_ERR_CUDA


def test_pool_create_rejects_bad_configs_before_touching_cuda():
    base = dict(n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, dtype=pie.PIE_F16, n_logical_blocks=8,
                n_gpu_slots=16, n_host_slots=16)
    for patch, code in [({"n_kv_heads": 3}, pie.PIE_ERR_INVALID), ({"head_dim": 96}, pie.PIE_ERR_UNSUPPORTED),
                        ({"n_q_heads": 64, "n_kv_heads": 4}, pie.PIE_ERR_UNSUPPORTED), ({"dtype": 5}, pie.PIE_ERR_INVALID),
                        ({"block_tokens": 32}, pie.PIE_ERR_UNSUPPORTED), ({"n_layers": 0}, pie.PIE_ERR_INVALID),
                        ({"split_tokens": 100}, pie.PIE_ERR_INVALID)]:
        with pytest.raises(pie.PieError) as e:
            pie.pie_pool_create(**{**base, **patch})
        assert e.value.status == code, patch


# ------------------------------------------------------------------------------- table vs oracle
def both_apply(o, t, op):
    """Apply one call to the oracle table and to the library's table; compare everything observable."""
    kind = op[0]
    if kind == "alloc":
        a, b = o.alloc(op[1], op[2]), t.alloc(op[1], op[2])
    elif kind == "free":
        a, b = o.free(op[1]), t.free(op[1])
    elif kind in ("out", "in"):
        q = otable.Q_OUT if kind == "out" else otable.Q_IN
        a, b = o.swap(q, op[1], list(op[2])), t.swap(q, op[1], list(op[2]))
        if a[0] == otable.OK:
            assert list(o.last_elided) == list(t.last_elided), op
    elif kind == "attn":
        ra, rb = o.attention(op[1], list(op[2])), t.attention(op[1], list(op[2]))
        ra[2].pop(otable.Q_COMPUTE, None)  # same stream as the call itself: the library drops it
        a, b = ra, rb
    elif kind == "confirm":
        q, frac = op[1], op[2]
        tk = int(o.issued[q] * frac)
        a, b = o.confirm(q, tk), t.confirm(q, tk)
    elif kind == "dirty":
        a, b = o.mark_dirty(op[1], list(op[2])), t.mark_dirty(op[1], list(op[2]))
    elif kind == "drop":
        a, b = o.drop_host_copy(op[1], op[2]), t.drop_host_copy(op[1], op[2])
    elif kind == "retain":
        o.retain = bool(op[1])
        a, b = 0, t.set_retention(op[1])
    elif kind == "resize":
        a, b = o.resize_begin(op[1]), t.resize_begin(op[1])
    elif kind == "pass":
        a, b = int(o.layer_pass(op[1])), t.layer_pass(op[1])
    assert a == b, (op, a, b)
    assert t.kept_copies() == o.kept_copies(), op
    st, cap = t.capacity()
    assert cap == {"visible": o.capacity, "alloc_limit": o.alloc_limit(), "target": -1 if o.target is None else o.target,
                   "layers_moved": len(o.moved)}, op
    for l in range(o.L):
        for blk in range(o.NB):
            u = o._u(l, blk)
            st, s, g, h = t.state(l, blk)
            assert (s, g, h) == (o.state(l, blk), o.gpu_slot[u], o.host_slot[u]), (op, l, blk)


def test_table_matches_oracle_exhaustive_tiny():
    alphabet = [("alloc", 0, False), ("alloc", 1, True), ("free", 0), ("out", 0, (0,)), ("out", 1, (0, 1)),
                ("in", 0, (0,)), ("in", 1, (1, 0)), ("attn", 0, (0,)), ("attn", 1, (0, 1)),
                ("confirm", otable.Q_OUT, 1.0), ("confirm", otable.Q_IN, 1.0), ("confirm", otable.Q_COMPUTE, 1.0)]
    n = 0
    for length in range(1, 5):
        for seq in itertools.product(alphabet, repeat=length):
            if seq[0][0] != "alloc" and length > 1:
                continue
            o, t = otable.MappingTable(2, 2, 3, 3), pie.Table(2, 2, 3, 3)
            for op in seq:
                both_apply(o, t, op)
            n += 1
    assert n > 3000


def test_table_with_kept_host_copies_matches_oracle_exhaustive_tiny():
    alphabet = [("alloc", 1, True), ("free", 0), ("out", 0, (0,)), ("out", 1, (0, 1)), ("in", 0, (0,)), ("in", 1, (1, 0)),
                ("attn", 0, (0,)), ("dirty", 0, (0,)), ("dirty", 1, (1, 0)), ("drop", 0, 0), ("confirm", otable.Q_OUT, 1.0),
                ("confirm", otable.Q_IN, 1.0), ("confirm", otable.Q_COMPUTE, 1.0)]
    n = 0
    for length in range(1, 5):
        for seq in itertools.product(alphabet, repeat=length):
            o, t = otable.MappingTable(2, 2, 4, 4, retain=True), pie.Table(2, 2, 4, 4)
            assert t.set_retention(True) == pie.PIE_OK
            for op in [("alloc", 0, True), ("in", 0, (0,)), ("in", 1, (0,)), ("confirm", otable.Q_IN, 1.0)] + list(seq):
                both_apply(o, t, op)
            n += 1
    assert n > 20000


@pytest.mark.parametrize("retain", [False, True])
def test_table_matches_oracle_random_long(retain):
    rng = random.Random(11)
    for trial in range(40):
        L, NB = rng.choice([(1, 6), (3, 5), (2, 9)])
        ng, nh = rng.randint(NB, L * NB), rng.randint(NB, L * NB) + (L * NB if retain else 0)
        o, t = otable.MappingTable(L, NB, ng, nh, retain=retain), pie.Table(L, NB, ng, nh)
        t.set_retention(retain)
        for _ in range(150):
            k = rng.random()
            if retain and rng.random() < 0.15:
                both_apply(o, t, ("dirty", rng.randrange(L), tuple(rng.sample(range(NB), rng.randint(1, NB)))))
            if retain and rng.random() < 0.05:
                both_apply(o, t, ("drop", rng.randrange(L), rng.randrange(NB)))
            if retain and rng.random() < 0.04:
                both_apply(o, t, ("retain", rng.random() < 0.5))      # the switch itself, while copies are kept
            ids = tuple(rng.sample(range(NB), rng.randint(1, NB)))
            if rng.random() < 0.05:
                ids = ids + (ids[0],) if rng.random() < 0.5 else ids + (NB + 3,)
            layer = rng.randrange(L) if rng.random() > 0.03 else L
            if rng.random() < 0.06:
                both_apply(o, t, ("resize", rng.randint(0, NB + 1)) if rng.random() < 0.5 else ("pass", rng.randrange(L)))
            op = (("alloc", rng.randrange(NB), rng.random() < 0.3) if k < 0.15 else ("free", rng.randrange(NB)) if k < 0.2
                  else ("out", layer, ids) if k < 0.45 else ("in", layer, ids) if k < 0.7
                  else ("attn", layer, ids) if k < 0.85 else ("confirm", rng.choice([1, 2, 3]), rng.random()))
            both_apply(o, t, op)
        o.check_invariants()


def test_table_resize_matches_oracle_exhaustive_tiny():
    """Every sequence of up to 5 calls over resize / layer pass / alloc / free / swap on a 2-layer table of width 3."""
    alphabet = [("resize", 3), ("resize", 1), ("resize", 2), ("pass", 0), ("pass", 1), ("alloc", 0, False), ("alloc", 2, True),
                ("free", 2), ("out", 0, (0,)), ("in", 1, (2,))]
    n = 0
    for length in range(1, 6):
        for seq in itertools.product(alphabet, repeat=length):
            if seq[0][0] not in ("resize", "alloc"):
                continue
            o, t = otable.MappingTable(2, 3, 4, 4, capacity=2), pie.Table(2, 3, 4, 4)
            assert t.init_capacity(2) == pie.PIE_OK
            for op in seq:
                both_apply(o, t, op)
            n += 1
    assert n > 20000


def test_table_attention_without_ids_waits_for_every_arriving_unit():
    t = pie.Table(1, 4, 4, 4)
    for b in range(4):
        assert t.alloc(b, on_host=(b >= 2)) == pie.PIE_OK
    st, tk, pairs, waits = t.swap(pie.PIE_Q_IN, 0, [2])
    assert st == pie.PIE_OK and tk == 1
    st, ctk, waits = t.attention(0, None)
    assert st == pie.PIE_OK and waits == {pie.PIE_Q_IN: 1}
    t.confirm(pie.PIE_Q_IN, 1)
    st, ctk, waits = t.attention(0, None)
    assert waits == {}


# ------------------------------------------------------------------------------- protocol scheduler
def drive_fifo(n, t_swap, gpu_regions, cpu_regions, cpu_layers, n_tokens):
    """Simulated clock around pie_fifo_*: returns (events, stall) like the oracle's simulator (1-based layers)."""
    f = pie.Fifo(n, gpu_regions, cpu_regions, [1 if (l + 1) in cpu_layers else 0 for l in range(n)])
    busy = {pie.PIE_Q_OUT: None, pie.PIE_Q_IN: None}
    now, stall, events = 0.0, 0.0, []

    def complete(t):
        for d in (pie.PIE_Q_OUT, pie.PIE_Q_IN):
            if busy[d] is not None and busy[d] <= t:
                assert f.complete(d) == pie.PIE_OK
                busy[d] = None

    def start(t, k):
        st, o, i = f.layer_start(k)
        assert st == pie.PIE_OK
        if o >= 0:
            busy[pie.PIE_Q_OUT] = t + t_swap
            events.append((t, "out", o + 1))
        if i >= 0:
            busy[pie.PIE_Q_IN] = t + t_swap
            events.append((t, "in", i + 1))

    for _ in range(n_tokens):
        for k in range(n):
            complete(now)
            start(now, k)
            while f.location(k) != 0:
                nxt = min(b for b in busy.values() if b is not None)
                stall += nxt - now
                now = nxt
                complete(now)
                start(now, k)
            now += 1.0
    drive_fifo.counters = f.counters()
    return events, stall


def test_fifo_reproduces_the_nine_layer_example():
    rows, totals = read_golden()
    events, stall = drive_fifo(9, 2.0, 7, 4, {8, 9}, 6)
    started = {}
    for t, kind, layer in events:
        started.setdefault(int(t), {})[kind] = layer
    for tag, t, layer_starting, out, inn in rows:
        assert started.get(t, {}).get("out", 0) == out, (tag, t)
        assert started.get(t, {}).get("in", 0) == inn, (tag, t)
    assert stall == totals["stall"]


@pytest.mark.parametrize("n,t_swap,g,c,cpu", [(9, 2.0, 7, 4, {8, 9}), (9, 3.0, 7, 4, {8, 9}), (9, 2.0, 6, 4, {7, 8, 9}),
                                              (9, 2.0, 8, 3, {9}), (6, 1.5, 4, 4, {5, 6}), (12, 2.5, 9, 6, {1, 5, 12}),
                                              (5, 1.0, 5, 2, set())])
def test_fifo_matches_oracle_protocol(n, t_swap, g, c, cpu):
    events, stall = drive_fifo(n, t_swap, g, c, cpu, 7)
    ref = policy.simulate_protocol(n, t_swap, g, c, cpu, 7)
    assert events == ref.events
    assert stall == pytest.approx(ref.stall)
    assert drive_fifo.counters == (ref.in_starts, ref.violations)     # swap-ins started, of which for the next token


@pytest.mark.parametrize("t_swap", [1.0, 1.5, 2.0, 3.0])
def test_layer_controller_rule_matches_oracle_on_the_protocol_simulator(t_swap):
    """Section 3.4.2's rule for the number of CPU layers: the library's against the oracle's, both fed by the protocol
    simulator window after window (and by random measurements afterwards)."""
    n = 9
    c = policy.LayerController(m_max=n - 2)
    state, m = np.zeros(4), 0
    rng = random.Random(int(t_swap * 10))
    for w in range(60):
        if w < 40:
            r = policy.simulate_protocol(n, t_swap, n - m, m + 2, set(range(n - m + 1, n + 1)), 5)
            meas = (r.stall, 5.0 * n, r.in_starts, r.violations)
        else:
            meas = (rng.choice([0.0, 0.0, 3.0]), 45.0, rng.randint(0, 30), rng.randint(0, 12))
        want = c.update(*meas)
        m = pie.pie_layer_controller_decide(state, m, n - 2, *meas)
        assert m == want, (w, meas)


# ------------------------------------------------------------------------------------ controller rule
@pytest.mark.parametrize("bw,tc,bytes_layer,L", [(50e9, 200e-6, 400e6, 32), (400e9, 300e-6, 400e6, 32), (1e12, 1e-3, 1e8, 8)])
def test_controller_rule_matches_oracle(bw, tc, bytes_layer, L):
    c = policy.Controller(step=1.0 / L)
    state = np.zeros(16)
    r = 0.0
    rng = random.Random(3)
    for i in range(600):
        b = bw * (0.4 if 100 <= i < 110 or 200 < i < 400 else 1.0) * (1.0 + 0.2 * (rng.random() - 0.5))
        m = policy.fake_clock_step(r, bytes_layer, b, tc, L)
        want = c.tick(*m)
        r = pie.pie_controller_decide(state, r, 1.0 / L, *m)
        assert r == pytest.approx(want, abs=1e-12), i


# ------------------------------------------------------------------- throughput governor: C++ against the oracle
@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_governor_matches_oracle_on_random_reports(seed):
    """Random walks of (ratio, throughput) reports - rising, flat, falling and noisy stretches, ratios that follow the
    cap and ratios that do not: state and cap agree after every report."""
    from oracle.policy import Governor
    rng = np.random.default_rng(seed)
    step = [0.01, 1.0 / 32, 0.002, 0.05][seed]
    og, cg = Governor(step), pie.Governor(step)
    k, base, slope, sat = 0, 100.0, 800.0, int(rng.integers(0, 12))
    for i in range(600):
        if i % 97 == 96:                                   # the workload changes
            sat, slope = int(rng.integers(0, 12)), float(rng.choice([0.0, 300.0, 3000.0]))
        t = (base + slope * step * min(k, sat)) * (1 + float(rng.uniform(-0.01, 0.01)))
        want = og.report(k * step, t)
        got = cg.report(k * step, t)
        state, cap = cg.state()
        assert (state, cap) == (og.state, -1 if og.cap >= og.k_max else og.cap), i
        assert got == want
        move = rng.integers(0, 4)
        target = og.cap if move else int(rng.integers(0, 14))     # mostly follow the cap, sometimes not
        if k < min(target, 20):
            k += 1
        elif k > target:
            k -= 1
    cg.close()


def test_header_is_plain_c_and_cxx(tmp_path):
    """include/pie.h must stand on its own for a C99 and a C++17 caller (no torch, no CUDA types in the signatures)."""
    import os
    import shutil
    import subprocess
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    for comp, name, std in (("gcc", "t.c", "-std=c99"), ("g++", "t.cpp", "-std=c++17")):
        if shutil.which(comp) is None:
            pytest.skip(f"{comp} not installed")
        src = tmp_path / name
        src.write_text('#include "pie.h"\nint main(void) { pie_pool_config c; (void)c; return sizeof(pie_stats) > 0 ? 0 : 1; }\n')
        subprocess.check_call([comp, std, "-Wall", "-Werror", "-pedantic", "-I", inc, "-fsyntax-only", str(src)])
