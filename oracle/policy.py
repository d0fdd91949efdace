"""Oracle of the swap protocol (Section 3.3) and of the adaptive-expansion controller (Section 3.4.2).

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA library.  Both are heuristics, so the oracle
takes the paper's steps in the paper's order, on a simulated clock.

Protocol, at the instant layer k starts computing (Section 3.3):
  1. completions are applied: a finished swap-out frees its GPU region, a finished swap-in makes its
     layer usable and frees its CPU region;
  2. if no swap-out is in flight, the coldest GPU layer (the one whose next use is farthest away,
     i.e. the layer that just finished) is swapped out, unless every CPU layer is colder than it or
     no CPU region is free;
  3. if no swap-in is in flight, the hottest CPU layer (next use nearest) is swapped in, unless no
     GPU region is free.
A layer in transit holds a region on both sides (Section 3.2).  If layer k is not on the GPU when its
turn comes the computation waits (Section 3.2) and the wait is counted as a stall.
"""
from __future__ import annotations

import dataclasses

GPU, CPU, OUT, IN = "GPU", "CPU", "OUT", "IN"


@dataclasses.dataclass
class ProtocolResult:
    events: list          # (time, "out"|"in", layer) in start order; layers are 1-based as in the paper
    stall: float          # total time computation waited
    trips: list           # (layer, out_start, in_finish)
    max_off_gpu: int      # most layers simultaneously on the CPU or in transit
    swaps_per_token: float
    finish_time: float
    in_starts: int = 0    # swap-ins started
    violations: int = 0   # ... of which for a layer the NEXT token needs (Section 3.4.2's allowed rule violation)


def simulate_protocol(n_layers, t_swap, gpu_regions, cpu_regions, cpu_layers, n_tokens, t_compute=1.0):
    loc = {l: (CPU if l in cpu_layers else GPU) for l in range(1, n_layers + 1)}
    assert sum(v == GPU for v in loc.values()) <= gpu_regions
    assert sum(v == CPU for v in loc.values()) <= cpu_regions
    out_busy = None  # (finish, layer)
    in_busy = None
    events, trips, open_trip = [], [], {}
    stall, now, max_off, n_swaps = 0.0, 0.0, 0, 0
    counts = {"in": 0, "violations": 0}

    def dist(l, k):  # compute-steps until layer l is needed again, seen from the start of layer k
        return (l - k) % n_layers

    def complete(t):
        nonlocal out_busy, in_busy
        if out_busy and out_busy[0] <= t:
            loc[out_busy[1]] = CPU
            out_busy = None
        if in_busy and in_busy[0] <= t:
            loc[in_busy[1]] = GPU
            trips.append((in_busy[1], open_trip.pop(in_busy[1], None), in_busy[0]))
            in_busy = None

    def start_swaps(t, k):
        nonlocal out_busy, in_busy, n_swaps
        gpu_used = sum(v in (GPU, OUT, IN) for v in loc.values())
        cpu_used = sum(v in (CPU, OUT, IN) for v in loc.values())
        if out_busy is None:
            cand = [l for l in loc if loc[l] == GPU and l != k]
            on_cpu = [l for l in loc if loc[l] == CPU]
            if cand and on_cpu and cpu_used < cpu_regions:
                victim = max(cand, key=lambda l: dist(l, k))
                if any(dist(c, k) < dist(victim, k) for c in on_cpu):
                    loc[victim] = OUT
                    out_busy = (t + t_swap, victim)
                    open_trip[victim] = t
                    events.append((t, "out", victim))
                    cpu_used += 1
                    n_swaps += 1
        if in_busy is None:
            on_cpu = [l for l in loc if loc[l] == CPU]
            if on_cpu and gpu_used < gpu_regions:
                hot = min(on_cpu, key=lambda l: dist(l, k))
                loc[hot] = IN
                in_busy = (t + t_swap, hot)
                events.append((t, "in", hot))
                counts["in"] += 1
                # the current token still needs layers k .. n; a lower one is fetched for the token after it
                counts["violations"] += hot < k

    for _tok in range(n_tokens):
        for k in range(1, n_layers + 1):
            complete(now)
            start_swaps(now, k)
            while loc[k] != GPU:  # presence check failed: wait for the next completion
                nxt = min(b[0] for b in (out_busy, in_busy) if b is not None)
                stall += nxt - now
                now = nxt
                complete(now)
                start_swaps(now, k)
            max_off = max(max_off, sum(v != GPU for v in loc.values()))
            now += t_compute
    return ProtocolResult(events, stall, trips, max_off, n_swaps / n_tokens, now, counts["in"], counts["violations"])


# ---------------------------------------------------------------------------------------------
# Adaptive expansion in whole layers (Section 3.4.2 as the paper states it): m = layers kept on the CPU.
#   - more swapping: whenever a swap could be started and no on-CPU layer is needed by the token being computed, the
#     expansion is too small.  Rather than leave the link idle the protocol then fetches a layer of the NEXT token (the
#     violation the paper allows "to prevent waiting"); the share of swap-ins that are such violations is high while m is
#     small and falls as m grows.  When it reaches the preset ratio (or nothing is on the CPU at all), m grows by one.
#     The link is as busy before as after (the protocol swaps all the time), so link slack cannot be the signal here.
#   - less swapping: the computation had to wait (stall above eps of the compute time): m shrinks by one, and the
#     value that stalled is left alone for `hold` windows, twice as long after every failed return (a performance
#     record, as for the block-granular controller).
# The paper gives no constants; these are the build's: v_trigger = 0.3, eps = 0.02, hold = 4 windows at first.
# ---------------------------------------------------------------------------------------------
@dataclasses.dataclass
class LayerController:
    m_max: int
    v_trigger: float = 0.3
    eps: float = 0.02
    m: int = 0
    bad: int = -1          # lowest m known to make the computation wait (-1: none)
    hold: int = 0          # windows left before `bad` may be tried again
    hold_len: int = 4

    def update(self, stall, compute, in_starts, violations):
        """One window's measurements -> the number of CPU layers for the next window."""
        if stall > self.eps * compute:
            self.bad = self.m if self.bad < 0 else min(self.bad, self.m)
            self.m = max(0, self.m - 1)
            self.hold, self.hold_len = self.hold_len, min(2 * self.hold_len, 96)
            return self.m
        too_small = in_starts == 0 or violations >= self.v_trigger * in_starts
        if too_small and self.m < self.m_max:
            if self.bad >= 0 and self.m + 1 >= self.bad:
                if self.hold > 0:
                    self.hold -= 1
                    return self.m
            self.m += 1
        return self.m


# ---------------------------------------------------------------------------------------------
# Adaptive expansion (Section 3.4.2), block-granular: r = fraction of units kept host resident.
#   - start with everything on the GPU (r = 0);
#   - decrease when the computation had to wait for a swap (stall above eps of compute time) in at
#     least k_dec of the last `window` steps - a single disturbed step is tolerated;
#   - increase by one step when there was no stall and the link was busy for less than u_hi of the
#     compute time (the link has slack and nothing on the host was needed late), but not within
#     `cooldown` steps of the previous increase (a change has to be observed before the next);
#   - hold otherwise.
# The paper gives no constants; these are the build's: step = 1/n_layers ("one layer"), eps = 0.02,
# k_dec = 2 of window = 4, u_hi = 0.9, cooldown = 3.
# ---------------------------------------------------------------------------------------------

@dataclasses.dataclass
class Controller:
    step: float
    eps: float = 0.02
    k_dec: int = 2
    window: int = 4
    u_hi: float = 0.9
    r_max: float = 1.0
    cooldown: int = 3
    hold_max: int = 96
    r: float = 0.0
    wait: int = 0
    history: list = dataclasses.field(default_factory=list)
    # performance record (Section 3.4.2): the lowest ratio known to make the computation wait, how long to leave it
    # alone before probing it again (doubles with every failed probe), steps since the last back-off, and unstalled
    # steps spent at or above that ratio (enough of them clear the record)
    r_bad: float = -1.0
    hold: int = 3
    since_dec: int = 0
    ok_at_bad: int = 0

    def tick(self, stall, compute, swap_busy):
        """One decode step's measurements (same time unit) -> new ratio."""
        stalled = stall > self.eps * compute
        self.history.append(stalled)
        self.history = self.history[-self.window:]
        self.since_dec += 1
        if self.r_bad >= 0:
            self.ok_at_bad = self.ok_at_bad + 1 if (not stalled and self.r >= self.r_bad - 1e-12) else 0
            if self.ok_at_bad >= self.window:           # the ratio that used to stall is fine now: forget the record
                self.r_bad, self.hold, self.ok_at_bad = -1.0, self.cooldown, 0
        if stalled:
            if sum(self.history) >= self.k_dec:
                # backing off from the known bad ratio (or below it) again: the next probe waits twice as long
                again = self.r_bad >= 0 and self.r <= self.r_bad + 1e-12
                self.hold = min(2 * self.hold, self.hold_max) if again else self.cooldown
                self.r_bad, self.since_dec, self.ok_at_bad = self.r, 0, 0
                self.r = max(0.0, self.r - self.step)
                self.history = []
        elif self.wait > 0:
            self.wait -= 1
        elif swap_busy < self.u_hi * compute and self.r < self.r_max:
            target = min(self.r_max, self.r + self.step)
            if not (self.r_bad >= 0 and target >= self.r_bad - 1e-12 and self.since_dec < self.hold):
                self.r = target
                self.wait = self.cooldown
        return self.r


def fake_clock_step(r, bytes_layer, bw, t_compute_layer, n_layers):
    """Timings of one decode step on an ideal machine: layer l+1's host-resident share streams in
    while layer l computes; computation waits for whatever has not arrived."""
    t_in = r * bytes_layer / bw
    stall_per_layer = max(0.0, t_in - t_compute_layer)
    return stall_per_layer * n_layers, t_compute_layer * n_layers, t_in * n_layers


# ---------------------------------------------------------------------------------------------
# Performance records against throughput (Section 3.4.2, last paragraph).  The serving system reports the
# throughput it saw over a window at the ratio then in force; the governor keeps the newest report per ratio
# (in units of the controller's step) and turns the paragraph's three sentences into a cap on the ratio,
# which the stall-driven controller above then respects (it may stay below the cap, never above):
#   NORMAL   no cap.  When a report at ratio k shows no gain over the record one step below
#            (T[k] <= T[k-1] (1 + tol)), the workload has stopped scaling with expansion: stop increasing and
#            test whether decreasing has any adverse effect -> TEST_DOWN with the cap one step lower.
#   TEST_DOWN a report at the lowered cap: not worse than the reference (>= ref (1 - tol)) -> no adverse effect,
#            keep it and try one step lower still (at 0: HOLD); worse -> one step back up, HOLD.
#   HOLD     the cap stays.  Every `period` reports (low demand, spare bandwidth) -> PROBE_UP: cap one step up.
#   PROBE_UP a report at the raised cap: better than the reference by more than tol -> the workload scales
#            again: NORMAL; else one step back down, HOLD ("reduces it if the workload remains low").
# Reports at a ratio other than the cap (the controller has not got there, or was pushed below it by stalls)
# only update the records; `patience` such reports in a row end a test (TEST_DOWN, PROBE_UP -> HOLD at the
# ratio reported).  Constants are the build's: tol = 0.02, period = 8, patience = 6.
# ---------------------------------------------------------------------------------------------

NORMAL, TEST_DOWN, HOLD, PROBE_UP = 0, 1, 2, 3


@dataclasses.dataclass
class Governor:
    step: float
    tol: float = 0.02
    period: int = 8
    patience: int = 6
    k_max: int = 1 << 30
    state: int = NORMAL
    cap: int = 1 << 30            # in steps; k_max = no cap
    ref: float = 0.0              # throughput the running test compares with
    since: int = 0                # reports since HOLD began
    off: int = 0                  # reports in a row at a ratio other than the cap during a test
    rec: dict = dataclasses.field(default_factory=dict)

    def cap_ratio(self):
        return 1.0 if self.cap >= self.k_max else self.cap * self.step

    def report(self, ratio, throughput):
        """One window's throughput at `ratio` -> the cap (as a ratio; 1.0 = none)."""
        k = int(round(ratio / self.step))
        self.rec[k] = throughput
        if self.state == NORMAL:
            if k > 0 and (k - 1) in self.rec and throughput <= self.rec[k - 1] * (1 + self.tol):
                self.state, self.cap, self.ref, self.off = TEST_DOWN, k - 1, throughput, 0
        elif self.state == TEST_DOWN:
            if k != self.cap:
                self.off += 1
                if self.off >= self.patience:
                    self.state, self.cap, self.since, self.off = HOLD, k, 0, 0
            elif throughput >= self.ref * (1 - self.tol):
                self.ref, self.off = max(self.ref, throughput), 0
                if self.cap > 0:
                    self.cap -= 1
                else:
                    self.state, self.since = HOLD, 0
            else:
                self.state, self.cap, self.since, self.off = HOLD, self.cap + 1, 0, 0
        elif self.state == HOLD:
            self.since += 1
            if self.since >= self.period:
                self.state, self.ref, self.cap, self.off = PROBE_UP, throughput, self.cap + 1, 0
        else:  # PROBE_UP
            if k != self.cap:
                self.off += 1
                if self.off >= self.patience:
                    self.state, self.cap, self.since, self.off = HOLD, k, 0, 0
            elif throughput > self.ref * (1 + self.tol):
                self.state, self.cap, self.rec = NORMAL, self.k_max, {k: throughput}
            else:
                self.state, self.cap, self.since, self.off = HOLD, self.cap - 1, 0, 0
        return self.cap_ratio()
