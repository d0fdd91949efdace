"""A synthetic arrival driver around the library: requests arrive as a Poisson process, are admitted while their
prompt's blocks fit the GPU pool, decode one token per step in a continuous batch and leave when their output is
complete (the serving loop of Section 5.1's experiments reduced to what touches this path; no scheduler policy beyond
first come, first served; no model: every layer is its attention).  The pool runs in adaptive mode: the controller
moves a share of every layer's blocks to the host pool while that stays hidden, which is what frees GPU slots for more
requests; every window the driver reports its tokens per second to the throughput governor (Section 3.4.2).

Contents are a pure function of (request, layer, position): the prompt's keys and values enter through pie_kv_write,
every later token through the decode step's append, so a test can rebuild any sequence's keys and values from the
generator and check sampled outputs against the oracle.

    python -m paper_2411_09317_b200.arrivals --rate 1.0 --requests 200 [--kept-copies] [--kv-gb 2.0] [--out file.jsonl]

--rate is in units of the service capacity estimated from the first steps (1.0 = arrivals as fast as a full GPU pool can
serve them).  Time is GPU time of the decode steps (CUDA events); prompt writes are not counted.  One JSON line per window.
"""
from __future__ import annotations

import argparse
import collections
import dataclasses
import json
import sys

import numpy as np
import torch

from . import binding as pie
from . import synth

MAXPOS = 4096          # positions per (request, layer) in the generator's index space


@dataclasses.dataclass
class Shape:
    n_layers: int = 8
    n_q_heads: int = 32
    n_kv_heads: int = 8
    head_dim: int = 128
    dtype: int = synth.BF16
    kv_fp8: bool = False      # 8-bit blocks (head_dim 128): prompts and appended tokens are quantised by the library


@dataclasses.dataclass
class Request:
    rid: int
    arrival: float
    prompt: int
    out_len: int
    blocks: list = dataclasses.field(default_factory=list)
    ctx: int = 0            # tokens whose keys and values are in the cache
    produced: int = 0


def element_offset(sh: Shape, rid: int, layer: int, pos: int, row_elems: int) -> int:
    return ((rid * sh.n_layers + layer) * MAXPOS + pos) * row_elems


def make_requests(seed: int, n: int, mean_gap: float, prompt_median=600.0, prompt_sigma=0.6, out_mean=96.0):
    rng = np.random.default_rng(seed)
    t = np.cumsum(rng.exponential(mean_gap, n))
    prompts = np.clip(np.round(np.exp(rng.normal(np.log(prompt_median), prompt_sigma, n))), 32, 2048).astype(int)
    outs = np.clip(rng.geometric(1.0 / out_mean, n), 8, 512).astype(int)
    return [Request(i, float(t[i]), int(prompts[i]), int(outs[i])) for i in range(n)]


class Driver:
    K_SCALE, V_SCALE = 0.25, 0.125     # scales of an 8-bit pool

    def __init__(self, sh: Shape, gpu_blocks_per_layer: int, host_blocks_per_layer: int, max_seqs=128, seed=11,
                 kept_copies=False, ctrl_step=1.0 / 512, window=16, sample_ids=()):
        self.sh, self.seed, self.window, self.max_seqs = sh, seed, window, max_seqs
        self.dev = torch.device("cuda", torch.cuda.current_device())
        L = sh.n_layers
        self.gpu_blocks = gpu_blocks_per_layer
        self.n_logical = gpu_blocks_per_layer + host_blocks_per_layer
        self.max_blocks = (MAXPOS + 15) // 16
        staging = 3 * max(64, host_blocks_per_layer // 4)
        self.pool = pie.pie_pool_create(
            n_layers=L, n_q_heads=sh.n_q_heads, n_kv_heads=sh.n_kv_heads, head_dim=sh.head_dim, dtype=sh.dtype,
            n_logical_blocks=self.n_logical, max_seqs=max_seqs, n_gpu_slots=L * gpu_blocks_per_layer + staging,
            n_host_slots=L * host_blocks_per_layer + staging, timing=1, kv_fp8=int(sh.kv_fp8))
        if sh.kv_fp8:
            pie.pie_set_kv_scales(self.pool, self.K_SCALE, self.V_SCALE)
        pie.pie_set_controller(self.pool, ctrl_step, 0.0, 0.0)
        pie.pie_set_extension_ratio(self.pool, -1.0)             # adaptive
        pie.pie_set_retention(self.pool, int(kept_copies))
        self.kept = kept_copies
        self.bt_host = np.full((max_seqs, self.max_blocks), -1, dtype=np.int32)
        self.bt_dev = torch.from_numpy(self.bt_host).to(self.dev)
        self.ctx_dev = torch.zeros(max_seqs, dtype=torch.int32, device=self.dev)
        qe, ke = sh.n_q_heads * sh.head_dim, sh.n_kv_heads * sh.head_dim
        self.q = torch.empty(L * max_seqs * qe, dtype=torch.int16, device=self.dev)
        self.out = torch.zeros(L * max_seqs * qe, dtype=torch.int16, device=self.dev)
        self.k_new = torch.empty(L * max_seqs * ke, dtype=torch.int16, device=self.dev)
        self.v_new = torch.empty(L * max_seqs * ke, dtype=torch.int16, device=self.dev)
        self.prompt_k = torch.empty(2048 * ke, dtype=torch.int16, device=self.dev)
        self.prompt_v = torch.empty(2048 * ke, dtype=torch.int16, device=self.dev)
        self.pos_dev = torch.arange(2048, dtype=torch.int32, device=self.dev)
        self.row_dev = torch.zeros(2048, dtype=torch.int32, device=self.dev)
        self.lib = pie.synth_lib()
        self.base = {s: int(synth.stream_base(seed, s)) for s in (synth.STREAM_Q, synth.STREAM_KNEW, synth.STREAM_VNEW)}
        self.scale = 1.0 / float(np.sqrt(sh.head_dim))
        self.running: list[Request] = []
        self.sample_ids = set(sample_ids)
        self.samples = []          # (rid, ctx, out bits [L][Hq][D]) of sampled requests at their last step
        self.log = []

    # ---- admission: the prompt's blocks must all land in the GPU pool (the prompt is written there) ------------
    def try_admit(self, r: Request) -> bool:
        sh, L = self.sh, self.sh.n_layers
        nb = (r.prompt + 1 + 15) // 16
        # capacity at the expansion in force: with the share `ratio` of every layer's blocks living on the host, the GPU
        # pool's blocks carry 1 / (1 - ratio) times as many; the slots beyond them stay free for blocks in transit, and
        # a margin stays free for the running requests' growth
        ratio = pie.pie_get_extension_ratio(self.pool)
        held = sum(len(x.blocks) for x in self.running)
        if (held + nb + 2 * len(self.running)) * (1.0 - ratio) > self.gpu_blocks:
            return False
        try:
            ids = pie.pie_block_alloc(self.pool, nb)
        except pie.PieError as e:
            if e.status == pie.PIE_ERR_NOMEM:
                return False
            raise
        # (the last unit allocated is the first to spill: checking the newest block of every layer is enough)
        if any(pie.pie_block_state(self.pool, l, int(ids[-1]))[0] != pie.PIE_GPU for l in range(L)) or \
                any(pie.pie_block_state(self.pool, l, int(ids[0]))[0] != pie.PIE_GPU for l in range(L)):
            pie.pie_block_free(self.pool, ids)
            return False
        row = len(self.running)
        r.blocks = [int(b) for b in ids]
        self.bt_host[row, :] = -1
        self.bt_host[row, :nb] = ids
        self.bt_dev[row].copy_(torch.from_numpy(self.bt_host[row]))
        self.row_dev[:r.prompt].fill_(row)
        ke = sh.n_kv_heads * sh.head_dim
        for l in range(L):
            off = element_offset(sh, r.rid, l, 0, ke)
            for buf, stream in ((self.prompt_k, synth.STREAM_KNEW), (self.prompt_v, synth.STREAM_VNEW)):
                rc = self.lib.pie_synth_fill_tensor(buf.data_ptr(), r.prompt * ke, self.base[stream], off, sh.dtype, 1.0, None)
                assert rc == 0
            torch.cuda.synchronize()       # the generator ran on the default stream, the write runs on the pool's
            pie.pie_kv_write(self.pool, l, self.prompt_k.data_ptr(), self.prompt_v.data_ptr(), self.row_dev.data_ptr(),
                             self.pos_dev.data_ptr(), r.prompt, self.bt_dev.data_ptr(), self.max_blocks, row + 1)
            pie.pie_sync(self.pool)        # the two prompt buffers are reused by the next layer
        r.ctx = r.prompt
        self.running.append(r)
        return True

    def grow(self, r: Request, row: int) -> None:
        """The next token needs position r.ctx: a new block when that starts one the request does not hold yet."""
        if r.ctx // 16 >= len(r.blocks):
            b = int(pie.pie_block_alloc(self.pool, 1)[0])       # GPU if there is room, else the host pool
            self.bt_host[row, len(r.blocks)] = b
            r.blocks.append(b)
            self.bt_dev[row].copy_(torch.from_numpy(self.bt_host[row]))

    # ---- one decode step over the running batch -----------------------------------------------------------------
    def step(self) -> float:
        sh, L, S = self.sh, self.sh.n_layers, len(self.running)
        for row, r in enumerate(self.running):
            self.grow(r, row)
        ctx_next = np.array([r.ctx + 1 for r in self.running], dtype=np.int32)
        self.ctx_dev[:S].copy_(torch.from_numpy(ctx_next))
        qe, ke = sh.n_q_heads * sh.head_dim, sh.n_kv_heads * sh.head_dim
        for buf, stream, re_ in ((self.q, synth.STREAM_Q, qe), (self.k_new, synth.STREAM_KNEW, ke), (self.v_new, synth.STREAM_VNEW, ke)):
            offs = np.array([element_offset(sh, r.rid, l, r.ctx, re_) for l in range(L) for r in self.running], dtype=np.int64)
            od = torch.from_numpy(offs).to(self.dev)
            rc = self.lib.pie_synth_fill_rows(buf.data_ptr(), od.data_ptr(), L * S, re_, self.base[stream], sh.dtype, 1.0, None)
            assert rc == 0
        torch.cuda.synchronize()
        if self.kept:
            pie.pie_declare_append_blocks(self.pool, np.array([r.blocks[r.ctx // 16] for r in self.running], dtype=np.int32))
        pie.pie_decode_step(self.pool, self.q.data_ptr(), self.out.data_ptr(), self.bt_dev.data_ptr(), self.max_blocks,
                            self.ctx_dev.data_ptr(), S, self.scale, self.k_new.data_ptr(), self.v_new.data_ptr())
        pie.pie_sync(self.pool)
        st = pie.pie_get_stats(self.pool)
        for r in self.running:
            r.ctx += 1
            r.produced += 1
        # sampled requests that end with this step: their outputs, by the rows the step ran with
        def finished(r):
            return r.produced >= r.out_len or r.ctx + 1 >= MAXPOS
        outs = self.out[:L * S * qe].view(L, S, qe)
        for row, r in enumerate(self.running):
            if finished(r) and r.rid in self.sample_ids:
                self.samples.append((r.rid, r.ctx, outs[:, row, :].cpu().numpy().view(np.uint16).copy()))
        # retire (a finished request's row is taken by the last row)
        row = 0
        while row < len(self.running):
            r = self.running[row]
            if finished(r):
                pie.pie_block_free(self.pool, np.array(r.blocks, dtype=np.int32))
                last = len(self.running) - 1
                if row != last:
                    self.running[row] = self.running[last]
                    self.bt_host[row] = self.bt_host[last]
                    self.bt_dev[row].copy_(torch.from_numpy(self.bt_host[row]))
                self.running.pop()
                continue
            row += 1
        return st["last_step_ms"]

    def close(self):
        if self.pool:
            pie.pie_pool_destroy(self.pool)
            self.pool = None


def run(driver: Driver, requests, max_steps=100000, emit=None):
    """Serve the requests; -> summary dict.  Time advances by the CUDA-event time of the decode steps."""
    pending = collections.deque(sorted(requests, key=lambda r: r.arrival))
    waiting: collections.deque = collections.deque()
    now, steps, tokens, done = 0.0, 0, 0, 0
    win_t, win_tok, latencies = 0.0, 0, []
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    while steps < max_steps and (pending or waiting or driver.running):
        while pending and pending[0].arrival <= now:
            waiting.append(pending.popleft())
        if not driver.running and not waiting:
            now = pending[0].arrival                      # idle until the next arrival
            continue
        while waiting and len(driver.running) < driver.max_seqs and driver.try_admit(waiting[0]):
            waiting.popleft()
        if not driver.running:
            # nothing fits although nothing runs: the request is larger than the GPU pool
            raise RuntimeError("a request's prompt does not fit the GPU pool")
        S = len(driver.running)
        before = {r.rid: r for r in driver.running}
        ev0.record()
        driver.step()
        ev1.record()
        torch.cuda.synchronize()
        dt = ev0.elapsed_time(ev1) * 1e-3
        now += dt
        steps += 1
        tokens += S
        win_t += dt
        win_tok += S
        still = {r.rid for r in driver.running}
        for rid, r in before.items():
            if rid not in still:
                done += 1
                latencies.append(now - r.arrival)
        if steps % driver.window == 0:
            tps = win_tok / win_t
            pie.pie_report_throughput(driver.pool, tps)
            st = pie.pie_get_stats(driver.pool)
            row = {"t": now, "step": steps, "running": len(driver.running), "waiting": len(waiting), "done": done,
                   "tokens_per_s": tps, "ratio": pie.pie_get_extension_ratio(driver.pool), "ratio_floor": st["ratio_floor"],
                   "cap": st["governor_cap"], "governor": int(st["governor_state"]), "ms_per_step": 1e3 * win_t / driver.window,
                   "swap_in_gb": st["bytes_in"] / 1e9, "swap_out_gb": st["bytes_out"] / 1e9}
            driver.log.append(row)
            if emit:
                emit(row)
            win_t, win_tok = 0.0, 0
    return {"steps": steps, "tokens": tokens, "done": done, "gpu_seconds": now, "tokens_per_s": tokens / max(now, 1e-9),
            "mean_latency_s": float(np.mean(latencies)) if latencies else None, "left_waiting": len(waiting) + len(pending),
            "left_running": len(driver.running)}


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--rate", type=float, default=1.0, help="arrival rate in units of the estimated service capacity")
    ap.add_argument("--requests", type=int, default=200)
    ap.add_argument("--kv-gb", type=float, default=2.0, help="size of the GPU pool")
    ap.add_argument("--host-frac", type=float, default=0.25, help="host pool as a fraction of the GPU pool")
    ap.add_argument("--kept-copies", action="store_true")
    ap.add_argument("--kv-fp8", action="store_true", help="8-bit KV blocks")
    ap.add_argument("--max-steps", type=int, default=4000)
    ap.add_argument("--out", default=None)
    args = ap.parse_args(argv)
    out = open(args.out, "w") if args.out else sys.stdout

    def emit(o):
        out.write(json.dumps(o) + "\n")
        out.flush()

    sh = Shape(kv_fp8=args.kv_fp8)
    block_bytes = 2 * 16 * sh.n_kv_heads * sh.head_dim * (1 if sh.kv_fp8 else 2)
    gpu_blocks = int(args.kv_gb * 1e9 / (sh.n_layers * block_bytes))
    # service capacity, roughly: a full pool holds gpu_blocks * 16 tokens; a request holds prompt + out/2 tokens for out steps
    mean_tokens, mean_out = 600 * np.exp(0.6 ** 2 / 2) + 48, 96.0
    conc = min(128, gpu_blocks * 16 / mean_tokens)
    step_s = 40e-6 * sh.n_layers + conc * mean_tokens * sh.n_layers * 2 * sh.n_kv_heads * sh.head_dim * (1 if sh.kv_fp8 else 2) / 5.5e12
    capacity = conc / (mean_out * step_s)                  # requests per GPU second
    reqs = make_requests(5, args.requests, 1.0 / (args.rate * capacity))
    d = Driver(sh, gpu_blocks, int(args.host_frac * gpu_blocks), kept_copies=args.kept_copies)
    emit({"shape": dataclasses.asdict(sh), "gpu_blocks_per_layer": gpu_blocks, "block_bytes": block_bytes, "rate": args.rate,
          "capacity_req_per_s": capacity, "requests": args.requests, "kept_copies": args.kept_copies})
    emit(run(d, reqs, args.max_steps, emit))
    d.close()


if __name__ == "__main__":
    main()
