"""Ratio sweep and controller trajectory on the larger workload shapes (the synthetic counterpart of the paper's
throughput-versus-expansion and adaptive-expansion experiments, Section 5.2 and 5.4; no request stream here, so
what is reported is the decode step itself).

    python -m paper_2411_09317_b200.sweep --workload llama3_8b  --mode ratios   [--layers N] [--steps K]
    python -m paper_2411_09317_b200.sweep --workload llama3_70b --mode adaptive [--layers N] [--steps K]

ratios:   the extension ratio is set to 0, 0.1, ... 1.0 (fraction of every layer's blocks kept host resident
          between uses); per ratio: median step time, attention GB/s, swap GB/s per direction, share of the step
          the computation spent waiting for blocks.
adaptive: the controller owns the ratio.  --host-frac 0.5 (default): half of the blocks start host resident and the GPU
          pool holds only the other half, so the ratio has a floor; --host-frac 0: everything starts on the GPU and the
          ratio climbs from 0 until waits or slow-down appear.  Per step: ratio, floor, step time, wait share.
expansion: tokens per second against expansion (the batch grows, the GPU pool does not; --ratios lists expansions).
layers:   whole layers on the CPU (the paper's protocol, Section 3.3) against the same share of every layer's blocks.
interference: adaptive, with foreign pinned-memory traffic on the host link during the middle third of the run.
Prints one JSON object per line.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import sys

import numpy as np
import torch

from . import binding as pie
from . import synth
from .harness import DeviceWorkload


OTHER = {"fn": None}   # stand-in for a model's other per-layer work (--other-mb): called after every layer's attention
SWAP_MODE = {"mode": pie.PIE_MODE_AUTO}   # --swap-mode: how swap lists are moved


def run_steps(dw, n):
    """n decode steps; -> (per-step ms by CUDA events, stats before, stats after, context lengths before)"""
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    dw.sync()
    dw.advance_context()
    dw.decode_step(between_layers=OTHER["fn"], mode=SWAP_MODE["mode"])
    before, ctx0 = pie.pie_get_stats(dw.pool), dw.ctx_lens.copy()
    with torch.cuda.stream(dw.s_compute):
        marks[0].record()
    per_stats = []
    for i in range(n):
        dw.advance_context()
        dw.decode_step(between_layers=OTHER["fn"], mode=SWAP_MODE["mode"])
        per_stats.append(pie.pie_get_stats(dw.pool))
        with torch.cuda.stream(dw.s_compute):
            marks[i + 1].record()
    dw.sync()
    pie.pie_controller_tick(dw.pool)
    return [marks[i].elapsed_time(marks[i + 1]) for i in range(n)], before, pie.pie_get_stats(dw.pool), ctx0, per_stats


def attention_bytes(wl, ctx):
    ctx = ctx.astype(np.int64)
    return wl.n_layers * (int(ctx.sum()) * 2 * wl.n_kv_heads * wl.head_dim * (1 if wl.kv_fp8 else 2) + 2 * wl.n_seqs * wl.n_q_heads * wl.head_dim * 2
                          + 4 * (int(((ctx + 15) // 16).sum()) + wl.n_seqs))


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="llama3_8b")
    ap.add_argument("--mode", default="ratios", choices=["ratios", "adaptive", "interference", "layers", "expansion"])
    ap.add_argument("--cpu-layers", default="1,2,4", help="layers: numbers of layers kept on the CPU, comma list")
    ap.add_argument("--background-mb", type=int, default=256,
                    help="interference: pinned-memory traffic per step and direction on two other streams, MB")
    ap.add_argument("--layers", type=int, default=0, help="use only this many layers (smaller pools)")
    ap.add_argument("--steps", type=int, default=6)
    ap.add_argument("--ratios", default="", help="ratios: comma list instead of 0, 0.1, ... 1.0")
    ap.add_argument("--host-frac", type=float, default=0.5, help="adaptive: share of the blocks that starts host resident")
    ap.add_argument("--ctrl-step", type=float, default=1.0 / 64.0, help="adaptive: the controller's ratio step")
    ap.add_argument("--kept-copies", action="store_true",
                    help="host copies are kept after a swap-in and the write-back of unwritten blocks is skipped (pie_set_retention)")
    ap.add_argument("--other-mb", type=int, default=0,
                    help="ratios / adaptive: after every layer's attention, an elementwise kernel that reads and writes this many MB "
                         "on the compute stream stands in for the model's projections and MLP (weights streamed from HBM); the "
                         "step then runs layer by layer through pie_decode_layer")
    ap.add_argument("--swap-mode", default="auto", choices=["auto", "kernel", "copy_engine", "bulk_kernel"],
                    help="how swap lists are moved (PIE_MODE_*)")
    ap.add_argument("--lookahead", type=int, default=0, help="layers per prefetch group (pie_set_lookahead; 0: the library chooses)")
    ap.add_argument("--run-ahead", type=int, default=1, help="decode steps the host may be ahead of the GPU (pie_set_run_ahead)")
    ap.add_argument("--split", type=int, default=0, help="split-K chunk in tokens (0: the library's default)")
    ap.add_argument("--attn-variant", type=int, default=0, help="attention kernel variant (tuning)")
    ap.add_argument("--kv-fp8", action="store_true", help="blocks of E4M3 bytes (half the bytes per token; head_dim 128)")
    ap.add_argument("--out", default=None)
    args = ap.parse_args(argv)
    out = open(args.out, "w") if args.out else sys.stdout

    def emit(obj):
        out.write(json.dumps(obj) + "\n")
        out.flush()

    SWAP_MODE["mode"] = {"auto": pie.PIE_MODE_AUTO, "kernel": pie.PIE_MODE_KERNEL, "copy_engine": pie.PIE_MODE_COPY_ENGINE,
                         "bulk_kernel": pie.PIE_MODE_KERNEL_BULK}[args.swap_mode]
    if args.other_mb > 0:
        # an elementwise kernel, not a memcpy: a device-to-device cudaMemcpyAsync may be served by the copy engines,
        # which the swaps need
        w_src = torch.zeros((args.other_mb << 20) // 4, dtype=torch.float32, device="cuda")
        w_dst = torch.empty_like(w_src)
        OTHER["fn"] = lambda l: torch.add(w_src, 1.0, out=w_dst)
    wl = synth.workload(args.workload)
    if args.kv_fp8:
        wl = dataclasses.replace(wl, kv_fp8=True)
    if args.layers:
        wl = dataclasses.replace(wl, n_layers=args.layers)
    L = wl.n_layers
    link = {"h2d": pie.pie_probe_link(256 << 20, pie.PIE_H2D, 3), "d2h": pie.pie_probe_link(256 << 20, pie.PIE_D2H, 3),
            "both_per_dir": pie.pie_probe_link(256 << 20, 2, 3)}
    if args.mode == "interference":
        interference(args, wl, link, emit)
        return
    if args.mode == "expansion":
        emit({"workload": args.workload, "layers": L, "base_seqs": wl.n_seqs, "block_bytes": wl.block_bytes, "kept_copies": args.kept_copies,
              "other_mb_per_layer": args.other_mb, "link": link})
        expansion_throughput(args, wl, link, emit)
        return
    if args.mode == "layers":
        layers_vs_blocks(args, wl, link, emit)
        return
    if args.mode == "ratios":
        ratios = [float(x) for x in args.ratios.split(",")] if args.ratios else [round(0.1 * i, 1) for i in range(11)]
        total = len(ratios) * (args.steps + 4) + 4
        wl = dataclasses.replace(wl, decode_steps=total)
        _, _, nb = wl.tables()
        # both pools can hold everything: ratio 0 needs it on the GPU side, ratio 1 on the host side
        dw = DeviceWorkload(wl, host_frac=0.0, timing=True, extra_gpu_slots=3 * nb + 64, extra_host_slots=(L + 3) * nb + 64,
                            split_tokens=args.split, attn_variant=args.attn_variant)
        dw.set_retention(args.kept_copies)
        pie.pie_set_lookahead(dw.pool, args.lookahead)
        pie.pie_set_run_ahead(dw.pool, args.run_ahead)
        emit({"workload": args.workload, "layers": L, "seqs": wl.n_seqs, "blocks_per_layer": nb, "block_bytes": wl.block_bytes,
              "kv_gb": L * nb * wl.block_bytes / 1e9, "kept_copies": args.kept_copies, "other_mb_per_layer": args.other_mb,
              "lookahead": args.lookahead,
              "link": link})
        first_gbs = None
        for r in ratios:
            pie.pie_set_extension_ratio(dw.pool, r)
            run_steps(dw, 2)
            per, sb, sa, ctx0, _ = run_steps(dw, args.steps)
            ms = float(np.median(per))
            tot = sum(per) * 1e-3
            by = attention_bytes(wl, ctx0 + (args.steps + 1) // 2)
            first_gbs = first_gbs or by / (ms * 1e-3) / 1e9
            emit({"ratio": r,
                  # the context grows a token per sequence per step: rows are comparable in bytes per second, not in ms
                  "slowdown_vs_first_row_at_equal_context": first_gbs / (by / (ms * 1e-3) / 1e9) - 1.0, "expansion": None if r >= 1.0 else 1.0 / (1.0 - r), "ms_per_step": ms,
                  "attn_gbs": by / (ms * 1e-3) / 1e9, "swap_in_gbs": (sa["bytes_in"] - sb["bytes_in"]) / tot / 1e9,
                  "swap_out_gbs": (sa["bytes_out"] - sb["bytes_out"]) / tot / 1e9,
                  "wait_share": sa["last_step_stall_ms"] / max(sa["last_step_ms"], 1e-9),
                  "last_step": {k: sa[k] for k in ("last_step_ms", "last_step_compute_ms", "last_step_stall_ms",
                                                   "last_step_swap_in_ms", "last_step_swap_out_ms")},
                  "elided_out_gbs": (sa["bytes_out_elided"] - sb["bytes_out_elided"]) / tot / 1e9,
                  "calls_kernel": sa["calls_kernel"] - sb["calls_kernel"],
                  "calls_copy_engine": sa["calls_copy_engine"] - sb["calls_copy_engine"],
                  "swap_frac_of_link": (sa["bytes_in"] - sb["bytes_in"]) / tot / 1e9 / link["both_per_dir"]})
    else:
        wl = dataclasses.replace(wl, decode_steps=args.steps + 8)
        _, _, nb = wl.tables()
        # host_frac > 0: the GPU pool is sized for the GPU-resident share only (the ratio cannot go below that share);
        # host_frac = 0: everything fits, the host pool has room for a quarter of the blocks and the ratio climbs from 0
        extra_host = 0 if args.host_frac > 0 else (L // 4 + 3) * nb
        dw = DeviceWorkload(wl, host_frac=args.host_frac, timing=True, extra_host_slots=extra_host,
                            extra_gpu_slots=0 if args.host_frac > 0 else 3 * nb)
        emit({"workload": args.workload, "layers": L, "seqs": wl.n_seqs, "blocks_per_layer": nb, "block_bytes": wl.block_bytes,
              "kv_gb": L * nb * wl.block_bytes / 1e9, "gpu_pool_gb": dw.n_gpu_slots * wl.block_bytes / 1e9,
              "host_pool_gb": dw.n_host_slots * wl.block_bytes / 1e9, "host_frac": args.host_frac,
              "ctrl_step": args.ctrl_step, "link": link})
        dw.set_retention(args.kept_copies)
        pie.pie_set_controller(dw.pool, args.ctrl_step, 0.0, 0.0)
        pie.pie_set_extension_ratio(dw.pool, -1.0)
        per, sb, sa, ctx0, per_stats = run_steps(dw, args.steps)
        for i, (ms, st) in enumerate(zip(per, per_stats)):
            emit({"step": i, "ratio": st["ratio"], "ratio_floor": st["ratio_floor"], "ms_per_step": ms,
                  "wait_share_of_last_measured_step": st["last_step_stall_ms"] / max(st["last_step_ms"], 1e-9),
                  "slowdown_share_of_last_measured_step": st["last_step_slowdown_ms"] / max(st["last_step_compute_ms"], 1e-9)})
        tot = sum(per) * 1e-3
        emit({"summary": True, "final_ratio": sa["ratio"], "ratio_floor": sa["ratio_floor"], "median_ms_per_step": float(np.median(per)),
              "swap_in_gbs": (sa["bytes_in"] - sb["bytes_in"]) / tot / 1e9, "swap_out_gbs": (sa["bytes_out"] - sb["bytes_out"]) / tot / 1e9,
              "attn_gbs": attention_bytes(wl, ctx0 + args.steps // 2) / (float(np.median(per)) * 1e-3) / 1e9})
    dw.close()


def layers_vs_blocks(args, wl, link, emit):
    """The paper's unit against this build's: m whole layers live on the CPU and rotate through n - m GPU regions and
    m + 2 CPU regions first in, first out (Section 3.3, pie_set_layer_policy) - against the same share m / n of every
    layer's blocks (the block-granular plan at extension ratio m / n).  Same bytes per token either way."""
    L = wl.n_layers
    ms_list = [int(x) for x in args.cpu_layers.split(",")]
    wl = dataclasses.replace(wl, decode_steps=len(ms_list) * 2 * (args.steps + 6) + 8)
    _, _, nb = wl.tables()
    m_max = max(ms_list)
    dw = DeviceWorkload(wl, host_frac=0.0, timing=True, extra_gpu_slots=3 * nb + 64, extra_host_slots=(2 * m_max + 6) * nb + 64)   # room for the change-over between the two plans
    emit({"workload": args.workload, "layers": L, "seqs": wl.n_seqs, "blocks_per_layer": nb, "block_bytes": wl.block_bytes,
          "kv_gb": L * nb * wl.block_bytes / 1e9, "link": link})
    ids = np.arange(nb, dtype=np.int32)
    for m in ms_list:
        # whole layers: the last m layers wholly onto the host, then the protocol takes over
        pie.pie_set_extension_ratio(dw.pool, 0.0)
        run_steps(dw, 2)                      # everything back on the GPU
        for l in range(L - m, L):
            pie.pie_swap_out(dw.pool, l, ids)
        dw.sync()
        pie.pie_set_layer_policy(dw.pool, L - m, m + 2)
        run_steps(dw, 2)
        per, sb, sa, ctx0, _ = run_steps(dw, args.steps)
        tot = sum(per) * 1e-3
        row = {"cpu_layers": m, "ratio": m / L, "whole_layers": {
            "ms_per_step": float(np.median(per)), "swap_in_gbs": (sa["bytes_in"] - sb["bytes_in"]) / tot / 1e9,
            "swap_out_gbs": (sa["bytes_out"] - sb["bytes_out"]) / tot / 1e9,
            "gb_in_per_step": (sa["bytes_in"] - sb["bytes_in"]) / args.steps / 1e9}}
        pie.pie_set_layer_policy(dw.pool, 0, 0)
        pie.pie_set_extension_ratio(dw.pool, m / L)
        run_steps(dw, 3)                      # the block plan redistributes: every layer keeps m / n of its blocks out
        per, sb, sa, ctx0, _ = run_steps(dw, args.steps)
        tot = sum(per) * 1e-3
        row["blocks"] = {"ms_per_step": float(np.median(per)), "swap_in_gbs": (sa["bytes_in"] - sb["bytes_in"]) / tot / 1e9,
                         "swap_out_gbs": (sa["bytes_out"] - sb["bytes_out"]) / tot / 1e9,
                         "gb_in_per_step": (sa["bytes_in"] - sb["bytes_in"]) / args.steps / 1e9}
        emit(row)
    dw.close()


def expansion_throughput(args, wl, link, emit):
    """The paper's throughput-versus-expansion experiment (Section 5.4) in this build's terms: the GPU pool is fixed at what
    the base batch needs; at expansion e the batch is e times as large (more sequences of the same length mix), the
    surplus share r = 1 - 1/e of every layer's blocks lives on the host between uses, and what is reported is tokens per
    second of the decode step (sequences / step time).  No request stream: the batch is full and steady, which is the
    regime the paper's curves flatten into."""
    base = wl.n_seqs
    exps = [float(x) for x in args.ratios.split(",")] if args.ratios else [1.0, 1.02, 1.05, 1.1, 1.25, 1.5, 2.0]
    _, _, nb_base = dataclasses.replace(wl, decode_steps=args.steps + 8).tables()
    first = None
    for e in exps:
        n = max(base, int(round(base * e)))
        big = dataclasses.replace(synth.workload(args.workload, scale=n / base), n_layers=wl.n_layers, decode_steps=args.steps + 8,
                                  kv_fp8=wl.kv_fp8)
        _, _, nb = big.tables()
        r = max(0.0, 1.0 - nb_base / nb)
        h = int(np.ceil(r * nb)) + 1
        # GPU side: the base batch's blocks per layer, plus three layers' shares in transit; host side: the surplus
        dw = DeviceWorkload(big, host_frac=0.0, timing=True, split_tokens=args.split, extra_gpu_slots=0, extra_host_slots=0,
                            gpu_slots_override=wl.n_layers * nb_base + 3 * h + 64, host_slots_override=(wl.n_layers + 3) * h + 64,
                            initial_host_blocks=h if r > 0 else 0)
        dw.set_retention(args.kept_copies)
        pie.pie_set_lookahead(dw.pool, args.lookahead)
        pie.pie_set_run_ahead(dw.pool, args.run_ahead)
        pie.pie_set_extension_ratio(dw.pool, r)
        run_steps(dw, 2)
        per, sb, sa, ctx0, _ = run_steps(dw, args.steps)
        ms = float(np.median(per))
        tot = sum(per) * 1e-3
        tps = big.n_seqs / (ms * 1e-3)
        first = first or tps
        emit({"expansion": nb / nb_base, "ratio": r, "seqs": big.n_seqs, "blocks_per_layer": nb, "ms_per_step": ms,
              "tokens_per_s": tps, "vs_expansion_1": tps / first, "swap_in_gbs": (sa["bytes_in"] - sb["bytes_in"]) / tot / 1e9,
              "swap_out_gbs": (sa["bytes_out"] - sb["bytes_out"]) / tot / 1e9,
              "wait_share": sa["last_step_stall_ms"] / max(sa["last_step_ms"], 1e-9),
              "gpu_pool_gb": dw.n_gpu_slots * big.block_bytes / 1e9, "host_pool_gb": dw.n_host_slots * big.block_bytes / 1e9})
        dw.close()
        for name in ("gpu_pool", "host_pool", "q_all", "out_all", "k_new", "v_new"):
            setattr(dw, name, None)
        del dw
        import gc
        gc.collect()
        torch.cuda.empty_cache()


def interference(args, wl, link, emit):
    """Section 3.4.2, last paragraph: other traffic on the host link takes bandwidth away; the controller is expected
    to notice (waits or slow-down appear) and give ground, and to come back when the traffic stops.  Three phases of
    --steps decode steps each: quiet, with --background-mb of pinned copies per step in each direction on two streams
    of their own, quiet again."""
    L = wl.n_layers
    wl = dataclasses.replace(wl, decode_steps=3 * args.steps + 16)
    _, _, nb = wl.tables()
    dw = DeviceWorkload(wl, host_frac=0.0, timing=True, extra_host_slots=(L // 4 + 3) * nb, extra_gpu_slots=3 * nb)
    dw.set_retention(args.kept_copies)
    pie.pie_set_controller(dw.pool, args.ctrl_step, 0.0, 0.0)
    pie.pie_set_extension_ratio(dw.pool, -1.0)
    n = args.background_mb << 20
    h_src = torch.empty(n, dtype=torch.uint8).pin_memory()
    h_dst = torch.empty(n, dtype=torch.uint8).pin_memory()
    d_a = torch.empty(n, dtype=torch.uint8, device=dw.dev)
    d_b = torch.empty(n, dtype=torch.uint8, device=dw.dev)
    s_bg_in, s_bg_out = torch.cuda.Stream(device=dw.dev), torch.cuda.Stream(device=dw.dev)
    emit({"workload": args.workload, "layers": L, "seqs": wl.n_seqs, "blocks_per_layer": nb, "ctrl_step": args.ctrl_step,
          "background_mb_per_step_and_direction": args.background_mb, "kept_copies": args.kept_copies, "link": link})
    run_steps(dw, 2)
    for phase in ("quiet", "background", "quiet_again"):
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        with torch.cuda.stream(dw.s_compute):
            marks[0].record()
        sb = pie.pie_get_stats(dw.pool)
        ratios, slow = [], []
        for i in range(args.steps):
            if phase == "background":
                # one step's worth of foreign traffic, released when the step starts
                s_bg_in.wait_event(marks[i])
                s_bg_out.wait_event(marks[i])
                with torch.cuda.stream(s_bg_in):
                    d_a.copy_(h_src, non_blocking=True)
                with torch.cuda.stream(s_bg_out):
                    h_dst.copy_(d_b, non_blocking=True)
            dw.advance_context()
            dw.decode_step()
            st = pie.pie_get_stats(dw.pool)
            ratios.append(st["ratio"])
            slow.append((st["last_step_stall_ms"] + st["last_step_slowdown_ms"]) / max(st["last_step_compute_ms"], 1e-9))
            with torch.cuda.stream(dw.s_compute):
                marks[i + 1].record()
        dw.sync()
        torch.cuda.synchronize()
        sa = pie.pie_get_stats(dw.pool)
        per = [marks[i].elapsed_time(marks[i + 1]) for i in range(args.steps)]
        tot = sum(per) * 1e-3
        emit({"phase": phase, "median_ms_per_step": float(np.median(per)), "ratio_first": ratios[0], "ratio_last": ratios[-1],
              "ratio_mean": float(np.mean(ratios)), "ratio_max": float(np.max(ratios)),
              "wait_plus_slowdown_share_mean": float(np.mean(slow)),
              "swap_in_gbs": (sa["bytes_in"] - sb["bytes_in"]) / tot / 1e9, "swap_out_gbs": (sa["bytes_out"] - sb["bytes_out"]) / tot / 1e9,
              "background_gbs_per_dir": (args.background_mb * 2**20 * args.steps / tot / 1e9) if phase == "background" else 0.0,
              "ratios": [round(r, 4) for r in ratios]})
    dw.close()


if __name__ == "__main__":
    main()
