"""Swap microbenchmark (the analogue of the paper's Figure 1 link measurement, Section 2.4) and the
hidden-swap measurement: how much host-link traffic the swap path moves behind a looping decode-attention
kernel, and what that costs the kernel.

    python -m paper_2411_09317_b200.microbench [--quick] [--out FILE]

Blocks are 16 tokens x 8 KV heads x 128 dims of bf16 K+V (64 KiB).  Part 1: 1..8192 blocks per call,
contiguous vs randomly scattered slot ids, host-to-device / device-to-host / both, gather-scatter kernel vs
copy engine (one cudaMemcpyAsync per run of consecutive slots), against a pinned-memcpy probe of the link.
Part 2: the same swap calls issued once per launch of a 128-sequence x 4096-token GQA (32/8 heads) decode
attention on another stream; reports swap GB/s per direction and the attention slowdown.
Prints one JSON object per line.
"""
from __future__ import annotations

import argparse
import json
import sys

import numpy as np
import torch

from . import binding as pie
from . import synth
from .harness import DeviceWorkload


def swap_lists(n, pattern, n_pool, seed):
    if pattern == "contiguous":
        return np.arange(n, dtype=np.int32), np.arange(n, dtype=np.int32)
    src = synth.seeded_permutation(seed, n_pool, salt=1)[:n].astype(np.int32)
    dst = synth.seeded_permutation(seed, n_pool, salt=2)[:n].astype(np.int32)
    return src, dst


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--out", default=None)
    ap.add_argument("--seqs", type=int, default=128)
    ap.add_argument("--ctx", type=int, default=4096)
    ap.add_argument("--swap-ctas", type=int, default=0)
    ap.add_argument("--part", default="12", help="1 swap alone, 2 behind attention, 3 prefill-side write, 4 pairings of movers for the two directions")
    ap.add_argument("--q-heads", type=int, default=32)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--fp16", action="store_true", help="fp16 instead of bf16")
    ap.add_argument("--kv-fp8", action="store_true", help="8-bit KV blocks (the attention beside the swaps, and part 3's write)")
    ap.add_argument("--blocks", default="", help="comma list of blocks per launch for part 2")
    ap.add_argument("--every", type=int, default=1, help="part 2: one swap call per this many launches, carrying as many times the blocks")
    args = ap.parse_args(argv)
    out = open(args.out, "w") if args.out else sys.stdout

    def emit(obj):
        out.write(json.dumps(obj) + "\n")
        out.flush()

    n_swap_slots = 16384 if not args.quick else 2048
    wl = synth.Workload("swap_attn", 4, 1, args.q_heads, args.kv_heads, 128, synth.F16 if args.fp16 else synth.BF16,
                        np.full(args.seqs, args.ctx, dtype=np.int32), 0, 0.0, kv_fp8=args.kv_fp8)
    dw = DeviceWorkload(wl, host_frac=0.0, timing=False, extra_gpu_slots=n_swap_slots, extra_host_slots=n_swap_slots,
                        swap_ctas=args.swap_ctas, extra_tokens=0)
    BB = wl.block_bytes
    gpu_lo = dw.n_gpu_slots - n_swap_slots     # the swap region: slots never handed to a unit
    host_lo = dw.n_host_slots - n_swap_slots
    link = {"h2d": pie.pie_probe_link(256 << 20, pie.PIE_H2D, 3), "d2h": pie.pie_probe_link(256 << 20, pie.PIE_D2H, 3),
            "both_per_dir": pie.pie_probe_link(256 << 20, 2, 3)}
    emit({"probe": "pinned cudaMemcpyAsync 256 MiB", **link, "block_bytes": BB})
    s_in, s_out, s_c = dw.s_in, dw.s_out, dw.s_compute

    def do_swap(direction, src, dst, mode):
        if direction == "h2d":
            pie.pie_swap_raw(dw.pool, pie.PIE_H2D, src + host_lo, dst + gpu_lo, mode, s_in.cuda_stream)
        else:
            pie.pie_swap_raw(dw.pool, pie.PIE_D2H, src + gpu_lo, dst + host_lo, mode, s_out.cuda_stream)

    # ---------------------------------------------------------------- part 1: swap alone
    if "1" in args.part:
        sizes = [1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096, 8192]
        if args.quick:
            sizes = [1, 16, 256, 2048]
        for pattern in ("contiguous", "scattered"):
            for direction in ("h2d", "d2h", "both"):
                for mode, mname in ((pie.PIE_MODE_KERNEL, "kernel"), (pie.PIE_MODE_KERNEL_BULK, "bulk_kernel"),
                                    (pie.PIE_MODE_COPY_ENGINE, "copy_engine")):
                    for n in sizes:
                        if n > n_swap_slots:
                            continue
                        src, dst = swap_lists(n, pattern, n_swap_slots, 100 + n)
                        reps = 3 if n >= 1024 else 8
                        best = None
                        for r in range(reps + 1):
                            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                            torch.cuda.synchronize()
                            e0.record(s_in)
                            s_out.wait_event(e0)
                            if direction in ("h2d", "both"):
                                do_swap("h2d", src, dst, mode)
                            e1.record(s_in)
                            if direction in ("d2h", "both"):
                                do_swap("d2h", src, dst, mode)
                            e2.record(s_out)
                            torch.cuda.synchronize()
                            ms = max(e0.elapsed_time(e1), e0.elapsed_time(e2))
                            if r > 0:
                                best = ms if best is None else min(best, ms)
                        gbs = n * BB / (best * 1e-3) / 1e9
                        ref = link["both_per_dir"] if direction == "both" else link[direction]
                        emit({"part": "swap_alone", "pattern": pattern, "dir": direction, "mode": mname, "blocks": n,
                              "bytes": n * BB, "ms": best, "gbs_per_dir": gbs, "frac_of_link": gbs / ref})

    # ---------------------------------------------------------------- part 2: behind attention
    if "2" in args.part:
        def attn_loop(n_launch, per_launch=None):
            """n_launch attention calls back to back; per_launch(i) may enqueue swaps.  -> ms per launch"""
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            dw.sync()
            e0.record(s_c)
            s_in.wait_event(e0)
            s_out.wait_event(e0)
            for i in range(n_launch):
                if per_launch:
                    per_launch(i)
                dw.attention(0)
            e1.record(s_c)
            ei, eo = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ei.record(s_in)
            eo.record(s_out)
            dw.sync()
            return e0.elapsed_time(e1) / n_launch, max(e0.elapsed_time(ei), e0.elapsed_time(eo)) / n_launch

        n_launch = 30 if args.quick else 60
        attn_loop(5)
        base = [attn_loop(n_launch)[0] for _ in range(3)]
        t0 = float(np.median(base))
        kv_bytes = dw.attention_bytes_per_layer()
        emit({"part": "attention_alone", "ms_per_launch": t0, "gbs": kv_bytes / (t0 * 1e-3) / 1e9, "runs": base})
        blocks = [8, 16, 32, 64, 128, 192, 256, 384] if not args.quick else [32, 128]
        if args.blocks:
            blocks = [int(x) for x in args.blocks.split(",")]
        for pattern in ("contiguous", "scattered"):
            for mode, mname in ((pie.PIE_MODE_KERNEL, "kernel"), (pie.PIE_MODE_KERNEL_BULK, "bulk_kernel"),
                                (pie.PIE_MODE_COPY_ENGINE, "copy_engine")):
                for direction in ("h2d", "d2h", "both"):
                    for n in blocks:
                        src, dst = swap_lists(n * args.every, pattern, n_swap_slots, 200 + n)

                        def per_launch(i):
                            if i % args.every:
                                return
                            if direction in ("h2d", "both"):
                                do_swap("h2d", src, dst, mode)
                            if direction in ("d2h", "both"):
                                do_swap("d2h", src, dst, mode)

                        t1, t_swap = attn_loop(n_launch, per_launch)
                        t0b = attn_loop(n_launch)[0]   # A/B/A: re-measure the baseline next to it
                        ref = 0.5 * (t0 + t0b)
                        gbs = n * BB / (max(t1, t_swap) * 1e-3) / 1e9
                        lref = link["both_per_dir"] if direction == "both" else link[direction]
                        emit({"part": "behind_attention", "pattern": pattern, "mode": mname, "dir": direction, "blocks_per_launch": n,
                              "swap_call_every": args.every,
                              "attn_ms": t1, "attn_ms_alone": ref, "slowdown": t1 / ref - 1.0, "swap_gbs_per_dir": gbs,
                              "frac_of_link": gbs / lref, "swap_keeps_up": t_swap <= t1 * 1.02})
    # ---------------------------------------------------------------- part 3: prefill-side KV write
    if "3" in args.part:
        # every position of every sequence of the attention workload, one layer, in one call: reads the K/V rows once
        # and writes them once (HBM-bound scatter of 2 * head_dim * 2-byte pieces)
        ctx = dw.ctx_lens.astype(np.int64)
        seq = np.repeat(np.arange(wl.n_seqs, dtype=np.int32), ctx)
        pos = np.concatenate([np.arange(c, dtype=np.int32) for c in ctx])
        T = len(seq)
        k = torch.empty((T, wl.n_kv_heads, wl.head_dim), dtype=torch.int16, device=dw.dev)
        v = torch.empty_like(k)
        lib = pie.synth_lib()
        for t_, stream in ((k, synth.STREAM_KNEW), (v, synth.STREAM_VNEW)):
            base = int(synth.stream_base(wl.seed, stream)) & 0xFFFFFFFFFFFFFFFF
            assert lib.pie_synth_fill_tensor(t_.data_ptr(), t_.numel(), base, 0, wl.dtype, 1.0, None) == 0
        seq_d, pos_d = torch.from_numpy(seq).to(dw.dev), torch.from_numpy(pos).to(dw.dev)
        torch.cuda.synchronize()
        times = []
        for r in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(s_c)
            pie.pie_kv_write(dw.pool, r % wl.n_layers, k.data_ptr(), v.data_ptr(), seq_d.data_ptr(), pos_d.data_ptr(), T,
                             dw.block_table_dev.data_ptr(), dw.max_blocks, wl.n_seqs)
            e1.record(s_c)
            dw.sync()
            times.append(e0.elapsed_time(e1))
        ms = float(np.median(times[1:]))
        # K and V rows read once (16-bit) and written once (16-bit, or one byte per value into an 8-bit pool)
        nbytes = 2 * T * wl.n_kv_heads * wl.head_dim * (2 + (1 if wl.kv_fp8 else 2))
        emit({"part": "kv_write", "tokens": T, "ms": ms, "gbs_read_plus_write": nbytes / (ms * 1e-3) / 1e9, "bytes": nbytes})
    # ---------------------------------------------------------------- part 4: both directions at once, every pairing of who moves
    # which direction (does host traffic issued by SMs slow the other direction down, whoever moves that one?)
    if "4" in args.part:
        n = 4096 if not args.quick else 1024
        modes = {"bulk_kernel": pie.PIE_MODE_KERNEL_BULK, "kernel": pie.PIE_MODE_KERNEL, "copy_engine": pie.PIE_MODE_COPY_ENGINE}
        for pattern in ("contiguous", "scattered"):
            src, dst = swap_lists(n, pattern, n_swap_slots, 100 + n)
            for m_in in (None, "bulk_kernel", "kernel", "copy_engine"):
                for m_out in (None, "bulk_kernel", "kernel", "copy_engine"):
                    if m_in is None and m_out is None:
                        continue
                    best = None
                    for r in range(4):
                        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                        torch.cuda.synchronize()
                        e0.record(s_in)
                        s_out.wait_event(e0)
                        if m_in:
                            pie.pie_swap_raw(dw.pool, pie.PIE_H2D, src + host_lo, dst + gpu_lo, modes[m_in], s_in.cuda_stream)
                        e1.record(s_in)
                        if m_out:
                            pie.pie_swap_raw(dw.pool, pie.PIE_D2H, src + gpu_lo, dst + host_lo, modes[m_out], s_out.cuda_stream)
                        e2.record(s_out)
                        torch.cuda.synchronize()
                        ms = max(e0.elapsed_time(e1), e0.elapsed_time(e2))
                        if r > 0:
                            best = ms if best is None else min(best, ms)
                    emit({"part": "swap_pairings", "pattern": pattern, "blocks": n, "in": m_in, "out": m_out, "swap_ctas": args.swap_ctas,
                          "gbs_per_dir": n * BB / (best * 1e-3) / 1e9})
    dw.close()


if __name__ == "__main__":
    main()
