"""Throughput of the chunked-prefill attention kernel (pie_prefill_attention, tcgen05 / TMEM) on synthetic shapes.

    python -m paper_2411_09317_b200.prefill_bench [--hq 32 --hkv 8 --seqs 16 --chunk 1024 --prefix 3072 --dtype 1]

A batch of `seqs` sequences, each with `prefix` cached tokens and a chunk of `chunk` query tokens behind them; K, V and q
are N(0,1) drawn on the device.  Prints one JSON line: time per call (CUDA events, mean of `reps` calls after 3 warm-up
calls), TFLOP/s over the algorithmic flops 4 * Hq * D * sum over chunk tokens of (position + 1) (the causal part counted as
what it needs, not as the tiles the kernel runs), and the largest difference from a plain fp32 evaluation of one head
(a sanity check beside the parity tests, which use the oracle).
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as pie
from . import synth


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--hq", type=int, default=32)
    ap.add_argument("--hkv", type=int, default=8)
    ap.add_argument("--head-dim", type=int, default=128)
    ap.add_argument("--seqs", type=int, default=16)
    ap.add_argument("--chunk", type=int, default=1024)
    ap.add_argument("--prefix", type=int, default=3072)
    ap.add_argument("--dtype", type=int, default=synth.BF16, help="0 fp16, 1 bf16")
    ap.add_argument("--reps", type=int, default=10)
    a = ap.parse_args(argv)
    D = a.head_dim
    dev = torch.device("cuda", torch.cuda.current_device())
    tdt = torch.bfloat16 if a.dtype == synth.BF16 else torch.float16
    ctx = np.full(a.seqs, a.prefix + a.chunk, np.int32)
    nblk = (ctx + 15) // 16
    NB, maxb = int(nblk.sum()), int(nblk.max())
    bt = np.zeros((a.seqs, maxb), np.int32)
    perm = synth.seeded_permutation(7, NB)     # scattered blocks, as a serving pool would have them
    k = 0
    for s in range(a.seqs):
        bt[s, :nblk[s]] = perm[k:k + nblk[s]]
        k += nblk[s]
    pool = pie.pie_pool_create(n_layers=1, n_q_heads=a.hq, n_kv_heads=a.hkv, head_dim=D, dtype=a.dtype, n_logical_blocks=NB,
                               max_seqs=a.seqs, n_gpu_slots=NB + 8, n_host_slots=8, timing=0)
    pie.pie_block_alloc(pool, NB, np.zeros(NB, np.uint8))
    torch.manual_seed(0)
    n_tok, n_kv = a.seqs * a.chunk, int(ctx.sum())
    q = torch.randn((n_tok, a.hq, D), device=dev).to(tdt)
    out = torch.empty_like(q)
    kk, vv = torch.randn((n_kv, a.hkv, D), device=dev).to(tdt), torch.randn((n_kv, a.hkv, D), device=dev).to(tdt)
    off = (np.arange(a.seqs + 1) * a.chunk).astype(np.int32)
    bt_d, ctx_d, off_d = torch.from_numpy(bt).to(dev), torch.from_numpy(ctx).to(dev), torch.from_numpy(off).to(dev)
    tseq = torch.from_numpy(np.repeat(np.arange(a.seqs), ctx).astype(np.int32)).to(dev)
    tpos = torch.from_numpy(np.concatenate([np.arange(c) for c in ctx]).astype(np.int32)).to(dev)
    pie.pie_kv_write(pool, 0, kk.data_ptr(), vv.data_ptr(), tseq.data_ptr(), tpos.data_ptr(), n_kv, bt_d.data_ptr(), maxb, a.seqs)
    pie.pie_sync(pool)
    stream = torch.cuda.current_stream()

    def call():
        pie.pie_prefill_attention(pool, 0, q.data_ptr(), out.data_ptr(), bt_d.data_ptr(), maxb, ctx_d.data_ptr(), off_d.data_ptr(),
                                  ctx, off, a.seqs, 1.0 / float(np.sqrt(D)))

    for _ in range(3):
        call()
    pie.pie_sync(pool)
    import time
    t0 = time.perf_counter()       # the pool's own compute stream carries the kernels: host clock around synchronised calls
    for _ in range(a.reps):
        call()
    pie.pie_sync(pool)
    ms = (time.perf_counter() - t0) * 1e3 / a.reps
    flops = a.seqs * 4.0 * a.hq * D * float((a.prefix + np.arange(a.chunk) + 1).sum())
    g = a.hq // a.hkv
    sc = (q[:a.chunk, 0].float() @ kk[:ctx[0], 0].float().T) / float(np.sqrt(D))
    mask = torch.arange(int(ctx[0]), device=dev)[None, :] <= (a.prefix + torch.arange(a.chunk, device=dev))[:, None]
    ref = torch.softmax(sc.masked_fill(~mask, float("-inf")), -1) @ vv[:ctx[0], 0].float()
    err = (out[:a.chunk, 0].float() - ref).abs().max().item()
    print(json.dumps({"n_q_heads": a.hq, "n_kv_heads": a.hkv, "head_dim": D, "seqs": a.seqs, "chunk": a.chunk, "prefix": a.prefix,
                      "dtype": "bf16" if a.dtype == synth.BF16 else "f16", "ms_per_call": ms, "tflops": flops / (ms * 1e-3) / 1e12,
                      "kv_gb": n_kv * 2 * a.hkv * D * 2 / 1e9, "group": g, "max_abs_diff_vs_fp32_one_head": err}))
    pie.pie_pool_destroy(pool)


if __name__ == "__main__":
    main()
