"""Oracle of chunked-prefill paged attention.  TEST INFRASTRUCTURE ONLY; shares no code with the CUDA library.

Section 2.1's prefill stage computes attention for all prompt tokens at once; with a paged cache (Section 2.2) and a
prompt fed in chunks, a chunk of C query tokens of a sequence whose context - chunk included - is ctx tokens long sits at
positions ctx - C .. ctx - 1, and its token i attends to every cached position up to its own:

    out[i][h] = sum_{t <= pos_i} softmax_t(scale * q[i][h] . K[t][kvh]) * V[t][kvh],   pos_i = ctx - C + i, kvh = h // (Hq / Hkv)

The chunk's own keys and values are in the cache already (the prefill-side write comes first).  This file is that
definition written out: gather the sequence's K and V rows through the block table, convert the 16-bit values exactly,
and evaluate the formula in fp64 (or fp32), token by token and head by head.  No blocking, no running maximum.
"""
from __future__ import annotations

import numpy as np

F16, BF16 = 0, 1


def bits_to_real(bits: np.ndarray, dtype: int, real=np.float64) -> np.ndarray:
    """fp16 / bf16 bit patterns -> their exact values (numpy's own conversions)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == F16:
        return bits.view(np.float16).astype(real)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(real)


def gather_kv(gpu_pool, host_pool, unit_side, unit_slot, blocks, ctx, n_kv_heads, head_dim, dtype, real):
    """K, V [ctx][Hkv][D] of one sequence (slot layout [Hkv][2][16][D]; a unit lives in the pool its side names)."""
    K = np.zeros((ctx, n_kv_heads, head_dim), dtype=real)
    V = np.zeros((ctx, n_kv_heads, head_dim), dtype=real)
    for j in range((ctx + 15) // 16):
        b = int(blocks[j])
        if not 0 <= b < len(unit_slot):
            raise ValueError("oracle: block id out of range")
        pool = host_pool if unit_side[b] else gpu_pool
        tile = bits_to_real(pool[int(unit_slot[b])], dtype, real).reshape(n_kv_heads, 2, 16, head_dim)
        n = min(16, ctx - 16 * j)
        K[16 * j:16 * j + n] = tile[:, 0, :n, :].transpose(1, 0, 2)
        V[16 * j:16 * j + n] = tile[:, 1, :n, :].transpose(1, 0, 2)
    return K, V


def prefill_attention(gpu_pool, host_pool, unit_side, unit_slot, q, q_offsets, block_table, ctx_lens, n_q_heads, n_kv_heads,
                      head_dim, dtype, scale, precision="f64"):
    """q: [n_tokens][Hq][D] 16-bit patterns, the chunks of all sequences one after the other; q_offsets [S + 1]: sequence
    s owns tokens q_offsets[s] .. q_offsets[s + 1] - 1; ctx_lens [S]: context lengths INCLUDING the chunk.
    -> out [n_tokens][Hq][D] in the requested precision (not rounded to 16 bits)."""
    real = np.float64 if precision == "f64" else np.float32
    q = np.ascontiguousarray(q, dtype=np.uint16).reshape(-1, n_q_heads, head_dim)
    out = np.zeros(q.shape, dtype=real)
    group = n_q_heads // n_kv_heads
    hp = host_pool if host_pool is not None else gpu_pool
    for s in range(len(ctx_lens)):
        t0, t1 = int(q_offsets[s]), int(q_offsets[s + 1])
        C, ctx = t1 - t0, int(ctx_lens[s])
        if C == 0:
            continue
        if C > ctx:
            raise ValueError("oracle: a chunk longer than its context")
        K, V = gather_kv(gpu_pool, hp, unit_side, unit_slot, block_table[s], ctx, n_kv_heads, head_dim, dtype, real)
        qs = bits_to_real(q[t0:t1], dtype, real)
        for i in range(C):
            pos = ctx - C + i
            for h in range(n_q_heads):
                kvh = h // group
                score = real(scale) * (K[:pos + 1, kvh, :] @ qs[i, h])
                p = np.exp(score - score.max())
                out[t0 + i, h] = (p / p.sum()) @ V[:pos + 1, kvh, :]
    return out
