"""Oracle of the 8-bit KV variant: blocks hold K and V as FP8 E4M3 bytes (a variant beyond the paper, whose blocks are
16-bit; it halves the bytes a token costs in HBM and on the link).

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA library.

E4M3 ("fn" flavour: no infinities): 1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits; exponent 0 is subnormal
(m / 8 * 2^-6); exponent 15 with mantissa 7 is NaN; the largest finite value is 448.  A stored byte b stands for
decode(b) * scale, with one scale for all keys and one for all values of a pool.  Attention over such blocks is, by
definition, attention over the decoded values: the oracle decodes the pools into 16-bit pools (every E4M3 value is
exactly representable in fp16 and in bf16) and calls the 16-bit oracle with the key scale folded into the softmax
scale and the value scale applied to the result.  The append quantises the new token's rows: value / scale rounded
to the nearest E4M3 value, ties to the even code, magnitudes beyond 448 saturating to 448.
"""
from __future__ import annotations

import numpy as np

import oracle

F16, BF16 = 0, 1   # the 16-bit type of q / out / the new token's rows, as in include/pie.h


def _bits16_to_f64(bits, dtype) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    if dtype == F16:
        return bits.view(np.float16).astype(np.float64)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _table() -> np.ndarray:
    t = np.zeros(256, dtype=np.float64)
    for b in range(256):
        sign = -1.0 if b & 0x80 else 1.0
        e, m = (b >> 3) & 0xF, b & 7
        if e == 15 and m == 7:
            t[b] = np.nan
        elif e == 0:
            t[b] = sign * (m / 8.0) * 2.0 ** -6
        else:
            t[b] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return t


E4M3 = _table()
_POS = E4M3[:127]            # codes 0 .. 126: the non-negative finite values, ascending


def decode(b) -> np.ndarray:
    """bytes -> float64 values (exact)"""
    return E4M3[np.asarray(b, dtype=np.uint8)]


def quantize(x) -> np.ndarray:
    """float values -> E4M3 bytes: nearest value, ties to the even code, saturating at +-448, NaN -> 0x7f"""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), 448.0)
    hi = np.clip(np.searchsorted(_POS, a, side="left"), 0, 126)      # first code whose value is >= a
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = _POS[hi] - a, a - _POS[lo]
    pick_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(pick_lo, lo, hi).astype(np.uint8)
    code = np.where(np.signbit(x), code | 0x80, code).astype(np.uint8)
    return np.where(np.isnan(x), np.uint8(0x7F), code).astype(np.uint8)


def to_bits16(b, dtype) -> np.ndarray:
    """E4M3 bytes -> the 16-bit patterns (fp16 or bf16) of the same values (exact in both formats)"""
    v = decode(b).astype(np.float32)
    if dtype == F16:
        return v.astype(np.float16).view(np.uint16)
    return (v.view(np.uint32) >> 16).astype(np.uint16)            # bf16: the value has at most 4 significant bits


def paged_attention(gpu_pool8, host_pool8, unit_side, unit_slot, q, block_table, ctx_lens, n_q_heads, n_kv_heads, head_dim,
                    dtype, scale, k_scale, v_scale, precision="f32"):
    """Pools are uint8 arrays [slots][Hkv * 2 * 16 * D]; q is 16-bit of `dtype`.  -> out [S][Hq][D]"""
    g16 = to_bits16(gpu_pool8, dtype)
    h16 = to_bits16(host_pool8, dtype) if host_pool8 is not None else None
    out = oracle.paged_attention(g16, h16, unit_side, unit_slot, q, block_table, ctx_lens, n_q_heads, n_kv_heads, head_dim,
                                 dtype, scale * k_scale, precision=precision)
    return out * v_scale


def append(gpu_pool8, host_pool8, unit_side, unit_slot, k_new, v_new, block_table, ctx_lens, n_kv_heads, head_dim, dtype,
           k_scale, v_scale):
    """The new token of every sequence (16-bit rows [S][Hkv][D]) is quantised and written at position ctx_len - 1."""
    # the division is a single-precision one (the precision the kernel takes this decision in); the rounding to E4M3
    # then starts from that fp32 quotient
    kf = _bits16_to_f64(k_new, dtype).astype(np.float32) / np.float32(k_scale)
    vf = _bits16_to_f64(v_new, dtype).astype(np.float32) / np.float32(v_scale)
    kq, vq = quantize(kf), quantize(vf)
    for s, ctx in enumerate(np.asarray(ctx_lens)):
        if ctx <= 0:
            continue
        pos = int(ctx) - 1
        b = int(block_table[s, pos // 16])
        pool = host_pool8 if unit_side[b] else gpu_pool8
        tile = pool[int(unit_slot[b])].reshape(n_kv_heads, 2, 16, head_dim)
        tile[:, 0, pos % 16, :] = kq[s]
        tile[:, 1, pos % 16, :] = vq[s]


def kv_write(gpu_pool8, host_pool8, unit_side, unit_slot, k, v, token_seq, token_pos, block_table, n_kv_heads, head_dim, dtype,
             k_scale, v_scale):
    """Prefill-side write into an 8-bit pool: token t is position token_pos[t] of sequence token_seq[t]; its 16-bit rows
    k[t], v[t] ([Hkv][D]) are quantised like the append's (fp32 quotient by the scale, nearest E4M3, ties to the even code,
    saturating) and land in row pos % 16 of the K and V halves of every head's tile in the block that holds the position.
    Returns -1 (nothing written) if a position is beyond the table or a block id out of range."""
    block_table = np.asarray(block_table, dtype=np.int32)
    k = np.ascontiguousarray(k, dtype=np.uint16).reshape(-1, n_kv_heads, head_dim)
    v = np.ascontiguousarray(v, dtype=np.uint16).reshape(-1, n_kv_heads, head_dim)
    for t in range(len(token_seq)):
        s, pos = int(token_seq[t]), int(token_pos[t])
        if not (0 <= s < block_table.shape[0] and 0 <= pos < 16 * block_table.shape[1]):
            return -1
        if not 0 <= block_table[s, pos // 16] < len(unit_slot):
            return -1
    kq = quantize(_bits16_to_f64(k, dtype).astype(np.float32) / np.float32(k_scale))
    vq = quantize(_bits16_to_f64(v, dtype).astype(np.float32) / np.float32(v_scale))
    for t in range(len(token_seq)):
        s, pos = int(token_seq[t]), int(token_pos[t])
        b = int(block_table[s, pos // 16])
        pool = host_pool8 if unit_side[b] else gpu_pool8
        tile = pool[int(unit_slot[b])].reshape(n_kv_heads, 2, 16, head_dim)
        tile[:, 0, pos % 16, :] = kq[t]
        tile[:, 1, pos % 16, :] = vq[t]
    return 0
