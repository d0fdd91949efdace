"""CPU oracle of the KV-swap + paged-decode-attention path.  TEST INFRASTRUCTURE ONLY.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product library never does, and the oracle imports nothing from the product.

``pie_oracle.c`` (+ ``pie_oracle_attention.inc``) holds swap semantics and paged attention in fp32 and
fp64; ``table.py`` the mapping-table state machine; ``policy.py`` the swap protocol and controller.
This file compiles the C with gcc on first use and wraps it with ctypes (argument marshalling only).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libpie_oracle.so")
_SRC = [os.path.join(_HERE, "pie_oracle.c"), os.path.join(_HERE, "pie_oracle_attention.inc")]
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or any(os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC[0], "-lm"])
        os.replace(tmp, _SO)
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.pie_oracle_bits_to_f32.restype = ctypes.c_float
        _lib.pie_oracle_bits_to_f32.argtypes = [ctypes.c_uint16, ctypes.c_int]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def bits_to_f32(bits: np.ndarray, dtype: int) -> np.ndarray:
    l = lib()
    flat = np.ascontiguousarray(bits, dtype=np.uint16).ravel()
    return np.array([l.pie_oracle_bits_to_f32(int(b), dtype) for b in flat], dtype=np.float32).reshape(np.shape(bits))


def swap_raw(dst_pool: np.ndarray, src_pool: np.ndarray, block_bytes: int, src, dst) -> int:
    """dst_pool[dst[i]] <- src_pool[src[i]]; pools are uint8 [n_slots * block_bytes] (dst modified in place)."""
    src, dst = _i32(src), _i32(dst)
    assert dst_pool.dtype == np.uint8 and src_pool.dtype == np.uint8 and len(src) == len(dst)
    return lib().pie_oracle_swap_raw(_p(dst_pool), ctypes.c_int64(dst_pool.size // block_bytes), _p(src_pool),
                                     ctypes.c_int64(src_pool.size // block_bytes), ctypes.c_int64(block_bytes),
                                     _p(src), _p(dst), ctypes.c_int64(len(src)))


def append(gpu_pool, host_pool, unit_side, unit_slot, k_new, v_new, block_table, ctx_lens, n_kv_heads, head_dim):
    block_table = _i32(block_table)
    lib().pie_oracle_append(_p(gpu_pool), _p(host_pool), _p(_i32(unit_side)), _p(_i32(unit_slot)),
                            _p(np.ascontiguousarray(k_new, dtype=np.uint16)), _p(np.ascontiguousarray(v_new, dtype=np.uint16)),
                            _p(block_table), block_table.shape[1], _p(_i32(ctx_lens)), len(ctx_lens), n_kv_heads, head_dim)


def kv_write(gpu_pool, host_pool, unit_side, unit_slot, k, v, token_seq, token_pos, block_table, n_kv_heads, head_dim):
    """Prefill-side write of a flat batch of tokens into the paged KV cache (the prompt's keys and values, Section 2.2):
    token t is position token_pos[t] of sequence token_seq[t]; k[t], v[t] are [Hkv][D] 16-bit rows.  Its K row of head
    h lands in row pos % 16 of the K half of head h's tile in the block that holds the position, its V row in the V
    half - in whichever pool the unit lives (slot layout [Hkv][2][16][D]).  Plain loops: the definition.
    Returns -1 (nothing written) if a position is beyond the table or a block id out of range."""
    block_table = _i32(block_table)
    k = np.ascontiguousarray(k, dtype=np.uint16).reshape(-1, n_kv_heads, head_dim)
    v = np.ascontiguousarray(v, dtype=np.uint16).reshape(-1, n_kv_heads, head_dim)
    for t in range(len(token_seq)):
        s, pos = int(token_seq[t]), int(token_pos[t])
        if not (0 <= s < block_table.shape[0] and 0 <= pos < 16 * block_table.shape[1]):
            return -1
        if not 0 <= block_table[s, pos // 16] < len(unit_slot):
            return -1
    for t in range(len(token_seq)):
        s, pos = int(token_seq[t]), int(token_pos[t])
        b = int(block_table[s, pos // 16])
        pool = host_pool if unit_side[b] else gpu_pool
        tile = pool[int(unit_slot[b])].reshape(n_kv_heads, 2, 16, head_dim)
        tile[:, 0, pos % 16, :] = k[t]
        tile[:, 1, pos % 16, :] = v[t]
    return 0


def paged_attention(gpu_pool, host_pool, unit_side, unit_slot, q, block_table, ctx_lens, n_q_heads, n_kv_heads,
                    head_dim, dtype, scale, precision="f32", nthreads=1, split_tokens=None):
    """Paged decode attention of one layer.  Pools are uint16 arrays (slot layout [Hkv][2][16][D]);
    unit_side/unit_slot give, per logical block, the pool (0 device, 1 host) and slot that hold it.
    Returns out [S][Hq][D] in the requested precision (not rounded to 16 bits)."""
    block_table = _i32(block_table)
    ctx_lens = _i32(ctx_lens)
    unit_side, unit_slot = _i32(unit_side), _i32(unit_slot)
    q = np.ascontiguousarray(q, dtype=np.uint16)
    S = len(ctx_lens)
    real = np.float32 if precision == "f32" else np.float64
    out = np.zeros((S, n_q_heads, head_dim), dtype=real)
    hp = host_pool if host_pool is not None else gpu_pool
    if split_tokens is None:
        fn = getattr(lib(), f"pie_oracle_paged_attention_{precision}")
        st = fn(_p(gpu_pool), _p(hp), _p(unit_side), _p(unit_slot), len(unit_side), _p(q), _p(block_table),
                block_table.shape[1], _p(ctx_lens), S, n_q_heads, n_kv_heads, head_dim, dtype,
                ctypes.c_double(scale), _p(out), nthreads)
    else:
        fn = getattr(lib(), f"pie_oracle_paged_attention_split_{precision}")
        st = fn(_p(gpu_pool), _p(hp), _p(unit_side), _p(unit_slot), _p(q), _p(block_table), block_table.shape[1],
                _p(ctx_lens), S, n_q_heads, n_kv_heads, head_dim, dtype, ctypes.c_double(scale), int(split_tokens),
                _p(out))
    if st != 0:
        raise ValueError("oracle: block id out of range")
    return out


def merge(m1, l1, acc1, m2, l2, acc2, precision="f32"):
    """Log-sum-exp merge of two split-K partials -> (m, l, acc)."""
    real, ct = (np.float32, ctypes.c_float) if precision == "f32" else (np.float64, ctypes.c_double)
    a1 = np.array(acc1, dtype=real)
    a2 = np.ascontiguousarray(acc2, dtype=real)
    m, l = ct(m1), ct(l1)
    getattr(lib(), f"pie_oracle_merge_{precision}")(ctypes.byref(m), ctypes.byref(l), _p(a1), ct(m2), ct(l2), _p(a2),
                                                    len(a1))
    return m.value, l.value, a1
