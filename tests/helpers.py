"""Builders of small paged-KV cases as numpy arrays, and the dense brute-force attention used as a pin."""
from __future__ import annotations

import numpy as np

from paper_2411_09317_b200 import synth


class Case:
    """One layer-set of paged KV with a placement of every (layer, block) unit in a device or host pool."""

    def __init__(self, n_layers, n_q_heads, n_kv_heads, head_dim, dtype, ctx_lens, seed=0, host_frac=0.0,
                 placement="identity", n_gpu_slots=None, n_host_slots=None, gain=1.0, q_gain=1.0,
                 shuffle_table=False, extra_tokens=0, kv_fp8=False, k_scale=0.25, v_scale=0.5):
        # kv_fp8: the pools hold one byte per element (the 8-bit variant); a byte stands for its value times the scale
        self.kv_fp8, self.k_scale, self.v_scale = kv_fp8, k_scale, v_scale
        self.L, self.Hq, self.Hkv, self.D, self.dtype = n_layers, n_q_heads, n_kv_heads, head_dim, dtype
        self.seed = seed
        self.ctx_lens = np.asarray(ctx_lens, dtype=np.int32)
        self.S = len(self.ctx_lens)
        self.block_table, self.nblk, self.NB = synth.build_block_table(
            self.ctx_lens, 16, extra_tokens=extra_tokens, shuffle_seed=seed if shuffle_table else None)
        self.NB = max(self.NB, 1)
        self.slot_elems = n_kv_heads * 2 * 16 * head_dim
        self.block_bytes = self.slot_elems * (1 if kv_fp8 else 2)
        host_ids = synth.pick_host_blocks(seed, self.block_table, self.nblk, host_frac)
        self.host_ids = host_ids
        on_host = np.zeros(self.NB, dtype=bool)
        on_host[host_ids] = True
        n_units = self.L * self.NB
        self.n_gpu_slots = n_gpu_slots or n_units
        self.n_host_slots = n_host_slots or max(1, n_units)
        self.gpu_pool = np.zeros((self.n_gpu_slots, self.slot_elems), dtype=np.uint8 if kv_fp8 else np.uint16)
        self.host_pool = np.zeros((self.n_host_slots, self.slot_elems), dtype=np.uint8 if kv_fp8 else np.uint16)
        self.unit_side = np.zeros((self.L, self.NB), dtype=np.int32)
        self.unit_slot = np.zeros((self.L, self.NB), dtype=np.int32)
        g_order = self._order(self.n_gpu_slots, placement, 11)
        h_order = self._order(self.n_host_slots, placement, 12)
        gi = hi = 0
        for l in range(self.L):
            for b in range(self.NB):
                if kv_fp8:
                    bits = synth.kv_unit_bytes(seed, l, b, self.NB, n_kv_heads, head_dim).ravel()
                else:
                    bits = synth.kv_unit_bits(seed, l, b, self.NB, n_kv_heads, head_dim, dtype, gain).ravel()
                if on_host[b]:
                    slot = int(h_order[hi]); hi += 1
                    self.host_pool[slot] = bits
                    self.unit_side[l, b] = 1
                else:
                    slot = int(g_order[gi]); gi += 1
                    self.gpu_pool[slot] = bits
                self.unit_slot[l, b] = slot
        self.q = synth.tensor_bits(seed, synth.STREAM_Q, (self.L, self.S, n_q_heads, head_dim), dtype, q_gain)
        self.scale = 1.0 / np.sqrt(head_dim)

    def _order(self, n, placement, salt):
        if placement == "identity":
            return np.arange(n)
        if placement == "reversed":
            return np.arange(n)[::-1]
        return synth.seeded_permutation(self.seed + 77, n, salt=salt)

    # contiguous K, V of one sequence as float64 [ctx][Hkv][D] (for brute-force checks)
    def dense_kv(self, layer, s):
        ctx = int(self.ctx_lens[s])
        K = np.zeros((ctx, self.Hkv, self.D))
        V = np.zeros((ctx, self.Hkv, self.D))
        for t in range(ctx):
            b = self.block_table[s, t // 16]
            pool = self.host_pool if self.unit_side[layer, b] else self.gpu_pool
            unit = pool[self.unit_slot[layer, b]].reshape(self.Hkv, 2, 16, self.D)
            K[t] = synth.bits16_to_f32(unit[:, 0, t % 16, :], self.dtype)
            V[t] = synth.bits16_to_f32(unit[:, 1, t % 16, :], self.dtype)
        return K, V

    def q_f(self, layer):
        return synth.bits16_to_f32(self.q[layer], self.dtype).astype(np.float64)


def dense_attention(q, K, V, scale):
    """Brute force on contiguous fp64 arrays: q [Hq][D], K/V [ctx][Hkv][D] -> [Hq][D]."""
    Hq, Hkv = q.shape[0], K.shape[1]
    g = Hq // Hkv
    out = np.zeros_like(q)
    for h in range(Hq):
        s = scale * (K[:, h // g, :] @ q[h])
        p = np.exp(s - s.max())
        p /= p.sum()
        out[h] = p @ V[:, h // g, :]
    return out


TOL = 2e-3   # max-abs bound on attention outputs (fp16 / bf16 inputs)


def tolerance(want, dtype):
    """Element-wise bound on |got - want|.  Flat 2e-3 wherever the exact output is small (|want| < 0.25: every element
    of the N(0,1) workloads with contexts of a hundred tokens or more).  Where |want| >= 0.25 (very short contexts,
    dominant keys, scaled inputs) rounding the output to 16 bits alone costs up to half an ulp - 2^-8 |want| in bf16
    (8 significant bits), 2^-11 |want| in fp16 (11 bits) - and the bound is 2e-3 plus that."""
    from paper_2411_09317_b200 import synth
    want = np.asarray(want)
    half_ulp = (2.0 ** -8 if dtype == synth.BF16 else 2.0 ** -11) * np.abs(want)
    return TOL + np.where(np.abs(want) >= 0.25, half_ulp, 0.0)
