"""GPU-side test helpers: load a numpy Case into a pie pool and run it (marshalling only)."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2411_09317_b200 import binding as pie
from paper_2411_09317_b200 import synth


class PoolCase:
    def __init__(self, case, n_gpu_slots=None, n_host_slots=None, split_tokens=0, timing=0, all_on_gpu=False,
                 visible_blocks=0):
        self.c = case
        L, NB = case.L, case.NB
        on_host = np.zeros(NB, dtype=np.uint8) if all_on_gpu else case.unit_side[0].astype(np.uint8)
        nh = int(on_host.sum())
        self.n_gpu_slots = n_gpu_slots or (L * (NB - nh) + 3 * max(nh, 1) + 2)
        self.n_host_slots = n_host_slots or (L * NB + 2)
        self.pool = pie.pie_pool_create(n_layers=L, n_q_heads=case.Hq, n_kv_heads=case.Hkv, head_dim=case.D,
                                        dtype=case.dtype, n_logical_blocks=NB, max_seqs=max(case.S, 1),
                                        n_gpu_slots=self.n_gpu_slots, n_host_slots=self.n_host_slots,
                                        split_tokens=split_tokens, timing=timing, visible_blocks=visible_blocks,
                                        kv_fp8=int(getattr(case, "kv_fp8", False)))
        if getattr(case, "kv_fp8", False):
            pie.pie_set_kv_scales(self.pool, case.k_scale, case.v_scale)
        n0 = visible_blocks or NB          # with a smaller visible size only that many blocks exist at first
        ids = pie.pie_block_alloc(self.pool, n0, on_host[:n0])
        assert np.array_equal(ids, np.arange(n0))
        self.write_blocks(range(n0))
        dev = torch.device("cuda:0")
        self.q = torch.from_numpy(case.q.view(np.int16)).to(dev)              # [L][S][Hq][D]
        self.out = torch.zeros_like(self.q)
        self.bt = torch.from_numpy(case.block_table).to(dev)
        self.ctx = torch.from_numpy(case.ctx_lens.astype(np.int32)).to(dev)
        torch.cuda.synchronize()

    def write_blocks(self, ids):
        for l in range(self.c.L):
            for b in ids:
                pie.pie_block_write(self.pool, l, int(b), self.unit_bits(l, int(b)))

    def unit_bits(self, l, b):
        c = self.c
        pool = c.host_pool if c.unit_side[l, b] else c.gpu_pool
        return pool[c.unit_slot[l, b]]

    def attention(self, layer, host_tables=True, k_new=None, v_new=None, ctx=None):
        c = self.c
        pie.pie_decode_attention(self.pool, layer, self.q[layer].data_ptr(), self.out[layer].data_ptr(), self.bt.data_ptr(),
                                 c.block_table.shape[1], (self.ctx if ctx is None else ctx).data_ptr(), c.S, c.scale,
                                 block_table_host=c.block_table if host_tables else None,
                                 ctx_lens_host=c.ctx_lens if host_tables else None,
                                 k_new=None if k_new is None else k_new.data_ptr(),
                                 v_new=None if v_new is None else v_new.data_ptr())

    def result(self, layer):
        pie.pie_sync(self.pool)
        bits = self.out[layer].cpu().numpy().view(np.uint16)
        return bits, synth.bits16_to_f32(bits, self.c.dtype)

    def read_unit(self, l, b):
        raw = pie.pie_block_read(self.pool, l, b)
        return raw if getattr(self.c, "kv_fp8", False) else raw.view(np.uint16)

    def close(self):
        if self.pool:
            pie.pie_pool_destroy(self.pool)
            self.pool = None


def oracle_attention(case, layer, precision="f32"):
    if getattr(case, "kv_fp8", False):
        from oracle import fp8
        return fp8.paged_attention(case.gpu_pool, case.host_pool, case.unit_side[layer], case.unit_slot[layer], case.q[layer],
                                   case.block_table, case.ctx_lens, case.Hq, case.Hkv, case.D, case.dtype, case.scale,
                                   case.k_scale, case.v_scale, precision=precision)
    return oracle.paged_attention(case.gpu_pool, case.host_pool, case.unit_side[layer], case.unit_slot[layer], case.q[layer],
                                  case.block_table, case.ctx_lens, case.Hq, case.Hkv, case.D, case.dtype, case.scale,
                                  precision=precision)
