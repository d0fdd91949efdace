"""Set-up helpers shared by the GPU tests and bench.py: put a synthetic workload into a pie pool.

torch is used for device / pinned memory and streams only; every step of the path runs in libpie.so.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as pie
from . import synth


def _u64(x) -> int:
    return int(x) & 0xFFFFFFFFFFFFFFFF


class DeviceWorkload:
    """A pool holding one workload's KV blocks, with the seeded host-resident choice established at
    allocation time and contents written by the generator kernels (so nothing is moved during set-up)."""

    K_SCALE, V_SCALE = 0.25, 0.125    # scales of an 8-bit pool: the generator's bytes (|decoded| < 15) then stand for |k| < 4, |v| < 2

    def __init__(self, wl: synth.Workload, host_frac=None, timing=True, split_tokens=0, swap_ctas=0,
                 attn_ctas_per_sm=0, staging_layers=3, shuffle_table=False, extra_gpu_slots=0, extra_host_slots=0,
                 extra_tokens=None, attn_variant=0, gpu_slots_override=0, host_slots_override=0, initial_host_blocks=0):
        self.wl = wl
        dev = torch.device("cuda", torch.cuda.current_device())
        self.dev = dev
        self.host_frac = wl.host_frac if host_frac is None else host_frac
        self.extra_tokens = wl.decode_steps if extra_tokens is None else extra_tokens
        self.block_table, self.nblk, self.NB = wl.tables(shuffle=shuffle_table, extra_tokens=self.extra_tokens)
        self.max_blocks = self.block_table.shape[1]
        self.host_ids = synth.pick_host_blocks(wl.seed, self.block_table, self.nblk, self.host_frac)
        if initial_host_blocks:      # a given number of blocks starts on the host (a GPU pool smaller than the batch)
            self.host_ids = synth.seeded_permutation(wl.seed, self.NB, salt=5)[:initial_host_blocks].astype(np.int32)
        on_host = np.zeros(self.NB, dtype=np.uint8)
        on_host[self.host_ids] = 1
        L, S = wl.n_layers, wl.n_seqs
        n_host_blocks = int(on_host.sum())
        staging = staging_layers * max(n_host_blocks, 1)
        self.n_gpu_slots = L * (self.NB - n_host_blocks) + staging + extra_gpu_slots
        self.n_host_slots = L * n_host_blocks + staging + extra_host_slots
        if gpu_slots_override:
            self.n_gpu_slots = max(gpu_slots_override, L * (self.NB - n_host_blocks) + 2)
        if host_slots_override:
            self.n_host_slots = max(host_slots_override, L * n_host_blocks + 2)
        BB = wl.block_bytes
        self.gpu_pool = torch.empty(self.n_gpu_slots * BB, dtype=torch.uint8, device=dev)
        self.host_pool = torch.empty(self.n_host_slots * BB, dtype=torch.uint8, pin_memory=True)
        self.s_compute = torch.cuda.Stream(device=dev, priority=0)
        self.s_in = torch.cuda.Stream(device=dev, priority=-1)
        self.s_out = torch.cuda.Stream(device=dev, priority=-1)
        self.pool = pie.pie_pool_create(
            n_layers=L, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim, dtype=wl.dtype,
            n_logical_blocks=self.NB, max_seqs=max(S, 1), n_gpu_slots=self.n_gpu_slots, n_host_slots=self.n_host_slots,
            gpu_base=self.gpu_pool.data_ptr(), host_base=self.host_pool.data_ptr(), own_streams=0,
            compute_stream=self.s_compute.cuda_stream, copy_in_stream=self.s_in.cuda_stream,
            copy_out_stream=self.s_out.cuda_stream, split_tokens=split_tokens, swap_ctas=swap_ctas,
            attn_ctas_per_sm=attn_ctas_per_sm, timing=int(timing), attn_variant=attn_variant, kv_fp8=int(wl.kv_fp8))
        if wl.kv_fp8:
            pie.pie_set_kv_scales(self.pool, self.K_SCALE, self.V_SCALE)
        ids = pie.pie_block_alloc(self.pool, self.NB, on_host)
        assert np.array_equal(ids, np.arange(self.NB))
        self.fill_pools()
        # per-step inputs
        shape_q = (L, S, wl.n_q_heads, wl.head_dim)
        shape_kv = (L, S, wl.n_kv_heads, wl.head_dim)
        self.q_all = torch.empty(shape_q, dtype=torch.int16, device=dev)
        self.out_all = torch.zeros(shape_q, dtype=torch.int16, device=dev)
        self.k_new = torch.empty(shape_kv, dtype=torch.int16, device=dev)
        self.v_new = torch.empty(shape_kv, dtype=torch.int16, device=dev)
        self.fill_step_inputs(0)
        self.block_table_dev = torch.from_numpy(self.block_table).to(dev)
        self.ctx_lens = wl.ctx_lens.astype(np.int32).copy()      # host mirror of the current context lengths
        self.ctx_lens_dev = torch.from_numpy(self.ctx_lens).to(dev)
        self.scale = 1.0 / float(np.sqrt(wl.head_dim))
        torch.cuda.synchronize()

    # ---- contents ------------------------------------------------------------------------------------
    def fill_pools(self):
        wl = self.wl
        side, slot = pie.pie_get_placement(self.pool, wl.n_layers, self.NB)
        elems = wl.block_bytes // (1 if wl.kv_fp8 else 2)
        base = _u64(synth.stream_base(wl.seed, synth.STREAM_KV))
        units = np.arange(wl.n_layers * self.NB, dtype=np.int64).reshape(wl.n_layers, self.NB)
        lib = pie.synth_lib()
        for which, n_slots, ptr in ((pie.PIE_GPU, self.n_gpu_slots, self.gpu_pool.data_ptr()),
                                    (pie.PIE_HOST, self.n_host_slots, self.host_pool.data_ptr())):
            slot_unit = np.full(n_slots, -1, dtype=np.int64)
            m = side == which
            slot_unit[slot[m]] = units[m]
            su = torch.from_numpy(slot_unit).to(self.dev)
            if wl.kv_fp8:
                rc = lib.pie_synth_fill_slots_bytes(ptr, su.data_ptr(), n_slots, elems, base, None)
            else:
                rc = lib.pie_synth_fill_slots(ptr, su.data_ptr(), n_slots, elems, base, wl.dtype, 1.0, None)
            assert rc == 0, f"fill_slots: cudaError {rc}"
            torch.cuda.synchronize()

    def fill_step_inputs(self, step: int):
        wl, lib = self.wl, pie.synth_lib()
        for t, stream in ((self.q_all, synth.STREAM_Q), (self.k_new, synth.STREAM_KNEW), (self.v_new, synth.STREAM_VNEW)):
            base = _u64(synth.stream_base(wl.seed, stream))
            rc = lib.pie_synth_fill_tensor(t.data_ptr(), t.numel(), base, step * t.numel(), wl.dtype, 1.0, None)
            assert rc == 0
        torch.cuda.synchronize()

    def step_inputs_host(self, step: int, layer: int):
        """The same q / k_new / v_new bits for one layer, drawn by the numpy generator."""
        wl = self.wl
        out = []
        for t, stream in ((self.q_all, synth.STREAM_Q), (self.k_new, synth.STREAM_KNEW), (self.v_new, synth.STREAM_VNEW)):
            per_layer = t[0].numel()
            out.append(synth.tensor_bits(wl.seed, stream, tuple(t.shape[1:]), wl.dtype,
                                         offset=step * t.numel() + layer * per_layer))
        return out

    # ---- running ---------------------------------------------------------------------------------------
    def set_retention(self, on: bool):
        """Kept host copies + write-back elision (pie_set_retention); the blocks each step's append writes are
        declared from the host mirror of the context lengths."""
        self.retention = bool(on)
        pie.pie_set_retention(self.pool, int(on))
        if not on:
            pie.pie_declare_append_blocks(self.pool, None)

    def advance_context(self):
        """One more token per sequence (the step's append position)."""
        self.ctx_lens += 1
        assert int(self.ctx_lens.max() - self.wl.ctx_lens.max()) <= self.extra_tokens, "block table has no room left"
        with torch.cuda.stream(self.s_compute):
            self.ctx_lens_dev += 1
        if getattr(self, "retention", False):
            tails = self.block_table[np.arange(self.wl.n_seqs), (self.ctx_lens - 1) // 16]
            pie.pie_declare_append_blocks(self.pool, tails)

    def decode_step(self, append=True, mode=pie.PIE_MODE_AUTO, between_layers=None):
        """One decode step.  between_layers(l), if given, is called after every layer's attention has been enqueued (the
        place of a model's projections and MLP): the step then goes layer by layer through pie_decode_layer."""
        if between_layers is None:
            pie.pie_decode_step(self.pool, self.q_all.data_ptr(), self.out_all.data_ptr(), self.block_table_dev.data_ptr(),
                                self.max_blocks, self.ctx_lens_dev.data_ptr(), self.wl.n_seqs, self.scale,
                                self.k_new.data_ptr() if append else None, self.v_new.data_ptr() if append else None, mode)
            return
        pie.pie_step_begin(self.pool)
        for l in range(self.wl.n_layers):
            pie.pie_decode_layer(self.pool, l, self.q_all[l].data_ptr(), self.out_all[l].data_ptr(),
                                 self.block_table_dev.data_ptr(), self.max_blocks, self.ctx_lens_dev.data_ptr(), self.wl.n_seqs,
                                 self.scale, self.k_new[l].data_ptr() if append else None,
                                 self.v_new[l].data_ptr() if append else None, mode)
            with torch.cuda.stream(self.s_compute):
                between_layers(l)
        pie.pie_controller_tick(self.pool)

    def attention(self, layer, append=False, host_tables=False):
        pie.pie_decode_attention(
            self.pool, layer, self.q_all[layer].data_ptr(), self.out_all[layer].data_ptr(), self.block_table_dev.data_ptr(),
            self.max_blocks, self.ctx_lens_dev.data_ptr(), self.wl.n_seqs, self.scale,
            block_table_host=self.block_table if host_tables else None, ctx_lens_host=self.ctx_lens if host_tables else None,
            k_new=self.k_new[layer].data_ptr() if append else None, v_new=self.v_new[layer].data_ptr() if append else None)

    def sync(self):
        pie.pie_sync(self.pool)
        torch.cuda.synchronize()

    def out_bits(self) -> np.ndarray:
        return self.out_all.cpu().numpy().view(np.uint16)

    def attention_bytes_per_layer(self) -> int:
        """Algorithmic bytes of one layer call: valid KV tokens + q + out + table and lengths."""
        wl = self.wl
        ctx = self.ctx_lens.astype(np.int64)
        kv = int(ctx.sum()) * 2 * wl.n_kv_heads * wl.head_dim * (1 if wl.kv_fp8 else 2)
        qo = 2 * wl.n_seqs * wl.n_q_heads * wl.head_dim * 2
        tab = 4 * (int(((ctx + 15) // 16).sum()) + wl.n_seqs)
        return kv + qo + tab

    def close(self):
        if self.pool:
            pie.pie_pool_destroy(self.pool)
            self.pool = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
