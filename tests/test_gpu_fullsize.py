"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: sampled outputs the oracle can
compute one (layer, sequence) at a time, plus properties that hold at any size (swapped vs resident bit-identity,
final placement, byte counters)."""
import dataclasses
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2411_09317_b200 import binding as pie
from paper_2411_09317_b200 import synth
from paper_2411_09317_b200.harness import DeviceWorkload

pytestmark = pytest.mark.gpu
TOL = 2e-3


def oracle_one_sequence(dw, layer, s, steps_done):
    """fp32 oracle output [Hq][D] for one (layer, sequence) after `steps_done` appended tokens, from regenerated inputs."""
    wl = dw.wl
    ctx = int(wl.ctx_lens[s]) + steps_done
    nb = (ctx + 15) // 16
    blocks = dw.block_table[s, :nb]
    elems = wl.block_bytes // 2
    pool = np.zeros((nb, elems), dtype=np.uint16)
    for i, b in enumerate(blocks):
        pool[i] = synth.kv_unit_bits(wl.seed, layer, int(b), dw.NB, wl.n_kv_heads, wl.head_dim, wl.dtype).ravel()
    q, k_new, v_new = dw.step_inputs_host(0, layer)      # the harness feeds the same per-layer inputs every step
    side = np.zeros(nb, dtype=np.int32)
    slot = np.arange(nb, dtype=np.int32)
    table = np.arange(nb, dtype=np.int32)[None, :]
    for t in range(1, steps_done + 1):                   # token t lands at position ctx0 + t - 1
        oracle.append(pool, pool, side, slot, k_new[s:s + 1], v_new[s:s + 1], table,
                      np.array([int(wl.ctx_lens[s]) + t], np.int32), wl.n_kv_heads, wl.head_dim)
    out = oracle.paged_attention(pool, pool, side, slot, q[s:s + 1], table, np.array([ctx], np.int32), wl.n_q_heads,
                                 wl.n_kv_heads, wl.head_dim, wl.dtype, 1.0 / np.sqrt(wl.head_dim))
    return out[0]


def check_samples(dw, samples, steps_done):
    got_all = dw.out_all.cpu().numpy().view(np.uint16)
    worst = 0.0
    for layer, s in samples:
        want = oracle_one_sequence(dw, layer, s, steps_done)
        got = synth.bits16_to_f32(got_all[layer, s], dw.wl.dtype)
        worst = max(worst, float(np.abs(got - want).max()))
    assert worst <= TOL, worst
    return worst


def free(dw):
    dw.close()
    for name in ("gpu_pool", "host_pool", "q_all", "out_all", "k_new", "v_new"):
        setattr(dw, name, None)
    gc.collect()
    torch.cuda.empty_cache()


def test_llama2_7b_full_size_swapped_matches_oracle_and_resident_run():
    wl = synth.workload("llama2_7b")
    steps = 2
    dw = DeviceWorkload(wl, host_frac=wl.host_frac, timing=True)          # 30 % of every sequence's blocks on the host
    host_ids = set(dw.host_ids.tolist())
    for _ in range(steps):
        dw.advance_context()
        dw.decode_step()
    dw.sync()
    short = int(np.argmin(wl.ctx_lens))
    check_samples(dw, [(0, short), (17, short), (wl.n_layers - 1, int(np.argsort(wl.ctx_lens)[1]))], steps)
    stats = pie.pie_get_stats(dw.pool)
    n_host = len(host_ids)
    # per step every layer's host set comes in and goes out once (layer 0 of the first step is fetched on demand)
    assert stats["bytes_out"] == steps * wl.n_layers * n_host * wl.block_bytes
    assert stats["bytes_in"] == stats["bytes_out"] + n_host * wl.block_bytes    # layer 0 already prefetched again
    side, _ = pie.pie_get_placement(dw.pool, wl.n_layers, dw.NB)
    mask = np.zeros(dw.NB, bool)
    mask[list(host_ids)] = True
    assert np.all(side[1:, mask] == pie.PIE_HOST) and np.all(side[:, ~mask] == pie.PIE_GPU) and np.all(side[0, mask] == pie.PIE_GPU)
    swapped = dw.out_all.cpu().numpy().copy()
    free(dw)
    # the same logical inputs, never swapped: bit-identical outputs
    dw2 = DeviceWorkload(wl, host_frac=0.0, timing=False)
    for _ in range(steps):
        dw2.advance_context()
        dw2.decode_step()
    dw2.sync()
    resident = dw2.out_all.cpu().numpy()
    assert np.array_equal(swapped, resident)
    free(dw2)


def test_llama3_8b_full_size_gqa_bf16_fixed_ratio():
    wl = synth.workload("llama3_8b")
    wl = dataclasses.replace(wl, decode_steps=4)            # room for the steps run here (the config decodes 256)
    # the host-resident share is established through the ratio knob, not the initial placement
    _, _, nb = wl.tables()
    dw = DeviceWorkload(wl, host_frac=0.0, timing=True, extra_gpu_slots=3 * int(0.1 * nb) + 64,
                        extra_host_slots=wl.n_layers * int(0.1 * nb) + 4 * int(0.1 * nb) + 64)
    pie.pie_set_extension_ratio(dw.pool, 0.1)
    steps = 3
    for _ in range(steps):
        dw.advance_context()
        dw.decode_step()
    dw.sync()
    assert abs(pie.pie_get_extension_ratio(dw.pool) - 0.1) < 1e-6
    stats = pie.pie_get_stats(dw.pool)
    assert stats["bytes_out"] >= (steps - 1) * wl.n_layers * int(0.1 * nb) * wl.block_bytes
    order = np.argsort(wl.ctx_lens)
    check_samples(dw, [(0, int(order[0])), (15, int(order[1])), (31, int(order[len(order) // 2]))], steps)
    free(dw)


def test_llama3_70b_shape_long_context_adaptive_controller():
    """GQA-8, contexts of 4k-32k tokens, half of the blocks host resident at the start (KV = 2x the HBM pool share),
    16 of the 80 layers to keep the pinned pool small; the adaptive controller owns the ratio."""
    wl = synth.workload("llama3_70b")
    wl = dataclasses.replace(wl, n_layers=16, decode_steps=12)
    dw = DeviceWorkload(wl, host_frac=0.5, timing=True)
    pie.pie_set_controller(dw.pool, 1.0 / 64.0, 0.0, 0.0)
    pie.pie_set_extension_ratio(dw.pool, -1.0)               # adaptive, starting from the ratio in place
    steps = 10
    ratios = []
    for _ in range(steps):
        dw.advance_context()
        dw.decode_step()
        ratios.append(pie.pie_get_extension_ratio(dw.pool))
    dw.sync()
    stats = pie.pie_get_stats(dw.pool)
    assert stats["steps_measured"] >= steps - 4
    # link-bound at 50 %: the computation waits, so the controller must have backed off
    assert ratios[-1] < ratios[0] <= 0.51
    short = int(np.argmin(wl.ctx_lens))
    check_samples(dw, [(0, short), (15, short)], steps)
    free(dw)
