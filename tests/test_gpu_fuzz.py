"""Seeded random cases of the attention path against the oracle: shapes, length mixes, split sizes, placements, with and
without the append, 16-bit and 8-bit blocks.  Every case is reproducible from its seed."""
import numpy as np
import pytest
import torch

import oracle
from helpers import Case, tolerance
from gpu_helpers import PoolCase, oracle_attention
from oracle import fp8
from paper_2411_09317_b200 import binding as pie
from paper_2411_09317_b200 import synth

pytestmark = pytest.mark.gpu
F16, BF16 = pie.PIE_F16, pie.PIE_BF16
TOL = 2e-3


def random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    kv8 = bool(rng.integers(0, 3) == 0)
    d = 128 if kv8 else int(rng.choice([64, 128]))
    hkv = int(rng.choice([1, 2, 4, 8]))
    group = int(rng.choice([1, 2, 4, 8]))
    dtype = int(rng.choice([F16, BF16]))
    n = int(rng.integers(1, 24))
    kind = rng.integers(0, 4)
    if kind == 0:
        lens = rng.integers(0, 80, n)
    elif kind == 1:
        lens = 16 * rng.integers(0, 40, n) + rng.choice([-1, 0, 1], n)
    elif kind == 2:
        lens = rng.integers(1, 3000, n)
    else:
        lens = np.concatenate([rng.integers(1, 64, n), [int(rng.integers(2000, 6000))]])
    lens = np.clip(lens, 0, None).astype(np.int32)
    split = int(rng.choice([0, 16, 48, 128, 512, 1024]))
    host_frac = float(rng.choice([0.0, 0.3, 0.7]))
    placement = str(rng.choice(["identity", "reversed", "random"]))
    append = bool(rng.integers(0, 2))
    return dict(kv8=kv8, d=d, hkv=hkv, hq=hkv * group, dtype=dtype, lens=lens, split=split, host_frac=host_frac,
                placement=placement, append=append, shuffle=bool(rng.integers(0, 2)))


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("PIE_FUZZ_CASES", "24"))))
def test_random_case_matches_oracle(seed):
    c = random_case(seed)
    kw = dict(kv_fp8=True, k_scale=0.25, v_scale=0.125) if c["kv8"] else {}
    case = Case(1, c["hq"], c["hkv"], c["d"], c["dtype"], c["lens"], seed=seed, host_frac=c["host_frac"], placement=c["placement"],
                shuffle_table=c["shuffle"], extra_tokens=1, **kw)
    pc = PoolCase(case, split_tokens=c["split"])
    if len(case.host_ids):
        pie.pie_swap_in(pc.pool, 0, case.host_ids, [pie.PIE_MODE_AUTO, pie.PIE_MODE_KERNEL, pie.PIE_MODE_KERNEL_BULK][seed % 3])
    dev = torch.device("cuda:0")
    if c["append"]:
        k_new = synth.tensor_bits(seed, synth.STREAM_KNEW, (case.S, case.Hkv, case.D), case.dtype)
        v_new = synth.tensor_bits(seed, synth.STREAM_VNEW, (case.S, case.Hkv, case.D), case.dtype, gain=0.5)
        cur = case.ctx_lens + 1
        ctx_dev = torch.from_numpy(cur.astype(np.int32)).to(dev)
        k_dev = torch.from_numpy(k_new.view(np.int16)).to(dev)
        v_dev = torch.from_numpy(v_new.view(np.int16)).to(dev)
        pie.pie_decode_attention(pc.pool, 0, pc.q[0].data_ptr(), pc.out[0].data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                                 ctx_dev.data_ptr(), case.S, case.scale, k_new=k_dev.data_ptr(), v_new=v_dev.data_ptr())
        # the oracle's pools follow: every unit sits in the GPU pool now (the host-resident ones were swapped in)
        side = np.zeros(case.NB, np.int32)
        # bring the oracle's view of the host-resident units over to its GPU pool copy at fresh slots
        g = np.concatenate([case.gpu_pool, case.host_pool[case.unit_slot[0][case.unit_side[0] == 1]]]) if len(case.host_ids) else case.gpu_pool
        slot = case.unit_slot[0].copy()
        if len(case.host_ids):
            moved = np.where(case.unit_side[0] == 1)[0]
            slot[moved] = len(case.gpu_pool) + np.arange(len(moved))
        if c["kv8"]:
            fp8.append(g, g, side, slot, k_new, v_new, case.block_table, cur, case.Hkv, case.D, case.dtype, case.k_scale, case.v_scale)
            want = fp8.paged_attention(g, g, side, slot, case.q[0], case.block_table, cur, case.Hq, case.Hkv, case.D, case.dtype,
                                       case.scale, case.k_scale, case.v_scale)
        else:
            oracle.append(g, g, side, slot, k_new, v_new, case.block_table, cur, case.Hkv, case.D)
            want = oracle.paged_attention(g, g, side, slot, case.q[0], case.block_table, cur, case.Hq, case.Hkv, case.D, case.dtype,
                                          case.scale)
        pie.pie_sync(pc.pool)
        # the appended rows, bit for bit, in the units that received them
        for s in range(case.S):
            b = int(case.block_table[s, (cur[s] - 1) // 16])
            got_unit = pc.read_unit(0, b)
            assert np.array_equal(got_unit, g[slot[b]]), (s, b)
    else:
        pc.attention(0, host_tables=False)
        want = oracle_attention(case, 0)
        pie.pie_sync(pc.pool)
    got = synth.bits16_to_f32(pc.out[0].cpu().numpy().view(np.uint16), case.dtype)
    bound = tolerance(want, case.dtype)
    assert np.all(np.abs(got - want) <= bound), (c, float(np.abs(got - want).max()))
    pc.close()


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("PIE_FUZZ_SEEDS", "12"))))
def test_random_decode_steps_with_changing_ratio_match_oracle(seed):
    """Several decode steps on a small model while the extension ratio, the look-ahead and the kept-copies switch change
    at random between steps: every step's outputs within tolerance, and at the end every unit's bytes equal the oracle's."""
    rng = np.random.default_rng(5000 + seed)
    kv8 = bool(seed % 3 == 1)
    dtype = int(rng.choice([F16, BF16]))
    L, hkv, group = int(rng.integers(2, 5)), int(rng.choice([1, 2, 4])), int(rng.choice([1, 2, 4]))
    d = 128 if kv8 else int(rng.choice([64, 128]))
    lens = rng.integers(1, 400, int(rng.integers(2, 9))).astype(np.int32)
    steps = 6
    kw = dict(kv_fp8=True, k_scale=0.25, v_scale=0.125) if kv8 else {}
    case = Case(L, hkv * group, hkv, d, dtype, lens, seed=seed, host_frac=float(rng.choice([0.0, 0.4])), placement="random",
                extra_tokens=steps, **kw)
    nh = len(case.host_ids)
    pc = PoolCase(case, timing=1, n_gpu_slots=L * case.NB + 6 * case.NB + 8, n_host_slots=L * case.NB + 6 * case.NB + 8)
    dev = torch.device("cuda:0")
    cur = lens.copy()
    ctx_dev = torch.from_numpy(cur).to(dev)
    for t in range(steps):
        pie.pie_set_extension_ratio(pc.pool, float(rng.choice([0.0, 0.1, 0.3, 0.6, 1.0])))
        pie.pie_set_lookahead(pc.pool, int(rng.integers(1, 4)))
        pie.pie_set_retention(pc.pool, int(rng.integers(0, 2)))
        k_new = synth.tensor_bits(seed, synth.STREAM_KNEW, (L, case.S, case.Hkv, case.D), dtype, offset=t * 10_000_000)
        v_new = synth.tensor_bits(seed, synth.STREAM_VNEW, (L, case.S, case.Hkv, case.D), dtype, gain=0.5, offset=t * 10_000_000)
        k_dev = torch.from_numpy(k_new.view(np.int16)).to(dev)
        v_dev = torch.from_numpy(v_new.view(np.int16)).to(dev)
        cur = cur + 1
        ctx_dev.copy_(torch.from_numpy(cur))
        torch.cuda.synchronize()
        api = int(rng.integers(0, 3))        # the whole step, the same layer by layer, or from host buffers
        if api == 0:
            pie.pie_decode_step(pc.pool, pc.q.data_ptr(), pc.out.data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                                ctx_dev.data_ptr(), case.S, case.scale, k_dev.data_ptr(), v_dev.data_ptr())
        elif api == 1:
            pie.pie_step_begin(pc.pool)
            for l in range(L):
                pie.pie_decode_layer(pc.pool, l, pc.q[l].data_ptr(), pc.out[l].data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                                     ctx_dev.data_ptr(), case.S, case.scale, k_dev[l].data_ptr(), v_dev[l].data_ptr())
            pie.pie_controller_tick(pc.pool)
        else:
            out_host = np.zeros(tuple(pc.q.shape), dtype=np.int16)
            pie.pie_decode_step_host(pc.pool, np.ascontiguousarray(case.q.view(np.int16)), out_host, case.block_table,
                                     case.block_table.shape[1], cur.astype(np.int32), case.S, case.scale,
                                     np.ascontiguousarray(k_new.view(np.int16)), np.ascontiguousarray(v_new.view(np.int16)))
            pc.out.copy_(torch.from_numpy(out_host))
        pie.pie_sync(pc.pool)
        case.ctx_lens = cur.copy()
        for l in range(L):
            if kv8:
                fp8.append(case.gpu_pool, case.host_pool, case.unit_side[l], case.unit_slot[l], k_new[l], v_new[l], case.block_table,
                           cur, case.Hkv, case.D, dtype, case.k_scale, case.v_scale)
            else:
                oracle.append(case.gpu_pool, case.host_pool, case.unit_side[l], case.unit_slot[l], k_new[l], v_new[l],
                              case.block_table, cur, case.Hkv, case.D)
            want = oracle_attention(case, l)
            got = synth.bits16_to_f32(pc.out[l].cpu().numpy().view(np.uint16), dtype)
            bound = tolerance(want, dtype)
            assert np.all(np.abs(got - want) <= bound), (seed, t, l, float(np.abs(got - want).max()))
    for l in range(L):
        for b in range(case.NB):
            assert np.array_equal(pc.read_unit(l, b), pc.unit_bits(l, b)), (seed, l, b)
    pc.close()


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("PIE_FUZZ_OPS", "6"))))
def test_random_pool_operations_keep_every_unit_and_attend_correctly(seed):
    """A random walk over the pool's calls - allocate (either side) and fill, free, swap lists out and in by any of the
    copy paths, read back, attend over sequences made of whatever blocks exist - against a plain dictionary of what every
    (layer, block) should hold.  Nothing is synchronised unless a call needs it."""
    rng = np.random.default_rng(9000 + seed)
    L, hkv, hq, d, dtype = int(rng.integers(1, 4)), 2, 4, 128, int(rng.choice([F16, BF16]))
    NB = 48
    elems = hkv * 2 * 16 * d
    pool = pie.pie_pool_create(n_layers=L, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, dtype=dtype, n_logical_blocks=NB, max_seqs=8,
                               n_gpu_slots=int(rng.integers(NB // 2, L * NB)) + 4, n_host_slots=L * NB + 8)
    content = {}                                   # (layer, block) -> uint16 [elems]
    live = []
    dev = torch.device("cuda:0")
    modes = [pie.PIE_MODE_AUTO, pie.PIE_MODE_KERNEL, pie.PIE_MODE_COPY_ENGINE, pie.PIE_MODE_KERNEL_BULK]
    fills = 0
    for step in range(120):
        k = rng.random()
        if k < 0.2 and len(live) < NB:
            n = int(rng.integers(1, min(6, NB - len(live)) + 1))
            try:
                ids = pie.pie_block_alloc(pool, n, rng.integers(0, 2, n).astype(np.uint8))
            except pie.PieError as e:
                assert e.status == pie.PIE_ERR_NOMEM
                continue
            for b in ids:
                for l in range(L):
                    bits = synth.normal_bits(seed, synth.STREAM_KV, np.arange(elems, dtype=np.uint64) + np.uint64(fills * elems), dtype)
                    fills += 1
                    pie.pie_block_write(pool, l, int(b), bits)
                    content[(l, int(b))] = bits
                live.append(int(b))
        elif k < 0.3 and live:
            gone = [live.pop(int(rng.integers(0, len(live)))) for _ in range(min(len(live), int(rng.integers(1, 4))))]
            pie.pie_sync(pool)                      # a block with a copy in flight cannot be freed
            pie.pie_block_free(pool, gone)
            for b in gone:
                for l in range(L):
                    del content[(l, b)]
        elif k < 0.65 and live:
            ids = rng.choice(live, int(rng.integers(1, len(live) + 1)), replace=False).astype(np.int32)
            layer, mode = int(rng.integers(0, L)), modes[int(rng.integers(0, 4))]
            try:
                (pie.pie_swap_out if rng.random() < 0.5 else pie.pie_swap_in)(pool, layer, ids, mode)
            except pie.PieError as e:
                assert e.status == pie.PIE_ERR_NOMEM
        elif k < 0.8 and live:
            l, b = int(rng.integers(0, L)), int(rng.choice(live))
            assert np.array_equal(pie.pie_block_read(pool, l, b).view(np.uint16), content[(l, b)]), (step, l, b)
        elif live:
            # attention over up to four sequences cut from a random order of the live blocks
            layer = int(rng.integers(0, L))
            order = rng.permutation(live)
            S = int(rng.integers(1, min(4, len(order)) + 1))
            parts = np.array_split(order, S)
            max_blocks = max(len(p) for p in parts)
            bt = np.full((S, max_blocks), -1, dtype=np.int32)
            lens = np.zeros(S, dtype=np.int32)
            for s, p in enumerate(parts):
                bt[s, :len(p)] = p
                lens[s] = 16 * len(p) - int(rng.integers(0, 16))
            try:
                pie.pie_swap_in(pool, layer, order.astype(np.int32), modes[int(rng.integers(0, 4))])
            except pie.PieError as e:
                assert e.status == pie.PIE_ERR_NOMEM
                continue
            q = synth.tensor_bits(seed, synth.STREAM_Q, (S, hq, d), dtype, offset=step * 100_000)
            q_dev = torch.from_numpy(q.view(np.int16)).to(dev)
            out_dev = torch.zeros_like(q_dev)
            bt_dev, len_dev = torch.from_numpy(bt).to(dev), torch.from_numpy(lens).to(dev)
            torch.cuda.synchronize()
            pie.pie_decode_attention(pool, layer, q_dev.data_ptr(), out_dev.data_ptr(), bt_dev.data_ptr(), max_blocks,
                                     len_dev.data_ptr(), S, 1.0 / np.sqrt(d), block_table_host=bt, ctx_lens_host=lens)
            pie.pie_sync(pool)
            store = np.stack([content[(layer, int(b))] for b in order])
            slot_of = np.full(NB, -1, dtype=np.int32)
            slot_of[order] = np.arange(len(order))
            want = oracle.paged_attention(store, store, np.zeros(NB, np.int32), slot_of, q, bt, lens, hq, hkv, d, dtype, 1.0 / np.sqrt(d))
            got = synth.bits16_to_f32(out_dev.cpu().numpy().view(np.uint16), dtype)
            bound = tolerance(want, dtype)
            assert np.all(np.abs(got - want) <= bound), (seed, step, float(np.abs(got - want).max()))
    pie.pie_sync(pool)
    for (l, b), bits in content.items():
        assert np.array_equal(pie.pie_block_read(pool, l, b).view(np.uint16), bits), (l, b)
    pie.pie_pool_destroy(pool)


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("PIE_FUZZ_LAYERS", "6"))))
def test_random_whole_layer_protocol_configurations_match_oracle(seed):
    """The paper's whole-layer protocol (Section 3.3) with a random number of layers, of layers that start on the CPU and
    of spare regions on either side: outputs of every step and the final bytes of every unit against the oracle."""
    rng = np.random.default_rng(7000 + seed)
    L = int(rng.integers(3, 11))
    m = int(rng.integers(1, L - 1))                       # layers on the CPU at the start: the last m
    gpu_regions = L - m + int(rng.integers(0, 2))
    cpu_regions = m + int(rng.integers(1, 4))
    dtype = int(rng.choice([F16, BF16]))
    hkv, group, d = int(rng.choice([1, 2, 4])), int(rng.choice([1, 2])), int(rng.choice([64, 128]))
    lens = rng.integers(1, 300, int(rng.integers(1, 6))).astype(np.int32)
    steps = 4
    case = Case(L, hkv * group, hkv, d, dtype, lens, seed=seed, host_frac=0.0, placement="identity", extra_tokens=steps)
    NB = case.NB
    pool = pie.pie_pool_create(n_layers=L, n_q_heads=case.Hq, n_kv_heads=hkv, head_dim=d, dtype=dtype, n_logical_blocks=NB,
                               max_seqs=case.S, n_gpu_slots=gpu_regions * NB, n_host_slots=max(cpu_regions, L) * NB, timing=1)
    pie.pie_block_alloc(pool, NB, np.ones(NB, np.uint8))
    for l in range(L):
        for b in range(NB):
            pie.pie_block_write(pool, l, b, case.gpu_pool[case.unit_slot[l, b]])
    for l in range(L - m):
        pie.pie_swap_in(pool, l, np.arange(NB))
    pie.pie_sync(pool)
    pie.pie_set_layer_policy(pool, gpu_regions, cpu_regions)
    dev = torch.device("cuda:0")
    q = torch.from_numpy(case.q.view(np.int16)).to(dev)
    out = torch.zeros_like(q)
    bt = torch.from_numpy(case.block_table).to(dev)
    cur = lens.copy()
    ctx_dev = torch.from_numpy(cur).to(dev)
    for t in range(steps):
        k_new = synth.tensor_bits(seed, synth.STREAM_KNEW, (L, case.S, case.Hkv, case.D), dtype, offset=t * 1_000_000)
        v_new = synth.tensor_bits(seed, synth.STREAM_VNEW, (L, case.S, case.Hkv, case.D), dtype, offset=t * 1_000_000)
        k_dev = torch.from_numpy(k_new.view(np.int16)).to(dev)
        v_dev = torch.from_numpy(v_new.view(np.int16)).to(dev)
        cur = cur + 1
        ctx_dev.copy_(torch.from_numpy(cur))
        torch.cuda.synchronize()
        pie.pie_decode_step(pool, q.data_ptr(), out.data_ptr(), bt.data_ptr(), case.block_table.shape[1], ctx_dev.data_ptr(),
                            case.S, case.scale, k_dev.data_ptr(), v_dev.data_ptr())
        pie.pie_sync(pool)
        case.ctx_lens = cur.copy()
        for l in range(L):
            oracle.append(case.gpu_pool, case.host_pool, case.unit_side[l], case.unit_slot[l], k_new[l], v_new[l],
                          case.block_table, cur, case.Hkv, case.D)
            want = oracle_attention(case, l)
            got = synth.bits16_to_f32(out[l].cpu().numpy().view(np.uint16), dtype)
            bound = tolerance(want, dtype)
            assert np.all(np.abs(got - want) <= bound), (seed, L, m, gpu_regions, cpu_regions, t, l)
    for l in range(L):
        for b in range(NB):
            assert np.array_equal(pie.pie_block_read(pool, l, b).view(np.uint16), case.gpu_pool[case.unit_slot[l, b]]), (seed, l, b)
    pie.pie_pool_destroy(pool)
