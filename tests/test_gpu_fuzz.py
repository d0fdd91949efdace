"""Seeded random cases of the attention path against the oracle: shapes, length mixes, split sizes, placements, with and
without the append, 16-bit and 8-bit blocks.  Every case is reproducible from its seed."""
import numpy as np
import pytest
import torch

import oracle
from helpers import Case
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


@pytest.mark.parametrize("seed", range(24))
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
    bound = TOL + (2.0 ** -8 if case.dtype == BF16 else 2.0 ** -11) * np.abs(want)
    assert np.all(np.abs(got - want) <= bound), (c, float(np.abs(got - want).max()))
    pc.close()


@pytest.mark.parametrize("seed", range(8))
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
        pie.pie_decode_step(pc.pool, pc.q.data_ptr(), pc.out.data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                            ctx_dev.data_ptr(), case.S, case.scale, k_dev.data_ptr(), v_dev.data_ptr())
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
            bound = TOL + (2.0 ** -8 if dtype == BF16 else 2.0 ** -11) * np.abs(want)
            assert np.all(np.abs(got - want) <= bound), (seed, t, l, float(np.abs(got - want).max()))
    for l in range(L):
        for b in range(case.NB):
            assert np.array_equal(pc.read_unit(l, b), pc.unit_bits(l, b)), (seed, l, b)
    pc.close()
