"""GPU parity of the 8-bit KV variant (blocks of E4M3 bytes) against its oracle: attention over decoded values within the
16-bit path's tolerance, appended bytes bit for bit, swapping unchanged."""
import numpy as np
import pytest
import torch

from helpers import Case, tolerance
from gpu_helpers import PoolCase, oracle_attention
from oracle import fp8
from paper_2411_09317_b200 import binding as pie
from paper_2411_09317_b200 import synth

pytestmark = pytest.mark.gpu
F16, BF16 = pie.PIE_F16, pie.PIE_BF16
TOL = 2e-3      # as for 16-bit pools: the decoded values times the scales are of the same magnitude (|k| < 4, |v| < 2)


def tol(want, dtype):
    return tolerance(want, dtype)


def fp8_case(*a, **kw):
    kw.setdefault("k_scale", 0.25)
    kw.setdefault("v_scale", 0.125)
    return Case(*a, kv_fp8=True, **kw)


def check(case, pc, layer):
    pc.attention(layer)
    bits, got = pc.result(layer)
    want = oracle_attention(case, layer, "f32")
    err = np.abs(got - want)
    assert np.all(err <= tol(want, case.dtype)), f"max-abs {err.max()}"
    return bits


def test_byte_generator_kernel_matches_numpy():
    lib = pie.synth_lib()
    elems, n_slots = 2 * 2 * 16 * 128, 6
    slot_unit = np.array([4, -1, 0, 9, 2, -1], dtype=np.int64)
    pool = torch.zeros(n_slots * elems, dtype=torch.uint8, device="cuda")
    su = torch.from_numpy(slot_unit).cuda()
    base = int(synth.stream_base(5, synth.STREAM_KV))
    assert lib.pie_synth_fill_slots_bytes(pool.data_ptr(), su.data_ptr(), n_slots, elems, base, None) == 0
    torch.cuda.synchronize()
    got = pool.cpu().numpy().reshape(n_slots, elems)
    for s, u in enumerate(slot_unit):
        if u < 0:
            assert not got[s].any()
        else:
            want = synth.kv_unit_bytes(5, 0, int(u), 100, 2, 128).ravel()      # unit index = layer * NB + block
            assert np.array_equal(got[s], want)
    assert not np.any((got & 0x78) == 0x78)      # never the all-ones exponent


@pytest.mark.parametrize("hq,hkv,dtype", [(8, 8, F16), (8, 2, BF16), (8, 1, BF16), (16, 2, F16), (32, 32, BF16), (8, 8, BF16)])
def test_attention_parity_edge_lengths(hq, hkv, dtype):
    lens = [1, 15, 16, 17, 31, 32, 33, 255, 256, 257, 511, 512, 513, 0, 100]
    case = fp8_case(1, hq, hkv, 128, dtype, lens, seed=21, placement="random", shuffle_table=True)
    pc = PoolCase(case)
    assert pie.pie_block_bytes(pc.pool) == 2 * 16 * hkv * 128
    check(case, pc, 0)
    pc.close()


@pytest.mark.parametrize("split", [16, 64, 256, 1024])
def test_attention_parity_split_sizes_and_long_context(split):
    case = fp8_case(1, 8, 2, 128, BF16, [4097, 3, 1500], seed=22, placement="reversed")
    pc = PoolCase(case, split_tokens=split)
    check(case, pc, 0)
    pc.close()


def test_attention_parity_batch_128_ragged_scales_not_powers_of_two():
    lens = synth.uniform_lengths(7, 128, 1, 200)
    case = fp8_case(1, 32, 8, 128, F16, lens, seed=23, placement="random", k_scale=0.3, v_scale=0.11)
    pc = PoolCase(case)
    check(case, pc, 0)
    pc.close()


def test_tail_bytes_beyond_the_context_are_excluded():
    case = fp8_case(1, 8, 4, 128, F16, [5, 17, 33, 250], seed=24)
    pc0 = PoolCase(case)
    clean = check(case, pc0, 0)
    pc0.close()
    for s in range(case.S):
        ctx = int(case.ctx_lens[s])
        b = case.block_table[s, (ctx - 1) // 16]
        unit = case.gpu_pool[case.unit_slot[0, b]].reshape(case.Hkv, 2, 16, case.D)
        if ctx % 16:
            unit[:, :, ctx % 16:, :] = 0x7F          # NaN in K and V tails
            unit[:, 1, ctx % 16:, ::2] = 0xFE        # -448
    pc = PoolCase(case)
    poisoned = check(case, pc, 0)
    pc.close()
    assert np.array_equal(clean, poisoned)


def test_resident_vs_swapped_bit_identical():
    lens = [100, 257, 31, 1024]
    a = fp8_case(2, 8, 2, 128, BF16, lens, seed=25, host_frac=0.0)
    b = fp8_case(2, 8, 2, 128, BF16, lens, seed=25, host_frac=0.5, placement="random")
    pa, pb = PoolCase(a), PoolCase(b)
    for l in range(2):
        ids = b.host_ids
        pie.pie_swap_in(pb.pool, l, ids)
        ra = check(a, pa, l)
        pb.attention(l)
        rb, _ = pb.result(l)
        assert np.array_equal(ra, rb)
        pie.pie_swap_out(pb.pool, l, ids)
    pie.pie_sync(pb.pool)
    for l in range(2):
        for blk in range(b.NB):
            assert np.array_equal(pb.read_unit(l, blk), pb.unit_bits(l, blk))
    pa.close()
    pb.close()


@pytest.mark.parametrize("retention", ["off", "declared"])
@pytest.mark.parametrize("dtype", [F16, BF16])
def test_multi_step_decode_with_append_matches_oracle_every_step(retention, dtype):
    """Five decode steps, 40 % of the blocks host resident: every step's outputs within tolerance and, at the end, every
    unit's bytes exactly the oracle's (the appended tokens quantised the same way, nothing lost in the swaps)."""
    lens = np.array([30, 63, 64, 65, 129, 7], dtype=np.int32)
    steps = 5
    case = fp8_case(3, 8, 2, 128, dtype, lens, seed=42, host_frac=0.4, placement="random", extra_tokens=steps)
    nh = len(case.host_ids)
    pc = PoolCase(case, timing=1, n_gpu_slots=case.L * (case.NB - nh) + 3 * nh + 2)
    if retention != "off":
        pie.pie_set_retention(pc.pool, 1)
    dev = torch.device("cuda:0")
    cur = lens.copy()
    ctx_dev = torch.from_numpy(cur).to(dev)
    for t in range(steps):
        k_new = synth.tensor_bits(42, synth.STREAM_KNEW, (case.L, case.S, case.Hkv, case.D), dtype, offset=t * 10_000_000)
        v_new = synth.tensor_bits(42, synth.STREAM_VNEW, (case.L, case.S, case.Hkv, case.D), dtype, gain=0.5, offset=t * 10_000_000)
        k_dev = torch.from_numpy(k_new.view(np.int16)).to(dev)
        v_dev = torch.from_numpy(v_new.view(np.int16)).to(dev)
        cur = cur + 1
        ctx_dev.copy_(torch.from_numpy(cur))
        torch.cuda.synchronize()
        if retention == "declared":
            pie.pie_declare_append_blocks(pc.pool, case.block_table[np.arange(case.S), (cur - 1) // 16])
        pie.pie_decode_step(pc.pool, pc.q.data_ptr(), pc.out.data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                            ctx_dev.data_ptr(), case.S, case.scale, k_dev.data_ptr(), v_dev.data_ptr())
        pie.pie_sync(pc.pool)
        case.ctx_lens = cur.copy()
        for l in range(case.L):
            fp8.append(case.gpu_pool, case.host_pool, case.unit_side[l], case.unit_slot[l], k_new[l], v_new[l],
                       case.block_table, cur, case.Hkv, case.D, dtype, case.k_scale, case.v_scale)
            want = oracle_attention(case, l)
            got = synth.bits16_to_f32(pc.out[l].cpu().numpy().view(np.uint16), dtype)
            assert np.all(np.abs(got - want) <= tol(want, dtype)), (t, l)
    for l in range(case.L):
        for b in range(case.NB):
            assert np.array_equal(pc.read_unit(l, b), pc.unit_bits(l, b)), (l, b)
    stats = pie.pie_get_stats(pc.pool)
    if retention == "off":
        assert stats["bytes_out_elided"] == 0
    else:
        assert stats["bytes_out_elided"] > 0
        assert stats["bytes_out_elided"] + stats["bytes_out"] == steps * case.L * nh * case.block_bytes
    pc.close()


@pytest.mark.parametrize("dtype", [F16, BF16])
def test_appended_bytes_at_ties_subnormals_saturation_and_nan(dtype):
    """The new token's 128 values per head are chosen: every midpoint between neighbouring E4M3 values (ties go to the
    even code), values just beside them, the subnormal range, magnitudes beyond 448 (saturate), infinities, signed zeros
    and a NaN.  Only the stored bytes are compared (a NaN row makes the outputs meaningless)."""
    pos = fp8.E4M3[:127]
    mids = (pos[:-1] + pos[1:]) / 2                                   # 126 midpoints: 5 significant bits, exact in 16 bits
    vals = np.concatenate([mids, [0.0, -0.0]])                        # 128 for K
    extra = np.concatenate([-mids[:60], mids[60:100] * (1 + 2.0 ** -7), mids[100:120] * (1 - 2.0 ** -7),
                            [448.0, 449.0, 464.0, 480.0, 1000.0, 60000.0, np.inf, -np.inf]])   # 128 for V
    assert len(vals) == 128 and len(extra) == 128
    k_scale, v_scale = 0.5, 2.0                                       # powers of two: x = value * scale is exact
    lens = np.array([17, 40], dtype=np.int32)
    case = fp8_case(1, 8, 2, 128, dtype, lens, seed=44, extra_tokens=1, k_scale=k_scale, v_scale=v_scale)
    pc = PoolCase(case)
    k_f = np.zeros((1, case.S, case.Hkv, 128), dtype=np.float32)
    v_f = np.zeros_like(k_f)
    k_f[0, :, 0, :] = vals * k_scale
    k_f[0, :, 1, :] = -vals[::-1] * k_scale
    v_f[0, :, 0, :] = extra * v_scale
    v_f[0, :, 1, :] = extra[::-1] * v_scale
    with np.errstate(over="ignore"):                                  # 120000 is an infinity in fp16: intended
        k_new = synth.f32_to_16_bits(k_f, dtype)
        v_new = synth.f32_to_16_bits(v_f, dtype)
    k_new[0, 1, 1, 5] = 0x7E00 if dtype == F16 else 0x7FC0            # a NaN
    # every chosen value must have survived the 16-bit rounding of the inputs, or the test would not test the ties
    assert np.array_equal(synth.bits16_to_f32(k_new, dtype)[0, 0, 0], (vals * k_scale).astype(np.float32))
    dev = torch.device("cuda:0")
    cur = lens + 1
    ctx_dev = torch.from_numpy(cur).to(dev)
    k_dev = torch.from_numpy(k_new.view(np.int16)).to(dev)
    v_dev = torch.from_numpy(v_new.view(np.int16)).to(dev)
    pie.pie_decode_attention(pc.pool, 0, pc.q[0].data_ptr(), pc.out[0].data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                             ctx_dev.data_ptr(), case.S, case.scale, k_new=k_dev.data_ptr(), v_new=v_dev.data_ptr())
    pie.pie_sync(pc.pool)
    fp8.append(case.gpu_pool, case.host_pool, case.unit_side[0], case.unit_slot[0], k_new[0], v_new[0], case.block_table, cur,
               case.Hkv, case.D, dtype, k_scale, v_scale)
    for b in range(case.NB):
        assert np.array_equal(pc.read_unit(0, b), pc.unit_bits(0, b)), b
    # spot values, written out: midpoint of codes 0x38 (1.0) and 0x39 (1.125) -> the even code; beyond 448 -> 0x7e / 0xfe
    s0 = case.block_table[0, (cur[0] - 1) // 16]
    unit = pc.read_unit(0, int(s0)).reshape(case.Hkv, 2, 16, 128)
    row = (cur[0] - 1) % 16
    assert unit[0, 0, row, 0x38] == 0x38 and unit[0, 0, row, 0x39] == 0x3A
    assert list(unit[0, 1, row, 120:128]) == [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE]
    pc.close()


def test_argument_checks():
    kw = dict(n_layers=1, n_q_heads=8, n_kv_heads=8, dtype=F16, n_logical_blocks=8, n_gpu_slots=8, n_host_slots=8)
    with pytest.raises(pie.PieError) as e:
        pie.pie_pool_create(head_dim=64, kv_fp8=1, **kw)
    assert e.value.status == pie.PIE_ERR_UNSUPPORTED
    with pytest.raises(pie.PieError) as e:
        pie.pie_pool_create(head_dim=128, kv_fp8=1, attn_variant=3, **kw)
    assert e.value.status == pie.PIE_ERR_UNSUPPORTED
    with pytest.raises(pie.PieError) as e:
        pie.pie_pool_create(head_dim=128, kv_fp8=2, **kw)
    assert e.value.status == pie.PIE_ERR_INVALID
    p16 = pie.pie_pool_create(head_dim=128, **kw)
    with pytest.raises(pie.PieError) as e:
        pie.pie_set_kv_scales(p16, 1.0, 1.0)
    assert e.value.status == pie.PIE_ERR_UNSUPPORTED
    pie.pie_pool_destroy(p16)
    p8 = pie.pie_pool_create(head_dim=128, kv_fp8=1, **kw)
    assert pie.pie_block_bytes(p8) == 2 * 16 * 8 * 128
    for ks, vs in ((0.0, 1.0), (1.0, -1.0), (float("nan"), 1.0), (1.0, float("inf"))):
        with pytest.raises(pie.PieError) as e:
            pie.pie_set_kv_scales(p8, ks, vs)
        assert e.value.status == pie.PIE_ERR_INVALID
    pie.pie_set_kv_scales(p8, 0.5, 0.25)
    pie.pie_pool_destroy(p8)


@pytest.mark.parametrize("hq,hkv,dtype", [(8, 8, BF16), (8, 1, F16), (16, 4, F16)])
def test_prompt_write_quantises_like_the_append_and_attention_reads_it(hq, hkv, dtype):
    """Whole prompts written token by token (flat batch, shuffled order) into an 8-bit pool that starts as a fill
    pattern: every byte of every unit equals the oracle's quantised write, and attention over them matches the oracle."""
    lens = np.array([1, 16, 17, 100, 45], dtype=np.int32)
    case = fp8_case(2, hq, hkv, 128, dtype, lens, seed=61)
    seqs, poss = [], []
    for s in range(case.S):
        for t in range(int(lens[s])):
            seqs.append(s); poss.append(t)
    order = synth.seeded_permutation(61, len(seqs), salt=9)
    seqs, poss = np.array(seqs, np.int32)[order], np.array(poss, np.int32)[order]
    case.gpu_pool[:] = 0x55
    pc = PoolCase(case)
    dev = torch.device("cuda:0")
    seq_dev, pos_dev = torch.from_numpy(seqs).to(dev), torch.from_numpy(poss).to(dev)
    for l in range(case.L):
        k = synth.tensor_bits(61, synth.STREAM_KNEW, (len(seqs), hkv, 128), dtype, offset=l * 1_000_000)
        v = synth.tensor_bits(61, synth.STREAM_VNEW, (len(seqs), hkv, 128), dtype, gain=0.5, offset=l * 1_000_000)
        k_dev, v_dev = torch.from_numpy(k.view(np.int16)).to(dev), torch.from_numpy(v.view(np.int16)).to(dev)
        torch.cuda.synchronize()
        pie.pie_kv_write(pc.pool, l, k_dev.data_ptr(), v_dev.data_ptr(), seq_dev.data_ptr(), pos_dev.data_ptr(), len(seqs),
                         pc.bt.data_ptr(), case.block_table.shape[1], case.S)
        assert fp8.kv_write(case.gpu_pool, case.host_pool, case.unit_side[l], case.unit_slot[l], k, v, seqs, poss,
                            case.block_table, hkv, 128, dtype, case.k_scale, case.v_scale) == 0
    pie.pie_sync(pc.pool)
    for l in range(case.L):
        for b in range(case.NB):
            assert np.array_equal(pc.read_unit(l, b), pc.unit_bits(l, b)), (l, b)     # written rows and the untouched fill alike
        check(case, pc, l)
    pc.close()
