"""Pins of the chunked-prefill oracle: against single-token decode calls of the (separately pinned) decode oracle, against
a library routine on dense arrays with an explicit causal mask, closed forms, and causality itself."""
import numpy as np
import pytest
import torch

import oracle
from oracle import prefill
from paper_2411_09317_b200 import synth
from tests.helpers import Case

F16, BF16 = synth.F16, synth.BF16


def chunked(case, chunk_lens, seed=3):
    """q for chunks of the given lengths at the end of each sequence's context -> (q bits [n_tokens][Hq][D], offsets)."""
    off = np.concatenate([[0], np.cumsum(chunk_lens)]).astype(np.int64)
    q = synth.tensor_bits(seed, synth.STREAM_Q, (int(off[-1]), case.Hq, case.D), case.dtype)
    return q, off


def run(case, layer, q, off, precision="f64"):
    return prefill.prefill_attention(case.gpu_pool, case.host_pool, case.unit_side[layer], case.unit_slot[layer], q, off,
                                     case.block_table, case.ctx_lens, case.Hq, case.Hkv, case.D, case.dtype, case.scale, precision)


@pytest.mark.parametrize("dtype", [F16, BF16])
def test_all_16_bit_patterns_convert_like_the_decode_oracle(dtype):
    bits = np.arange(65536, dtype=np.uint16)
    a = prefill.bits_to_real(bits, dtype, np.float32)
    b = oracle.bits_to_f32(bits, dtype)
    nan = np.isnan(b)
    assert np.array_equal(np.isnan(a), nan) and nan.sum() > 0                        # NaN patterns stay NaN (payloads aside)
    assert np.array_equal(a[~nan].view(np.uint32), b[~nan].view(np.uint32))          # everything else bit for bit


@pytest.mark.parametrize("hq,hkv,d,dtype", [(4, 4, 64, F16), (8, 2, 128, BF16), (8, 1, 64, F16)])
def test_each_chunk_token_is_a_decode_call_at_its_own_length(hq, hkv, d, dtype):
    case = Case(2, hq, hkv, d, dtype, [37, 5, 64, 130], seed=21, host_frac=0.4, placement="random")
    chunk = [9, 5, 17, 33]
    q, off = chunked(case, chunk)
    got = run(case, 1, q, off)
    for s, C in enumerate(chunk):
        for i in range(C):
            pos = int(case.ctx_lens[s]) - C + i
            want = oracle.paged_attention(case.gpu_pool, case.host_pool, case.unit_side[1], case.unit_slot[1], q[off[s] + i][None],
                                          case.block_table[s:s + 1], [pos + 1], hq, hkv, d, dtype, case.scale, "f64")[0]
            assert np.abs(got[off[s] + i] - want).max() < 1e-12, (s, i)


@pytest.mark.parametrize("hq,hkv", [(4, 4), (8, 2)])
def test_dense_causal_attention_by_a_library_routine(hq, hkv):
    """torch's scaled_dot_product_attention in fp64 on contiguous K, V with an explicit boolean mask (row i of the chunk
    sees columns 0 .. p0 + i) - a different formulation (matrix form, masked softmax) of the same thing."""
    d, dtype = 64, F16
    case = Case(1, hq, hkv, d, dtype, [50, 23, 16], seed=22, host_frac=0.5, placement="reversed")
    chunk = [20, 23, 1]
    q, off = chunked(case, chunk)
    got = run(case, 0, q, off)
    g = hq // hkv
    for s, C in enumerate(chunk):
        ctx = int(case.ctx_lens[s])
        K, V = prefill.gather_kv(case.gpu_pool, case.host_pool, case.unit_side[0], case.unit_slot[0], case.block_table[s], ctx, hkv, d,
                                 dtype, np.float64)
        Q = torch.from_numpy(prefill.bits_to_real(q[off[s]:off[s + 1]], dtype)).permute(1, 0, 2)                 # [Hq][C][D]
        Kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(g, dim=0)                                    # [Hq][ctx][D]
        Vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(g, dim=0)
        mask = torch.arange(ctx)[None, :] <= (ctx - C + torch.arange(C))[:, None]
        want = torch.nn.functional.scaled_dot_product_attention(Q, Kt, Vt, attn_mask=mask, scale=case.scale).permute(1, 0, 2).numpy()
        assert np.abs(got[off[s]:off[s + 1]] - want).max() < 1e-12, s


def test_closed_forms_and_causality():
    case = Case(1, 4, 2, 64, F16, [40, 12], seed=23, host_frac=0.0, placement="identity")
    chunk = [40, 12]                      # whole prompts: the first token of each sees only itself
    q, off = chunked(case, chunk)
    out = run(case, 0, q, off)
    for s in range(2):
        _, V = prefill.gather_kv(case.gpu_pool, case.host_pool, case.unit_side[0], case.unit_slot[0], case.block_table[s],
                                 int(case.ctx_lens[s]), 2, 64, F16, np.float64)
        for h in range(4):
            assert np.array_equal(out[off[s], h], V[0, h // 2])                      # one key: weight 1, out = its value
    # causality: scrambling the keys and values of positions after a token leaves that token's output bit for bit
    blk = int(case.block_table[0, 2])                                                 # positions 32 .. 39 of sequence 0
    tile = case.gpu_pool[case.unit_slot[0, blk]].reshape(2, 2, 16, 64)
    tile[:, :, 4:, :] ^= 0x1234                                                       # positions 36 .. 47
    out2 = run(case, 0, q, off)
    assert np.array_equal(out2[:36], out[:36]) and not np.array_equal(out2[36:40], out[36:40])
    assert np.array_equal(out2[40:], out[40:])                                        # the other sequence is untouched
    # weights sum to one: constant values give that constant, whatever the keys
    tile2 = case.gpu_pool.reshape(-1, 2, 2, 16, 64)
    tile2[:, :, 1, :, :] = synth.f32_to_16_bits(np.array([0.375], np.float32), F16)[0]
    assert np.allclose(run(case, 0, q, off), 0.375, rtol=0, atol=1e-15)


def test_a_chunk_of_one_token_is_decode_and_residency_does_not_matter():
    a = Case(1, 8, 4, 64, BF16, [33, 100], seed=24, host_frac=0.0, placement="identity")
    b = Case(1, 8, 4, 64, BF16, [33, 100], seed=24, host_frac=0.7, placement="random")
    q, off = chunked(a, [1, 1])
    oa, ob = run(a, 0, q, off), run(b, 0, q, off)
    assert np.array_equal(oa, ob)
    want = oracle.paged_attention(a.gpu_pool, a.host_pool, a.unit_side[0], a.unit_slot[0], q, a.block_table, a.ctx_lens, 8, 4, 64,
                                  BF16, a.scale, "f64")
    assert np.abs(oa - want).max() < 1e-12
    with pytest.raises(ValueError):
        run(a, 0, *chunked(a, [34, 1]))                                              # a chunk longer than its context
