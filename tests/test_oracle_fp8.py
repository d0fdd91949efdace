"""Pins of the 8-bit KV oracle: the E4M3 table and the quantiser against an independent implementation (torch's CPU
float8_e4m3fn), the saturation and tie rules by hand, and attention over E4M3 blocks against the dense brute force on
the decoded values."""
import numpy as np
import pytest
import torch

import oracle
from oracle import fp8
from paper_2411_09317_b200 import synth
from tests.helpers import dense_attention

F16, BF16 = synth.F16, synth.BF16


def test_e4m3_table_matches_an_independent_decoder_for_all_256_codes():
    want = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = fp8.decode(np.arange(256)).astype(np.float32)
    assert np.array_equal(np.isnan(got), np.isnan(want)) and int(np.isnan(got).sum()) == 2
    assert np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
    assert fp8.decode([0x7E, 0xFE, 0x01, 0x08, 0x38])[...].tolist() == [448.0, -448.0, 2.0 ** -9, 2.0 ** -6, 1.0]


def test_quantiser_nearest_even_saturating():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(4000) * 3, rng.uniform(-448, 448, 4000), rng.uniform(-2 ** -5, 2 ** -5, 2000)])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = fp8.quantize(x.astype(np.float32))
    assert np.array_equal(got, want)                      # in range, the two agree everywhere (round to nearest even)
    # every representable value is a fixed point; exact midpoints go to the even code
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    assert np.array_equal(fp8.quantize(fp8.decode(codes)) & 0x7F, codes & 0x7F)
    pos = fp8.decode(np.arange(127))
    mid = (pos[:-1] + pos[1:]) / 2
    q = fp8.quantize(mid)
    assert np.all(q % 2 == 0) and np.all((q == np.arange(126)) | (q == np.arange(1, 127)))
    # beyond the largest finite value: saturate (the fn format has no infinity), keep the sign; NaN stays NaN
    assert fp8.quantize([449.0, 1e9, -500.0, np.inf, -np.inf]).tolist() == [0x7E, 0x7E, 0xFE, 0x7E, 0xFE]
    assert fp8.quantize([np.nan])[0] == 0x7F
    assert fp8.quantize([0.0, -0.0, 1e-6]).tolist() == [0x00, 0x80, 0x00]


@pytest.mark.parametrize("dtype", [F16, BF16])
def test_16_bit_images_of_e4m3_values_are_exact(dtype):
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    back = synth.bits16_to_f32(fp8.to_bits16(codes, dtype), dtype)
    assert np.array_equal(back.astype(np.float64), fp8.decode(codes))


@pytest.mark.parametrize("dtype,hq,hkv", [(F16, 8, 4), (BF16, 8, 1)])
def test_attention_over_e4m3_blocks_equals_dense_attention_on_the_decoded_values(dtype, hq, hkv):
    rng = np.random.default_rng(11)
    D, lens = 64, np.array([1, 16, 17, 50], dtype=np.int32)
    table, nblk, NB = synth.build_block_table(lens, 16)
    side = rng.integers(0, 2, NB).astype(np.int32)
    slot = rng.permutation(NB).astype(np.int32)
    g8 = rng.integers(0, 256, (NB, hkv * 2 * 16 * D)).astype(np.uint8)
    h8 = rng.integers(0, 256, (NB, hkv * 2 * 16 * D)).astype(np.uint8)
    for pool in (g8, h8):                                  # no NaN codes, moderate magnitudes
        pool[(pool & 0x7F) == 0x7F] ^= 1
        pool &= 0xBF                                       # clear the top exponent bit: |value| < 2
    q = synth.tensor_bits(5, synth.STREAM_Q, (len(lens), hq, D), dtype)
    k_scale, v_scale, scale = 0.5, 2.0, 1.0 / 8.0
    out = fp8.paged_attention(g8, h8, side, slot, q, table, lens, hq, hkv, D, dtype, scale, k_scale, v_scale, precision="f64")
    qf = synth.bits16_to_f32(q, dtype).astype(np.float64)
    for s, ctx in enumerate(lens):
        K = np.zeros((ctx, hkv, D))
        V = np.zeros((ctx, hkv, D))
        for t in range(ctx):
            b = table[s, t // 16]
            tile = (h8 if side[b] else g8)[slot[b]].reshape(hkv, 2, 16, D)
            K[t] = fp8.decode(tile[:, 0, t % 16, :]) * k_scale
            V[t] = fp8.decode(tile[:, 1, t % 16, :]) * v_scale
        want = dense_attention(qf[s], K, V, scale)
        assert np.abs(out[s] - want).max() < 1e-12


def test_append_quantises_and_writes_position_ctx_minus_one():
    rng = np.random.default_rng(2)
    hkv, D, lens = 2, 64, np.array([17, 1, 32], dtype=np.int32)
    table, nblk, NB = synth.build_block_table(lens, 16)
    side = np.zeros(NB, np.int32)
    slot = np.arange(NB, dtype=np.int32)
    g8 = np.full((NB, hkv * 2 * 16 * D), 0x7F, np.uint8)
    k_new = synth.tensor_bits(9, synth.STREAM_KNEW, (len(lens), hkv, D), F16)
    v_new = synth.tensor_bits(9, synth.STREAM_VNEW, (len(lens), hkv, D), F16)
    before = g8.copy()
    fp8.append(g8, None, side, slot, k_new, v_new, table, lens, hkv, D, F16, 0.25, 4.0)
    assert int((g8 != before).sum()) <= len(lens) * hkv * D * 2
    for s, ctx in enumerate(lens):
        pos = ctx - 1
        tile = g8[slot[table[s, pos // 16]]].reshape(hkv, 2, 16, D)
        kf = synth.bits16_to_f32(k_new[s], F16).astype(np.float64)
        vf = synth.bits16_to_f32(v_new[s], F16).astype(np.float64)
        # the stored value times the scale is within half an E4M3 step of the input (relative 2^-4, absolute 2^-10 * scale)
        assert np.all(np.abs(fp8.decode(tile[:, 0, pos % 16, :]) * 0.25 - kf) <= np.maximum(np.abs(kf) * 2.0 ** -4, 0.25 * 2.0 ** -10))
        assert np.all(np.abs(fp8.decode(tile[:, 1, pos % 16, :]) * 4.0 - vf) <= np.maximum(np.abs(vf) * 2.0 ** -4, 4.0 * 2.0 ** -10))


def test_generated_bytes_are_finite_values_of_both_signs():
    from paper_2411_09317_b200 import synth
    b = synth.kv_unit_bytes(3, 1, 2, 10, 4, 128)
    assert b.shape == (4, 2, 16, 128) and b.dtype == np.uint8
    v = fp8.decode(b)
    assert np.all(np.isfinite(v)) and (v < 0).any() and (v > 0).any()
    assert 2.0 ** -4 <= np.abs(v).min() and np.abs(v).max() <= 15.0
    assert len(np.unique(b)) > 100                       # signs, mantissas and eight exponents all occur
    assert not np.array_equal(b, synth.kv_unit_bytes(3, 1, 3, 10, 4, 128))


def test_prompt_write_equals_token_by_token_append_and_reads_back_through_attention():
    """The prefill-side write of a whole prompt leaves the bytes the append leaves when the same tokens arrive one by one,
    touches nothing else, and rejects positions beyond the table."""
    rng = np.random.default_rng(4)
    hkv, d, n_tok = 2, 128, 37
    nb = (n_tok + 15) // 16
    k = rng.normal(0, 2.0, (n_tok, hkv, d)).astype(np.float16).view(np.uint16)
    v = rng.normal(0, 1.0, (n_tok, hkv, d)).astype(np.float16).view(np.uint16)
    table = np.arange(nb, dtype=np.int32)[::-1].copy()[None, :]          # blocks in reverse order
    side, slot = np.zeros(nb, np.int32), np.arange(nb, dtype=np.int32)
    a = np.full((nb, hkv * 2 * 16 * d), 0x55, dtype=np.uint8)
    b = a.copy()
    order = rng.permutation(n_tok)
    assert fp8.kv_write(a, a, side, slot, k[order], v[order], np.zeros(n_tok, np.int32), order.astype(np.int32), table, hkv, d,
                        fp8.F16, 0.25, 0.5) == 0
    for t in range(n_tok):
        fp8.append(b, b, side, slot, k[t:t + 1], v[t:t + 1], table, np.array([t + 1], np.int32), hkv, d, fp8.F16, 0.25, 0.5)
    assert np.array_equal(a, b)
    tail = a[slot[table[0, nb - 1]]].reshape(hkv, 2, 16, d)[:, :, n_tok % 16:, :]
    assert np.all(tail == 0x55)                                            # rows beyond the prompt untouched
    assert fp8.kv_write(a, a, side, slot, k[:1], v[:1], np.zeros(1, np.int32), np.array([16 * nb], np.int32), table, hkv, d,
                        fp8.F16, 0.25, 0.5) == -1
    assert np.array_equal(a, b)
