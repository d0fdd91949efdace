"""Pins of the oracle's paged attention against things other than itself: numpy's half conversion,
dense brute force on contiguous arrays, closed forms and invariances."""
import numpy as np
import pytest

import oracle
from paper_2411_09317_b200 import synth
from tests.helpers import Case, dense_attention

F16, BF16 = synth.F16, synth.BF16


def run(case, layer=0, precision="f32", **kw):
    return oracle.paged_attention(case.gpu_pool, case.host_pool, case.unit_side[layer], case.unit_slot[layer],
                                  case.q[layer], case.block_table, case.ctx_lens, case.Hq, case.Hkv, case.D,
                                  case.dtype, case.scale, precision=precision, **kw)


def test_half_conversion_all_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    for dtype, want in ((F16, bits.view(np.float16).astype(np.float32)),
                        (BF16, (bits.astype(np.uint32) << 16).view(np.float32))):
        got = oracle.bits_to_f32(bits, dtype)
        nan = np.isnan(want)
        assert np.array_equal(np.isnan(got), nan)  # NaN payloads may be quieted on the way back
        assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


@pytest.mark.parametrize("dtype", [F16, BF16])
@pytest.mark.parametrize("hq,hkv,d", [(8, 4, 64), (4, 4, 128), (8, 1, 128)])
def test_against_dense_brute_force(dtype, hq, hkv, d):
    case = Case(2, hq, hkv, d, dtype, [1, 15, 16, 17, 100, 33], seed=3, host_frac=0.5, placement="random",
                shuffle_table=True)
    for layer in range(case.L):
        o64 = run(case, layer, "f64")
        o32 = run(case, layer, "f32")
        for s in range(case.S):
            K, V = case.dense_kv(layer, s)
            want = dense_attention(case.q_f(layer)[s], K, V, case.scale)
            assert np.abs(o64[s] - want).max() < 1e-12
            assert np.abs(o32[s] - want).max() < 2e-6


def test_residency_and_placement_invariance_bit_exact():
    base = Case(2, 8, 4, 64, F16, [100, 231, 300, 17], seed=0, host_frac=0.0, placement="identity")
    ref = [run(base, l) for l in range(base.L)]
    for frac, placement in [(0.5, "random"), (1.0, "reversed"), (0.3, "identity")]:
        c = Case(2, 8, 4, 64, F16, [100, 231, 300, 17], seed=0, host_frac=frac, placement=placement)
        for l in range(c.L):
            assert np.array_equal(run(c, l).view(np.uint32), ref[l].view(np.uint32))


def _set_rows(case, layer, s, kv, fn):
    """Overwrite K (kv=0) or V (kv=1) rows of sequence s: fn(t, kvh) -> float row [D]."""
    for t in range(int(case.ctx_lens[s])):
        b = case.block_table[s, t // 16]
        pool = case.host_pool if case.unit_side[layer, b] else case.gpu_pool
        unit = pool[case.unit_slot[layer, b]].reshape(case.Hkv, 2, 16, case.D)
        for h in range(case.Hkv):
            unit[h, kv, t % 16] = synth.f32_to_16_bits(np.asarray(fn(t, h), dtype=np.float32), case.dtype)


def test_closed_forms():
    c = Case(1, 4, 2, 64, F16, [1, 40, 40, 40, 0], seed=5, host_frac=0.5, placement="random")
    # all K rows equal -> uniform weights -> mean of V (sequence 1)
    _set_rows(c, 0, 1, 0, lambda t, h: np.full(64, 0.25))
    # V constant -> that constant (sequence 2)
    _set_rows(c, 0, 2, 1, lambda t, h: np.full(64, -1.5))
    # one key aligned with q and huge, the others zero -> output = that token's V (sequence 3)
    qf = c.q_f(0)
    _set_rows(c, 0, 3, 0, lambda t, h: (qf[3, 2 * h] * 64.0 if t == 7 else np.zeros(64)))
    out = run(c, 0, "f64")
    K, V = c.dense_kv(0, 0)
    assert np.allclose(out[0], np.repeat(V[0], 2, axis=0), atol=0)          # ctx = 1 -> V[0] exactly
    K, V = c.dense_kv(0, 1)
    assert np.allclose(out[1], np.repeat(V.mean(axis=0), 2, axis=0), atol=1e-13)
    assert np.allclose(out[2], -1.5, atol=1e-13)
    K, V = c.dense_kv(0, 3)
    assert np.abs(out[3, 0] - V[7, 0]).max() < 1e-9                          # head 0 uses its own q
    assert np.array_equal(out[4], np.zeros_like(out[4]))                     # ctx = 0 -> zeros


def test_weights_sum_to_one_and_shift_invariance():
    c = Case(1, 8, 4, 64, BF16, [77, 130], seed=9)
    ref = run(c, 0, "f64")
    # adding the same vector to every key shifts every score by a constant: output unchanged
    c2 = Case(1, 8, 4, 64, BF16, [77, 130], seed=9)
    u = np.linspace(-1, 1, 64).astype(np.float32)
    for s in range(2):
        K, _ = c2.dense_kv(0, s)
        _set_rows(c2, 0, s, 0, lambda t, h: K[t, h] + u)
    # keys were re-rounded to bf16, so compare against brute force on the re-rounded keys
    out = run(c2, 0, "f64")
    for s in range(2):
        K, V = c2.dense_kv(0, s)
        assert np.abs(out[s] - dense_attention(c2.q_f(0)[s], K, V, c2.scale)).max() < 1e-12
    # V == 1 -> out == 1 (weights sum to one)
    for s in range(2):
        _set_rows(c, 0, s, 1, lambda t, h: np.ones(64))
    assert np.allclose(run(c, 0, "f64"), 1.0, atol=1e-13)
    assert np.allclose(run(c, 0, "f32"), 1.0, atol=1e-5)
    assert ref.shape == (2, 8, 64)


def test_gqa_equals_mha_with_replicated_heads():
    g = Case(1, 8, 2, 64, F16, [50, 19], seed=4)
    m = Case(1, 8, 8, 64, F16, [50, 19], seed=4)
    for b in range(g.NB):
        src = g.gpu_pool[g.unit_slot[0, b]].reshape(2, 2, 16, 64)
        m.gpu_pool[m.unit_slot[0, b]] = np.repeat(src, 4, axis=0).ravel()
    m.q = g.q
    assert np.array_equal(run(g, 0).view(np.uint32), run(m, 0).view(np.uint32))


def test_sequence_permutation():
    c = Case(1, 4, 4, 64, F16, [30, 64, 5], seed=6)
    ref = run(c, 0)
    perm = [2, 0, 1]
    out = oracle.paged_attention(c.gpu_pool, c.host_pool, c.unit_side[0], c.unit_slot[0], c.q[0][perm],
                                 c.block_table[perm], c.ctx_lens[perm], c.Hq, c.Hkv, c.D, c.dtype, c.scale)
    assert np.array_equal(out.view(np.uint32), ref[perm].view(np.uint32))


def test_tail_poison_is_never_read():
    c = Case(1, 4, 2, 64, F16, [5, 17, 33], seed=8)
    ref = run(c, 0)
    for s in range(c.S):
        ctx = int(c.ctx_lens[s])
        b = c.block_table[s, (ctx - 1) // 16]
        unit = c.gpu_pool[c.unit_slot[0, b]].reshape(c.Hkv, 2, 16, c.D)
        unit[:, :, ctx % 16 or 16:, :] = 0x7E00  # fp16 NaN
        if ctx % 16:
            unit[:, 1, ctx % 16:, 0] = 0x7C00     # +inf
    assert np.array_equal(run(c, 0).view(np.uint32), ref.view(np.uint32))


@pytest.mark.parametrize("chunk", [16, 48, 512])
def test_split_invariance_and_merge_rule(chunk):
    c = Case(1, 8, 4, 64, BF16, [1, 16, 100, 513], seed=2, host_frac=0.4, placement="random")
    full64 = run(c, 0, "f64")
    split64 = run(c, 0, "f64", split_tokens=chunk)
    assert np.abs(full64 - split64).max() < 1e-13
    split32 = run(c, 0, "f32", split_tokens=chunk)
    assert np.abs(full64 - split32).max() < 2e-6


def test_merge_rule_by_hand():
    # partial 1: one token with score 0 and value 1; partial 2: one token with score ln 3 and value 5.
    # softmax weights are 1/4 and 3/4 -> out = 0.25 * 1 + 0.75 * 5 = 4.
    m, l, acc = oracle.merge(0.0, 1.0, [1.0], np.log(3.0), 1.0, [5.0], "f64")
    assert m == pytest.approx(np.log(3.0)) and l == pytest.approx(4.0 / 3.0)
    assert acc[0] / l == pytest.approx(4.0, abs=1e-14)
    # order reversed gives the same
    m, l, acc = oracle.merge(np.log(3.0), 1.0, [5.0], 0.0, 1.0, [1.0], "f64")
    assert acc[0] / l == pytest.approx(4.0, abs=1e-14)
    # an empty partial (-inf, 0, 0) is the identity on either side and never yields NaN
    m, l, acc = oracle.merge(-np.inf, 0.0, [0.0], 2.0, 3.0, [7.0], "f32")
    assert (m, l, acc[0]) == (2.0, 3.0, 7.0)
    m, l, acc = oracle.merge(2.0, 3.0, [7.0], -np.inf, 0.0, [0.0], "f32")
    assert (m, l, acc[0]) == (2.0, 3.0, 7.0)
    m, l, acc = oracle.merge(-np.inf, 0.0, [0.0], -np.inf, 0.0, [0.0], "f32")
    assert l == 0.0 and not np.isnan(acc[0])


def test_append_writes_position_ctx_minus_one():
    c = Case(1, 4, 2, 64, F16, [16, 17, 1], seed=12, host_frac=0.5, placement="random", extra_tokens=1)
    k_new = synth.tensor_bits(12, synth.STREAM_KNEW, (c.S, c.Hkv, c.D), F16)
    v_new = synth.tensor_bits(12, synth.STREAM_VNEW, (c.S, c.Hkv, c.D), F16)
    g0, h0 = c.gpu_pool.copy(), c.host_pool.copy()
    lens = c.ctx_lens + 1
    oracle.append(c.gpu_pool, c.host_pool, c.unit_side[0], c.unit_slot[0], k_new, v_new, c.block_table, lens, c.Hkv, c.D)
    changed = int((c.gpu_pool != g0).sum() + (c.host_pool != h0).sum())
    assert changed <= c.S * c.Hkv * c.D * 2 and changed > 0
    c.ctx_lens = lens
    for s in range(c.S):
        K, V = c.dense_kv(0, s)
        assert np.array_equal(K[-1], synth.bits16_to_f32(k_new[s], F16))
        assert np.array_equal(V[-1], synth.bits16_to_f32(v_new[s], F16))


# ---- prefill-side write of many tokens (the oracle's definition against an independent reader) ----------------
def test_kv_write_then_paged_attention_equals_dense_attention_on_the_source_arrays():
    """The writer is tied to the reader, which is itself pinned against the dense brute force: a prompt written token
    by token from dense K/V arrays must attend exactly like those arrays (a swapped K/V half, a transposed head/row
    index or an off-by-one position fails)."""
    rng = np.random.default_rng(5)
    c = Case(1, 8, 4, 64, F16, [1, 16, 17, 45], seed=21, host_frac=0.5, placement="random", shuffle_table=True)
    c.gpu_pool[:] = 0x7e00          # NaN everywhere: whatever is not written must not be read
    c.host_pool[:] = 0x7e00
    dense = {}
    seqs, poss, ks, vs = [], [], [], []
    for s in range(c.S):
        ctx = int(c.ctx_lens[s])
        K = rng.standard_normal((ctx, c.Hkv, c.D)).astype(np.float16)
        V = rng.standard_normal((ctx, c.Hkv, c.D)).astype(np.float16)
        dense[s] = (K, V)
        for t in range(ctx):
            seqs.append(s); poss.append(t); ks.append(K[t].view(np.uint16)); vs.append(V[t].view(np.uint16))
    order = rng.permutation(len(seqs))         # any order of the flat batch
    st = oracle.kv_write(c.gpu_pool, c.host_pool, c.unit_side[0], c.unit_slot[0], np.stack(ks)[order], np.stack(vs)[order],
                         np.array(seqs)[order], np.array(poss)[order], c.block_table, c.Hkv, c.D)
    assert st == 0
    out = run(c, 0, "f64")
    for s in range(c.S):
        K, V = dense[s]
        want = dense_attention(c.q_f(0)[s], K.astype(np.float64), V.astype(np.float64), c.scale)
        assert np.abs(out[s] - want).max() < 1e-12


def test_kv_write_of_one_token_per_sequence_is_the_append_and_touches_nothing_else():
    c = Case(1, 4, 2, 64, F16, [16, 17, 1, 40], seed=12, host_frac=0.5, placement="random", extra_tokens=1)
    k_new = synth.tensor_bits(12, synth.STREAM_KNEW, (c.S, c.Hkv, c.D), F16)
    v_new = synth.tensor_bits(12, synth.STREAM_VNEW, (c.S, c.Hkv, c.D), F16)
    g1, h1 = c.gpu_pool.copy(), c.host_pool.copy()
    lens = c.ctx_lens + 1
    oracle.append(g1, h1, c.unit_side[0], c.unit_slot[0], k_new, v_new, c.block_table, lens, c.Hkv, c.D)
    g2, h2 = c.gpu_pool.copy(), c.host_pool.copy()
    assert oracle.kv_write(g2, h2, c.unit_side[0], c.unit_slot[0], k_new, v_new, np.arange(c.S), lens - 1, c.block_table,
                           c.Hkv, c.D) == 0
    assert np.array_equal(g1, g2) and np.array_equal(h1, h2)
    assert int((g2 != c.gpu_pool).sum() + (h2 != c.host_pool).sum()) <= c.S * c.Hkv * c.D * 2
    # a position beyond the table, a sequence that does not exist: nothing is written
    g3, h3 = c.gpu_pool.copy(), c.host_pool.copy()
    for seq, pos in ((0, 16 * c.block_table.shape[1]), (c.S, 0), (0, -1)):
        assert oracle.kv_write(g3, h3, c.unit_side[0], c.unit_slot[0], k_new[:2], v_new[:2], [1, seq], [3, pos],
                               c.block_table, c.Hkv, c.D) == -1
    assert np.array_equal(g3, c.gpu_pool) and np.array_equal(h3, c.host_pool)
