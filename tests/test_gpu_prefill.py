"""Chunked-prefill paged attention (tcgen05 / TMEM kernel) against the prefill oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from oracle import prefill
from paper_2411_09317_b200 import binding as pie
from paper_2411_09317_b200 import synth
from tests.gpu_helpers import PoolCase
from tests.helpers import Case, tolerance

pytestmark = pytest.mark.gpu
F16, BF16 = synth.F16, synth.BF16


def run_prefill(case, pc, layer, chunk_lens, seed=9, ctx_lens=None):
    """-> (got fp32 [n_tokens][Hq][D], want fp64) for chunks of the given lengths at the end of each context"""
    ctx = np.asarray(case.ctx_lens if ctx_lens is None else ctx_lens, dtype=np.int32)
    off = np.concatenate([[0], np.cumsum(chunk_lens)]).astype(np.int32)
    n_tok = int(off[-1])
    q = synth.tensor_bits(seed, synth.STREAM_Q, (n_tok, case.Hq, case.D), case.dtype)
    dev = torch.device("cuda:0")
    q_dev = torch.from_numpy(q.view(np.int16)).to(dev)
    out_dev = torch.full_like(q_dev, 0x7e00 if case.dtype == F16 else 0x7fc0)     # NaN: every valid row must be written
    off_dev = torch.from_numpy(off).to(dev)
    ctx_dev = torch.from_numpy(ctx).to(dev)
    pie.pie_prefill_attention(pc.pool, layer, q_dev.data_ptr(), out_dev.data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                              ctx_dev.data_ptr(), off_dev.data_ptr(), ctx, off, len(ctx), case.scale)
    pie.pie_sync(pc.pool)
    got = synth.bits16_to_f32(out_dev.cpu().numpy().view(np.uint16), case.dtype)
    want = prefill.prefill_attention(case.gpu_pool, case.host_pool, case.unit_side[layer], case.unit_slot[layer], q, off, case.block_table,
                                     ctx, case.Hq, case.Hkv, case.D, case.dtype, case.scale)
    return got, want


def check(case, pc, layer, chunk_lens, **kw):
    got, want = run_prefill(case, pc, layer, chunk_lens, **kw)
    err = np.abs(got - want)
    assert np.all(np.isfinite(got))
    assert np.all(err <= tolerance(want, case.dtype)), float(err.max())
    return float(err.max())


def test_one_full_prompt_of_one_tile():
    """The smallest case: one sequence, one KV head, 64 tokens fed as one chunk (one stage, one tile)."""
    case = Case(1, 1, 1, 128, F16, [64], seed=61, host_frac=0.0, placement="identity")
    pc = PoolCase(case, all_on_gpu=True)
    check(case, pc, 0, [64])
    pc.close()


@pytest.mark.parametrize("hq,hkv,d,dtype", [(4, 4, 128, F16), (8, 2, 128, BF16), (8, 1, 128, F16), (4, 2, 64, BF16), (2, 2, 64, F16)])
@pytest.mark.parametrize("chunk", [16, 64, 256])
def test_chunks_after_ragged_prefixes(hq, hkv, d, dtype, chunk):
    """Chunks of one length behind prefixes of every kind: none, shorter than a block, not a multiple of anything, several
    stages long; group sizes 1, 2, 4 and 8, both types, both head sizes; scattered slots."""
    prefixes = [0, 5, 100, 333, 16, 1000]
    ctx = [p + chunk for p in prefixes]
    case = Case(2, hq, hkv, d, dtype, ctx, seed=62, host_frac=0.0, placement="random")
    pc = PoolCase(case, all_on_gpu=True)
    check(case, pc, 1, [chunk] * len(prefixes))
    pc.close()


def test_ragged_chunk_lengths_in_one_call():
    """Chunks of 1 to 1024 tokens in one batch (tiles with a single valid row, tiles that end mid-way, an empty chunk)."""
    chunks = [1, 1024, 0, 37, 130, 64, 257]
    prefixes = [50, 0, 200, 0, 7, 1, 700]
    ctx = [p + c for p, c in zip(prefixes, chunks)]
    case = Case(1, 8, 2, 128, BF16, ctx, seed=63, host_frac=0.0, placement="reversed")
    pc = PoolCase(case, all_on_gpu=True)
    check(case, pc, 0, chunks)
    pc.close()


def test_tail_garbage_and_future_tokens_do_not_leak():
    """Causality and the tail rule on the device: NaN and Inf patterns in the cache beyond a chunk's last position (the
    rest of its last block, and whole blocks of tokens that come later) change nothing."""
    case = Case(1, 4, 2, 128, F16, [300, 90], seed=64, host_frac=0.0, placement="identity")
    chunks = [100, 40]
    clean = Case(1, 4, 2, 128, F16, [300, 90], seed=64, host_frac=0.0, placement="identity")
    # the chunks end at positions 199 and 59: poison everything after them
    for s, last in ((0, 199), (1, 59)):
        for pos in range(last + 1, int(case.ctx_lens[s])):
            tile = case.gpu_pool[case.unit_slot[0, case.block_table[s, pos // 16]]].reshape(2, 2, 16, 128)
            tile[:, :, pos % 16, :] = np.array([0x7e00, 0x7c00, 0xfc00, 0x7bff], dtype=np.uint16)[pos % 4]
    pc, pc_clean = PoolCase(case, all_on_gpu=True), PoolCase(clean, all_on_gpu=True)
    ctx_now = np.array([200, 60], dtype=np.int32)
    got, want = run_prefill(case, pc, 0, chunks, ctx_lens=ctx_now)
    got_clean, _ = run_prefill(clean, pc_clean, 0, chunks, ctx_lens=ctx_now)
    assert np.array_equal(got, got_clean)
    assert np.all(np.abs(got - want) <= tolerance(want, F16))
    pc.close()
    pc_clean.close()


def test_several_waves_of_tiles_sampled_against_the_decode_oracle():
    """More CTAs than the GPU holds at once (fourteen sequences x sixteen tiles x two KV heads), chunks of 512 tokens behind
    1536 cached ones, 32 stages per tile: the warps of a CTA run at their own pace here (softmax warps a stage apart, the
    loading warp behind or ahead of the issuing one).  Sampled rows - first, last and seeded tokens of the chunks - against
    single-token calls of the decode oracle at the token's own context length; every row finite."""
    n_seqs, prefix, chunk = 14, 1536, 512
    ctx = [prefix + chunk] * (n_seqs - 2) + [prefix + chunk - 7, 40 + chunk]
    case = Case(1, 8, 2, 128, BF16, ctx, seed=68, host_frac=0.0, placement="random")
    pc = PoolCase(case, all_on_gpu=True)
    chunks = [chunk] * n_seqs
    off = np.concatenate([[0], np.cumsum(chunks)]).astype(np.int32)
    n_tok = int(off[-1])
    q = synth.tensor_bits(19, synth.STREAM_Q, (n_tok, case.Hq, case.D), case.dtype)
    dev = torch.device("cuda:0")
    q_dev = torch.from_numpy(q.view(np.int16)).to(dev)
    out_dev = torch.full_like(q_dev, 0x7fc0)
    off_dev = torch.from_numpy(off).to(dev)
    ctx_np = np.asarray(ctx, dtype=np.int32)
    ctx_dev = torch.from_numpy(ctx_np).to(dev)
    for _ in range(3):      # (repeated: the failure this guards against depended on timing)
        pie.pie_prefill_attention(pc.pool, 0, q_dev.data_ptr(), out_dev.data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                                  ctx_dev.data_ptr(), off_dev.data_ptr(), ctx_np, off, n_seqs, case.scale)
    pie.pie_sync(pc.pool)
    got = synth.bits16_to_f32(out_dev.cpu().numpy().view(np.uint16), case.dtype)
    assert np.all(np.isfinite(got))
    rng = np.random.default_rng(5)
    samples = [(0, 0), (0, chunk - 1), (n_seqs - 1, 0), (n_seqs - 1, chunk - 1), (n_seqs - 2, 255), (5, 31), (5, 32), (7, 480)]
    samples += [(int(rng.integers(0, n_seqs)), int(rng.integers(0, chunk))) for _ in range(8)]
    for s, i in samples:
        pos = ctx[s] - chunk + i
        want = oracle.paged_attention(case.gpu_pool, case.host_pool, case.unit_side[0], case.unit_slot[0], q[off[s] + i][None],
                                      case.block_table[s:s + 1], np.array([pos + 1], np.int32), case.Hq, case.Hkv, case.D,
                                      case.dtype, case.scale, "f64")[0]
        err = np.abs(got[off[s] + i] - want)
        assert np.all(err <= tolerance(want, case.dtype)), (s, i, float(err.max()))
    pc.close()


def test_rejected_arguments_enqueue_nothing():
    case = Case(1, 4, 2, 128, F16, [64, 64], seed=65, host_frac=0.0, placement="identity")
    pc = PoolCase(case, all_on_gpu=True)
    dev = torch.device("cuda:0")
    q = torch.zeros((80, 4, 128), dtype=torch.int16, device=dev)
    out = torch.zeros_like(q)
    ctx = np.array([64, 64], np.int32)
    ctx_dev = torch.from_numpy(ctx).to(dev)
    for off in ([0, 70, 80], [1, 40, 80], [0, 40, 30]):               # chunk longer than its context; first offset; decreasing
        off = np.array(off, np.int32)
        with pytest.raises(pie.PieError) as e:
            pie.pie_prefill_attention(pc.pool, 0, q.data_ptr(), out.data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                                      ctx_dev.data_ptr(), torch.from_numpy(off).to(dev).data_ptr(), ctx, off, 2, case.scale)
        assert e.value.status == pie.PIE_ERR_INVALID
    too_long = np.array([16 * case.block_table.shape[1] + 1, 64], np.int32)
    with pytest.raises(pie.PieError):
        pie.pie_prefill_attention(pc.pool, 0, q.data_ptr(), out.data_ptr(), pc.bt.data_ptr(), case.block_table.shape[1],
                                  ctx_dev.data_ptr(), ctx_dev.data_ptr(), too_long, np.array([0, 40, 80], np.int32), 2, case.scale)
    pie.pie_sync(pc.pool)
    assert int(out.abs().sum()) == 0
    pc.close()


def test_prompt_in_chunks_through_write_swap_and_attend():
    """The serving order of a chunked prefill: the prompt's K and V enter the cache chunk by chunk (pie_kv_write), blocks of
    earlier chunks are swapped out to the host and brought back before the layer is used again, and each chunk attends to
    everything cached so far.  Outputs of every chunk match the oracle fed the same K and V."""
    hq, hkv, d, dtype = 8, 2, 128, BF16
    lens = [700, 333]
    case = Case(1, hq, hkv, d, dtype, lens, seed=66, host_frac=0.0, placement="identity")
    pc = PoolCase(case, all_on_gpu=True, n_host_slots=case.NB + 4)
    dev = torch.device("cuda:0")
    # the prompt's K and V rows, written by the library instead of by the test's set-up: clear the pool first
    k_all = synth.tensor_bits(66, synth.STREAM_KNEW, (sum(lens), hkv, d), dtype)
    v_all = synth.tensor_bits(66, synth.STREAM_VNEW, (sum(lens), hkv, d), dtype)
    case.gpu_pool[:] = 0
    for b in range(case.NB):
        pie.pie_block_write(pc.pool, 0, b, case.gpu_pool[case.unit_slot[0, b]])
    starts = np.concatenate([[0], np.cumsum(lens)])
    done = np.zeros(2, np.int32)
    chunk = 256
    while np.any(done < lens):
        c = np.minimum(chunk, np.array(lens) - done).astype(np.int32)
        seq = np.concatenate([np.full(c[s], s, np.int32) for s in range(2)])
        pos = np.concatenate([done[s] + np.arange(c[s], dtype=np.int32) for s in range(2)])
        rows = np.concatenate([starts[s] + done[s] + np.arange(c[s]) for s in range(2)])
        k_dev = torch.from_numpy(k_all[rows].view(np.int16)).to(dev)
        v_dev = torch.from_numpy(v_all[rows].view(np.int16)).to(dev)
        seq_dev, pos_dev = torch.from_numpy(seq).to(dev), torch.from_numpy(pos).to(dev)   # (kept alive until the sync below)
        pie.pie_kv_write(pc.pool, 0, k_dev.data_ptr(), v_dev.data_ptr(), seq_dev.data_ptr(), pos_dev.data_ptr(), len(seq),
                         pc.bt.data_ptr(), case.block_table.shape[1], 2)
        assert oracle.kv_write(case.gpu_pool, case.host_pool, case.unit_side[0], case.unit_slot[0], k_all[rows], v_all[rows], seq, pos,
                               case.block_table, hkv, d) == 0
        ctx = (done + c).astype(np.int32)
        got, want = run_prefill(case, pc, 0, c.tolist(), seed=100 + int(done[0]), ctx_lens=ctx)
        assert np.all(np.abs(got - want) <= tolerance(want, dtype)), (done, float(np.abs(got - want).max()))
        done = done + c
        # the blocks written so far leave for the host and come back into other slots before the next chunk
        used = np.unique(np.concatenate([case.block_table[s, :(done[s] + 15) // 16] for s in range(2)]))
        pie.pie_swap_out(pc.pool, 0, used)
        pie.pie_swap_in(pc.pool, 0, used[::-1].copy())
    pie.pie_sync(pc.pool)
    pc.close()
