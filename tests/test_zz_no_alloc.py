"""The allocation-free attention entry point against the regular one.

Some users of the library cannot allocate device memory at the point where they need attention (another
component owns the arena, or they run inside a loop that must not synchronise the device), so
pie_decode_attention_noalloc takes every buffer from the caller and keeps its split-K scratch in a fixed
device array inside the library.  It runs the same kernels, so its output must equal the pool entry point's
bit for bit; two calls in a row check that the shared scratch carries nothing over from one call to the next.
This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2411_09317_b200 import binding as pie
from paper_2411_09317_b200 import synth
from tests.gpu_helpers import oracle_attention
from tests.helpers import Case, tolerance

pytestmark = pytest.mark.gpu


def run_both(case, split=0, break_block=None, ctx_dev_override=None):
    """-> (bits from pie_decode_attention, bits from pie_decode_attention_noalloc, the four status words) for layer 0.
    break_block: that logical block's slot-table entry is -1 in the table the second entry point gets;
    ctx_dev_override: the device copy of the lengths the second entry point gets (the host copy stays the case's)."""
    dev = torch.device("cuda:0")
    n_slots = case.NB + 3
    BB = case.block_bytes
    kv = torch.zeros(n_slots * BB, dtype=torch.uint8, device=dev)
    pool = pie.pie_pool_create(n_layers=1, n_q_heads=case.Hq, n_kv_heads=case.Hkv, head_dim=case.D, dtype=case.dtype,
                               n_logical_blocks=case.NB, max_seqs=case.S, n_gpu_slots=n_slots, n_host_slots=1,
                               gpu_base=kv.data_ptr(), split_tokens=split)
    pie.pie_block_alloc(pool, case.NB)
    for b in range(case.NB):
        pie.pie_block_write(pool, 0, b, case.gpu_pool[case.unit_slot[0, b]])
    side, slot = pie.pie_get_placement(pool, 1, case.NB)
    q = torch.from_numpy(case.q[0].view(np.int16)).to(dev)
    bt = torch.from_numpy(case.block_table).to(dev)
    ctx = torch.from_numpy(case.ctx_lens.astype(np.int32)).to(dev)
    out_a = torch.zeros_like(q)
    out_b = torch.full_like(q, 0x5555)
    slots = slot[0].astype(np.int32)
    if break_block is not None:
        slots[break_block] = -1
    slot_table = torch.from_numpy(slots).to(dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    ctx_b = ctx if ctx_dev_override is None else torch.from_numpy(np.asarray(ctx_dev_override, np.int32)).to(dev)
    torch.cuda.synchronize()
    pie.pie_decode_attention(pool, 0, q.data_ptr(), out_a.data_ptr(), bt.data_ptr(), case.block_table.shape[1],
                             ctx.data_ptr(), case.S, case.scale, block_table_host=case.block_table,
                             ctx_lens_host=case.ctx_lens)
    pie.pie_sync(pool)
    stream = torch.cuda.Stream()
    pie.pie_decode_attention_noalloc(kv.data_ptr(), n_slots, slot_table.data_ptr(), case.NB, q.data_ptr(), out_b.data_ptr(),
                                     bt.data_ptr(), case.block_table.shape[1], ctx_b.data_ptr(), case.ctx_lens, case.S,
                                     case.Hq, case.Hkv, case.D, case.dtype, case.scale, split_tokens=split,
                                     status_dev=status.data_ptr(), stream=stream.cuda_stream)
    stream.synchronize()
    a = out_a.cpu().numpy().view(np.uint16)
    b = out_b.cpu().numpy().view(np.uint16)
    pie.pie_pool_destroy(pool)
    return a, b, status.cpu().numpy()


def test_noalloc_matches_pool_entry_point_on_two_calls_in_a_row():
    # first call: long ragged batch; second call: a different, smaller shape that reuses the same scratch
    first = Case(1, 8, 2, 128, synth.BF16, [513, 17, 1, 300, 0, 2049], seed=31, placement="random")
    second = Case(1, 8, 4, 64, synth.F16, [100, 231, 33], seed=32, placement="reversed")
    for case, split in ((first, 0), (second, 64)):
        a, b, status = run_both(case, split)
        assert np.array_equal(a, b)
        assert status[:3].tolist() == [0, 0, 0] and status[3] == int(case.ctx_lens.sum())
        want = oracle_attention(case, 0)
        got = synth.bits16_to_f32(b, case.dtype)
        bound = tolerance(want, case.dtype)
        assert np.all(np.abs(got - want) <= bound)


def test_noalloc_beyond_1024_sequences_takes_its_chunk_offsets_from_the_static_array():
    """More sequences than the kernel scans in shared memory: the chunk offsets come from a plan kernel that writes them
    into the static scratch.  Short contexts keep the case at a few MB."""
    rng = np.random.default_rng(7)
    case = Case(1, 4, 2, 64, synth.F16, rng.integers(0, 40, size=1025).astype(np.int32), seed=33, placement="random")
    a, b, status = run_both(case, 0)
    assert np.array_equal(a, b) and status[:3].tolist() == [0, 0, 0]
    want = oracle_attention(case, 0)
    assert np.all(np.abs(synth.bits16_to_f32(b, case.dtype) - want) <= tolerance(want, case.dtype))


def test_noalloc_flags_what_only_the_device_can_see():
    """A block without a slot, and device lengths that disagree with the host copy the scratch was sized from: flags in the
    caller's status words (no fault: the tile reads slot 0 / nothing is computed), PIE_OK from the call."""
    case = Case(1, 8, 2, 128, synth.BF16, [100, 231, 33], seed=34, placement="random")
    blk = int(case.block_table[1, 3])
    a, b, status = run_both(case, 0, break_block=blk)
    assert status[0] == 1 and status[1] == 0 and status[2] == 0
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[2], b[2])        # the other sequences are as they should be
    # the device says every sequence is 700 tokens long (two chunks each), the host said one chunk each: more chunks than
    # the scratch was sized for -> flagged, nothing computed
    big = Case(1, 8, 2, 128, synth.BF16, [100, 231, 33], seed=34, placement="random", extra_tokens=700)
    _, _, status = run_both(big, 0, ctx_dev_override=[700, 700, 700])
    assert status[1] == 1 and status[2] == 0


def test_noalloc_rejects_what_does_not_fit():
    dev = torch.device("cuda:0")
    dummy = torch.zeros(4096, dtype=torch.uint8, device=dev)
    args = dict(n_logical_blocks=8, q=dummy.data_ptr(), out=dummy.data_ptr(), block_table_dev=dummy.data_ptr(),
                ctx_lens_dev=dummy.data_ptr(), n_q_heads=8, n_kv_heads=8, head_dim=128, dtype=pie.PIE_F16, scale=1.0)
    # more sequences than the fixed scratch is laid out for
    with pytest.raises(pie.PieError) as e:
        pie.pie_decode_attention_noalloc(dummy.data_ptr(), 8, dummy.data_ptr(), max_blocks_per_seq=1,
                                         ctx_lens_host=np.ones(5000, np.int32), n_seqs=5000, **args)
    assert e.value.status == pie.PIE_ERR_NOMEM
    # partials beyond 16 MiB: 64 sequences x 4096 chunks of 16 tokens x 8 heads
    with pytest.raises(pie.PieError) as e:
        pie.pie_decode_attention_noalloc(dummy.data_ptr(), 8, dummy.data_ptr(), max_blocks_per_seq=4096,
                                         ctx_lens_host=np.full(64, 65536, np.int32), n_seqs=64, split_tokens=16, **args)
    assert e.value.status == pie.PIE_ERR_NOMEM
    # a length beyond the table is an argument error
    with pytest.raises(pie.PieError) as e:
        pie.pie_decode_attention_noalloc(dummy.data_ptr(), 8, dummy.data_ptr(), max_blocks_per_seq=2,
                                         ctx_lens_host=np.array([33], np.int32), n_seqs=1, **args)
    assert e.value.status == pie.PIE_ERR_INVALID
