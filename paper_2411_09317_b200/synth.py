"""Seeded synthetic inputs for the KV-swap + paged-decode-attention path.

This module is the only code shared by the tests' CPU oracle side and the CUDA
side.  It holds none of the method's arithmetic: it only draws numbers and
builds integer tables (lengths, block tables, host-resident sets).

Generator (counter based, so that the CUDA fill kernel in ``csrc/pie_synth.cu``
reproduces the same bits): for element index ``i`` of stream ``stream`` under
``seed`` three 64-bit hashes ``mix64(base + GOLDEN * (3 i + j + 1))`` are drawn,
their twelve 16-bit fields are summed, 393210 (the mean) is subtracted and the
integer is scaled by 2**-16 in fp32: an Irwin-Hall(12) variate with mean 0 and
variance 1 - 2**-32, exact in integer/fp32 arithmetic.  It is then rounded
(nearest even) to fp16 or bf16.  ``mix64`` is the SplitMix64 finaliser.

The workloads stand in for the request-length mixes of the paper's serving
traces (Section 5.1); no item of those traces is used.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)

F16 = 0
BF16 = 1

# stream ids (one per tensor kind)
STREAM_KV = 1
STREAM_Q = 2
STREAM_KNEW = 3
STREAM_VNEW = 4
STREAM_LEN = 5
STREAM_PICK = 6
STREAM_BYTES = 7


def mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function on uint64 arrays (wrapping arithmetic)."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        z = z ^ (z >> np.uint64(31))
    return z


def stream_base(seed: int, stream: int) -> np.uint64:
    with np.errstate(over="ignore"):
        s = np.uint64(seed) * GOLDEN + np.uint64(stream)
    return mix64(np.array([s], dtype=np.uint64))[0]


def irwin_hall_int(seed: int, stream: int, idx: np.ndarray) -> np.ndarray:
    """Centred integer sum of twelve 16-bit uniforms for each index (int32)."""
    idx = np.asarray(idx, dtype=np.uint64)
    base = stream_base(seed, stream)
    acc = np.zeros(idx.shape, dtype=np.int64)
    with np.errstate(over="ignore"):
        for j in range(3):
            h = mix64(base + GOLDEN * (idx * np.uint64(3) + np.uint64(j + 1)))
            for k in range(4):
                acc += ((h >> np.uint64(16 * k)) & np.uint64(0xFFFF)).astype(np.int64)
    return (acc - 393210).astype(np.int32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    b = np.asarray(x, dtype=np.float32).view(np.uint32)
    r = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + r) >> np.uint32(16)).astype(np.uint16)


def f32_to_16_bits(x: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == F16:
        return np.asarray(x, dtype=np.float32).astype(np.float16).view(np.uint16)
    return f32_to_bf16_bits(x)


def bits16_to_f32(bits: np.ndarray, dtype: int) -> np.ndarray:
    bits = np.asarray(bits, dtype=np.uint16)
    if dtype == F16:
        return bits.view(np.float16).astype(np.float32)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bits(seed: int, stream: int, idx: np.ndarray, dtype: int, gain: float = 1.0) -> np.ndarray:
    """16-bit patterns of ~N(0,1) values (times ``gain``, a power of two keeps it exact)."""
    v = irwin_hall_int(seed, stream, idx).astype(np.float32) * np.float32(2.0 ** -16)
    if gain != 1.0:
        v = v * np.float32(gain)
    return f32_to_16_bits(v, dtype)


def uniform_u32(seed: int, stream: int, idx: np.ndarray) -> np.ndarray:
    idx = np.asarray(idx, dtype=np.uint64)
    base = stream_base(seed, stream)
    with np.errstate(over="ignore"):
        h = mix64(base + GOLDEN * (idx + np.uint64(1)))
    return (h >> np.uint64(32)).astype(np.uint32)


# --------------------------------------------------------------------------------------
# KV element indexing: content is a function of the LOGICAL identity of an element only
# (layer, logical block, kv head, k-or-v, row in block, d), never of the slot it sits in.
# --------------------------------------------------------------------------------------

def kv_unit_indices(layer: int, block: int, n_logical_blocks: int, n_kv_heads: int, head_dim: int,
                    block_tokens: int = 16) -> np.ndarray:
    """Element indices of one (layer, logical block) unit in slot order [Hkv][kv][T][D]."""
    per_unit = n_kv_heads * 2 * block_tokens * head_dim
    unit = np.uint64(layer) * np.uint64(n_logical_blocks) + np.uint64(block)
    return unit * np.uint64(per_unit) + np.arange(per_unit, dtype=np.uint64)


def kv_unit_bits(seed: int, layer: int, block: int, n_logical_blocks: int, n_kv_heads: int, head_dim: int,
                 dtype: int, gain: float = 1.0) -> np.ndarray:
    """uint16 [Hkv][2][16][D] contents of one (layer, logical block) unit."""
    idx = kv_unit_indices(layer, block, n_logical_blocks, n_kv_heads, head_dim)
    return normal_bits(seed, STREAM_KV, idx, dtype, gain).reshape(n_kv_heads, 2, 16, head_dim)


def kv_unit_bytes(seed: int, layer: int, block: int, n_logical_blocks: int, n_kv_heads: int, head_dim: int) -> np.ndarray:
    """uint8 [Hkv][2][16][D] contents of one (layer, logical block) unit of an 8-bit pool: bytes with a random sign bit,
    a random 3-bit mantissa and an exponent field of 3 .. 10 (so never the all-ones exponent)."""
    idx = kv_unit_indices(layer, block, n_logical_blocks, n_kv_heads, head_dim)
    base = stream_base(seed, STREAM_KV)
    with np.errstate(over="ignore"):
        h = mix64(base + GOLDEN * (idx + np.uint64(1)))
    b = ((h >> np.uint64(32)) & np.uint64(0x87)) | ((((h >> np.uint64(40)) & np.uint64(7)) + np.uint64(3)) << np.uint64(3))
    return b.astype(np.uint8).reshape(n_kv_heads, 2, 16, head_dim)


def tensor_bits(seed: int, stream: int, shape, dtype: int, gain: float = 1.0, offset: int = 0) -> np.ndarray:
    n = int(np.prod(shape))
    idx = np.arange(n, dtype=np.uint64) + np.uint64(offset)
    return normal_bits(seed, stream, idx, dtype, gain).reshape(shape)


# --------------------------------------------------------------------------------------
# integer structure: lengths, block tables, host-resident sets
# --------------------------------------------------------------------------------------

def uniform_lengths(seed: int, n: int, lo: int, hi: int) -> np.ndarray:
    u = uniform_u32(seed, STREAM_LEN, np.arange(n)).astype(np.uint64)
    return (lo + (u * np.uint64(hi - lo + 1) >> np.uint64(32))).astype(np.int32)


def lognormal_lengths(seed: int, n: int, median: float, sigma: float, lo: int, hi: int) -> np.ndarray:
    z = irwin_hall_int(seed, STREAM_LEN, np.arange(n)).astype(np.float64) * 2.0 ** -16
    v = np.exp(math.log(median) + sigma * z)
    return np.clip(np.rint(v), lo, hi).astype(np.int32)


def build_block_table(ctx_lens: np.ndarray, block_tokens: int = 16, extra_tokens: int = 0,
                      shuffle_seed: int | None = None):
    """Assign logical block ids to sequences.

    Every sequence gets ceil((ctx + extra_tokens) / block_tokens) blocks.  Ids are handed out
    in sequence order, or in a seeded random permutation when ``shuffle_seed`` is given.
    Returns (block_table int32 [S][max_blocks] padded with -1, n_blocks_per_seq, n_logical).
    """
    ctx_lens = np.asarray(ctx_lens, dtype=np.int64)
    nblk = (ctx_lens + extra_tokens + block_tokens - 1) // block_tokens
    total = int(nblk.sum())
    ids = np.arange(total, dtype=np.int32)
    if shuffle_seed is not None:
        ids = ids[seeded_permutation(shuffle_seed, total, salt=17)]
    max_blocks = int(nblk.max()) if len(nblk) else 0
    table = np.full((len(ctx_lens), max(max_blocks, 1)), -1, dtype=np.int32)
    p = 0
    for s, nb in enumerate(nblk):
        table[s, :nb] = ids[p:p + nb]
        p += int(nb)
    return table, nblk.astype(np.int32), total


def seeded_permutation(seed: int, n: int, salt: int = 0) -> np.ndarray:
    """Fisher-Yates shuffle driven by the counter-based generator."""
    perm = np.arange(n, dtype=np.int64)
    if n <= 1:
        return perm
    u = uniform_u32(seed, STREAM_PICK, np.arange(n, dtype=np.uint64) + np.uint64(salt) * np.uint64(1 << 32))
    for i in range(n - 1, 0, -1):
        j = int((int(u[i]) * (i + 1)) >> 32)
        perm[i], perm[j] = perm[j], perm[i]
    return perm


def pick_host_blocks(seed: int, block_table: np.ndarray, nblk: np.ndarray, frac: float) -> np.ndarray:
    """Per sequence, a seeded choice of round(frac * n_blocks) of its blocks (sorted ids)."""
    out = []
    for s in range(block_table.shape[0]):
        nb = int(nblk[s])
        k = int(round(frac * nb))
        if k <= 0:
            continue
        perm = seeded_permutation(seed, nb, salt=1000 + s)
        out.append(block_table[s, np.sort(perm[:k])])
    if not out:
        return np.zeros(0, dtype=np.int32)
    return np.sort(np.concatenate(out)).astype(np.int32)


def random_bytes(seed: int, n: int, offset: int = 0) -> np.ndarray:
    """Opaque bytes for swap tests (n must be a multiple of 8)."""
    assert n % 8 == 0
    idx = np.arange(n // 8, dtype=np.uint64) + np.uint64(offset)
    base = stream_base(seed, STREAM_BYTES)
    with np.errstate(over="ignore"):
        h = mix64(base + GOLDEN * (idx + np.uint64(1)))
    return h.view(np.uint8)


# --------------------------------------------------------------------------------------
# named workloads (shapes of the benchmark configurations)
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class Workload:
    name: str
    seed: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: int
    ctx_lens: np.ndarray          # int32 [S], context BEFORE the first decode step's append
    decode_steps: int
    host_frac: float
    block_tokens: int = 16
    kv_fp8: bool = False          # blocks hold one byte per element (an 8-bit variant) instead of the 16-bit type

    @property
    def n_seqs(self) -> int:
        return int(len(self.ctx_lens))

    @property
    def block_bytes(self) -> int:
        return 2 * self.block_tokens * self.n_kv_heads * self.head_dim * (1 if self.kv_fp8 else 2)

    def tables(self, shuffle: bool = False, extra_tokens: int | None = None):
        """Block table with room for `extra_tokens` decoded tokens per sequence (default: decode_steps)."""
        return build_block_table(self.ctx_lens, self.block_tokens,
                                 extra_tokens=self.decode_steps if extra_tokens is None else extra_tokens,
                                 shuffle_seed=self.seed if shuffle else None)


def workload(name: str, scale: float = 1.0) -> Workload:
    """The benchmark configurations; ``scale`` < 1 keeps shapes but uses fewer sequences/layers."""
    def sc(n, lo=1):
        return max(lo, int(round(n * scale)))
    if name == "tiny":
        return Workload("tiny", 0, 2, 8, 4, 64, F16, uniform_lengths(0, 4, 100, 300), 1, 0.5)
    if name == "llama2_7b":
        return Workload("llama2_7b", 1, sc(32, 2), 32, 32, 128, F16,
                        uniform_lengths(1, sc(64, 2), 512, 2048), 16, 0.3)
    if name == "llama3_8b":
        return Workload("llama3_8b", 2, sc(32, 2), 32, 8, 128, BF16,
                        lognormal_lengths(2, sc(128, 2), 1000.0, 0.8, 32, 8192), 256, 0.0)
    if name == "llama3_70b":
        lens = uniform_lengths(3, 32, 4096, 32768)
        # keep the longest prefix of the seeded batch whose KV fits 2 x 40 GB (80 layers x 4 KiB/token)
        per_tok = 80 * 2 * 8 * 128 * 2
        keep = int(np.searchsorted(np.cumsum(lens.astype(np.int64)) * per_tok, 80e9, side="right"))
        return Workload("llama3_70b", 3, sc(80, 2), 64, 8, 128, BF16, lens[:max(1, sc(keep))], 16, 0.5)
    if name == "swap_attn":
        # the attention kernel the swap microbenchmark runs beside: 128 sequences x 4096 tokens
        return Workload("swap_attn", 4, 1, 32, 8, 128, BF16, np.full(sc(128, 2), 4096, dtype=np.int32), 0, 0.0)
    raise ValueError(name)
