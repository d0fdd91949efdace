// sm_100a kernels: block gather/scatter swap, slot-table patch, KV append, split-K paged decode
// attention (TMA-staged, mma.sync with the KV tokens on the M axis) and the split-K combine.
#include "pie_kernels.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "../../include/pie.h"

namespace pie {

// =====================================================================================================
// Swap kernel (Section 4: "a CUDA kernel for efficient per-layer KV cache swapping"; here per block list)
// One work item = one 32 KiB chunk of one block.  Each thread issues UNROLL 16-byte loads before its
// stores so that a CTA keeps 32 KiB in flight on the host link; a warp touches 512 contiguous bytes.
// =====================================================================================================
constexpr int SWAP_THREADS = 256;
constexpr int SWAP_UNROLL = 8;
constexpr int SWAP_CHUNK_VECS = SWAP_THREADS * SWAP_UNROLL;  // 16-byte vectors per chunk

__global__ void __launch_bounds__(SWAP_THREADS)
swap_kernel(const uint4 *__restrict__ src_pool, uint4 *__restrict__ dst_pool, const int32_t *__restrict__ list,
            int64_t n, int32_t vecs_per_block, int32_t chunks_per_block, int32_t *slot_table, int table_mode) {
    const int64_t n_items = n * chunks_per_block;
    for (int64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
        const int64_t pair = item / chunks_per_block;
        const int32_t chunk = (int32_t)(item - pair * chunks_per_block);
        const int32_t s = list[3 * pair + 0];
        const int32_t d = list[3 * pair + 1];
        const uint4 *sp = src_pool + (int64_t)s * vecs_per_block;
        uint4 *dp = dst_pool + (int64_t)d * vecs_per_block;
        const int32_t base = chunk * SWAP_CHUNK_VECS + threadIdx.x;
        uint4 v[SWAP_UNROLL];
#pragma unroll
        for (int u = 0; u < SWAP_UNROLL; ++u) {
            const int32_t i = base + u * SWAP_THREADS;
            if (i < vecs_per_block) v[u] = __ldcs(sp + i);
        }
#pragma unroll
        for (int u = 0; u < SWAP_UNROLL; ++u) {
            const int32_t i = base + u * SWAP_THREADS;
            if (i < vecs_per_block) dp[i] = v[u];
        }
        if (slot_table != nullptr && chunk == 0 && threadIdx.x == 0)
            slot_table[list[3 * pair + 2]] = table_mode == 1 ? d : -1;
    }
}

cudaError_t launch_swap(const void *src_pool, void *dst_pool, const int32_t *list, int64_t n, int64_t block_bytes,
                        int32_t *slot_table, int table_mode, int n_ctas, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    const int32_t vecs = (int32_t)(block_bytes / 16);
    const int32_t chunks = (vecs + SWAP_CHUNK_VECS - 1) / SWAP_CHUNK_VECS;
    int64_t items = n * chunks;
    int grid = (int)(items < n_ctas ? items : n_ctas);
    swap_kernel<<<grid, SWAP_THREADS, 0, stream>>>((const uint4 *)src_pool, (uint4 *)dst_pool, list, n, vecs, chunks,
                                                   slot_table, table_mode);
    return cudaGetLastError();
}

__global__ void patch_kernel(int32_t *table, const int32_t *__restrict__ entries, int64_t n) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        table[entries[2 * i]] = entries[2 * i + 1];
}

cudaError_t launch_patch(int32_t *table, const int32_t *entries, int64_t n, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    int grid = (int)((n + 255) / 256 < 64 ? (n + 255) / 256 : 64);
    patch_kernel<<<grid, 256, 0, stream>>>(table, entries, n);
    return cudaGetLastError();
}

__global__ void patch_from_list_kernel(int32_t *slot_table, const int32_t *__restrict__ list, int64_t n, int mode) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        slot_table[list[3 * i + 2]] = mode == 1 ? list[3 * i + 1] : -1;
}

cudaError_t launch_patch_from_list(int32_t *slot_table, const int32_t *list, int64_t n, int table_mode,
                                   cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    int grid = (int)((n + 255) / 256 < 64 ? (n + 255) / 256 : 64);
    patch_from_list_kernel<<<grid, 256, 0, stream>>>(slot_table, list, n, table_mode);
    return cudaGetLastError();
}

// =====================================================================================================
// PTX helpers
// =====================================================================================================
// The status words live in mapped pinned host memory: plain stores only (one word per flag), no atomics.
__device__ __forceinline__ void raise_status(int32_t *status, int32_t flag) {
    *reinterpret_cast<volatile int32_t *>(status + (flag == STATUS_MISSING_UNIT ? 0 : flag == STATUS_CTX_TOO_LONG ? 1 : 2)) = 1;
}
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after ~1 s of polling and reports false (the caller flags an error and leaves).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) __nanosleep(200);
    }
    return false;
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
template <bool BF16>
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if (BF16)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                     : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <bool BF16>
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    if (BF16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&v);
    } else {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&v);
    }
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// =====================================================================================================
// Plan: chunk_off[s] = number of split-K chunks of sequences before s (exclusive scan), chunk_off[S] = total.
// =====================================================================================================
__global__ void __launch_bounds__(1024)
plan_kernel(const int32_t *__restrict__ ctx_lens, int32_t n_seqs, int32_t max_tokens, int32_t split_tokens,
            int32_t max_chunks, int32_t *__restrict__ chunk_off, int32_t *status) {
    __shared__ int32_t warp_sums[32];
    __shared__ int32_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int32_t base = 0; base < n_seqs; base += 1024) {
        const int32_t s = base + threadIdx.x;
        int32_t v = 0;
        if (s < n_seqs) {
            int32_t ctx = ctx_lens[s];
            if (ctx > max_tokens) {
                ctx = max_tokens;
                raise_status(status, STATUS_CTX_TOO_LONG);
            }
            v = ctx > 0 ? (ctx + split_tokens - 1) / split_tokens : 0;
        }
        int32_t x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int32_t y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
        }
        if (lane == 31) warp_sums[warp] = x;
        __syncthreads();
        if (warp == 0) {
            int32_t w = warp_sums[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                int32_t y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += y;
            }
            warp_sums[lane] = w;
        }
        __syncthreads();
        const int32_t incl = x + (warp > 0 ? warp_sums[warp - 1] : 0) + carry;
        if (s < n_seqs) chunk_off[s] = incl - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry = incl;
        __syncthreads();
    }
    if (carry > max_chunks) {
        // more chunks than the partials buffer holds (sequences sharing blocks): compute nothing, flag it
        for (int32_t s = threadIdx.x; s <= n_seqs; s += 1024) chunk_off[s] = 0;
        if (threadIdx.x == 0) raise_status(status, STATUS_CTX_TOO_LONG);
    } else if (threadIdx.x == 0) {
        chunk_off[n_seqs] = carry;
    }
}

// =====================================================================================================
// KV append (Section 3.2: each token iteration updates each layer's cache): K and V rows of the new token
// go to position ctx_len-1 of the sequence's tail block.  grid (S, Hkv), block 2 * D/8 threads.
// =====================================================================================================
__global__ void append_kernel(uint4 *__restrict__ pool, const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                              const int32_t *__restrict__ block_table, int32_t max_blocks,
                              const int32_t *__restrict__ ctx_lens, const int32_t *__restrict__ slot_table,
                              int32_t n_kv_heads, int32_t head_dim, int32_t n_logical, int64_t n_gpu_slots,
                              int32_t *status) {
    const int s = blockIdx.x, kvh = blockIdx.y;
    const int vecs = head_dim / 8;
    const int kv = threadIdx.x / vecs, v = threadIdx.x % vecs;
    int32_t pos = ctx_lens[s] - 1;
    if (pos < 0) return;
    if (pos >= max_blocks * 16) return;  // flagged by the plan kernel
    const int32_t blk = block_table[(int64_t)s * max_blocks + pos / 16];
    int32_t slot = (blk >= 0 && blk < n_logical) ? slot_table[blk] : -1;
    if (slot < 0 || slot >= n_gpu_slots) {
        if (threadIdx.x == 0) raise_status(status, STATUS_MISSING_UNIT);
        return;
    }
    const uint4 *src = (kv == 0 ? k_new : v_new) + ((int64_t)s * n_kv_heads + kvh) * vecs + v;
    uint4 *dst = pool + ((((int64_t)slot * n_kv_heads + kvh) * 2 + kv) * 16 + (pos & 15)) * vecs + v;
    *dst = *src;
}

// =====================================================================================================
// Paged decode attention, split-K.
//
// Work item = (sequence, KV head, chunk of `split_tokens` tokens); items are dealt round-robin to a
// persistent grid.  Per item a CTA streams the chunk's 16-token tiles (K rows 0-15 and V rows 16-31 of
// one head: one contiguous 2*16*D*2-byte piece of the slot) through a ring of shared-memory stages:
//   - warp NW (producer): resolves block_table -> slot table -> slot for 32 tiles at a time and issues
//     one TMA tile copy per stage (128-byte swizzle), completion on the stage's "full" mbarrier;
//   - warps 0..NW-1 (consumers): tile i of an item goes to warp i % NW.  The KV tokens sit on the M axis
//     of mma.m16n8k16 and the (up to 8) query heads of the KV head's group on the N axis, so a tile costs
//     D/16 MMAs for S^T = K q^T and D/16 for O^T += V^T P^T whatever the group size.  Online softmax in
//     fp32 per warp; P^T reaches the B-operand layout with two movmatrix transposes.
// The NW per-warp partials are merged in warp order through shared memory and written as one fp32 partial
// (m, l, unnormalised acc) per item; combine_kernel merges a sequence's chunks in chunk order.  Every
// reduction order depends only on the logical token order and on ctx_len, never on slot ids or timing, so
// a run with swapped blocks reproduces a resident run bit for bit.
// =====================================================================================================
constexpr int ATT_NW = 4;
constexpr int ATT_THREADS = (ATT_NW + 1) * 32;
constexpr int ATT_STAGES = 8;

struct AttnParams {
    const uint16_t *q;
    const int32_t *block_table;
    const int32_t *ctx_lens;
    const int32_t *slot_table;
    const int32_t *chunk_off;
    float *part_o;
    float *part_ml;
    int32_t *status;
    int64_t n_gpu_slots;
    int32_t max_blocks, n_seqs, n_q_heads, n_kv_heads, group, n_logical, split_tokens, use3d;
    float scale_log2e;
};

template <int D>
struct AttnSmem {
    static constexpr int TILE_BYTES = 2 * 16 * D * 2;
    static constexpr int HALF_BYTES = 32 * 128;  // 32 rows x 128 bytes
    static constexpr int MO_STRIDE = D + 4;      // floats per (warp, head) row; +4 keeps the scatter conflict-free
    static constexpr int OFF_MO = ATT_STAGES * TILE_BYTES;
    static constexpr int OFF_ML = OFF_MO + ATT_NW * 8 * MO_STRIDE * 4;
    static constexpr int OFF_BAR = OFF_ML + ATT_NW * 8 * 2 * 4;
    static constexpr int OFF_ABORT = OFF_BAR + 2 * ATT_STAGES * 8;
    static constexpr int BYTES = OFF_ABORT + 16;
};

struct ItemInfo {
    int32_t s, kvh, t0, t1, ntiles;
};

__device__ __forceinline__ ItemInfo decode_item(const AttnParams &p, int32_t item) {
    ItemInfo it;
    const int32_t ci = item / p.n_kv_heads;
    it.kvh = item - ci * p.n_kv_heads;
    int32_t lo = 0, hi = p.n_seqs;  // largest s with chunk_off[s] <= ci
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (__ldg(p.chunk_off + mid) <= ci) lo = mid;
        else hi = mid;
    }
    it.s = lo;
    const int32_t c = ci - __ldg(p.chunk_off + lo);
    int32_t ctx = __ldg(p.ctx_lens + lo);
    ctx = min(ctx, p.max_blocks * 16);
    it.t0 = c * p.split_tokens;
    it.t1 = min(ctx, it.t0 + p.split_tokens);
    it.ntiles = (it.t1 - it.t0 + 15) >> 4;
    return it;
}

template <int D, bool BF16>
__global__ void __launch_bounds__(ATT_THREADS)
paged_decode_attn_kernel(const __grid_constant__ CUtensorMap tmap, const AttnParams p) {
    using SM = AttnSmem<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_full = smem_base + SM::OFF_BAR;
    const uint32_t bar_empty = bar_full + ATT_STAGES * 8;
    volatile int32_t *abort_flag = reinterpret_cast<volatile int32_t *>(smem + SM::OFF_ABORT);

    if (tid == 0) {
        for (int s = 0; s < ATT_STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int32_t n_items = __ldg(p.chunk_off + p.n_seqs) * p.n_kv_heads;
    uint32_t gt = 0;  // tiles this CTA has streamed so far (same count in producer and consumers)

    if (warp == ATT_NW) {
        // ------------------------------------------------------------------ producer warp
        for (int32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
            const ItemInfo it = decode_item(p, item);
            const int32_t *bt = p.block_table + (int64_t)it.s * p.max_blocks + (it.t0 >> 4);
            for (int32_t base = 0; base < it.ntiles; base += 32) {
                int32_t slot = -1;
                if (base + lane < it.ntiles) {
                    const int32_t blk = __ldg(bt + base + lane);
                    if (blk >= 0 && blk < p.n_logical) slot = __ldg(p.slot_table + blk);
                    if (slot >= p.n_gpu_slots) slot = -1;
                }
                const int32_t cnt = min(32, it.ntiles - base);
                for (int32_t j = 0; j < cnt; ++j, ++gt) {
                    int32_t sl = __shfl_sync(0xffffffffu, slot, j);
                    if (lane == 0) {
                        const uint32_t stage = gt % ATT_STAGES;
                        const uint32_t phase = (gt / ATT_STAGES) & 1u;
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u)) {
                            raise_status(p.status, STATUS_WAIT_TIMEOUT);
                            *abort_flag = 1;
                        }
                        if (sl < 0) {  // unit not on the GPU: flag it, stream slot 0 so the ring stays in step
                            raise_status(p.status, STATUS_MISSING_UNIT);
                            sl = 0;
                        }
                        if (*abort_flag == 0) {
                            const uint32_t dst = smem_base + stage * SM::TILE_BYTES;
                            const uint32_t bar = bar_full + 8 * stage;
                            const int32_t row0 = (sl * p.n_kv_heads + it.kvh) * 32;
                            mbar_expect_tx(bar, SM::TILE_BYTES);
                            if (p.use3d) {
                                tma_load_3d(dst, &tmap, 0, row0, 0, bar);
                            } else {
#pragma unroll
                                for (int h = 0; h < D / 64; ++h)
                                    tma_load_2d(dst + h * SM::HALF_BYTES, &tmap, h * 64, row0, bar);
                            }
                        }
                    }
                    if (__shfl_sync(0xffffffffu, (int)*abort_flag, 0)) return;
                }
            }
        }
        return;
    }

    // ---------------------------------------------------------------------- consumer warps
    const int c2 = (lane & 3) * 2;  // this thread's head pair {c2, c2+1} in the S^T and O^T fragments
    const int r0 = lane >> 2;       // this thread's token rows {r0, r0+8} in S^T, d rows in O^T
    float *mo = reinterpret_cast<float *>(smem + SM::OFF_MO);
    float *ml = reinterpret_cast<float *>(smem + SM::OFF_ML);
    // ldmatrix source coordinates of this lane
    const int lm = lane >> 3, lr = lane & 7;
    const int k_tok = lr + (lm & 1) * 8, k_csel = lm >> 1;   // K: matrices {tok 0-7, tok 8-15} x {chunk, chunk+1}
    const int v_tok = lr + (lm >> 1) * 8, v_csel = lm & 1;   // V (transposed): {chunk, chunk+1} x {tok 0-7, tok 8-15}

    for (int32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
        const ItemInfo it = decode_item(p, item);
        // q as the B operand of S^T = K q^T: b0 = q[g][16 ks + c2 .. +1], b1 = q[g][16 ks + 8 + c2 .. +1], g = lane / 4
        uint32_t bq[D / 16][2];
        {
            const int g = lane >> 2;
            const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
                p.q + ((int64_t)it.s * p.n_q_heads + (int64_t)it.kvh * p.group + g) * D);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                bq[ks][0] = g < p.group ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
                bq[ks][1] = g < p.group ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
            }
        }
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[D / 16][4];
#pragma unroll
        for (int j = 0; j < D / 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

        for (int32_t i = warp; i < it.ntiles; i += ATT_NW) {
            const uint32_t tg = gt + (uint32_t)i;
            const uint32_t stage = tg % ATT_STAGES;
            const uint32_t phase = (tg / ATT_STAGES) & 1u;
            if (!mbar_wait(bar_full + 8 * stage, phase)) {
                raise_status(p.status, STATUS_WAIT_TIMEOUT);
                *abort_flag = 1;
            }
            __syncwarp();
            if (*abort_flag) break;  // leave through the item's barriers so that no warp is left waiting
            uint8_t *tile = smem + stage * SM::TILE_BYTES;
            const uint32_t tile_u32 = smem_base + stage * SM::TILE_BYTES;
            const int nvalid = min(16, it.t1 - (it.t0 + 16 * i));
            if (nvalid < 16) {
                // masked tokens are excluded, not multiplied by zero: clear their V rows so that 0 * garbage
                // (possibly NaN/Inf) never enters the PV product.  A row is 128 contiguous bytes per half.
                const int nvec = (16 - nvalid) * (D / 64) * 8;
                for (int e = lane; e < nvec; e += 32) {
                    const int row = 16 + nvalid + e / ((D / 64) * 8);
                    const int rem = e % ((D / 64) * 8);
                    *reinterpret_cast<uint4 *>(tile + (rem >> 3) * SM::HALF_BYTES + row * 128 + (rem & 7) * 16) =
                        make_uint4(0, 0, 0, 0);
                }
                __syncwarp();
            }
            // ---- S^T[16 tokens][8 heads] = K[16][D] . q^T[D][8]
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const int chunk = 2 * ks + k_csel;
                uint32_t a[4];
                ldmatrix_x4(tile_u32 + (chunk >> 3) * SM::HALF_BYTES + k_tok * 128 + (((chunk & 7) ^ (k_tok & 7)) << 4), a);
                if (ks & 1) mma_16816<BF16>(sb, a, bq[ks][0], bq[ks][1]);
                else mma_16816<BF16>(sa, a, bq[ks][0], bq[ks][1]);
            }
            float v0 = (sa[0] + sb[0]) * p.scale_log2e, v1 = (sa[1] + sb[1]) * p.scale_log2e;
            float v2 = (sa[2] + sb[2]) * p.scale_log2e, v3 = (sa[3] + sb[3]) * p.scale_log2e;
            if (r0 >= nvalid) v0 = v1 = -INFINITY;
            if (r0 + 8 >= nvalid) v2 = v3 = -INFINITY;
            float x0 = fmaxf(v0, v2), x1 = fmaxf(v1, v3);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, off));
                x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, off));
            }
            const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);  // finite: token 0 of a tile is always valid
            const float a0 = fast_exp2(m0 - n0), a1 = fast_exp2(m1 - n1);
            const float p0 = fast_exp2(v0 - n0), p1 = fast_exp2(v1 - n1);
            const float p2 = fast_exp2(v2 - n0), p3 = fast_exp2(v3 - n1);
            m0 = n0;
            m1 = n1;
            l0 = l0 * a0 + (p0 + p2);
            l1 = l1 * a1 + (p1 + p3);
#pragma unroll
            for (int j = 0; j < D / 16; ++j) {
                o[j][0] *= a0;
                o[j][1] *= a1;
                o[j][2] *= a0;
                o[j][3] *= a1;
            }
            // P^T as the B operand of O^T += V^T P^T: transpose the two 8x8 (token x head) blocks
            const uint32_t h01 = pack2<BF16>(p0, p1), h23 = pack2<BF16>(p2, p3);
            const uint32_t pb0 = movmatrix_trans(h01);
            const uint32_t pb1 = movmatrix_trans(h23);
            // bf16 keeps 8 significant bits: carry the rounding remainder of P in a second bf16 term so that the
            // PV product sees ~16 bits (fp16's 11 bits need no correction)
            uint32_t pl0 = 0, pl1 = 0;
            if (BF16) {
                pl0 = movmatrix_trans(pack2<true>(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xffff0000u)));
                pl1 = movmatrix_trans(pack2<true>(p2 - __uint_as_float(h23 << 16), p3 - __uint_as_float(h23 & 0xffff0000u)));
            }
#pragma unroll
            for (int j = 0; j < D / 16; ++j) {
                const int chunk = 2 * j + v_csel;
                uint32_t a[4];
                ldmatrix_x4_trans(
                    tile_u32 + (chunk >> 3) * SM::HALF_BYTES + (16 + v_tok) * 128 + (((chunk & 7) ^ (v_tok & 7)) << 4), a);
                mma_16816<BF16>(o[j], a, pb0, pb1);
                if (BF16) mma_16816<BF16>(o[j], a, pl0, pl1);
            }
            __syncwarp();
            if (nvalid < 16) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            if (lane == 0) mbar_arrive(bar_empty + 8 * stage);
        }
        gt += (uint32_t)it.ntiles;

        // ---- merge the NW warps' partials in warp order
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, off);
            l1 += __shfl_xor_sync(0xffffffffu, l1, off);
        }
        {
            float *w = mo + warp * 8 * SM::MO_STRIDE;
#pragma unroll
            for (int j = 0; j < D / 16; ++j) {
                w[c2 * SM::MO_STRIDE + 16 * j + r0] = o[j][0];
                w[(c2 + 1) * SM::MO_STRIDE + 16 * j + r0] = o[j][1];
                w[c2 * SM::MO_STRIDE + 16 * j + 8 + r0] = o[j][2];
                w[(c2 + 1) * SM::MO_STRIDE + 16 * j + 8 + r0] = o[j][3];
            }
            if (lane < 4) {
                ml[(warp * 8 + c2) * 2 + 0] = m0;
                ml[(warp * 8 + c2) * 2 + 1] = l0;
                ml[(warp * 8 + c2 + 1) * 2 + 0] = m1;
                ml[(warp * 8 + c2 + 1) * 2 + 1] = l1;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(ATT_NW * 32) : "memory");
        for (int e = tid; e < p.group * D; e += ATT_NW * 32) {
            const int g = e / D, d = e - g * D;
            float mm = -INFINITY;
#pragma unroll
            for (int w = 0; w < ATT_NW; ++w) mm = fmaxf(mm, ml[(w * 8 + g) * 2]);
            float acc = 0.f, ll = 0.f;
#pragma unroll
            for (int w = 0; w < ATT_NW; ++w) {
                const float mw = ml[(w * 8 + g) * 2];
                const float wt = mw == -INFINITY ? 0.f : fast_exp2(mw - mm);
                acc += mo[(w * 8 + g) * SM::MO_STRIDE + d] * wt;
                ll += ml[(w * 8 + g) * 2 + 1] * wt;
            }
            p.part_o[((int64_t)item * p.group + g) * D + d] = acc;
            if (d == 0) {
                p.part_ml[((int64_t)item * p.group + g) * 2 + 0] = mm;
                p.part_ml[((int64_t)item * p.group + g) * 2 + 1] = ll;
            }
        }
        // second barrier (partials buffer free again) doubles as a uniform vote on the abort flag
        uint32_t any_abort;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 q, %1, 0;\n\t"
            "bar.red.or.pred p, 1, %2, q;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(any_abort)
            : "r"((uint32_t)*abort_flag), "n"(ATT_NW * 32)
            : "memory");
        if (any_abort) return;
    }
}

// =====================================================================================================
// Combine: one warp per (sequence, query head) merges that sequence's chunk partials in chunk order with the
// log-sum-exp rule, normalises and rounds to the 16-bit output type (nearest even).  No chunk -> zeros.
// =====================================================================================================
template <int D, bool BF16>
__global__ void __launch_bounds__(128)
combine_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml, const int32_t *__restrict__ chunk_off,
               uint16_t *__restrict__ out, int32_t n_seqs, int32_t n_q_heads, int32_t n_kv_heads, int32_t group) {
    constexpr int EPL = D / 32;  // elements per lane
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * 4 + (threadIdx.x >> 5);
    if (row >= (int64_t)n_seqs * n_q_heads) return;
    const int32_t s = (int32_t)(row / n_q_heads), h = (int32_t)(row % n_q_heads);
    const int32_t kvh = h / group, g = h % group;
    const int32_t c0 = chunk_off[s], c1 = chunk_off[s + 1];
    float mm = -INFINITY;
    for (int32_t c = c0; c < c1; ++c) mm = fmaxf(mm, part_ml[(((int64_t)c * n_kv_heads + kvh) * group + g) * 2]);
    float acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    float ll = 0.f;
    for (int32_t c = c0; c < c1; ++c) {
        const int64_t idx = ((int64_t)c * n_kv_heads + kvh) * group + g;
        const float mc = part_ml[idx * 2];
        const float wt = mc == -INFINITY ? 0.f : fast_exp2(mc - mm);
        ll += part_ml[idx * 2 + 1] * wt;
        const float *po = part_o + idx * D + lane * EPL;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] += po[e] * wt;
    }
    const float inv = ll > 0.f ? 1.f / ll : 0.f;
    uint16_t *dst = out + row * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; e += 2) {
        const uint32_t v = pack2<BF16>(acc[e] * inv, acc[e + 1] * inv);
        *reinterpret_cast<uint32_t *>(dst + e) = v;
    }
}

// =====================================================================================================
// Host side: descriptors and launches
// =====================================================================================================
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cudaError_t make_pool_tensor_maps(void *gpu_pool, int64_t n_gpu_slots, int n_kv_heads, int head_dim, CUtensorMap *map3d,
                                  CUtensorMap *map2d, int *use3d) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fn);
    const cuuint64_t rows = (cuuint64_t)n_gpu_slots * (cuuint64_t)n_kv_heads * 32u;
    const cuuint32_t halves = (cuuint32_t)(head_dim / 64);
    {
        // one 128-byte half-row is the inner dimension; the tile lands as [half][32 rows][128 B], swizzled
        cuuint64_t dims[3] = {64, rows, halves};
        cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, 128};
        cuuint32_t box[3] = {64, 32, halves};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = encode(map3d, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, gpu_pool, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        *use3d = r == CUDA_SUCCESS ? 1 : 0;
    }
    {
        cuuint64_t dims[2] = {(cuuint64_t)head_dim, rows};
        cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
        cuuint32_t box[2] = {64, 32};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = encode(map2d, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, gpu_pool, dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    return cudaSuccess;
}

int attn_smem_bytes(int head_dim) { return head_dim == 128 ? AttnSmem<128>::BYTES : AttnSmem<64>::BYTES; }

template <int D, bool BF16>
static cudaError_t configure_one(int *ctas_per_sm) {
    cudaError_t e = cudaFuncSetAttribute(paged_decode_attn_kernel<D, BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         AttnSmem<D>::BYTES);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, paged_decode_attn_kernel<D, BF16>, ATT_THREADS,
                                                         AttnSmem<D>::BYTES);
}

cudaError_t attn_configure(int head_dim, int dtype, int *ctas_per_sm) {
    if (head_dim == 128) return dtype == PIE_BF16 ? configure_one<128, true>(ctas_per_sm) : configure_one<128, false>(ctas_per_sm);
    return dtype == PIE_BF16 ? configure_one<64, true>(ctas_per_sm) : configure_one<64, false>(ctas_per_sm);
}

template <int D, bool BF16>
static cudaError_t launch_one(const AttnShape &sh, const AttnScratch &sc, const AttnLaunch &a, const CUtensorMap &map,
                              int use3d, cudaStream_t stream) {
    AttnParams p;
    p.q = (const uint16_t *)a.q;
    p.block_table = a.block_table;
    p.ctx_lens = a.ctx_lens;
    p.slot_table = a.slot_table;
    p.chunk_off = sc.chunk_off;
    p.part_o = sc.part_o;
    p.part_ml = sc.part_ml;
    p.status = a.status;
    p.n_gpu_slots = sh.n_gpu_slots;
    p.max_blocks = a.max_blocks;
    p.n_seqs = a.n_seqs;
    p.n_q_heads = sh.n_q_heads;
    p.n_kv_heads = sh.n_kv_heads;
    p.group = sh.n_q_heads / sh.n_kv_heads;
    p.n_logical = sh.n_logical;
    p.split_tokens = a.split_tokens;
    p.use3d = use3d;
    p.scale_log2e = a.scale * 1.4426950408889634f;
    paged_decode_attn_kernel<D, BF16><<<a.grid, ATT_THREADS, AttnSmem<D>::BYTES, stream>>>(map, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const int64_t rows = (int64_t)a.n_seqs * sh.n_q_heads;
    combine_kernel<D, BF16><<<(unsigned)((rows + 3) / 4), 128, 0, stream>>>(sc.part_o, sc.part_ml, sc.chunk_off,
                                                                           (uint16_t *)a.out, a.n_seqs, sh.n_q_heads,
                                                                           sh.n_kv_heads, p.group);
    return cudaGetLastError();
}

cudaError_t launch_attention(const AttnShape &sh, const AttnScratch &sc, const AttnLaunch &a, const CUtensorMap &map,
                             int use3d, cudaStream_t stream) {
    if (a.n_seqs <= 0) return cudaSuccess;
    plan_kernel<<<1, 1024, 0, stream>>>(a.ctx_lens, a.n_seqs, a.max_blocks * 16, a.split_tokens,
                                        (int32_t)(sc.max_items / sh.n_kv_heads), sc.chunk_off, a.status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (a.k_new != nullptr && a.v_new != nullptr) {
        dim3 grid((unsigned)a.n_seqs, (unsigned)sh.n_kv_heads);
        append_kernel<<<grid, 2 * sh.head_dim / 8, 0, stream>>>((uint4 *)a.gpu_pool, (const uint4 *)a.k_new,
                                                                (const uint4 *)a.v_new, a.block_table, a.max_blocks,
                                                                a.ctx_lens, a.slot_table, sh.n_kv_heads, sh.head_dim,
                                                                sh.n_logical, sh.n_gpu_slots, a.status);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (sh.head_dim == 128)
        return sh.dtype == PIE_BF16 ? launch_one<128, true>(sh, sc, a, map, use3d, stream)
                                    : launch_one<128, false>(sh, sc, a, map, use3d, stream);
    return sh.dtype == PIE_BF16 ? launch_one<64, true>(sh, sc, a, map, use3d, stream)
                                : launch_one<64, false>(sh, sc, a, map, use3d, stream);
}

}  // namespace pie
