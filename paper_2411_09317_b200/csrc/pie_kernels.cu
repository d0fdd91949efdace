// sm_100a kernels: block gather/scatter swap, slot-table patch, KV append, split-K paged decode
// attention (TMA-staged, mma.sync with the KV tokens on the M axis) and the split-K combine.
#include "pie_kernels.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "../../include/pie.h"

namespace pie {

// =====================================================================================================
// Swap kernel (the per-layer swap kernel of Section 4, here per block list)
// One work item = one 32 KiB chunk of one block.  Each thread issues UNROLL 16-byte loads before its
// stores so that a CTA keeps 32 KiB in flight on the host link; a warp touches 512 contiguous bytes.
// =====================================================================================================
constexpr int SWAP_THREADS = 256;
constexpr int SWAP_UNROLL = 8;
constexpr int SWAP_CHUNK_VECS = SWAP_THREADS * SWAP_UNROLL;  // 16-byte vectors per chunk

// Time stamps: kernels note the GPU's nanosecond timer in host-visible memory instead of the host putting timing
// events between the kernels of the compute stream (a timing event there costs the stream 2-3 us per record).
__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

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

__device__ __forceinline__ void raise_status(int32_t *status, int32_t flag);  // defined with the other helpers below

// Prefill-side write: a CTA takes a few consecutive tokens of a flat batch (about 16 KiB of rows) and copies each
// token's K and V rows of every KV head into the block that holds its position (slot layout [Hkv][2][16][D], 16-byte
// vectors).  A token whose block is not on the GPU, or whose position lies beyond the table, is skipped and flagged.
__global__ void __launch_bounds__(256)
kv_write_kernel(const uint4 *__restrict__ k, const uint4 *__restrict__ v, const int32_t *__restrict__ token_seq,
                const int32_t *__restrict__ token_pos, int64_t n_tokens, int32_t tokens_per_cta,
                const int32_t *__restrict__ block_table, int32_t max_blocks, int32_t n_seqs,
                const int32_t *__restrict__ slot_table, int32_t n_logical, int64_t n_gpu_slots, uint4 *__restrict__ pool,
                int32_t n_kv_heads, int32_t vecs_per_row, int32_t *status) {
    const int32_t per_token = n_kv_heads * vecs_per_row;                  // vectors of K (and of V) per token
    const int64_t slot_vecs = (int64_t)n_kv_heads * 2 * 16 * vecs_per_row;
    const int64_t t0 = (int64_t)blockIdx.x * tokens_per_cta;
    for (int32_t i = threadIdx.x; i < tokens_per_cta * 2 * per_token; i += blockDim.x) {
        const int32_t tt = i / (2 * per_token), r = i - tt * 2 * per_token;
        const int64_t t = t0 + tt;
        if (t >= n_tokens) break;
        const int32_t s = token_seq[t], pos = token_pos[t];
        if (s < 0 || s >= n_seqs || pos < 0 || pos >= max_blocks * 16) {
            if (r == 0) raise_status(status, STATUS_CTX_TOO_LONG);
            continue;
        }
        const int32_t b = block_table[(int64_t)s * max_blocks + (pos >> 4)];
        const int32_t slot = (b >= 0 && b < n_logical) ? slot_table[b] : -1;
        if (slot < 0 || slot >= n_gpu_slots) {
            if (r == 0) raise_status(status, STATUS_MISSING_UNIT);
            continue;
        }
        const int32_t kv = r >= per_token, j = r - kv * per_token;
        const int32_t h = j / vecs_per_row, c = j - h * vecs_per_row;
        const uint4 val = (kv ? v : k)[t * per_token + j];
        pool[(int64_t)slot * slot_vecs + (((int64_t)h * 2 + kv) * 16 + (pos & 15)) * vecs_per_row + c] = val;
    }
}

cudaError_t launch_kv_write(const void *k, const void *v, const int32_t *token_seq, const int32_t *token_pos, int64_t n_tokens,
                            const int32_t *block_table, int32_t max_blocks, int32_t n_seqs, const int32_t *slot_table,
                            int32_t n_logical, int64_t n_gpu_slots, void *gpu_pool, int32_t n_kv_heads, int32_t head_dim,
                            int32_t *status, cudaStream_t stream) {
    if (n_tokens <= 0) return cudaSuccess;
    const int32_t vecs_per_row = head_dim * 2 / 16;
    const int32_t per_cta = std::max(1, 1024 / (2 * n_kv_heads * vecs_per_row));   // ~1024 vectors = 4 per thread
    const int64_t grid = (n_tokens + per_cta - 1) / per_cta;
    kv_write_kernel<<<(unsigned)grid, 256, 0, stream>>>((const uint4 *)k, (const uint4 *)v, token_seq, token_pos, n_tokens, per_cta,
                                                       block_table, max_blocks, n_seqs, slot_table, n_logical, n_gpu_slots,
                                                       (uint4 *)gpu_pool, n_kv_heads, vecs_per_row, status);
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
// Programmatic dependent launch: a kernel launched with the stream-serialization attribute may become resident while
// the kernel before it in the stream still runs; nothing that kernel wrote may be touched before this wait, which
// returns once it has completed (at once for an ordinary launch).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
// slot-table entries are written by the copy streams while kernels run: read them from L2, never from a stale L1 line
__device__ __forceinline__ int32_t ld_slot(const int32_t *p) { return __ldcg(p); }
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
// Swap by bulk copies: the same lists as swap_kernel, moved by the TMA unit instead of by loads and stores.  One
// thread per CTA drives a ring of 4 KiB shared-memory stages: a bulk copy brings a chunk of a source slot in
// (host memory or HBM, completing on the stage's mbarrier), a bulk copy sends it on to the destination slot, and
// a stage is loaded again once the store that last used it has finished reading it.  No registers hold data and
// no load/store unit is kept busy: the SM footprint is one warp and the stages.
// =====================================================================================================
// Small stages on purpose: the persistent attention kernel leaves about 24 KiB of shared memory per SM, and a swap
// CTA that does not fit beside it would only run between two attention launches.
constexpr int BULK_STAGES = 4;
constexpr int BULK_CHUNK_BYTES = 4 * 1024;

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(32)
swap_bulk_kernel(const uint8_t *__restrict__ src_pool, uint8_t *__restrict__ dst_pool, const int32_t *__restrict__ list,
                 int64_t n, int64_t block_bytes, int32_t chunks_per_block, int32_t *slot_table, int table_mode,
                 int32_t *status) {
    extern __shared__ __align__(128) uint8_t bulk_smem[];
    __shared__ __align__(8) uint64_t bars[BULK_STAGES];
    if (threadIdx.x != 0) return;  // one thread drives the copies
    const uint32_t smem_base = smem_u32(bulk_smem), bar0 = smem_u32(bars);
    for (int s = 0; s < BULK_STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const int64_t n_items = n * chunks_per_block;
    const int64_t mine = n_items > blockIdx.x ? (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    auto chunk_of = [&](int64_t k, const uint8_t *&sp, uint8_t *&dp, uint32_t &bytes, int32_t &pair_block, int32_t &d_slot, bool &last) {
        const int64_t item = blockIdx.x + k * gridDim.x;
        const int64_t pair = item / chunks_per_block;
        const int32_t chunk = (int32_t)(item - pair * chunks_per_block);
        const int32_t s_slot = list[3 * pair + 0];
        d_slot = list[3 * pair + 1];
        pair_block = list[3 * pair + 2];
        const int64_t off = (int64_t)chunk * BULK_CHUNK_BYTES;
        bytes = (uint32_t)min((int64_t)BULK_CHUNK_BYTES, block_bytes - off);
        sp = src_pool + (int64_t)s_slot * block_bytes + off;
        dp = dst_pool + (int64_t)d_slot * block_bytes + off;
        last = chunk == chunks_per_block - 1;
    };
    bool ok = true;
    // loads run BULK_STAGES - 1 chunks ahead of the stores
    for (int64_t k = 0; k < mine + BULK_STAGES - 1 && ok; ++k) {
        if (k < mine) {
            const uint32_t stage = (uint32_t)(k % BULK_STAGES);
            // the store that last used this stage (chunk k - BULK_STAGES) is the newest one issued: wait for its reads
            if (k >= BULK_STAGES) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
            const uint8_t *sp;
            uint8_t *dp;
            uint32_t bytes;
            int32_t blk, d_slot;
            bool last;
            chunk_of(k, sp, dp, bytes, blk, d_slot, last);
            mbar_expect_tx(bar0 + 8 * stage, bytes);
            bulk_load(smem_base + stage * BULK_CHUNK_BYTES, sp, bytes, bar0 + 8 * stage);
        }
        const int64_t j = k - (BULK_STAGES - 1);
        if (j >= 0) {
            const uint32_t stage = (uint32_t)(j % BULK_STAGES);
            if (!mbar_wait(bar0 + 8 * stage, (uint32_t)((j / BULK_STAGES) & 1))) {
                raise_status(status, STATUS_WAIT_TIMEOUT);
                ok = false;
                break;
            }
            const uint8_t *sp;
            uint8_t *dp;
            uint32_t bytes;
            int32_t blk, d_slot;
            bool last;
            chunk_of(j, sp, dp, bytes, blk, d_slot, last);
            bulk_store(dp, smem_base + stage * BULK_CHUNK_BYTES, bytes);
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            if (slot_table != nullptr && last) slot_table[blk] = table_mode == 1 ? d_slot : -1;
        }
    }
    // everything this CTA stored must have landed before the kernel counts as complete; after a wait that ran out the
    // loads still in flight get their (bounded) time to arrive before the stages go away
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (!ok) {
        const int64_t issued = min(mine, (int64_t)BULK_STAGES);
        for (int64_t t = 0; t < issued; ++t) mbar_wait(bar0 + 8 * (uint32_t)(t % BULK_STAGES), 0);
    }
}

cudaError_t launch_swap_bulk(const void *src_pool, void *dst_pool, const int32_t *list, int64_t n, int64_t block_bytes,
                             int32_t *slot_table, int table_mode, int n_ctas, int32_t *status, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    if (block_bytes % 16 != 0) return cudaErrorInvalidValue;
    const int32_t chunks = (int32_t)((block_bytes + BULK_CHUNK_BYTES - 1) / BULK_CHUNK_BYTES);
    const int64_t items = n * chunks;
    const int grid = (int)(items < n_ctas ? items : n_ctas);
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(swap_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, BULK_STAGES * BULK_CHUNK_BYTES);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    swap_bulk_kernel<<<grid, 32, BULK_STAGES * BULK_CHUNK_BYTES, stream>>>((const uint8_t *)src_pool, (uint8_t *)dst_pool, list, n,
                                                                          block_bytes, chunks, slot_table, table_mode, status);
    return cudaGetLastError();
}

// =====================================================================================================
// Paged decode attention, split-K, one kernel per layer call.
//
// Work item = (sequence, KV head, chunk of `split_tokens` tokens).  A persistent grid pulls items from a
// global counter (so an SM that is slowed down, e.g. by a co-resident copy kernel, simply takes fewer).
// Per item a CTA streams the chunk's 16-token tiles (K rows 0-15 and V rows 16-31 of one head: one
// contiguous 2*16*D*2-byte piece of the slot) through a ring of shared-memory stages:
//   - warp NW (producer): fetches the next item, publishes it to the consumers through a small queue,
//     resolves block_table -> slot table -> slot for 32 tiles at a time and issues one TMA tile copy per
//     stage (128-byte swizzle), completion on the stage's "full" mbarrier;
//   - warps 0..NW-1 (consumers): tile i of an item goes to warp i % NW.  The KV tokens sit on the M axis of
//     mma.m16n8k16 and the (up to 8) query heads of the KV head's group on the N axis, so a tile costs D/16
//     MMAs for S^T = K q^T and D/16 for O^T += V^T P^T whatever the group size.  Online softmax in fp32
//     per warp; P^T reaches the B-operand layout with two movmatrix transposes.
// Fused into the same kernel:
//   - the split-K plan: every CTA builds the chunk offsets of the batch in shared memory (exclusive scan of
//     ceil(ctx / split) over the sequences);
//   - the KV append (Section 3.2: each token iteration updates each layer's cache): the warp that owns the
//     tile holding position ctx-1 patches the new token's K and V rows into the staged tile and into the pool;
//   - the combine of single-chunk sequences: normalised and rounded to 16 bits (nearest even) right here.  A
//     sequence with several chunks gets one fp32 partial (m, l, unnormalised acc) per item, merged in chunk order
//     by combine_kernel right after - or, inside a decode step, by the NEXT layer's launch of this kernel: a CTA that
//     has run out of attention work merges pieces of the previous layer's partials (the other pair of partial buffers)
//     while the launch's last CTAs finish, so that between two layers there is one kernel boundary and the merge costs
//     no time of its own.  (A fused "last CTA to finish the pair merges it" variant was measured: its per-item
//     release/acquire atomics and the serial merges cost more than the extra launch, badly so for 8-head groups and
//     long contexts.)
// Every reduction order depends only on the logical token order and on ctx_len (tile -> warp by index, warps
// merged in warp order, chunks merged in chunk order), never on slot ids, on which CTA ran an item or on
// timing, so a run with swapped blocks reproduces a resident run bit for bit.
// All waits are bounded: a wait that runs out raises a status word and the CTA leaves through its barriers.
// =====================================================================================================
constexpr int ATT_QD = 2;           // depth of the producer -> consumer item queue (item id + its query rows)
constexpr int ATT_SMEM_SEQS = 1024; // largest batch whose chunk offsets are built in shared memory

struct AttnParams {
    const uint16_t *q;
    uint16_t *out;
    const int32_t *block_table;
    const int32_t *ctx_lens;
    const int32_t *slot_table;
    const int32_t *chunk_off_global;  // used when n_seqs > ATT_SMEM_SEQS (filled by plan_kernel)
    int32_t *chunk_off_out;           // [n_seqs + 1]: the plan, written by CTA 0 for the combine kernel
    const uint4 *k_new, *v_new;       // optional append
    uint4 *pool;
    float *part_o;
    float *part_ml;
    // Deferred combine: the partials the call BEFORE this one left (same batch, same lengths, the other pair of partial
    // buffers) are merged into prev_out by this kernel's consumer warps once their CTA has run out of attention work -
    // in the tail of the launch, where SMs would idle - instead of by a kernel of its own between the two layers.
    const float *prev_part_o;
    const float *prev_part_ml;
    uint16_t *prev_out;  // NULL: nothing to merge
    int32_t early_trigger;  // the kernel after this one in the stream is the next layer's launch of this kernel: let it start
                            // beside this launch's tail (see below)
    int32_t *counters;  // this call's set: [0] next item, [1] CTAs that have left, [2] next piece of the deferred combine
    uint64_t *stamps;   // optional, host visible: [0] when CTA 0 started its main work, [1] when the last CTA left
                        // (globaltimer ns), [2] how long CTA 0 waited for the layer's arriving units (ns), [3] the
                        // batch's context tokens
    int32_t *status;
    // Presence wait inside the kernel (Section 3.2): the copy-in stream stores a list's ticket into *arrive once the
    // list's blocks and table entries have landed; no slot-table entry is read before *arrive >= arrive_need.
    int32_t *tokens_out;               // optional: receives the batch's context-token count
    // Completion word: the last CTA to leave stores done_value there once every CTA's writes (the appended rows among
    // them) are visible; the copy streams wait for it by value instead of by an event on the compute stream.
    unsigned long long *done_word;     // device memory, or NULL
    unsigned long long done_value;
    const unsigned long long *arrive;  // device word of this layer, or NULL
    unsigned long long arrive_need;    // 0: nothing to wait for
    // the same for the call's own inputs (q, k_new, v_new), where a copy stream brings them (host-buffer entry point)
    const unsigned long long *inputs_arrive;
    unsigned long long inputs_need;
    int64_t n_gpu_slots;
    int32_t max_blocks, n_seqs, n_q_heads, n_kv_heads, group, n_logical, split_tokens, use3d, max_chunks;
    float scale_log2e;      // softmax scale * log2(e) (* the key scale of an 8-bit pool)
    float out_scale = 1.f;  // 8-bit pools: the value scale (times what the kernel's 16-bit images of the bytes leave out)
    float k_scale = 1.f, v_scale = 1.f;  // 8-bit pools: the append stores E4M3(x / scale)
};

// KV8: the pool holds E4M3 bytes; a ring stage is then the 4 KiB byte tile as the TMA unit delivers it, and the consumer
// warps build their tensor-core operands from those bytes in registers.
template <int D, int STAGES, int NW, bool KV8 = false>
struct AttnSmem {
    static constexpr int TILE_BYTES = 2 * 16 * D * 2;
    static constexpr int RING_BYTES = KV8 ? 2 * 16 * D : TILE_BYTES;       // one ring stage
    static constexpr int HALF_BYTES = 32 * 128;  // 32 rows x 128 bytes
    static constexpr int MO_STRIDE = D + 4;      // floats per (warp, head) row; +4 keeps the scatter conflict-free
    static constexpr int Q_BYTES = 8 * D * 2;    // query rows of one item (up to 8 heads)
    static constexpr int OFF_Q = STAGES * RING_BYTES;
    static constexpr int OFF_MO = OFF_Q + ATT_QD * Q_BYTES;
    static constexpr int OFF_ML = OFF_MO + NW * 8 * MO_STRIDE * 4;
    static constexpr int OFF_BAR = OFF_ML + NW * 8 * 2 * 4;              // full[STAGES], empty[STAGES], qfull[QD], qempty[QD]
    static constexpr int OFF_MISC = OFF_BAR + (2 * STAGES + 2 * ATT_QD) * 8;  // abort, -, token count, -, q_item[QD]
    static constexpr int OFF_CO = OFF_MISC + 64;                          // chunk offsets [ATT_SMEM_SEQS + 1]
    static constexpr int BYTES = OFF_CO + (ATT_SMEM_SEQS + 1) * 4 + 12;
};

struct ItemInfo {
    int32_t s, kvh, ctx, t0, t1, ntiles, nchunks, chunk0;
};

__device__ __forceinline__ ItemInfo decode_item(const AttnParams &p, const int32_t *co, int32_t item) {
    ItemInfo it;
    const int32_t ci = item / p.n_kv_heads;
    it.kvh = item - ci * p.n_kv_heads;
    int32_t lo = 0, hi = p.n_seqs;  // largest s with co[s] <= ci
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (co[mid] <= ci) lo = mid;
        else hi = mid;
    }
    it.s = lo;
    it.chunk0 = co[lo];
    it.nchunks = co[lo + 1] - it.chunk0;
    const int32_t c = ci - it.chunk0;
    it.ctx = min(__ldg(p.ctx_lens + lo), p.max_blocks * 16);
    it.t0 = c * p.split_tokens;
    it.t1 = min(it.ctx, it.t0 + p.split_tokens);
    it.ntiles = (it.t1 - it.t0 + 15) >> 4;
    return it;
}

// barrier over the consumer warps that also ORs a predicate: every consumer thread gets the same answer
template <int NTHREADS>
__device__ __forceinline__ bool consumer_vote(bool pred) {
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(any)
        : "r"((uint32_t)pred), "n"(NTHREADS)
        : "memory");
    return any != 0;
}
template <int NTHREADS>
__device__ __forceinline__ void consumer_sync() {
    asm volatile("bar.sync 1, %0;" ::"n"(NTHREADS) : "memory");
}

// The two low (HI = false) or high bytes of a word -> fp16 x 2 (exact) by the conversion instruction.  The 8-bit kernel
// computes in fp16 whatever the pool's 16-bit type is: every E4M3 value is an fp16 number, the conversion has a pipe of
// its own, and fp16 keeps 11 bits of P where bf16 needs a second product for P's rounding remainder.  A bf16 query is
// brought into fp16's range by a power of two per work item (exact; undone in the softmax scale).  Measured on the way:
// decoding by bit moves (shift exponent and mantissa into place, fix the bias by a factor) in the ALU 3.5-3.8 TB/s on the
// fp16 MHA shape against 4.35-4.5 TB/s with the conversion instruction; bf16 operands built that way 3.0 TB/s.
template <bool HI>
__device__ __forceinline__ uint32_t e4m3x2_cvt_f16x2(uint32_t w) {
    uint32_t r;
    if (HI) asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, hi;\n\t}" : "=r"(r) : "r"(w));
    else asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, lo;\n\t}" : "=r"(r) : "r"(w));
    return r;
}
// two floats -> two E4M3 bytes (lo in the low byte): nearest even, saturating to +-448
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// Prefill-side write into an 8-bit pool: as kv_write_kernel, but every 16-byte vector of 16-bit values becomes eight
// E4M3 bytes (fp32 quotient by the scale, nearest even, saturating - the append's rule); rows are 128 bytes.
template <bool BF16>
__global__ void __launch_bounds__(256)
kv_write8_kernel(const uint4 *__restrict__ k, const uint4 *__restrict__ v, const int32_t *__restrict__ token_seq,
                 const int32_t *__restrict__ token_pos, int64_t n_tokens, int32_t tokens_per_cta,
                 const int32_t *__restrict__ block_table, int32_t max_blocks, int32_t n_seqs,
                 const int32_t *__restrict__ slot_table, int32_t n_logical, int64_t n_gpu_slots, uint8_t *__restrict__ pool,
                 int32_t n_kv_heads, float k_scale, float v_scale, int32_t *status) {
    constexpr int32_t vecs_per_row = 16;                                  // head_dim 128: 16 vectors of eight values
    const int32_t per_token = n_kv_heads * vecs_per_row;
    const int64_t slot_bytes = (int64_t)n_kv_heads * 2 * 16 * 128;
    const int64_t t0 = (int64_t)blockIdx.x * tokens_per_cta;
    for (int32_t i = threadIdx.x; i < tokens_per_cta * 2 * per_token; i += blockDim.x) {
        const int32_t tt = i / (2 * per_token), r = i - tt * 2 * per_token;
        const int64_t t = t0 + tt;
        if (t >= n_tokens) break;
        const int32_t s = token_seq[t], pos = token_pos[t];
        if (s < 0 || s >= n_seqs || pos < 0 || pos >= max_blocks * 16) {
            if (r == 0) raise_status(status, STATUS_CTX_TOO_LONG);
            continue;
        }
        const int32_t b = block_table[(int64_t)s * max_blocks + (pos >> 4)];
        const int32_t slot = (b >= 0 && b < n_logical) ? slot_table[b] : -1;
        if (slot < 0 || slot >= n_gpu_slots) {
            if (r == 0) raise_status(status, STATUS_MISSING_UNIT);
            continue;
        }
        const int32_t kv = r >= per_token, j = r - kv * per_token;
        const int32_t h = j / vecs_per_row, c = j - h * vecs_per_row;
        const uint4 val = (kv ? v : k)[t * per_token + j];
        const float sc = kv ? v_scale : k_scale;
        const uint32_t w[4] = {val.x, val.y, val.z, val.w};
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float lo, hi;
            if (BF16) {
                lo = __uint_as_float(w[q] << 16);
                hi = __uint_as_float(w[q] & 0xffff0000u);
            } else {
                const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[q]));
                lo = f.x;
                hi = f.y;
            }
            o[q] = f32x2_to_e4m3x2(__fdiv_rn(lo, sc), __fdiv_rn(hi, sc));
        }
        *reinterpret_cast<uint2 *>(pool + (int64_t)slot * slot_bytes + (((int64_t)h * 2 + kv) * 16 + (pos & 15)) * 128 + 8 * c) =
            make_uint2(o[0] | (o[1] << 16), o[2] | (o[3] << 16));
    }
}

cudaError_t launch_kv_write8(const void *k, const void *v, const int32_t *token_seq, const int32_t *token_pos, int64_t n_tokens,
                             const int32_t *block_table, int32_t max_blocks, int32_t n_seqs, const int32_t *slot_table,
                             int32_t n_logical, int64_t n_gpu_slots, void *gpu_pool, int32_t n_kv_heads, int32_t dtype,
                             float k_scale, float v_scale, int32_t *status, cudaStream_t stream) {
    if (n_tokens <= 0) return cudaSuccess;
    const int32_t per_cta = std::max(1, 1024 / (2 * n_kv_heads * 16));
    const int64_t grid = (n_tokens + per_cta - 1) / per_cta;
    if (dtype == PIE_BF16)
        kv_write8_kernel<true><<<(unsigned)grid, 256, 0, stream>>>((const uint4 *)k, (const uint4 *)v, token_seq, token_pos, n_tokens,
                                                                  per_cta, block_table, max_blocks, n_seqs, slot_table, n_logical,
                                                                  n_gpu_slots, (uint8_t *)gpu_pool, n_kv_heads, k_scale, v_scale, status);
    else
        kv_write8_kernel<false><<<(unsigned)grid, 256, 0, stream>>>((const uint4 *)k, (const uint4 *)v, token_seq, token_pos, n_tokens,
                                                                   per_cta, block_table, max_blocks, n_seqs, slot_table, n_logical,
                                                                   n_gpu_slots, (uint8_t *)gpu_pool, n_kv_heads, k_scale, v_scale, status);
    return cudaGetLastError();
}

// One 16-byte piece (four consecutive d of head g) of a sequence's output from its chunk partials: log-sum-exp merge in
// chunk order, normalised, rounded to the 16-bit type.  get_ml(c) -> {m, l} of chunk c for this head.  Used by the combine
// kernel and by the deferred combine in the attention kernel's tail: the same arithmetic in the same order, so the same
// bits whoever merges.
template <int D, bool BF16, typename GetML>
__device__ __forceinline__ uint2 merge_piece(const float *__restrict__ part_o, int32_t chunk0, int32_t nchunks, int32_t n_kv_heads,
                                             int32_t kvh, int32_t group, int g, int d, GetML get_ml) {
    float mm = -INFINITY;
    for (int32_t c = 0; c < nchunks; ++c) mm = fmaxf(mm, get_ml(c).x);
    float ll = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int32_t c0 = 0; c0 < nchunks; c0 += 8) {
        float4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (c0 + j < nchunks) {
                const int64_t id = ((int64_t)(chunk0 + c0 + j) * n_kv_heads + kvh) * group + g;
                v[j] = *reinterpret_cast<const float4 *>(part_o + id * D + d);
            }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (c0 + j < nchunks) {
                const float2 w = get_ml(c0 + j);
                const float wt = w.x == -INFINITY ? 0.f : fast_exp2(w.x - mm);
                ll += w.y * wt;
                acc.x += v[j].x * wt;
                acc.y += v[j].y * wt;
                acc.z += v[j].z * wt;
                acc.w += v[j].w * wt;
            }
    }
    const float inv = ll > 0.f ? 1.f / ll : 0.f;
    uint2 r;
    r.x = pack2<BF16>(acc.x * inv, acc.y * inv);
    r.y = pack2<BF16>(acc.z * inv, acc.w * inv);
    return r;
}

// The second launch bound: for 16-bit pools it only tells the assembler that it need not hold registers back for more
// CTAs per SM than shared memory lets in anyway (four of 50 KiB; without it some instantiations were capped at 96
// registers and spilled).  The 8-bit kernel is bound by instruction latency, not by bytes in flight, and its CTAs need
// less than half of the shared memory: five per SM (128 registers) measured 3-6 % faster than four.
template <int D, bool BF16, int STAGES, int NW, bool KV8 = false>
__global__ void __launch_bounds__((NW + 1) * 32, KV8 ? 5 : 1)
paged_decode_attn_kernel(const __grid_constant__ CUtensorMap tmap, const AttnParams p) {
    using SM = AttnSmem<D, STAGES, NW, KV8>;
    constexpr bool MB = BF16 && !KV8;  // the tensor-core products run in bf16 (else fp16: always so for 8-bit pools)
    static_assert(!KV8 || D == 128, "8-bit blocks: head_dim 128 (one 128-byte row per token)");
    // A stage must always be consumed by the same warp: tile i goes to warp i % NW and to stage i % STAGES.  If two
    // warps alternated on a stage, the one running ahead could pass a parity wait on the phase before the one it
    // needs (an mbarrier waiter may be at most one phase ahead).
    static_assert(STAGES % NW == 0, "ring stages must be a multiple of the consumer warps");
    constexpr int ATT_NW = NW;
    constexpr int ATT_THREADS = (NW + 1) * 32;
    constexpr int NCONS = NW * 32;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t bar_full = smem_base + SM::OFF_BAR;
    const uint32_t bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_qfull = bar_empty + STAGES * 8;
    const uint32_t bar_qempty = bar_qfull + ATT_QD * 8;
    volatile int32_t *misc = reinterpret_cast<volatile int32_t *>(smem + SM::OFF_MISC);
    volatile int32_t *abort_flag = misc;      // [0]
    volatile int32_t *q_item = misc + 4;      // [4 .. 4 + QD)
    int32_t *co_smem = reinterpret_cast<int32_t *>(smem + SM::OFF_CO);

    // Everything up to the dependency wait below touches only shared memory and the call's own inputs (lengths and
    // tables, which no kernel of the path writes): under a programmatic dependent launch it overlaps the tail of the
    // kernel before it in the stream.
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int s = 0; s < ATT_QD; ++s) {
            mbar_init(bar_qfull + 8 * s, 1);
            mbar_init(bar_qempty + 8 * s, ATT_NW);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // Presence, first look (the thread that would poll below): the arrival words are stored by copies, not by the kernel
    // before this one, so they may be read ahead of the dependency wait.  A list that has landed by now - the usual case,
    // the lists run a group of layers ahead - costs the kernel nothing: the load's latency hides behind the plan.
    bool there_early = false;
    if (tid == ATT_NW * 32 && (p.arrive_need != 0 || p.inputs_need != 0))
        there_early = (p.arrive_need == 0 || ld_acquire_u64(p.arrive) >= p.arrive_need) &&
                      (p.inputs_need == 0 || ld_acquire_u64(p.inputs_arrive) >= p.inputs_need);
    // ---- plan: chunk offsets of the batch (exclusive scan of the per-sequence chunk counts)
    const bool co_in_smem = p.n_seqs <= ATT_SMEM_SEQS;
    if (co_in_smem) {
        int32_t my_tokens = 0;
        for (int32_t s = tid; s < p.n_seqs; s += ATT_THREADS) {
            int32_t ctx = __ldg(p.ctx_lens + s);
            if (ctx > p.max_blocks * 16) {
                ctx = p.max_blocks * 16;
                if (blockIdx.x == 0) raise_status(p.status, STATUS_CTX_TOO_LONG);
            }
            co_smem[s + 1] = ctx > 0 ? (ctx + p.split_tokens - 1) / p.split_tokens : 0;
            my_tokens += max(ctx, 0);
        }
        if (blockIdx.x == 0) {  // the batch's context tokens, for the host's time-per-token record (status word 3)
            if (tid == 0) misc[2] = 0;
            __syncthreads();
            atomicAdd(const_cast<int32_t *>(misc + 2), my_tokens);
            __syncthreads();
            if (tid == 0) {
                if (p.tokens_out != nullptr) *reinterpret_cast<volatile int32_t *>(p.tokens_out) = misc[2];
                if (p.stamps != nullptr) *reinterpret_cast<volatile uint64_t *>(p.stamps + 3) = (uint64_t)misc[2];
            }
        }
        __syncthreads();
        if (warp == 0) {
            int32_t carry = 0;
            for (int32_t base = 0; base < p.n_seqs; base += 32) {
                const int32_t s = base + lane;
                const int32_t v = s < p.n_seqs ? co_smem[s + 1] : 0;
                int32_t x = v;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int32_t y = __shfl_up_sync(0xffffffffu, x, o);
                    if (lane >= o) x += y;
                }
                if (s < p.n_seqs) co_smem[s + 1] = carry + x;
                carry += __shfl_sync(0xffffffffu, x, 31);
            }
            if (lane == 0) co_smem[0] = 0;
        }
    }
    __syncthreads();
    // Programmatic dependent launch, layer after layer.  Nothing in a layer's attention depends on the layer before it: its
    // own keys and values, query rows, slot-table row, partial buffers and counters (three sets, taken in turn) - so
    // the dependency wait comes AFTER the launch's attention work, in front of the two things that do depend on the
    // launch before (merging that layer's partials, and the completion word, which must not overtake that layer's), and
    // the trigger comes first: the next layer's CTAs take the place of this launch's CTAs as these leave and go straight
    // to work, so the tail of one launch and the head of the next overlap.  A launch never gets two launches ahead: its
    // dependents start only when all its CTAs are resident, that is when the launch before it has left the SMs.
    if (p.early_trigger) grid_launch_dependents();
    if (!co_in_smem) grid_dependency_wait();   // (the chunk offsets come from plan_kernel, the launch before this one)
    if (tid == 0 && p.stamps != nullptr && blockIdx.x == 0) {
        *reinterpret_cast<volatile uint64_t *>(p.stamps) = globaltimer_ns();
        if (p.arrive_need == 0 && p.inputs_need == 0) *reinterpret_cast<volatile uint64_t *>(p.stamps + 2) = 0;   // every launch writes all its stamps
    }
    const int32_t *co = co_in_smem ? co_smem : p.chunk_off_global;
    int32_t n_chunks_total = co[p.n_seqs];
    if (n_chunks_total > p.max_chunks) {  // more chunks than the partials buffer holds: compute nothing, flag it
        if (blockIdx.x == 0 && tid == 0) raise_status(p.status, STATUS_CTX_TOO_LONG);
        n_chunks_total = 0;
    }
    const int32_t n_items = n_chunks_total * p.n_kv_heads;
    uint32_t gt = 0;  // tiles this CTA has streamed so far (same count in producer and consumers)
    uint32_t qn = 0;  // items this CTA has taken so far

    if (warp == ATT_NW) {
        // ------------------------------------------------------------------ producer warp
        // presence wait (Section 3.2): no slot-table entry of this layer is read before the list that brings the
        // layer's units has landed.  Bounded (about half a second of polling): then the CTA flags it and leaves.
        if (p.arrive_need != 0 || p.inputs_need != 0) {
            if (lane == 0 && there_early) {
                if (p.stamps != nullptr && blockIdx.x == 0) *reinterpret_cast<volatile uint64_t *>(p.stamps + 2) = 0;
            } else if (lane == 0) {
                const uint64_t t_begin = globaltimer_ns();
                bool there = false;
                for (uint32_t i = 0; i < (1u << 21); ++i) {
                    if ((p.arrive_need == 0 || ld_acquire_u64(p.arrive) >= p.arrive_need) &&
                        (p.inputs_need == 0 || ld_acquire_u64(p.inputs_arrive) >= p.inputs_need)) {
                        there = true;
                        break;
                    }
                    if (i > 16) __nanosleep(250);
                }
                if (!there) {
                    raise_status(p.status, STATUS_WAIT_TIMEOUT);
                    *abort_flag = 1;
                }
                if (p.stamps != nullptr && blockIdx.x == 0)
                    *reinterpret_cast<volatile uint64_t *>(p.stamps + 2) = p.arrive_need != 0 ? globaltimer_ns() - t_begin : 0;
            }
            __syncwarp();
        }
        // the first item is the CTA's own number, the later ones come from the global counter
        int32_t next = lane == 0 ? (int32_t)blockIdx.x : 0;
        for (;;) {
            int32_t item = -1;
            if (lane == 0) {
                const uint32_t qs = qn % ATT_QD;
                if (!mbar_wait(bar_qempty + 8 * qs, ((qn / ATT_QD) & 1u) ^ 1u)) {
                    raise_status(p.status, STATUS_WAIT_TIMEOUT);
                    *abort_flag = 1;
                }
                if (*abort_flag == 0 && next < n_items) item = next;
                q_item[qs] = item;
                if (item >= 0) {
                    // the item's query rows travel with its id: one bulk copy that completes on the same barrier
                    const int32_t ci = item / p.n_kv_heads, kvh = item - ci * p.n_kv_heads;
                    int32_t lo = 0, hi = p.n_seqs;
                    while (hi - lo > 1) {
                        const int32_t mid = (lo + hi) >> 1;
                        if (co[mid] <= ci) lo = mid;
                        else hi = mid;
                    }
                    const uint32_t bytes = (uint32_t)p.group * D * 2;
                    mbar_expect_tx(bar_qfull + 8 * qs, bytes);
                    bulk_load(smem_base + SM::OFF_Q + qs * SM::Q_BYTES,
                              p.q + ((int64_t)lo * p.n_q_heads + (int64_t)kvh * p.group) * D, bytes, bar_qfull + 8 * qs);
                    next = (int32_t)gridDim.x + atomicAdd(p.counters, 1);  // the next item's id: its latency hides behind this item's tiles
                } else {
                    mbar_arrive(bar_qfull + 8 * qs);
                }
            }
            item = __shfl_sync(0xffffffffu, item, 0);
            ++qn;
            if (item < 0) {
                // No work is left for this CTA.  Where the combine kernel follows, it may become resident once every CTA
                // has got here (its CTAs wait for this grid to complete before they read anything): its launch then costs
                // nothing at the end of this kernel.  (Signalled at the kernel's start, its small CTAs sat beside the
                // attention warps for the kernel's whole duration and cost 8-head groups 9 %.)
                if (!p.early_trigger) grid_launch_dependents();
                break;
            }
            const ItemInfo it = decode_item(p, co, item);
            const int32_t *bt = p.block_table + (int64_t)it.s * p.max_blocks + (it.t0 >> 4);
            for (int32_t base = 0; base < it.ntiles; base += 32) {
                int32_t slot = -1;
                if (base + lane < it.ntiles) {
                    const int32_t blk = __ldg(bt + base + lane);
                    if (blk >= 0 && blk < p.n_logical) slot = ld_slot(p.slot_table + blk);
                    if (slot >= p.n_gpu_slots) slot = -1;
                }
                const int32_t cnt = min(32, it.ntiles - base);
                for (int32_t j = 0; j < cnt; ++j, ++gt) {
                    int32_t sl = __shfl_sync(0xffffffffu, slot, j);
                    if (lane == 0) {
                        const uint32_t stage = gt % STAGES;
                        const uint32_t phase = (gt / STAGES) & 1u;
                        if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1u)) {
                            raise_status(p.status, STATUS_WAIT_TIMEOUT);
                            *abort_flag = 1;
                        }
                        if (sl < 0) {  // unit not on the GPU: flag it, stream slot 0 so the ring stays in step
                            raise_status(p.status, STATUS_MISSING_UNIT);
                            sl = 0;
                        }
                        if (*abort_flag == 0) {
                            const uint32_t dst = smem_base + stage * SM::RING_BYTES;
                            const uint32_t bar = bar_full + 8 * stage;
                            const int32_t row0 = (sl * p.n_kv_heads + it.kvh) * 32;
                            mbar_expect_tx(bar, SM::RING_BYTES);
                            if (KV8) {
                                tma_load_2d(dst, &tmap, 0, row0, bar);  // 32 rows (16 K, 16 V) of 128 bytes
                            } else if (p.use3d) {
                                tma_load_3d(dst, &tmap, 0, row0, 0, bar);
                            } else {
#pragma unroll
                                for (int h = 0; h < D / 64; ++h)
                                    tma_load_2d(dst + h * SM::HALF_BYTES, &tmap, h * 64, row0, bar);
                            }
                        }
                    }
                    if (__shfl_sync(0xffffffffu, (int)*abort_flag, 0)) {
                        // give the copies still in flight a bounded time to land before the CTA's memory goes away
                        if (lane == 0) {
                            const uint32_t first = gt > (uint32_t)STAGES ? gt - STAGES : 0u;
                            for (uint32_t t = first; t < gt; ++t) mbar_wait(bar_full + 8 * (t % STAGES), (t / STAGES) & 1u);
                        }
                        return;
                    }
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

    // CTA 0: the chunk offsets for the combine kernel; sequences without any token get a zero row (nobody else writes them)
    if (blockIdx.x == 0 && co_in_smem)
        for (int32_t s = tid; s <= p.n_seqs; s += ATT_NW * 32) p.chunk_off_out[s] = n_items == 0 ? 0 : co[s];
    if (blockIdx.x == 0)
        for (int32_t s = 0; s < p.n_seqs; ++s)
            if (co[s + 1] == co[s] || n_items == 0)
                for (int e = tid; e < p.n_q_heads * D; e += ATT_NW * 32) p.out[(int64_t)s * p.n_q_heads * D + e] = 0;

    for (;;) {
        const uint32_t qs = qn % ATT_QD;
        const bool late = !mbar_wait(bar_qfull + 8 * qs, (qn / ATT_QD) & 1u);
        if (consumer_vote<NCONS>(late || *abort_flag != 0)) {  // uniform: either every consumer goes on or none does
            if (late) raise_status(p.status, STATUS_WAIT_TIMEOUT);
            break;
        }
        const int32_t item = q_item[qs];
        if (item < 0) break;  // end marker: all consumers read the same queue entry
        const ItemInfo it = decode_item(p, co, item);
        // q as the B operand of S^T = K q^T: b0 = q[g][16 ks + c2 .. +1], b1 = q[g][16 ks + 8 + c2 .. +1], g = lane / 4
        uint32_t bq[D / 16][2];
        {
            const int g = lane >> 2;
            const uint32_t *qrow = reinterpret_cast<const uint32_t *>(smem + SM::OFF_Q + qs * SM::Q_BYTES) + g * (D / 2);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                if (KV8) {  // step 4 j + s reads d0 = 16 (4 j + t) + 4 s .. + 3 as k = d0, d0 + 1 | d0 + 2, d0 + 3: the K bytes' order below
                    const int w = 8 * (4 * (ks >> 2) + (lane & 3)) + 2 * (ks & 3);
                    bq[ks][0] = g < p.group ? qrow[w] : 0u;
                    bq[ks][1] = g < p.group ? qrow[w + 1] : 0u;
                } else {
                    bq[ks][0] = g < p.group ? qrow[ks * 8 + (lane & 3)] : 0u;
                    bq[ks][1] = g < p.group ? qrow[ks * 8 + 4 + (lane & 3)] : 0u;
                }
            }
        }
        float sl2e = p.scale_log2e;
        if constexpr (KV8 && BF16) {
            // bf16 query, fp16 products: scale the item's query rows by the power of two that puts their largest magnitude
            // into [2^14, 2^15) (exact; what falls below fp16's subnormals is 2^-38 of the largest and cannot show in an
            // fp32 sum), convert, and give the factor back through the softmax scale
            float mx = 0.f;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    mx = fmaxf(mx, fmaxf(fabsf(__uint_as_float(bq[ks][h] << 16)), fabsf(__uint_as_float(bq[ks][h] & 0xffff0000u))));
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
            int sh = mx > 0.f ? (int)((__float_as_uint(mx) >> 23) & 0xffu) - 127 - 14 : 0;
            sh = max(-100, min(100, sh));
            const float down = __uint_as_float((uint32_t)(127 - sh) << 23);
            sl2e *= __uint_as_float((uint32_t)(127 + sh) << 23);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    bq[ks][h] = pack2<false>(__uint_as_float(bq[ks][h] << 16) * down, __uint_as_float(bq[ks][h] & 0xffff0000u) * down);
        }
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[D / 16][4];
#pragma unroll
        for (int j = 0; j < D / 16; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;

        for (int32_t i = warp; i < it.ntiles; i += ATT_NW) {
            const uint32_t tg = gt + (uint32_t)i;
            const uint32_t stage = tg % STAGES;
            const uint32_t phase = (tg / STAGES) & 1u;
            if (!mbar_wait(bar_full + 8 * stage, phase)) {
                raise_status(p.status, STATUS_WAIT_TIMEOUT);
                *abort_flag = 1;
            }
            __syncwarp();
            if (*abort_flag) break;  // leave through the item's barriers so that no warp is left waiting
            const int nvalid = min(16, it.t1 - (it.t0 + 16 * i));
            bool touched = false;
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
            [[maybe_unused]] uint4 vv[4];  // 8-bit path: this lane's 16 bytes of the V rows of tokens 2t, 2t+1, 2t+8, 2t+9
            if constexpr (KV8) {
                // The stage holds the tile as bytes: 32 rows (16 K, 16 V) of 128, 16-byte pieces swizzled by the row.  The
                // operands are built in registers, straight from the bytes.  The sums over head_dim (scores) and over the
                // tokens (output) do not care in which order their terms are fed to the tensor core, and neither does the
                // output care which accumulator row holds which d, so every lane reads whole 16-byte pieces:
                //   K: lane (g, t) reads pieces t and 4 + t of rows g and g + 8; word s of piece 4 j + t feeds step 4 j + s,
                //      bytes 0, 1 as k = 2t, 2t+1 and bytes 2, 3 as k = 2t+8, 2t+9 (q is read with the same assignment);
                //   V (after the softmax): lane (g, t) reads piece g of the rows of tokens 2t, 2t+1, 2t+8, 2t+9; byte 2i (2i+1) of the piece is
                //      accumulator row g (g + 8) of product i, that is d = 16 g + 2 i (+ 1).
                uint8_t *ring = smem + stage * SM::RING_BYTES;
                if (p.k_new != nullptr && it.t1 == it.ctx && i == it.ntiles - 1) {
                    // append: quantise the new token's rows (fp32 quotient by the scale, nearest-even E4M3, saturating) and
                    // put the bytes into the pool and into the staged tile (lanes 0-15: K, 16-31: V, eight values each)
                    const int32_t pos = it.ctx - 1, r = pos & 15;
                    int32_t slot = -1;
                    if (lane == 0) {
                        const int32_t blk = __ldg(p.block_table + (int64_t)it.s * p.max_blocks + (pos >> 4));
                        if (blk >= 0 && blk < p.n_logical) slot = ld_slot(p.slot_table + blk);
                        if (slot >= p.n_gpu_slots) slot = -1;
                    }
                    slot = __shfl_sync(0xffffffffu, slot, 0);
                    const int kv = lane >> 4, c = lane & 15;
                    const uint4 val = __ldg((kv ? p.v_new : p.k_new) + ((int64_t)it.s * p.n_kv_heads + it.kvh) * (D / 8) + c);
                    const float sc = kv ? p.v_scale : p.k_scale;
                    const uint32_t w[4] = {val.x, val.y, val.z, val.w};
                    uint32_t b[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        float lo, hi;
                        if (BF16) {
                            lo = __uint_as_float(w[j] << 16);
                            hi = __uint_as_float(w[j] & 0xffff0000u);
                        } else {
                            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[j]));
                            lo = f.x;
                            hi = f.y;
                        }
                        b[j] = f32x2_to_e4m3x2(__fdiv_rn(lo, sc), __fdiv_rn(hi, sc));
                    }
                    const uint2 bytes = make_uint2(b[0] | (b[1] << 16), b[2] | (b[3] << 16));
                    if (slot >= 0)
                        *reinterpret_cast<uint2 *>(reinterpret_cast<uint8_t *>(p.pool) +
                                                   ((((int64_t)slot * p.n_kv_heads + it.kvh) * 2 + kv) * 16 + r) * D + 8 * c) = bytes;
                    *reinterpret_cast<uint2 *>(ring + (kv * 16 + r) * 128 + (((c >> 1) ^ (r & 7)) << 4) + (c & 1) * 8) = bytes;
                    touched = true;
                    __syncwarp();
                }
                const int g = lane >> 2, t = lane & 3;
                uint4 kg[2], kh[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int off = ((4 * j + t) ^ g) << 4;  // rows g and g + 8 are swizzled alike
                    kg[j] = *reinterpret_cast<const uint4 *>(ring + g * 128 + off);
                    kh[j] = *reinterpret_cast<const uint4 *>(ring + (g + 8) * 128 + off);
                }
                // ---- S^T[16 tokens][8 heads] = K . q^T
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint32_t wg[4] = {kg[j].x, kg[j].y, kg[j].z, kg[j].w};
                    const uint32_t wh[4] = {kh[j].x, kh[j].y, kh[j].z, kh[j].w};
#pragma unroll
                    for (int s4 = 0; s4 < 4; ++s4) {
                        const int ks = 4 * j + s4;
                        uint32_t a[4];
                        a[0] = e4m3x2_cvt_f16x2<false>(wg[s4]);
                        a[1] = e4m3x2_cvt_f16x2<false>(wh[s4]);
                        a[2] = e4m3x2_cvt_f16x2<true>(wg[s4]);
                        a[3] = e4m3x2_cvt_f16x2<true>(wh[s4]);
                        if (ks & 1) mma_16816<MB>(sb, a, bq[ks][0], bq[ks][1]);
                        else mma_16816<MB>(sa, a, bq[ks][0], bq[ks][1]);
                    }
                }
            } else {
                uint8_t *tile = smem + stage * SM::RING_BYTES;
                const uint32_t tile_u32 = smem_base + stage * SM::RING_BYTES;
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
                    touched = true;
                }
                if (p.k_new != nullptr && it.t1 == it.ctx && i == it.ntiles - 1) {
                    // append: this tile holds position ctx-1; put the new token's K and V rows into the staged tile
                    // (lanes 0-15: K, lanes 16-31: V, one 16-byte piece each) and into the pool
                    const int32_t pos = it.ctx - 1, r = pos & 15;
                    int32_t slot = -1;
                    if (lane == 0) {
                        const int32_t blk = __ldg(p.block_table + (int64_t)it.s * p.max_blocks + (pos >> 4));
                        if (blk >= 0 && blk < p.n_logical) slot = ld_slot(p.slot_table + blk);
                        if (slot >= p.n_gpu_slots) slot = -1;
                    }
                    slot = __shfl_sync(0xffffffffu, slot, 0);
                    const int kv = lane >> 4, c = lane & 15;
                    if (c < D / 8) {
                        const uint4 val = __ldg((kv ? p.v_new : p.k_new) + ((int64_t)it.s * p.n_kv_heads + it.kvh) * (D / 8) + c);
                        if (slot >= 0) {
                            p.pool[((((int64_t)slot * p.n_kv_heads + it.kvh) * 2 + kv) * 16 + r) * (D / 8) + c] = val;
                        }
                        *reinterpret_cast<uint4 *>(tile + (c >> 3) * SM::HALF_BYTES + (kv * 16 + r) * 128 + (((c & 7) ^ (r & 7)) << 4)) = val;
                    }
                    touched = true;
                }
                if (touched) __syncwarp();
                // ---- S^T[16 tokens][8 heads] = K[16][D] . q^T[D][8]
    #pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const int chunk = 2 * ks + k_csel;
                    uint32_t a[4];
                    ldmatrix_x4(tile_u32 + (chunk >> 3) * SM::HALF_BYTES + k_tok * 128 + (((chunk & 7) ^ (k_tok & 7)) << 4), a);
                    if (ks & 1) mma_16816<MB>(sb, a, bq[ks][0], bq[ks][1]);
                    else mma_16816<MB>(sa, a, bq[ks][0], bq[ks][1]);
                }
            }
            float v0 = (sa[0] + sb[0]) * sl2e, v1 = (sa[1] + sb[1]) * sl2e;
            float v2 = (sa[2] + sb[2]) * sl2e, v3 = (sa[3] + sb[3]) * sl2e;
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
            // (8-bit kernel, bound by its instruction stream: once the running maxima have settled both factors are exactly 1
            // in every lane and the 32 multiplications can go - the same bits either way)
            if (!KV8 || __any_sync(0xffffffffu, a0 != 1.f || a1 != 1.f)) {
#pragma unroll
                for (int j = 0; j < D / 16; ++j) {
                    o[j][0] *= a0;
                    o[j][1] *= a1;
                    o[j][2] *= a0;
                    o[j][3] *= a1;
                }
            }
            // P^T as the B operand of O^T += V^T P^T: transpose the two 8x8 (token x head) blocks
            const uint32_t h01 = pack2<MB>(p0, p1), h23 = pack2<MB>(p2, p3);
            const uint32_t pb0 = movmatrix_trans(h01);
            const uint32_t pb1 = movmatrix_trans(h23);
            // bf16 keeps 8 significant bits: carry the rounding remainder of P in a second bf16 term so that the
            // PV product sees ~16 bits (fp16's 11 bits need no correction)
            uint32_t pl0 = 0, pl1 = 0;
            if (MB) {
                pl0 = movmatrix_trans(pack2<true>(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xffff0000u)));
                pl1 = movmatrix_trans(pack2<true>(p2 - __uint_as_float(h23 << 16), p3 - __uint_as_float(h23 & 0xffff0000u)));
            }
            if constexpr (KV8) {
                {
                    // the V bytes are fetched only now: 16 fewer registers live across the softmax, so the 128 that five CTAs
                    // per SM allow hold everything without spills (+3-4 % over fetching them with the K bytes)
                    const uint8_t *ring = smem + stage * SM::RING_BYTES;
                    const int g = lane >> 2, t = lane & 3;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int tok = 2 * t + (j & 1) + 8 * (j >> 1);
                        vv[j] = *reinterpret_cast<const uint4 *>(ring + (16 + tok) * 128 + ((g ^ (tok & 7)) << 4));
                    }
                    if (nvalid < 16) {
                        // masked tokens are excluded, not multiplied by zero (a NaN byte stays a NaN): clear their V bytes
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (2 * t + (j & 1) + 8 * (j >> 1) >= nvalid) vv[j] = make_uint4(0u, 0u, 0u, 0u);
                    }
                    __syncwarp();
                    if (touched) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    if (lane == 0) mbar_arrive(bar_empty + 8 * stage);  // everything is in registers: the stage may be refilled
                }
                const uint32_t v0w[4] = {vv[0].x, vv[0].y, vv[0].z, vv[0].w}, v1w[4] = {vv[1].x, vv[1].y, vv[1].z, vv[1].w};
                const uint32_t v2w[4] = {vv[2].x, vv[2].y, vv[2].z, vv[2].w}, v3w[4] = {vv[3].x, vv[3].y, vv[3].z, vv[3].w};
#pragma unroll
                for (int j = 0; j < D / 16; ++j) {
                    const int w = j >> 1;
                    const uint32_t sel = (j & 1) ? 0x7362u : 0x5140u;  // byte 2j (mod 4) of both tokens, then byte 2j+1 of both
                    const uint32_t z01 = __byte_perm(v0w[w], v1w[w], sel), z23 = __byte_perm(v2w[w], v3w[w], sel);
                    uint32_t a[4];
                    a[0] = e4m3x2_cvt_f16x2<false>(z01);  // d = 16 g + 2 j of tokens 2t, 2t+1
                    a[1] = e4m3x2_cvt_f16x2<true>(z01);   // d = 16 g + 2 j + 1
                    a[2] = e4m3x2_cvt_f16x2<false>(z23);  // the same of tokens 2t+8, 2t+9
                    a[3] = e4m3x2_cvt_f16x2<true>(z23);
                    mma_16816<MB>(o[j], a, pb0, pb1);
                    if (MB) mma_16816<MB>(o[j], a, pl0, pl1);
                }
                __syncwarp();
            } else {
                const uint32_t tile_u32 = smem_base + stage * SM::RING_BYTES;
#pragma unroll
                for (int j = 0; j < D / 16; ++j) {
                    const int chunk = 2 * j + v_csel;
                    uint32_t a[4];
                    ldmatrix_x4_trans(
                        tile_u32 + (chunk >> 3) * SM::HALF_BYTES + (16 + v_tok) * 128 + (((chunk & 7) ^ (v_tok & 7)) << 4), a);
                    mma_16816<MB>(o[j], a, pb0, pb1);
                    if (MB) mma_16816<MB>(o[j], a, pl0, pl1);
                }
                __syncwarp();
                if (touched) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                if (lane == 0) mbar_arrive(bar_empty + 8 * stage);
            }
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
                // accumulator rows r0 and r0 + 8 of product j: d = 16 j + r0 (+ 8); 8-bit path: d = 16 r0 + 2 j (+ 1)
                const int d0 = KV8 ? 16 * r0 + 2 * j : 16 * j + r0, d1 = KV8 ? d0 + 1 : d0 + 8;
                w[c2 * SM::MO_STRIDE + d0] = o[j][0];
                w[(c2 + 1) * SM::MO_STRIDE + d0] = o[j][1];
                w[c2 * SM::MO_STRIDE + d1] = o[j][2];
                w[(c2 + 1) * SM::MO_STRIDE + d1] = o[j][3];
            }
            if (lane < 4) {
                ml[(warp * 8 + c2) * 2 + 0] = m0;
                ml[(warp * 8 + c2) * 2 + 1] = l0;
                ml[(warp * 8 + c2 + 1) * 2 + 0] = m1;
                ml[(warp * 8 + c2 + 1) * 2 + 1] = l1;
            }
        }
        consumer_sync<NCONS>();
        const int64_t out_row0 = ((int64_t)it.s * p.n_q_heads + (int64_t)it.kvh * p.group) * D;
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
            acc *= p.out_scale;  // 1 for 16-bit pools
            if (it.nchunks == 1) {
                // the whole context in one chunk: normalise and round here
                const float r = acc * (ll > 0.f ? 1.f / ll : 0.f);
                p.out[out_row0 + e] = BF16 ? __bfloat16_as_ushort(__float2bfloat16_rn(r)) : __half_as_ushort(__float2half_rn(r));
            } else {
                p.part_o[((int64_t)item * p.group + g) * D + d] = acc;
                if (d == 0) {
                    p.part_ml[((int64_t)item * p.group + g) * 2 + 0] = mm;
                    p.part_ml[((int64_t)item * p.group + g) * 2 + 1] = ll;
                }
            }
        }
        // last barrier of the item (merge buffer free again) doubles as a uniform vote on the abort flag
        if (consumer_vote<NCONS>(*abort_flag != 0)) break;
        if (lane == 0) mbar_arrive(bar_qempty + 8 * qs);
        ++qn;
    }
    // ---- from here on the launch before this one must have completed
    grid_dependency_wait();
    // ---- deferred combine of the call before this one (its partials are complete: that grid has finished).  Pieces of
    // 32 float4 each, handed out warp by warp from a counter of their own; sequences of a single chunk were finished by
    // their own kernel.
    if (p.prev_out != nullptr && n_items > 0 && *abort_flag == 0) {
        constexpr int PIECES = D / 4;
        const int per_pair = p.group * PIECES;
        const int slices = (per_pair + 31) / 32;
        const int32_t total = p.n_seqs * p.n_kv_heads * slices;
        for (;;) {
            int32_t ci = 0;
            if (lane == 0) ci = atomicAdd(p.counters + 2, 1);
            ci = __shfl_sync(0xffffffffu, ci, 0);
            if (ci >= total) break;
            const int32_t pair = ci / slices, e4 = (ci - pair * slices) * 32 + lane;
            const int32_t s = pair / p.n_kv_heads, kvh = pair - s * p.n_kv_heads;
            const int32_t chunk0 = co[s], nchunks = co[s + 1] - chunk0;
            if (nchunks >= 2 && e4 < per_pair) {
                const int g = e4 / PIECES, d = (e4 - g * PIECES) * 4;
                const float *pml = p.prev_part_ml;
                const int32_t hkv = p.n_kv_heads, grp = p.group;
                const uint2 r = merge_piece<D, BF16>(p.prev_part_o, chunk0, nchunks, hkv, kvh, grp, g, d, [&](int32_t c) {
                    return *reinterpret_cast<const float2 *>(pml + ((((int64_t)(chunk0 + c) * hkv + kvh) * grp + g) << 1));
                });
                *reinterpret_cast<uint2 *>(p.prev_out + ((int64_t)s * p.n_q_heads + (int64_t)kvh * grp + g) * D + d) = r;
            }
        }
    }
    // the last CTA to leave resets the work counter for the next launch (every CTA has drawn its end marker by then)
    if (p.done_word != nullptr || p.prev_out != nullptr) {
        consumer_sync<NCONS>();   // the CTA's consumer warps have issued all their writes (and drawn their last piece)
    }
    if (tid == 0) {
        if (p.done_word != nullptr) __threadfence();   // ... and they are visible before this CTA counts as gone
        const int32_t old = atomicAdd(p.counters + 1, 1);
        if (old == (int32_t)gridDim.x - 1) {
            p.counters[0] = 0;
            p.counters[1] = 0;
            p.counters[2] = 0;
            if (p.stamps != nullptr) *reinterpret_cast<volatile uint64_t *>(p.stamps + 1) = globaltimer_ns();
            if (p.done_word != nullptr) {
                __threadfence();
                *reinterpret_cast<volatile unsigned long long *>(p.done_word) = p.done_value;
            }
        }
    }
}

// =====================================================================================================
// Combine: one CTA per (sequence, KV head, slice of head_dim) merges the sequence's chunk partials in chunk order with
// the log-sum-exp rule, normalises and rounds to the 16-bit output type (nearest even).  Sequences with fewer than two
// chunks were finished by the attention kernel.  The chunks' (m, l) pairs go through shared memory (sized by the launch
// for the longest sequence the table allows, so that the whole grid is resident at once: the kernel sits between two
// layers' attention kernels and every wave of it is dead time); the accumulation keeps eight 16-byte loads in flight
// per thread.
// =====================================================================================================
constexpr int COMB_THREADS = 64;
constexpr int COMB_CAP = 256;  // chunks per sequence handled through shared memory; beyond that, plain loops

template <int D, bool BF16>
__global__ void __launch_bounds__(COMB_THREADS)
combine_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml, const int32_t *__restrict__ chunk_off,
               uint16_t *__restrict__ out, int32_t n_q_heads, int32_t n_kv_heads, int32_t group, int32_t cap) {
    extern __shared__ __align__(16) float comb_smem[];   // wbuf[group][cap], lbuf[group][cap]
    float *wbuf = comb_smem, *lbuf = comb_smem + group * cap;
    // Launched with programmatic stream serialization: CTAs may become resident while the attention kernel still runs
    // (which hides the launch); nothing that kernel wrote is read before the wait, which returns once the attention
    // grid has completed and its writes are visible.  The kernel after this one may be launched the same way: let its
    // CTAs become resident as soon as this grid's have started (it touches nothing of ours before its own wait).
    grid_launch_dependents();
    grid_dependency_wait();
    const int tid = threadIdx.x;
    const int32_t s = blockIdx.x / n_kv_heads, kvh = blockIdx.x - s * n_kv_heads;
    const int32_t chunk0 = chunk_off[s], nchunks = chunk_off[s + 1] - chunk0;
    if (nchunks < 2) return;
    const int width = D / (int)gridDim.y;  // this CTA's slice of head_dim
    const int d_lo = blockIdx.y * width;
    const int64_t row0 = ((int64_t)s * n_q_heads + (int64_t)kvh * group) * D;
    if (nchunks <= cap) {
        for (int idx = tid; idx < group * nchunks; idx += COMB_THREADS) {
            const int g = idx / nchunks, c = idx - g * nchunks;
            const int64_t id = ((int64_t)(chunk0 + c) * n_kv_heads + kvh) * group + g;
            wbuf[g * cap + c] = part_ml[id * 2];
            lbuf[g * cap + c] = part_ml[id * 2 + 1];
        }
        __syncthreads();
        // every thread works the weights of its head out for itself (a few exponentials, in chunk order: the same
        // sums whichever thread forms them), so there is no serial pass over the chunks between two barriers
        const int per_head = width / 4;   // float4 pieces per head in the slice
        for (int e4 = tid; e4 < group * per_head; e4 += COMB_THREADS) {
            const int g = e4 / per_head, d = d_lo + (e4 - g * per_head) * 4;
            const float *w = wbuf + g * cap, *l = lbuf + g * cap;
            const uint2 r = merge_piece<D, BF16>(part_o, chunk0, nchunks, n_kv_heads, kvh, group, g, d,
                                                 [&](int32_t c) { return make_float2(w[c], l[c]); });
            *reinterpret_cast<uint2 *>(out + row0 + g * D + d) = r;
        }
        return;
    }
    for (int e = tid; e < group * width; e += COMB_THREADS) {  // very many chunks: plain loops
        const int g = e / width, d = d_lo + (e - g * width);
        float mm = -INFINITY;
        for (int32_t c = 0; c < nchunks; ++c) mm = fmaxf(mm, part_ml[(((int64_t)(chunk0 + c) * n_kv_heads + kvh) * group + g) * 2]);
        float acc = 0.f, ll = 0.f;
        for (int32_t c = 0; c < nchunks; ++c) {
            const int64_t idx = ((int64_t)(chunk0 + c) * n_kv_heads + kvh) * group + g;
            const float mc = part_ml[idx * 2];
            const float wt = mc == -INFINITY ? 0.f : fast_exp2(mc - mm);
            ll += part_ml[idx * 2 + 1] * wt;
            acc += part_o[idx * D + d] * wt;
        }
        const float r = acc * (ll > 0.f ? 1.f / ll : 0.f);
        out[row0 + g * D + d] = BF16 ? __bfloat16_as_ushort(__float2bfloat16_rn(r)) : __half_as_ushort(__float2half_rn(r));
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

// 8-bit pools: rows of 128 bytes (one token's K or V of one head, head_dim 128), 32 rows per tile.
cudaError_t make_pool_tensor_map_fp8(void *gpu_pool, int64_t n_gpu_slots, int n_kv_heads, CUtensorMap *map2d) {
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fn);
    cuuint64_t dims[2] = {128, (cuuint64_t)n_gpu_slots * (cuuint64_t)n_kv_heads * 32u};
    cuuint64_t strides[1] = {128};
    cuuint32_t box[2] = {128, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map2d, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, gpu_pool, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// Kernel variants (consumer warps, ring stages): more stages keep more bytes in flight per CTA, fewer let a third
// CTA share the SM.  Variant 0 is the default.
struct AttnVariant {
    int nw, stages;
};
static const AttnVariant kVariants[] = {{2, 4}, {4, 8}, {2, 12}, {2, 6}, {4, 4}, {2, 8}, {1, 5}, {3, 6}, {1, 7}, {2, 4}, {1, 4}, {3, 3}, {1, 3}, {2, 2}};
constexpr int kNumVariants = (int)(sizeof(kVariants) / sizeof(kVariants[0]));
constexpr int kNumVariants8 = 3;

template <typename F>
static cudaError_t dispatch_variant(int head_dim, int dtype, int variant, int kv_fp8, F &&f) {
    if (variant < 0 || variant >= kNumVariants) return cudaErrorInvalidValue;
    if (kv_fp8) {  // 8-bit blocks: head_dim 128; variants (consumer warps, stages of 4 KiB)
        if (head_dim != 128 || variant >= kNumVariants8) return cudaErrorInvalidValue;
#define PIE_VARIANT8(IDX, NWV, STV)                                                                                                      \
    if (variant == IDX)                                                                                                                  \
        return dtype == PIE_BF16 ? f(paged_decode_attn_kernel<128, true, STV, NWV, true>, AttnSmem<128, STV, NWV, true>::BYTES, NWV)   \
                                 : f(paged_decode_attn_kernel<128, false, STV, NWV, true>, AttnSmem<128, STV, NWV, true>::BYTES, NWV);
        PIE_VARIANT8(0, 2, 6)  // the most stages that still let five CTAs share an SM's shared memory
        PIE_VARIANT8(1, 2, 4)
        PIE_VARIANT8(2, 2, 8)
#undef PIE_VARIANT8
        return cudaErrorInvalidValue;
    }
#define PIE_VARIANT(NWV, STV)                                                                       \
    if (kVariants[variant].nw == NWV && kVariants[variant].stages == STV) {                         \
        if (head_dim == 128) return dtype == PIE_BF16 ? f(paged_decode_attn_kernel<128, true, STV, NWV>, AttnSmem<128, STV, NWV>::BYTES, NWV) \
                                                      : f(paged_decode_attn_kernel<128, false, STV, NWV>, AttnSmem<128, STV, NWV>::BYTES, NWV); \
        return dtype == PIE_BF16 ? f(paged_decode_attn_kernel<64, true, STV, NWV>, AttnSmem<64, STV, NWV>::BYTES, NWV)   \
                                 : f(paged_decode_attn_kernel<64, false, STV, NWV>, AttnSmem<64, STV, NWV>::BYTES, NWV); \
    }
    PIE_VARIANT(2, 12)
    PIE_VARIANT(4, 8)
    PIE_VARIANT(2, 6)
    PIE_VARIANT(4, 4)
    PIE_VARIANT(2, 8)
    PIE_VARIANT(1, 5)
    PIE_VARIANT(3, 6)
    PIE_VARIANT(1, 7)
    PIE_VARIANT(2, 4)
    PIE_VARIANT(1, 4)
    PIE_VARIANT(3, 3)
    PIE_VARIANT(1, 3)
    PIE_VARIANT(2, 2)
#undef PIE_VARIANT
    return cudaErrorInvalidValue;
}

int attn_smem_bytes(int head_dim) { return head_dim == 128 ? AttnSmem<128, 4, 2>::BYTES : AttnSmem<64, 4, 2>::BYTES; }

// The attention kernel needs the SM's largest shared-memory carve-out.  An SM cannot change its carve-out while
// any CTA is resident, so every other kernel of the path asks for the same one: otherwise a small kernel that
// lands on an idle SM first could keep attention CTAs off that SM until it has finished.
static cudaError_t prefer_max_shared() {
    const void *fns[] = {(const void *)swap_kernel, (const void *)patch_kernel, (const void *)patch_from_list_kernel,
                         (const void *)kv_write_kernel, (const void *)kv_write8_kernel<true>, (const void *)kv_write8_kernel<false>, (const void *)swap_bulk_kernel, (const void *)plan_kernel, (const void *)combine_kernel<128, true>, (const void *)combine_kernel<128, false>,
                         (const void *)combine_kernel<64, true>, (const void *)combine_kernel<64, false>};
    for (const void *f : fns) {
        cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t attn_configure(int head_dim, int dtype, int variant, int *ctas_per_sm, int kv_fp8) {
    cudaError_t e0 = prefer_max_shared();
    if (e0 != cudaSuccess) return e0;
    return dispatch_variant(head_dim, dtype, variant, kv_fp8, [&](auto kernel, int smem, int nw) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, kernel, (nw + 1) * 32, smem);
    });
}

int64_t attn_counter_words(int32_t, int32_t) { return 64; }  // [0] next item, [1] CTAs that have left

cudaError_t launch_attention(const AttnShape &sh, const AttnScratch &sc, const AttnLaunch &a, const CUtensorMap &map,
                             int use3d, cudaStream_t stream) {
    if (a.n_seqs <= 0) return cudaSuccess;
    if (a.n_seqs > ATT_SMEM_SEQS) {  // batch too large for the in-kernel plan: build the chunk offsets first
        plan_kernel<<<1, 1024, 0, stream>>>(a.ctx_lens, a.n_seqs, a.max_blocks * 16, a.split_tokens,
                                            (int32_t)(sc.max_items / sh.n_kv_heads), sc.chunk_off, a.status);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    AttnParams p;
    p.q = (const uint16_t *)a.q;
    p.out = (uint16_t *)a.out;
    p.block_table = a.block_table;
    p.ctx_lens = a.ctx_lens;
    p.slot_table = a.slot_table;
    p.chunk_off_global = sc.chunk_off;
    p.chunk_off_out = sc.chunk_off;
    p.k_new = (const uint4 *)a.k_new;
    p.v_new = (const uint4 *)a.v_new;
    p.pool = (uint4 *)a.gpu_pool;
    // two pairs of partial buffers where the pool has them: a call whose merge is deferred leaves its partials in the pair
    // of its parity, and the next call (the other parity) merges them while it fills its own
    const int turn = sc.part_o_more[0] != nullptr ? a.parity % 3 : 0, before = (turn + 2) % 3;
    auto buf_o = [&](int t) { return t == 0 ? sc.part_o : sc.part_o_more[t - 1]; };
    auto buf_ml = [&](int t) { return t == 0 ? sc.part_ml : sc.part_ml_more[t - 1]; };
    p.part_o = buf_o(turn);
    p.part_ml = buf_ml(turn);
    p.prev_part_o = buf_o(before);
    p.prev_part_ml = buf_ml(before);
    const bool can_defer = sc.part_o_more[0] != nullptr;
    p.prev_out = can_defer ? (uint16_t *)a.prev_out : nullptr;
    p.early_trigger = can_defer && a.defer_combine ? 1 : 0;
    p.counters = sc.counters + 4 * turn;
    p.stamps = a.stamps;
    p.status = a.status;
    p.tokens_out = a.tokens_out;
    p.done_word = a.done_word;
    p.done_value = a.done_value;
    p.arrive = a.arrive;
    p.arrive_need = a.arrive != nullptr ? a.arrive_need : 0ull;
    p.inputs_arrive = a.inputs_arrive;
    p.inputs_need = a.inputs_arrive != nullptr ? a.inputs_need : 0ull;
    p.n_gpu_slots = sh.n_gpu_slots;
    p.max_blocks = a.max_blocks;
    p.n_seqs = a.n_seqs;
    p.n_q_heads = sh.n_q_heads;
    p.n_kv_heads = sh.n_kv_heads;
    p.group = sh.n_q_heads / sh.n_kv_heads;
    p.n_logical = sh.n_logical;
    p.split_tokens = a.split_tokens;
    p.use3d = use3d;
    p.max_chunks = (int32_t)(sc.max_items / sh.n_kv_heads);
    p.scale_log2e = a.scale * 1.4426950408889634f;
    if (sh.kv_fp8) {
        p.k_scale = a.k_scale;
        p.v_scale = p.out_scale = a.v_scale;
        p.scale_log2e *= a.k_scale;  // scores over the stored keys are scores over the keys / k_scale
    }
    if (a.k_new == nullptr || a.v_new == nullptr) p.k_new = p.v_new = nullptr;
    cudaError_t e = dispatch_variant(sh.head_dim, sh.dtype, a.variant, sh.kv_fp8, [&](auto kernel, int smem, int nw) -> cudaError_t {
        if (!a.dependent_launch) {
            kernel<<<a.grid, (nw + 1) * 32, smem, stream>>>(map, p);
            return cudaGetLastError();
        }
        // behind the previous layer's last kernel (its attention kernel, where the merge is deferred): the CTAs may
        // become resident, set their barriers up and scan the batch's lengths while that kernel drains; they wait for
        // it before anything else
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3((unsigned)a.grid);
        lc.blockDim = dim3((unsigned)((nw + 1) * 32));
        lc.dynamicSmemBytes = (size_t)smem;
        lc.stream = stream;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        lc.attrs = at;
        lc.numAttrs = 1;
        return cudaLaunchKernelEx(&lc, kernel, map, p);
    });
    if (e != cudaSuccess) return e;
    if (a.defer_combine && can_defer) return cudaSuccess;   // the next call's kernel merges them
    return launch_combine(sh, sc, a.out, a.n_seqs, a.max_blocks, a.split_tokens, turn, stream);
}

// merge the partials of sequences that span several chunks (CTAs of single-chunk sequences return at once)
cudaError_t launch_combine(const AttnShape &sh, const AttnScratch &sc, void *out_ptr, int32_t n_seqs, int32_t max_blocks,
                           int32_t split_tokens, int parity, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    const int32_t group = sh.n_q_heads / sh.n_kv_heads;
    // chunks of the longest sequence the table allows (rounded up to a multiple of 8: the loads go in eights)
    const int64_t longest = ((int64_t)max_blocks * 16 + split_tokens - 1) / split_tokens;
    const int32_t cap = (int32_t)std::min<int64_t>(COMB_CAP, (longest + 7) / 8 * 8);
    // slices of head_dim such that a thread merges one 16-byte piece of one head (the merge is a chain of dependent
    // loads: what counts is how many rounds of them a thread makes), whole head_dim per CTA at most
    const int64_t pairs = (int64_t)n_seqs * sh.n_kv_heads;
    int slices = 1;
    while (slices < sh.head_dim / 32 && group * (sh.head_dim / 4) / slices > COMB_THREADS) slices *= 2;
    cfg.gridDim = dim3((unsigned)pairs, (unsigned)slices);
    cfg.blockDim = dim3(COMB_THREADS);
    cfg.dynamicSmemBytes = (size_t)(2 * group * cap) * sizeof(float);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    uint16_t *out = (uint16_t *)out_ptr;
    const int turn = sc.part_o_more[0] != nullptr ? parity % 3 : 0;
    const float *po = turn == 0 ? sc.part_o : sc.part_o_more[turn - 1], *pml = turn == 0 ? sc.part_ml : sc.part_ml_more[turn - 1];
    const int32_t *co = sc.chunk_off;
    const int32_t hq = sh.n_q_heads, hkv = sh.n_kv_heads;
    if (sh.head_dim == 128)
        return sh.dtype == PIE_BF16 ? cudaLaunchKernelEx(&cfg, combine_kernel<128, true>, po, pml, co, out, hq, hkv, group, cap)
                                    : cudaLaunchKernelEx(&cfg, combine_kernel<128, false>, po, pml, co, out, hq, hkv, group, cap);
    return sh.dtype == PIE_BF16 ? cudaLaunchKernelEx(&cfg, combine_kernel<64, true>, po, pml, co, out, hq, hkv, group, cap)
                                : cudaLaunchKernelEx(&cfg, combine_kernel<64, false>, po, pml, co, out, hq, hkv, group, cap);
}

}  // namespace pie
