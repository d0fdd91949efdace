// Chunked-prefill paged attention (Section 2.1: the prefill stage; Section 2.2: the paged KV cache) on the fifth-
// generation tensor cores: tcgen05.mma issued by one thread per CTA, operands staged in shared memory by TMA,
// accumulators in tensor memory (TMEM), read back with tcgen05.ld for the softmax.
//
// A chunk of C query tokens of a sequence whose context (chunk included) is ctx tokens long sits at positions
// ctx - C .. ctx - 1; token i attends to every cached position up to its own.  The chunk's own K and V are in the cache
// already (pie_kv_write comes first).
//
// Work item = (sequence, KV head, tile of 128 query rows).  A row is a (token, query head of the KV head's group) pair,
// token-major, so a tile holds 128 / G tokens; the rows of a tile share every K and V tile they read, which is what makes
// this a dense contraction: 128 rows per K and V tile against the decode kernel's G.  Per 64-token stage (four
// 16-token blocks of the paged pool):
//   - the loading warp (warp 5) resolves the blocks' slots several stages ahead and issues the TMA copies of their K and V
//     rows, eight lanes at once (two-dimensional tiles of 16 rows x 64 elements, 128-byte swizzle, straight into the layout
//     the tensor core's shared-memory descriptors expect: K as the K-major B operand of S = Q K^T, V as the MN-major B
//     operand of O += P V), double buffered: K(j + 2) once S(j) is complete, V(j + 1) once O += P V of stage j - 1 is;
//   - one thread of the issuing warp (warp 4) issues D / 16 MMAs of shape 128 x 64 x 16 for S (fp32, 64 TMEM columns, two
//     buffers: the scores of stage j + 1 are computed while the softmax of stage j runs) and commits them to an mbarrier;
//   - the four softmax warps read their 32 rows of S from TMEM (a thread holds one whole row: the softmax needs no
//     shuffles), apply the causal mask by selection, update the running maximum (lazily) and the sum, write P in the 16-bit
//     type back over the scores in TMEM as the next MMA's A operand, and rescale O in TMEM where a row's maximum moved;
//   - the issuing thread issues four MMAs (bf16: eight, the second operand carrying P's rounding remainder) of shape
//     128 x D x 16 for O += P V (fp32, D TMEM columns), A operand from TMEM.
// At the end every thread reads its row of O, divides by the row's sum and stores the 16-bit result.
// Every mbarrier exists once per stage parity and the end of the last product has a barrier of its own (a parity wait may
// be at most one phase behind, and the warps run at their own pace).  Every wait is bounded; a wait that runs out raises
// the status word, the loading warp waits (bounded) for its copies in flight, and the CTA still frees its TMEM before it
// leaves.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>

#include "../../include/pie.h"
#include "pie_kernels.h"

namespace pie {

namespace {

constexpr int PF_M = 128;        // query rows per CTA (the MMA's M)
constexpr int PF_KV = 64;        // KV tokens per stage
constexpr int PF_ROWS_THREADS = 128;  // four softmax warps: warp w owns TMEM lanes 32 w .. 32 w + 31 (one thread per query row)
constexpr int PF_THREADS = 192;       // + a warp that issues the MMAs (warp 4) and one that loads: block-table look-ups, TMA copies (warp 5)
constexpr int PF_TMEM_COLS = 256;
// The running maximum of a row is only raised - and the row's O and sum rescaled, a round trip through tensor memory for
// the whole warp - when the stage's maximum exceeds it by more than this (in log2 units): until then the probabilities
// are taken against the older maximum and may reach 2^8, which fp32 sums and both 16-bit types hold without loss.  With
// an exact running maximum some row of a warp moves its maximum in most stages, even hundreds of stages in.
constexpr float PF_LAZY = 8.f;

__device__ __forceinline__ uint32_t pf_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void pf_raise(int32_t *status, int32_t flag) {
    *reinterpret_cast<volatile int32_t *>(status + (flag == STATUS_MISSING_UNIT ? 0 : flag == STATUS_CTX_TOO_LONG ? 1 : 2)) = 1;
}
__device__ __forceinline__ void pf_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void pf_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void pf_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool pf_mbar_try_wait(uint32_t bar, uint32_t parity) {
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
// bounded: about a second of polling, then false
__device__ __forceinline__ bool pf_mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 22); ++i) {
        if (pf_mbar_try_wait(bar, parity)) return true;
        if (i > 64) __nanosleep(200);
    }
    return false;
}
__device__ __forceinline__ void pf_tma_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

// ---- tensor memory ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (base lane + i), v[c] = column (base column + c)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]),
          "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]),
          "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]),
          "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
          "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]),
          "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]),
          "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- MMA descriptors ---------------------------------------------------------------------------------------------------
// Shared-memory operand descriptor, 128-byte swizzle: start address, leading-dimension and stride byte offsets in units
// of 16 bytes, descriptor version 1, layout type 2.  For a K-major operand (rows of 128 bytes along the contraction) the
// leading offset is not used (1) and the stride offset is the distance between groups of eight rows (1024 bytes); for an
// MN-major operand the leading offset is the distance between 64-element chunks along MN.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(sbo_bytes >> 4) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}
// Instruction descriptor of kind::f16: fp32 accumulator, A and B both fp16 or both bf16, A K-major, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(bool bf16, int n, bool b_mn_major) {
    return (1u << 4) | ((bf16 ? 1u : 0u) << 7) | ((bf16 ? 1u : 0u) << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(PF_M >> 4) << 24);
}
__device__ __forceinline__ void mma_f16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// the same with the A operand in tensor memory (row r in lane r, two 16-bit elements of the contraction per 32-bit column)
__device__ __forceinline__ void mma_f16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ float pf_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
template <bool BF16>
__device__ __forceinline__ uint32_t pf_pack2(float lo, float hi) {
    if (BF16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&v);
    } else {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t *>(&v);
    }
}

struct PrefillParams {
    const uint16_t *q;
    uint16_t *out;
    const int32_t *block_table, *ctx_lens, *q_offsets, *tile_off, *slot_table;
    int32_t *status;
    int64_t n_gpu_slots;
    int32_t max_blocks, n_seqs, n_q_heads, n_kv_heads, group, n_logical;
    float scale_log2e;
};

template <int D>
struct PfSmem {
    static constexpr int Q_BYTES = PF_M * D * 2;        // [D / 64][128 rows][128 B]
    static constexpr int KV_BYTES = PF_KV * D * 2;      // [D / 64][64 tokens][128 B]
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + Q_BYTES;       // two stages
    static constexpr int OFF_V = OFF_K + 2 * KV_BYTES;  // two stages
    static constexpr int OFF_BAR = OFF_V + 2 * KV_BYTES; // k_full[2], v_full[2], s_done[2], o_done[2], p_done[2], done
    static constexpr int OFF_MISC = OFF_BAR + 128;      // [0] TMEM base, [1] abort, [4 .. 35] slots of eight stages' blocks
    static constexpr int BYTES = OFF_MISC + 256;        // two CTAs per SM (with TMEM for two: 2 x 256 of 512 columns)
};

template <int D, bool BF16>
__global__ void __launch_bounds__(PF_THREADS)
prefill_attn_kernel(const __grid_constant__ CUtensorMap tmap, const PrefillParams p) {
    using SM = PfSmem<D>;
    constexpr int HALVES = D / 64;
    extern __shared__ __align__(1024) uint8_t pf_smem[];
    uint8_t *smem = pf_smem;
    const uint32_t base = pf_smem_u32(pf_smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (base & 1023u) {   // the swizzled tiles need a 1024-byte boundary: never seen otherwise, but do not compute garbage
        if (tid == 0) pf_raise(p.status, STATUS_WAIT_TIMEOUT);
        return;
    }
    // Every barrier exists once per stage parity.  A parity wait may be at most one phase behind, and the warps of this
    // kernel run at their own pace (a softmax warp may be a stage ahead of another, the loading warp behind the issuing
    // one): with a barrier per parity, the next phase of the barrier a warp waits on cannot complete before that warp
    // has passed its wait (it needs what the warp does afterwards), whoever is slow.
    const uint32_t bar_k = base + SM::OFF_BAR, bar_v = bar_k + 16, bar_s = bar_k + 32, bar_o2 = bar_k + 48, bar_p = bar_k + 64;
    const uint32_t bar_p2[2] = {bar_p, bar_p + 8};
    const uint32_t bar_done = bar_k + 80;   // O is final (used once)
    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + SM::OFF_MISC);

    // ---- which tile
    const int32_t item = blockIdx.x;
    const int32_t tile_g = item / p.n_kv_heads, kvh = item - tile_g * p.n_kv_heads;
    int32_t lo = 0, hi = p.n_seqs;  // largest s with tile_off[s] <= tile_g
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (__ldg(p.tile_off + mid) <= tile_g) lo = mid;
        else hi = mid;
    }
    const int32_t s = lo;
    const int32_t G = p.group, tile_tokens = PF_M / G;
    const int32_t q0 = __ldg(p.q_offsets + s), C = __ldg(p.q_offsets + s + 1) - q0;
    const int32_t ctx = min(__ldg(p.ctx_lens + s), p.max_blocks * 16);
    const int32_t tok0 = (tile_g - __ldg(p.tile_off + s)) * tile_tokens;   // first chunk token of the tile
    const int32_t ntok = min(tile_tokens, C - tok0);
    const int32_t p0 = ctx - C;                                            // tokens cached before the chunk
    const int32_t kv_len = p0 + tok0 + ntok;                               // what the tile's last token sees
    const bool bad = C > ctx || ntok <= 0;                                 // (flagged by the host where it has the lengths)
    const int32_t n_stages = bad ? 0 : (kv_len + PF_KV - 1) / PF_KV;

    if (tid == 0) {
        for (int i = 0; i < 8; ++i) pf_mbar_init(bar_k + 8 * i, 1);   // k_full[2], v_full[2], s_done[2], o_done[2]
        pf_mbar_init(bar_p2[0], PF_ROWS_THREADS);                      // P of a stage is in place: every row's thread arrives
        pf_mbar_init(bar_p2[1], PF_ROWS_THREADS);
        pf_mbar_init(bar_done, 1);
        misc[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(base + SM::OFF_MISC, PF_TMEM_COLS);
    // ---- block table -> slot table -> slot: lanes of the loading warp resolve the blocks of a stage well ahead of the
    // stage's copies into a ring in shared memory (two dependent global loads each; done serially by the thread that
    // issues the copies they cost ten microseconds per stage)
    volatile int32_t *slot_ring = reinterpret_cast<volatile int32_t *>(smem + SM::OFF_MISC + 16);   // [8 stages][4 blocks]
    const int32_t n_blocks = (kv_len + 15) / 16;
    auto load_blk = [&](int32_t j, int32_t i) -> int32_t {   // the block's logical id, -1: the stage has no such block
        const int32_t b = j * (PF_KV / 16) + i;
        if (j >= n_stages || b >= n_blocks) return -1;
        const int32_t blk = __ldg(p.block_table + (int64_t)s * p.max_blocks + b);
        return blk < 0 ? p.n_logical : blk;   // an id that names nothing is a missing unit, not a missing block
    };
    auto load_slot = [&](int32_t blk) -> int32_t {           // its slot, -2: no such unit on the GPU
        if (blk < 0) return -1;
        const int32_t v = blk < p.n_logical ? __ldcg(p.slot_table + blk) : -2;
        return v < 0 ? -2 : v;
    };
    auto store_slot = [&](int32_t j, int32_t i, int32_t slot) {
        if (slot < -1 || slot >= p.n_gpu_slots) {  // unit not on the GPU: flag it, stream slot 0 so the barriers complete
            pf_raise(p.status, STATUS_MISSING_UNIT);
            slot = 0;
        }
        slot_ring[(j & 7) * 4 + i] = slot;
    };
    if (warp == 5 && lane < 16) store_slot(lane >> 2, lane & 3, load_slot(load_blk(lane >> 2, lane & 3)));   // stages 0 .. 3
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc[0];
    const uint32_t tmem_o = tmem + 2 * PF_KV;   // S (and then P) of even stages: columns 0 .. 63, of odd stages: 64 .. 127; O: 128 .. 128 + D - 1
    constexpr uint32_t IDESC_S = instr_desc(BF16, PF_KV, false), IDESC_O = instr_desc(BF16, D, true);

    // ---- Q: thread r brings row r (token tok0 + r / G, head kvh * G + r % G) into the K-major swizzled layout
    const int r = tid;
    const int32_t my_tok = r / G, my_g = r - my_tok * G;
    const bool row_valid = !bad && tid < PF_ROWS_THREADS && my_tok < ntok;
    if (tid < PF_ROWS_THREADS) {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.q + ((int64_t)(q0 + tok0 + my_tok) * p.n_q_heads + kvh * G + my_g) * D);
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
            const uint4 v = row_valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4 *>(smem + SM::OFF_Q + (c >> 3) * (PF_M * 128) + (r >> 3) * 1024 + (r & 7) * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    auto dead = [&]() { return __shfl_sync(0xffffffffu, misc[1] != 0 ? 1 : 0, 0) != 0; };
    auto wait_all = [&](uint32_t bar, uint32_t parity) {   // by every lane of a warp
        if (!pf_mbar_wait(bar, parity)) {
            pf_raise(p.status, STATUS_WAIT_TIMEOUT);
            misc[1] = 1;
        }
        __syncwarp();
    };
    if (warp == 5) {
        // =============================================================================== the loading warp
        // A stage's K (or V) tiles - one TMA copy per (block, 64-element half), up to eight - are issued by as many lanes at
        // once.  K(j + 2) goes out as soon as the scores of stage j are complete (its buffer is free then), V(j + 1) as soon
        // as O += P V of stage j - 1 is.  The TMA unit takes a stage's 32 KiB at its own pace (the issue blocks meanwhile),
        // which is why this is a warp of its own: the MMAs must not queue behind it.
        int32_t last_k[2] = {-1, -1}, last_v[2] = {-1, -1};   // newest stage issued into each buffer
        auto issue_tiles = [&](int32_t j, bool v_rows) {
            const uint32_t buf = (uint32_t)(j & 1);
            const uint32_t bar = (v_rows ? bar_v : bar_k) + 8 * buf;
            const uint32_t dst0 = base + (v_rows ? SM::OFF_V : SM::OFF_K) + buf * SM::KV_BYTES;
            const int32_t nb = min(PF_KV / 16, n_blocks - j * (PF_KV / 16));
            if (lane == 0) pf_mbar_expect_tx(bar, (uint32_t)nb * 16u * D * 2u);
            __syncwarp();
            const int32_t i = lane / HALVES, h = lane - i * HALVES;
            if (i < nb) {
                const int32_t row0 = (slot_ring[(j & 7) * 4 + i] * p.n_kv_heads + kvh) * 32 + (v_rows ? 16 : 0);
                pf_tma_2d(dst0 + h * (PF_KV * 128) + i * 2048, &tmap, h * 64, row0, bar);
            }
            __syncwarp();
            (v_rows ? last_v : last_k)[buf] = j;
        };
        for (int32_t j = 0; j < min(n_stages, 2); ++j) {
            issue_tiles(j, false);
            issue_tiles(j, true);
        }
        __syncthreads();   // (Q is in shared memory: nothing of this warp's depends on it)
        // look-ups in flight across iterations: lanes 0 .. 3 hold the slot of a block of stage j + 4 and the id of one of
        // stage j + 5; their loads are issued in one iteration and used in the next
        int32_t slot_pend = -1, blk_pend = -1;
        if (lane < 4) {
            slot_pend = load_slot(load_blk(4, lane));
            blk_pend = load_blk(5, lane);
        }
        for (int32_t j = 0; j < n_stages; ++j) {
            if (lane < 4) {
                store_slot(j + 4, lane, slot_pend);
                slot_pend = load_slot(blk_pend);
                blk_pend = load_blk(j + 6, lane);
            }
            __syncwarp();
            if (dead()) break;
            if (j + 2 < n_stages) {
                wait_all(bar_s + 8 * (j & 1), (uint32_t)((j >> 1) & 1));
                if (dead()) break;
                issue_tiles(j + 2, false);
            }
            if (j >= 1 && j + 1 < n_stages) {
                wait_all(bar_o2 + 8 * ((j - 1) & 1), (uint32_t)(((j - 1) >> 1) & 1));
                if (dead()) break;
                issue_tiles(j + 1, true);
            }
        }
        if (dead()) {
            // giving up: the copies already issued still write into this CTA's shared memory - wait (bounded) for them
            for (int b2 = 0; b2 < 2; ++b2) {
                if (last_k[b2] >= 0) pf_mbar_wait(bar_k + 8 * b2, (uint32_t)((last_k[b2] >> 1) & 1));
                if (last_v[b2] >= 0) pf_mbar_wait(bar_v + 8 * b2, (uint32_t)((last_v[b2] >> 1) & 1));
            }
        }
        __syncwarp();
    } else if (warp == 4) {
        // =============================================================================== the issuing warp
        // (operand descriptors are formed by the whole warp, outside the branch of the lane that issues: values every lane
        // holds alike can live in the uniform registers the MMA instruction takes its operands from)
        uint64_t q_desc[D / 16];
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) q_desc[ks] = smem_desc(base + SM::OFF_Q + (ks >> 2) * (PF_M * 128) + (ks & 3) * 32, 16, 1024);
        // S(j) = Q K(j)^T into the stage's half of the score columns (K(j) must have landed)
        auto issue_qk = [&](int32_t j) {
            const uint32_t buf = (uint32_t)(j & 1);
            wait_all(bar_k + 8 * buf, (uint32_t)((j >> 1) & 1));
            if (dead()) return;
            uint64_t k_desc[D / 16];
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks)
                k_desc[ks] = smem_desc(base + SM::OFF_K + buf * SM::KV_BYTES + (ks >> 2) * (PF_KV * 128) + (ks & 3) * 32, 16, 1024);
            const uint32_t d_addr = tmem + buf * PF_KV;
            if (lane == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) mma_f16(d_addr, q_desc[ks], k_desc[ks], IDESC_S, ks > 0 ? 1u : 0u);
                tc_commit(bar_s + 8 * buf);
            }
            __syncwarp();
        };
        __syncthreads();   // Q is in shared memory
        if (n_stages > 0) issue_qk(0);
        // Software pipeline: while the four softmax warps work on the scores of stage j, the tensor core computes those of
        // stage j + 1 (into the other half of the score columns) and, before that, finishes O += P V of stage j - 1.
        for (int32_t j = 0; j < n_stages; ++j) {
            if (dead()) break;
            const uint32_t buf = (uint32_t)(j & 1);
            // the other half of the score columns held P(j - 1): O += P V of stage j - 1 must have completed
            if (j >= 1) {
                wait_all(bar_o2 + 8 * ((j - 1) & 1), (uint32_t)(((j - 1) >> 1) & 1));
                if (dead()) break;
            }
            if (j + 1 < n_stages) {
                issue_qk(j + 1);
                if (dead()) break;
            }
            // P(j) is in tensor memory (every row's thread has arrived) and V(j) has landed: O += P V
            wait_all(bar_p2[buf], (uint32_t)((j >> 1) & 1));
            wait_all(bar_v + 8 * buf, (uint32_t)((j >> 1) & 1));
            if (dead()) break;
            // V: 16 tokens (two groups of eight rows) further per step; 64-element chunks of D are PF_KV * 128 bytes apart
            uint64_t v_desc[PF_KV / 16];
#pragma unroll
            for (int ks = 0; ks < PF_KV / 16; ++ks) v_desc[ks] = smem_desc(base + SM::OFF_V + buf * SM::KV_BYTES + ks * 2048, PF_KV * 128, 1024);
            const uint32_t tmem_sj = tmem + buf * PF_KV;
            const uint32_t acc0 = j > 0 ? 1u : 0u;
            if (lane == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < PF_KV / 16; ++ks) {
                    mma_f16_ts(tmem_o, tmem_sj + ks * 8, v_desc[ks], IDESC_O, ks > 0 ? 1u : acc0);
                    if (BF16) mma_f16_ts(tmem_o, tmem_sj + 32 + ks * 8, v_desc[ks], IDESC_O, 1u);
                }
                tc_commit(bar_o2 + 8 * buf);
                if (j + 1 == n_stages) tc_commit(bar_done);   // O is final
            }
            __syncwarp();
        }
        __syncwarp();
    } else {
        // =============================================================================== the softmax warps
        __syncthreads();   // Q is in shared memory
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const int32_t my_pos = p0 + tok0 + my_tok;   // this row's position: it sees tokens 0 .. my_pos
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int32_t j = 0; j < n_stages; ++j) {
            const uint32_t buf = (uint32_t)(j & 1);
            const uint32_t tmem_sj = tmem + buf * PF_KV;
            // ---- the scores of stage j
            if (!pf_mbar_wait(bar_s + 8 * buf, (uint32_t)((j >> 1) & 1))) {
                pf_raise(p.status, STATUS_WAIT_TIMEOUT);
                misc[1] = 1;
            }
            if (__any_sync(0xffffffffu, misc[1] != 0)) { ok = false; break; }
            tc_fence_after();
            uint32_t sv[2][32];
            tmem_ld32(tmem_sj + lane_addr, sv[0]);
            tmem_ld32(tmem_sj + lane_addr + 32, sv[1]);
            tmem_wait_ld();
            const int32_t t_base = j * PF_KV;
            float m_new, alpha, sum;
            uint32_t ph[32];
            [[maybe_unused]] uint32_t pl[32];
            // P in the 16-bit type, two tokens per 32-bit word: the A operand of O += P V, kept in tensor memory where the
            // scores were.  bf16 keeps 8 significant bits: the rounding remainder of P goes into a second bf16 operand, so
            // that the product sees about 16 bits (fp16's 11 bits need no correction).
            if (t_base + PF_KV - 1 <= p0 + tok0 && p.scale_log2e > 0.f) {
                // Every row of the tile sees every token of the stage (all stages but the last one or two of a tile): no
                // mask, and the softmax is what bounds this kernel - 64 exponentials per row and stage on four warps - so it
                // is written for the instruction count: the maximum over the raw scores (four chains), one fused
                // multiply-add and one ex2 per element, sums in four chains over the unrounded probabilities (they differ from
                // what the tensor core sees by the operand's rounding, 2^-12 or 2^-17 relative: nothing beside 2e-3).
                float a0 = -INFINITY, a1 = -INFINITY, a2 = -INFINITY, a3 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 64; c += 4) {
                    a0 = fmaxf(a0, __uint_as_float(sv[c >> 5][c & 31]));
                    a1 = fmaxf(a1, __uint_as_float(sv[(c + 1) >> 5][(c + 1) & 31]));
                    a2 = fmaxf(a2, __uint_as_float(sv[(c + 2) >> 5][(c + 2) & 31]));
                    a3 = fmaxf(a3, __uint_as_float(sv[(c + 3) >> 5][(c + 3) & 31]));
                }
                const float m_cand = fmaxf(m_run, fmaxf(fmaxf(a0, a1), fmaxf(a2, a3)) * p.scale_log2e);
                const bool grow = m_cand > m_run + PF_LAZY;   // (true at the first stage: m_run = -inf)
                m_new = grow ? m_cand : m_run;
                alpha = grow ? pf_exp2(m_run - m_cand) : 1.f;
                const float neg_m = -m_new;
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                for (int w = 0; w < 32; ++w) {
                    const int c = 2 * w;
                    const float e0 = pf_exp2(fmaf(__uint_as_float(sv[c >> 5][c & 31]), p.scale_log2e, neg_m));
                    const float e1 = pf_exp2(fmaf(__uint_as_float(sv[(c + 1) >> 5][(c + 1) & 31]), p.scale_log2e, neg_m));
                    ph[w] = pf_pack2<BF16>(e0, e1);
                    if (BF16) pl[w] = pf_pack2<true>(e0 - __uint_as_float(ph[w] << 16), e1 - __uint_as_float(ph[w] & 0xffff0000u));
                    if (w & 1) {
                        s2 += e0;
                        s3 += e1;
                    } else {
                        s0 += e0;
                        s1 += e1;
                    }
                }
                sum = (s0 + s1) + (s2 + s3);
            } else {
                float mx = -INFINITY;
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        float x = __uint_as_float(sv[h][c]) * p.scale_log2e;
                        x = (row_valid && t_base + h * 32 + c <= my_pos) ? x : -INFINITY;   // masked by selection (NaN scores too)
                        sv[h][c] = __float_as_uint(x);
                        mx = fmaxf(mx, x);
                    }
                const float m_cand = fmaxf(m_run, mx);
                const bool grow = m_cand > m_run + PF_LAZY;   // (m_run = -inf: true unless the row has seen nothing yet)
                m_new = grow ? m_cand : m_run;
                alpha = grow ? pf_exp2(m_run - m_cand) : 1.f;   // (m_run = -inf gives 0: nothing accumulated yet)
                sum = 0.f;
#pragma unroll
                for (int w = 0; w < 32; ++w) {
                    const int c = 2 * w;
                    const float x0 = __uint_as_float(sv[c >> 5][c & 31]), x1 = __uint_as_float(sv[(c + 1) >> 5][(c + 1) & 31]);
                    const float e0 = m_new == -INFINITY ? 0.f : pf_exp2(x0 - m_new), e1 = m_new == -INFINITY ? 0.f : pf_exp2(x1 - m_new);
                    ph[w] = pf_pack2<BF16>(e0, e1);
                    if (BF16) pl[w] = pf_pack2<true>(e0 - __uint_as_float(ph[w] << 16), e1 - __uint_as_float(ph[w] & 0xffff0000u));
                    sum += e0 + e1;
                }
            }
            l_run = l_run * alpha + sum;
            m_run = m_new;
            tmem_st32(tmem_sj + lane_addr, ph);            // a thread overwrites only its own row's scores, which it has read
            if (BF16) tmem_st32(tmem_sj + lane_addr + 32, pl);
            // ---- O *= alpha where a row's maximum moved (skipped by warps in which none did); O += P V of stage j - 1 first
            if (j >= 1 && __any_sync(0xffffffffu, alpha != 1.f)) {
                if (!pf_mbar_wait(bar_o2 + 8 * ((j - 1) & 1), (uint32_t)(((j - 1) >> 1) & 1))) {
                    pf_raise(p.status, STATUS_WAIT_TIMEOUT);
                    misc[1] = 1;
                }
                tc_fence_after();
                {
#pragma unroll
                    for (int c0 = 0; c0 < D; c0 += 32) {
                        uint32_t ov[32];
                        tmem_ld32(tmem_o + lane_addr + c0, ov);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
                        tmem_st32(tmem_o + lane_addr + c0, ov);
                    }
                }
            }
            tmem_wait_st();
            // ---- this stage's V has landed?  Rows of V beyond what the tile may see hold whatever was there (a tail
            // block's garbage, an earlier stage): masked tokens are excluded, not multiplied by zero, so clear them before
            // they meet P = 0
            const int32_t n_seen = min(PF_KV, kv_len - j * PF_KV);
            if (n_seen < PF_KV) {
                if (!pf_mbar_wait(bar_v + 8 * buf, (uint32_t)((j >> 1) & 1))) {
                    pf_raise(p.status, STATUS_WAIT_TIMEOUT);
                    misc[1] = 1;
                }
                for (int e = tid; e < (PF_KV - n_seen) * HALVES * 8; e += PF_ROWS_THREADS) {
                    const int row = n_seen + e / (HALVES * 8), rem = e % (HALVES * 8);
                    *reinterpret_cast<uint4 *>(smem + SM::OFF_V + buf * SM::KV_BYTES + (rem >> 3) * (PF_KV * 128) + row * 128 + ((rem & 7) << 4)) =
                        make_uint4(0u, 0u, 0u, 0u);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            tc_fence_before();
            pf_mbar_arrive(bar_p2[buf]);
        }
        if (ok && n_stages > 0) {
            if (!pf_mbar_wait(bar_done, 0u)) {
                pf_raise(p.status, STATUS_WAIT_TIMEOUT);
                misc[1] = 1;
            }
            tc_fence_after();
            ok = !__any_sync(0xffffffffu, misc[1] != 0);
        }
        // ---- out = O / l, rounded to the 16-bit type (nearest even).  The TMEM loads are warp-wide: rows beyond the chunk
        // take part in them and store nothing.
        if (ok && n_stages > 0) {
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            uint4 *dst = reinterpret_cast<uint4 *>(p.out + ((int64_t)(q0 + tok0 + my_tok) * p.n_q_heads + kvh * G + my_g) * D);
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t ov[32];
                tmem_ld32(tmem_o + lane_addr + c0, ov);
                tmem_wait_ld();
                if (row_valid) {
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {
                        uint4 v;
                        v.x = pf_pack2<BF16>(__uint_as_float(ov[c]) * inv, __uint_as_float(ov[c + 1]) * inv);
                        v.y = pf_pack2<BF16>(__uint_as_float(ov[c + 2]) * inv, __uint_as_float(ov[c + 3]) * inv);
                        v.z = pf_pack2<BF16>(__uint_as_float(ov[c + 4]) * inv, __uint_as_float(ov[c + 5]) * inv);
                        v.w = pf_pack2<BF16>(__uint_as_float(ov[c + 6]) * inv, __uint_as_float(ov[c + 7]) * inv);
                        dst[(c0 + c) >> 3] = v;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, PF_TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------------------------------
// The same tile with stages of 128 KV tokens and ONE score buffer of 128 columns (fp16 pools).  A stage's scores are then
// eight MMAs of 128 x 128 x 16: the Q tile is re-read from shared memory half as often per token as with 64-token stages,
// which is what held the tensor pipe.  A CTA's stages run strictly one after the other - S(j), softmax(j), O += P V (j),
// then S(j + 1) over the columns P(j) lay in - and the overlap comes from the SM's other CTA: while one CTA's warps do
// the softmax, the other's MMAs run.  K and V need one buffer each (K(j + 1) is loaded during the softmax and O += P V
// of stage j, V(j + 1) during the scores and the softmax of stage j + 1).  The softmax takes a row's 128 scores in two
// halves of 64 and in two passes (the maximum, then the probabilities: a thread cannot hold the whole row).  bf16 pools
// keep the 64-token kernel above: with their second P operand O += P V is sixteen MMAs per stage, and strictly serial
// stages lose more there than the wider score tile gains (602 against 642 TFLOP/s; fp16: 816 against 698).
constexpr int PFW_KV = 128;
constexpr int PFW_TMEM_COLS = 256;

template <int D>
struct PfSmemWide {
    static constexpr int Q_BYTES = PF_M * D * 2;        // [D / 64][128 rows][128 B]
    static constexpr int KV_BYTES = PFW_KV * D * 2;      // [D / 64][128 tokens][128 B]
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + Q_BYTES;       // one stage
    static constexpr int OFF_V = OFF_K + KV_BYTES;      // one stage
    static constexpr int OFF_BAR = OFF_V + KV_BYTES;    // k_full, v_full, s_done, o_done, p_done, done
    static constexpr int OFF_MISC = OFF_BAR + 128;      // [0] TMEM base, [1] abort, [4 .. 35] slots of eight stages' blocks
    static constexpr int BYTES = OFF_MISC + 256;        // two CTAs per SM (with TMEM for two: 2 x 256 of 512 columns)
};

template <int D, bool BF16>
__global__ void __launch_bounds__(PF_THREADS)
prefill_attn_wide_kernel(const __grid_constant__ CUtensorMap tmap, const PrefillParams p) {
    using SM = PfSmemWide<D>;
    constexpr int HALVES = D / 64;
    extern __shared__ __align__(1024) uint8_t pf_smem[];
    uint8_t *smem = pf_smem;
    const uint32_t base = pf_smem_u32(pf_smem);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (base & 1023u) {   // the swizzled tiles need a 1024-byte boundary: never seen otherwise, but do not compute garbage
        if (tid == 0) pf_raise(p.status, STATUS_WAIT_TIMEOUT);
        return;
    }
    // One barrier of each kind, phase = stage parity.  A CTA's stages run one after the other - S(j), softmax(j), O += P V
    // (j), then S(j + 1) over the same columns - so no waiter can fall two phases behind the barrier it waits on: the next
    // phase of each needs what the waiter does after its wait.  (The overlap comes from the SM's other CTA: while one
    // CTA's warps do the softmax, the other's MMAs run.)
    const uint32_t bar_k = base + SM::OFF_BAR, bar_v = bar_k + 8, bar_s = bar_k + 16, bar_o = bar_k + 24, bar_p = bar_k + 32;
    const uint32_t bar_done = bar_k + 40;   // O is final (used once: the softmax warps do not follow bar_o)
    volatile uint32_t *misc = reinterpret_cast<volatile uint32_t *>(smem + SM::OFF_MISC);

    // ---- which tile
    const int32_t item = blockIdx.x;
    const int32_t tile_g = item / p.n_kv_heads, kvh = item - tile_g * p.n_kv_heads;
    int32_t lo = 0, hi = p.n_seqs;  // largest s with tile_off[s] <= tile_g
    while (hi - lo > 1) {
        const int32_t mid = (lo + hi) >> 1;
        if (__ldg(p.tile_off + mid) <= tile_g) lo = mid;
        else hi = mid;
    }
    const int32_t s = lo;
    const int32_t G = p.group, tile_tokens = PF_M / G;
    const int32_t q0 = __ldg(p.q_offsets + s), C = __ldg(p.q_offsets + s + 1) - q0;
    const int32_t ctx = min(__ldg(p.ctx_lens + s), p.max_blocks * 16);
    const int32_t tok0 = (tile_g - __ldg(p.tile_off + s)) * tile_tokens;   // first chunk token of the tile
    const int32_t ntok = min(tile_tokens, C - tok0);
    const int32_t p0 = ctx - C;                                            // tokens cached before the chunk
    const int32_t kv_len = p0 + tok0 + ntok;                               // what the tile's last token sees
    const bool bad = C > ctx || ntok <= 0;                                 // (flagged by the host where it has the lengths)
    const int32_t n_stages = bad ? 0 : (kv_len + PFW_KV - 1) / PFW_KV;

    if (tid == 0) {
        for (int i = 0; i < 4; ++i) pf_mbar_init(bar_k + 8 * i, 1);   // k_full, v_full, s_done, o_done
        pf_mbar_init(bar_p, PF_ROWS_THREADS);                          // P of a stage is in place: every row's thread arrives
        pf_mbar_init(bar_done, 1);
        misc[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 4) tmem_alloc(base + SM::OFF_MISC, PFW_TMEM_COLS);
    // ---- block table -> slot table -> slot: lanes of the loading warp resolve the blocks of a stage well ahead of the
    // stage's copies into a ring in shared memory (two dependent global loads each; done serially by the thread that
    // issues the copies they cost ten microseconds per stage)
    volatile int32_t *slot_ring = reinterpret_cast<volatile int32_t *>(smem + SM::OFF_MISC + 16);   // [4 stages][8 blocks]
    const int32_t n_blocks = (kv_len + 15) / 16;
    auto load_blk = [&](int32_t j, int32_t i) -> int32_t {   // the block's logical id, -1: the stage has no such block
        const int32_t b = j * (PFW_KV / 16) + i;
        if (j >= n_stages || b >= n_blocks) return -1;
        const int32_t blk = __ldg(p.block_table + (int64_t)s * p.max_blocks + b);
        return blk < 0 ? p.n_logical : blk;   // an id that names nothing is a missing unit, not a missing block
    };
    auto load_slot = [&](int32_t blk) -> int32_t {           // its slot, -2: no such unit on the GPU
        if (blk < 0) return -1;
        const int32_t v = blk < p.n_logical ? __ldcg(p.slot_table + blk) : -2;
        return v < 0 ? -2 : v;
    };
    auto store_slot = [&](int32_t j, int32_t i, int32_t slot) {
        if (slot < -1 || slot >= p.n_gpu_slots) {  // unit not on the GPU: flag it, stream slot 0 so the barriers complete
            pf_raise(p.status, STATUS_MISSING_UNIT);
            slot = 0;
        }
        slot_ring[(j & 3) * 8 + i] = slot;
    };
    if (warp == 5 && lane < 16) store_slot(lane >> 3, lane & 7, load_slot(load_blk(lane >> 3, lane & 7)));   // stages 0 and 1
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc[0];
    const uint32_t tmem_o = tmem + PFW_KV;   // S (and then P): columns 0 .. 127; O: 128 .. 128 + D - 1
    constexpr uint32_t IDESC_S = instr_desc(BF16, PFW_KV, false), IDESC_O = instr_desc(BF16, D, true);

    // ---- Q: thread r brings row r (token tok0 + r / G, head kvh * G + r % G) into the K-major swizzled layout
    const int r = tid;
    const int32_t my_tok = r / G, my_g = r - my_tok * G;
    const bool row_valid = !bad && tid < PF_ROWS_THREADS && my_tok < ntok;
    if (tid < PF_ROWS_THREADS) {
        const uint4 *src = reinterpret_cast<const uint4 *>(p.q + ((int64_t)(q0 + tok0 + my_tok) * p.n_q_heads + kvh * G + my_g) * D);
#pragma unroll
        for (int c = 0; c < D / 8; ++c) {
            const uint4 v = row_valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4 *>(smem + SM::OFF_Q + (c >> 3) * (PF_M * 128) + (r >> 3) * 1024 + (r & 7) * 128 + (((c & 7) ^ (r & 7)) << 4)) = v;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    auto dead = [&]() { return __shfl_sync(0xffffffffu, misc[1] != 0 ? 1 : 0, 0) != 0; };
    auto wait_all = [&](uint32_t bar, uint32_t parity) {   // by every lane of a warp
        if (!pf_mbar_wait(bar, parity)) {
            pf_raise(p.status, STATUS_WAIT_TIMEOUT);
            misc[1] = 1;
        }
        __syncwarp();
    };
    if (warp == 5) {
        // =============================================================================== the loading warp
        // A stage's K (or V) tiles - one TMA copy per (block, 64-element half), up to sixteen - are issued by as many lanes
        // at once.  K(j + 1) goes out as soon as the scores of stage j are complete (the buffer is free then: the softmax and
        // O += P V of stage j give it time to land), V(j + 1) as soon as O += P V of stage j is.  The TMA unit takes a stage's
        // 32 KiB at its own pace (the issue blocks meanwhile), which is why this is a warp of its own.
        int32_t last_k = -1, last_v = -1;   // newest stage issued into each buffer
        auto issue_tiles = [&](int32_t j, bool v_rows) {
            const uint32_t bar = v_rows ? bar_v : bar_k;
            const uint32_t dst0 = base + (v_rows ? SM::OFF_V : SM::OFF_K);
            const int32_t nb = min(PFW_KV / 16, n_blocks - j * (PFW_KV / 16));
            if (lane == 0) pf_mbar_expect_tx(bar, (uint32_t)nb * 16u * D * 2u);
            __syncwarp();
            const int32_t i = lane / HALVES, h = lane - i * HALVES;
            if (i < nb) {
                const int32_t row0 = (slot_ring[(j & 3) * 8 + i] * p.n_kv_heads + kvh) * 32 + (v_rows ? 16 : 0);
                pf_tma_2d(dst0 + h * (PFW_KV * 128) + i * 2048, &tmap, h * 64, row0, bar);
            }
            __syncwarp();
            (v_rows ? last_v : last_k) = j;
        };
        if (n_stages > 0) {
            issue_tiles(0, false);
            issue_tiles(0, true);
        }
        __syncthreads();   // (Q is in shared memory: nothing of this warp's depends on it)
        // look-ups in flight across iterations: lanes 0 .. 7 hold the slot of a block of stage j + 2 and the id of one of
        // stage j + 3; their loads are issued in one iteration and used in the next
        int32_t slot_pend = -1, blk_pend = -1;
        if (lane < 8) {
            slot_pend = load_slot(load_blk(2, lane));
            blk_pend = load_blk(3, lane);
        }
        for (int32_t j = 0; j < n_stages; ++j) {
            if (lane < 8) {
                store_slot(j + 2, lane, slot_pend);
                slot_pend = load_slot(blk_pend);
                blk_pend = load_blk(j + 4, lane);
            }
            __syncwarp();
            if (dead() || j + 1 >= n_stages) break;
            wait_all(bar_s, (uint32_t)(j & 1));
            if (dead()) break;
            issue_tiles(j + 1, false);
            wait_all(bar_o, (uint32_t)(j & 1));
            if (dead()) break;
            issue_tiles(j + 1, true);
        }
        if (dead()) {
            // giving up: the copies already issued still write into this CTA's shared memory - wait (bounded) for them
            if (last_k >= 0) pf_mbar_wait(bar_k, (uint32_t)(last_k & 1));
            if (last_v >= 0) pf_mbar_wait(bar_v, (uint32_t)(last_v & 1));
        }
        __syncwarp();
    } else if (warp == 4) {
        // =============================================================================== the issuing warp
        // (operand descriptors are formed by the whole warp, outside the branch of the lane that issues: values every lane
        // holds alike can live in the uniform registers the MMA instruction takes its operands from)
        uint64_t q_desc[D / 16];
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) q_desc[ks] = smem_desc(base + SM::OFF_Q + (ks >> 2) * (PF_M * 128) + (ks & 3) * 32, 16, 1024);
        // S(j) = Q K(j)^T (K(j) must have landed)
        auto issue_qk = [&](int32_t j) {
            wait_all(bar_k, (uint32_t)(j & 1));
            if (dead()) return;
            uint64_t k_desc[D / 16];
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) k_desc[ks] = smem_desc(base + SM::OFF_K + (ks >> 2) * (PFW_KV * 128) + (ks & 3) * 32, 16, 1024);
            if (lane == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) mma_f16(tmem, q_desc[ks], k_desc[ks], IDESC_S, ks > 0 ? 1u : 0u);
                tc_commit(bar_s);
            }
            __syncwarp();
        };
        __syncthreads();   // Q is in shared memory
        if (n_stages > 0) issue_qk(0);
        // V: 16 tokens (two groups of eight rows) further per step; 64-element chunks of D are PFW_KV * 128 bytes apart
        uint64_t v_desc[PFW_KV / 16];
#pragma unroll
        for (int ks = 0; ks < PFW_KV / 16; ++ks) v_desc[ks] = smem_desc(base + SM::OFF_V + ks * 2048, PFW_KV * 128, 1024);
        for (int32_t j = 0; j < n_stages; ++j) {
            if (dead()) break;
            // P(j) is in tensor memory (every row's thread has arrived) and V(j) has landed: O += P V.  P of the stage's
            // half h lies where the half's scores were: 32 columns of 16-bit pairs (bf16: 32 more with the remainders)
            wait_all(bar_p, (uint32_t)(j & 1));
            wait_all(bar_v, (uint32_t)(j & 1));
            if (dead()) break;
            const uint32_t acc0 = j > 0 ? 1u : 0u;
            if (lane == 0) {
                tc_fence_after();
#pragma unroll
                for (int ks = 0; ks < PFW_KV / 16; ++ks) {
                    const uint32_t a_addr = tmem + (ks >> 2) * 64 + (ks & 3) * 8;
                    mma_f16_ts(tmem_o, a_addr, v_desc[ks], IDESC_O, ks > 0 ? 1u : acc0);
                    if (BF16) mma_f16_ts(tmem_o, a_addr + 32, v_desc[ks], IDESC_O, 1u);
                }
                tc_commit(bar_o);
                if (j + 1 == n_stages) tc_commit(bar_done);   // O is final
            }
            __syncwarp();
            if (j + 1 < n_stages) {
                // the scores of the next stage go where P(j) lies: O += P V of stage j must have completed
                wait_all(bar_o, (uint32_t)(j & 1));
                if (dead()) break;
                issue_qk(j + 1);
            }
        }
        __syncwarp();
    } else {
        // =============================================================================== the softmax warps
        __syncthreads();   // Q is in shared memory
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        const int32_t my_pos = p0 + tok0 + my_tok;   // this row's position: it sees tokens 0 .. my_pos
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int32_t j = 0; j < n_stages; ++j) {
            // ---- the scores of stage j: 128 columns, taken in two halves of 64 (a thread holds one half of its row at a time)
            if (!pf_mbar_wait(bar_s, (uint32_t)(j & 1))) {
                pf_raise(p.status, STATUS_WAIT_TIMEOUT);
                misc[1] = 1;
            }
            if (__any_sync(0xffffffffu, misc[1] != 0)) { ok = false; break; }
            tc_fence_after();
            const int32_t t_base = j * PFW_KV;
            // Every row of the tile sees every token of the stage (all stages but the last one or two of a tile): no mask, and
            // the softmax is written for the instruction count - the maximum over the raw scores (four chains), one fused
            // multiply-add and one ex2 per element, sums in four chains over the unrounded probabilities (they differ from
            // what the tensor core sees by the operand's rounding, 2^-12 or 2^-17 relative: nothing beside 2e-3).
            const bool plain = t_base + PFW_KV - 1 <= p0 + tok0 && p.scale_log2e > 0.f;
            // ---- first pass: the row's maximum over the stage
            float mx = -INFINITY;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t sv[2][32];
                tmem_ld32(tmem + lane_addr + 64 * h, sv[0]);
                tmem_ld32(tmem + lane_addr + 64 * h + 32, sv[1]);
                tmem_wait_ld();
                if (plain) {
                    float a0 = -INFINITY, a1 = -INFINITY, a2 = -INFINITY, a3 = -INFINITY;
#pragma unroll
                    for (int c = 0; c < 64; c += 4) {
                        a0 = fmaxf(a0, __uint_as_float(sv[c >> 5][c & 31]));
                        a1 = fmaxf(a1, __uint_as_float(sv[(c + 1) >> 5][(c + 1) & 31]));
                        a2 = fmaxf(a2, __uint_as_float(sv[(c + 2) >> 5][(c + 2) & 31]));
                        a3 = fmaxf(a3, __uint_as_float(sv[(c + 3) >> 5][(c + 3) & 31]));
                    }
                    mx = fmaxf(mx, fmaxf(fmaxf(a0, a1), fmaxf(a2, a3)) * p.scale_log2e);
                } else {
#pragma unroll
                    for (int c = 0; c < 64; ++c) {
                        const float x = __uint_as_float(sv[c >> 5][c & 31]) * p.scale_log2e;
                        // masked by selection (NaN scores too)
                        mx = fmaxf(mx, (row_valid && t_base + 64 * h + c <= my_pos) ? x : -INFINITY);
                    }
                }
            }
            const float m_cand = fmaxf(m_run, mx);
            const bool grow = m_cand > m_run + PF_LAZY;   // (m_run = -inf: true unless the row has seen nothing yet)
            const float m_new = grow ? m_cand : m_run;
            const float alpha = grow ? pf_exp2(m_run - m_cand) : 1.f;   // (m_run = -inf gives 0: nothing accumulated yet)
            // ---- second pass: P in the 16-bit type, two tokens per 32-bit word: the A operand of O += P V, kept in tensor
            // memory where the half's scores were.  bf16 keeps 8 significant bits: the rounding remainder of P goes into a
            // second bf16 operand, so that the product sees about 16 bits (fp16's 11 bits need no correction).
            float sum = 0.f;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t sv[2][32];
                tmem_ld32(tmem + lane_addr + 64 * h, sv[0]);
                tmem_ld32(tmem + lane_addr + 64 * h + 32, sv[1]);
                tmem_wait_ld();
                uint32_t ph[32];
                [[maybe_unused]] uint32_t pl[32];
                if (plain) {
                    const float neg_m = -m_new;
                    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                    for (int w = 0; w < 32; ++w) {
                        const int c = 2 * w;
                        const float e0 = pf_exp2(fmaf(__uint_as_float(sv[c >> 5][c & 31]), p.scale_log2e, neg_m));
                        const float e1 = pf_exp2(fmaf(__uint_as_float(sv[(c + 1) >> 5][(c + 1) & 31]), p.scale_log2e, neg_m));
                        ph[w] = pf_pack2<BF16>(e0, e1);
                        if (BF16) pl[w] = pf_pack2<true>(e0 - __uint_as_float(ph[w] << 16), e1 - __uint_as_float(ph[w] & 0xffff0000u));
                        if (w & 1) {
                            s2 += e0;
                            s3 += e1;
                        } else {
                            s0 += e0;
                            s1 += e1;
                        }
                    }
                    sum += (s0 + s1) + (s2 + s3);
                } else {
#pragma unroll
                    for (int w = 0; w < 32; ++w) {
                        const int c = 2 * w;
                        const bool see0 = row_valid && t_base + 64 * h + c <= my_pos, see1 = row_valid && t_base + 64 * h + c + 1 <= my_pos;
                        const float x0 = __uint_as_float(sv[c >> 5][c & 31]) * p.scale_log2e;
                        const float x1 = __uint_as_float(sv[(c + 1) >> 5][(c + 1) & 31]) * p.scale_log2e;
                        const float e0 = (see0 && m_new != -INFINITY) ? pf_exp2(x0 - m_new) : 0.f;
                        const float e1 = (see1 && m_new != -INFINITY) ? pf_exp2(x1 - m_new) : 0.f;
                        ph[w] = pf_pack2<BF16>(e0, e1);
                        if (BF16) pl[w] = pf_pack2<true>(e0 - __uint_as_float(ph[w] << 16), e1 - __uint_as_float(ph[w] & 0xffff0000u));
                        sum += e0 + e1;
                    }
                }
                tmem_st32(tmem + lane_addr + 64 * h, ph);   // a thread overwrites only its own row's scores, which it has read
                if (BF16) tmem_st32(tmem + lane_addr + 64 * h + 32, pl);
            }
            l_run = l_run * alpha + sum;
            m_run = m_new;
            // ---- O *= alpha where a row's maximum moved (skipped by warps in which none did).  O += P V of stage j - 1 is
            // complete: this stage's scores were issued behind it.
            if (j >= 1 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t ov[32];
                    tmem_ld32(tmem_o + lane_addr + c0, ov);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
                    tmem_st32(tmem_o + lane_addr + c0, ov);
                }
            }
            tmem_wait_st();
            // ---- this stage's V has landed?  Rows of V beyond what the tile may see hold whatever was there (a tail
            // block's garbage, an earlier stage): masked tokens are excluded, not multiplied by zero, so clear them before
            // they meet P = 0
            const int32_t n_seen = min(PFW_KV, kv_len - j * PFW_KV);
            if (n_seen < PFW_KV) {
                if (!pf_mbar_wait(bar_v, (uint32_t)(j & 1))) {
                    pf_raise(p.status, STATUS_WAIT_TIMEOUT);
                    misc[1] = 1;
                }
                for (int e = tid; e < (PFW_KV - n_seen) * HALVES * 8; e += PF_ROWS_THREADS) {
                    const int row = n_seen + e / (HALVES * 8), rem = e % (HALVES * 8);
                    *reinterpret_cast<uint4 *>(smem + SM::OFF_V + (rem >> 3) * (PFW_KV * 128) + row * 128 + ((rem & 7) << 4)) =
                        make_uint4(0u, 0u, 0u, 0u);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
            tc_fence_before();
            pf_mbar_arrive(bar_p);
        }
        if (ok && n_stages > 0) {
            if (!pf_mbar_wait(bar_done, 0u)) {
                pf_raise(p.status, STATUS_WAIT_TIMEOUT);
                misc[1] = 1;
            }
            tc_fence_after();
            ok = !__any_sync(0xffffffffu, misc[1] != 0);
        }
        // ---- out = O / l, rounded to the 16-bit type (nearest even).  The TMEM loads are warp-wide: rows beyond the chunk
        // take part in them and store nothing.
        if (ok && n_stages > 0) {
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            uint4 *dst = reinterpret_cast<uint4 *>(p.out + ((int64_t)(q0 + tok0 + my_tok) * p.n_q_heads + kvh * G + my_g) * D);
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t ov[32];
                tmem_ld32(tmem_o + lane_addr + c0, ov);
                tmem_wait_ld();
                if (row_valid) {
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {
                        uint4 v;
                        v.x = pf_pack2<BF16>(__uint_as_float(ov[c]) * inv, __uint_as_float(ov[c + 1]) * inv);
                        v.y = pf_pack2<BF16>(__uint_as_float(ov[c + 2]) * inv, __uint_as_float(ov[c + 3]) * inv);
                        v.z = pf_pack2<BF16>(__uint_as_float(ov[c + 4]) * inv, __uint_as_float(ov[c + 5]) * inv);
                        v.w = pf_pack2<BF16>(__uint_as_float(ov[c + 6]) * inv, __uint_as_float(ov[c + 7]) * inv);
                        dst[(c0 + c) >> 3] = v;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, PFW_TMEM_COLS);
}

}  // namespace

int prefill_smem_bytes(int head_dim) { return head_dim == 128 ? PfSmem<128>::BYTES : PfSmem<64>::BYTES; }
static int prefill_wide_smem_bytes(int head_dim) { return head_dim == 128 ? PfSmemWide<128>::BYTES : PfSmemWide<64>::BYTES; }

// K and V rows of the pool as 16-row tiles: rows of head_dim elements, 32 per (slot, KV head): 16 of K, 16 of V.
cudaError_t make_prefill_tensor_map(void *gpu_pool, int64_t n_gpu_slots, int n_kv_heads, int head_dim, CUtensorMap *map) {
    typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                      const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (fn == nullptr || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
    cuuint64_t dims[2] = {(cuuint64_t)head_dim, (cuuint64_t)n_gpu_slots * (cuuint64_t)n_kv_heads * 32u};
    cuuint64_t strides[1] = {(cuuint64_t)head_dim * 2};
    cuuint32_t box[2] = {64, 16};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, gpu_pool, dims, strides, box, estr,
                                                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t prefill_configure(int head_dim, int dtype) {
    // bf16 pools: stages of 64 tokens, two score buffers; fp16 pools: stages of 128 tokens, one score buffer
    const bool wide = dtype != PIE_BF16;
    const int smem = wide ? prefill_wide_smem_bytes(head_dim) : prefill_smem_bytes(head_dim);
    const void *k = wide ? (head_dim == 128 ? (const void *)prefill_attn_wide_kernel<128, false> : (const void *)prefill_attn_wide_kernel<64, false>)
                         : (head_dim == 128 ? (const void *)prefill_attn_kernel<128, true> : (const void *)prefill_attn_kernel<64, true>);
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
}

cudaError_t launch_prefill_attention(const AttnShape &sh, const PrefillLaunch &a, const CUtensorMap &map, cudaStream_t stream) {
    if (a.n_tiles <= 0) return cudaSuccess;
    PrefillParams p;
    p.q = (const uint16_t *)a.q;
    p.out = (uint16_t *)a.out;
    p.block_table = a.block_table;
    p.ctx_lens = a.ctx_lens;
    p.q_offsets = a.q_offsets;
    p.tile_off = a.tile_off;
    p.slot_table = a.slot_table;
    p.status = a.status;
    p.n_gpu_slots = sh.n_gpu_slots;
    p.max_blocks = a.max_blocks;
    p.n_seqs = a.n_seqs;
    p.n_q_heads = sh.n_q_heads;
    p.n_kv_heads = sh.n_kv_heads;
    p.group = sh.n_q_heads / sh.n_kv_heads;
    p.n_logical = sh.n_logical;
    p.scale_log2e = a.scale * 1.4426950408889634f;
    const unsigned grid = (unsigned)((int64_t)a.n_tiles * sh.n_kv_heads);
    if (sh.dtype == PIE_BF16) {
        const int smem = prefill_smem_bytes(sh.head_dim);
        if (sh.head_dim == 128) prefill_attn_kernel<128, true><<<grid, PF_THREADS, smem, stream>>>(map, p);
        else prefill_attn_kernel<64, true><<<grid, PF_THREADS, smem, stream>>>(map, p);
    } else {
        const int smem = prefill_wide_smem_bytes(sh.head_dim);
        if (sh.head_dim == 128) prefill_attn_wide_kernel<128, false><<<grid, PF_THREADS, smem, stream>>>(map, p);
        else prefill_attn_wide_kernel<64, false><<<grid, PF_THREADS, smem, stream>>>(map, p);
    }
    return cudaGetLastError();
}

}  // namespace pie
