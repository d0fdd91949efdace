/*
 * CPU oracle for the KV-block swap + paged decode-attention path.  TEST INFRASTRUCTURE ONLY:
 * it is called by the tests, by the smoke check and by the benchmark's cpu_baseline leg, never
 * by the product library, and it shares no code with the CUDA path.
 *
 * What it states, and from where:
 *   - swap = byte copy of whole blocks between a device pool and a host pool, the source left
 *     as it was (Section 3.2: a swapped unit is copied in the background and the mapping table
 *     is switched over once the copy is confirmed; Section 4: a kernel that copies the cache).
 *   - paged decode attention = softmax(scale * q.K^T).V of one query token per sequence over the
 *     tokens held in that sequence's blocks (Section 2.1 decode stage; Section 2.3 paged,
 *     non-contiguous KV storage).  The paper inherits this kernel and prints no formula, so the
 *     textbook definition is written out: two passes (max, then exp/sum), index order, no blocking.
 *   - a block is reached through a mapping table (Section 3.2): logical block -> {side, slot}.
 *     The oracle reads a block wherever it lives, so its result cannot depend on residency.
 *
 * Slot layout (this build's choice, the paper states none): one slot holds one layer's K and V of
 * one 16-token block as 16-bit elements [Hkv][kv=2][16][D]; kv=0 is K, kv=1 is V.
 *
 * Every floating-point routine exists twice, in fp32 ("_f32", the precision the method computes
 * in) and in fp64 ("_f64", used to show the fp32 one is itself accurate).  Inputs are fp16/bf16
 * bit patterns converted exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define BLOCK_TOKENS 16

/* ---- exact 16-bit -> float conversions ------------------------------------------------ */

static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static float f16_to_f32(uint16_t h) {
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    int exp = (h >> 10) & 0x1F;
    uint32_t man = h & 0x3FFu;
    if (exp == 0) { /* zero or subnormal: man * 2^-24 exactly */
        float f = (float)man * 5.9604644775390625e-08f;
        return sign ? -f : f;
    }
    uint32_t u;
    if (exp == 31) u = sign | 0x7F800000u | (man << 13);
    else u = sign | ((uint32_t)(exp + 112) << 23) | (man << 13);
    float f;
    memcpy(&f, &u, 4);
    return f;
}

float pie_oracle_bits_to_f32(uint16_t bits, int dtype) {
    return dtype == 0 ? f16_to_f32(bits) : bf16_to_f32(bits);
}

/* ---- swap semantics -------------------------------------------------------------------- */

/* for i < n: dst_pool[dst[i]] <- src_pool[src[i]], whole blocks of block_bytes.  Returns -1 and
 * copies nothing when an id is out of range or two destinations coincide. */
int pie_oracle_swap_raw(uint8_t *dst_pool, int64_t n_dst_slots, const uint8_t *src_pool, int64_t n_src_slots,
                        int64_t block_bytes, const int32_t *src, const int32_t *dst, int64_t n) {
    for (int64_t i = 0; i < n; ++i) {
        if (src[i] < 0 || src[i] >= n_src_slots || dst[i] < 0 || dst[i] >= n_dst_slots) return -1;
        for (int64_t j = 0; j < i; ++j)
            if (dst[j] == dst[i]) return -1;
    }
    for (int64_t i = 0; i < n; ++i)
        memcpy(dst_pool + (int64_t)dst[i] * block_bytes, src_pool + (int64_t)src[i] * block_bytes, (size_t)block_bytes);
    return 0;
}

/* ---- locating one token's K or V row --------------------------------------------------- */

typedef struct {
    const uint16_t *gpu_pool;
    const uint16_t *host_pool;
    const int32_t *unit_side; /* [n_logical] of this layer: 0 -> gpu_pool, 1 -> host_pool */
    const int32_t *unit_slot; /* [n_logical] slot index inside that pool */
    int n_kv_heads, head_dim, dtype;
} kv_view;

static const uint16_t *kv_row(const kv_view *v, int32_t block, int kvh, int kv, int row) {
    const uint16_t *pool = v->unit_side[block] == 0 ? v->gpu_pool : v->host_pool;
    int64_t slot_elems = (int64_t)v->n_kv_heads * 2 * BLOCK_TOKENS * v->head_dim;
    return pool + (int64_t)v->unit_slot[block] * slot_elems +
           (((int64_t)kvh * 2 + kv) * BLOCK_TOKENS + row) * v->head_dim;
}

/* write the new token's K and V rows at position ctx_len-1 (the per-iteration cache update of
 * Section 3.2); pools are written in place. */
void pie_oracle_append(uint16_t *gpu_pool, uint16_t *host_pool, const int32_t *unit_side, const int32_t *unit_slot,
                       const uint16_t *k_new, const uint16_t *v_new, const int32_t *block_table, int max_blocks,
                       const int32_t *ctx_lens, int n_seqs, int n_kv_heads, int head_dim) {
    kv_view v = {gpu_pool, host_pool, unit_side, unit_slot, n_kv_heads, head_dim, 0};
    for (int s = 0; s < n_seqs; ++s) {
        int pos = ctx_lens[s] - 1;
        if (pos < 0) continue;
        int32_t blk = block_table[(int64_t)s * max_blocks + pos / BLOCK_TOKENS];
        for (int h = 0; h < n_kv_heads; ++h) {
            uint16_t *kr = (uint16_t *)kv_row(&v, blk, h, 0, pos % BLOCK_TOKENS);
            uint16_t *vr = (uint16_t *)kv_row(&v, blk, h, 1, pos % BLOCK_TOKENS);
            memcpy(kr, k_new + ((int64_t)s * n_kv_heads + h) * head_dim, (size_t)head_dim * 2);
            memcpy(vr, v_new + ((int64_t)s * n_kv_heads + h) * head_dim, (size_t)head_dim * 2);
        }
    }
}

/* ---- the two precisions ----------------------------------------------------------------- */

#define REAL float
#define EXP expf
#define SUFFIX(name) name##_f32
#include "pie_oracle_attention.inc"
#undef REAL
#undef EXP
#undef SUFFIX

#define REAL double
#define EXP exp
#define SUFFIX(name) name##_f64
#include "pie_oracle_attention.inc"
#undef REAL
#undef EXP
#undef SUFFIX
