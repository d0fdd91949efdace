// Launch interface between the pool (host control) and the sm_100a kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace pie {

// device status word bits (written by kernels into mapped pinned memory, read by the host later)
enum : int32_t {
    STATUS_MISSING_UNIT = 1,   // a block id or slot was out of range / not on the GPU
    STATUS_CTX_TOO_LONG = 2,   // ctx_len exceeded 16 * max_blocks_per_seq (clamped)
    STATUS_WAIT_TIMEOUT = 4    // a bounded mbarrier wait ran out
};

// ---- swap ----------------------------------------------------------------------------------------
// list: device int32 triples {src_slot, dst_slot, logical_block} x n.  slot_table may be NULL;
// table_mode 1: slot_table[block] = dst_slot (swap-in), 2: slot_table[block] = -1 (swap-out).
cudaError_t launch_swap(const void *src_pool, void *dst_pool, const int32_t *list, int64_t n, int64_t block_bytes,
                        int32_t *slot_table, int table_mode, int n_ctas, cudaStream_t stream);
// the same lists moved by bulk (TMA) copies through shared-memory stages: one warp per CTA, no data in registers.
// status: device-visible status words (a bounded wait that runs out raises STATUS_WAIT_TIMEOUT).
cudaError_t launch_swap_bulk(const void *src_pool, void *dst_pool, const int32_t *list, int64_t n, int64_t block_bytes,
                             int32_t *slot_table, int table_mode, int n_ctas, int32_t *status, cudaStream_t stream);
// table update only (copy-engine path, alloc/free): entries = device int32 pairs {index, value} x n.
cudaError_t launch_patch(int32_t *table, const int32_t *entries, int64_t n, cudaStream_t stream);
// same, from triples {src, dst, block} as launch_swap
cudaError_t launch_patch_from_list(int32_t *slot_table, const int32_t *list, int64_t n, int table_mode,
                                   cudaStream_t stream);

// ---- prefill-side KV write -------------------------------------------------------------------------
// k, v: device [n_tokens][n_kv_heads][head_dim] 16-bit; token t is position token_pos[t] of sequence token_seq[t].
cudaError_t launch_kv_write(const void *k, const void *v, const int32_t *token_seq, const int32_t *token_pos, int64_t n_tokens,
                            const int32_t *block_table, int32_t max_blocks, int32_t n_seqs, const int32_t *slot_table,
                            int32_t n_logical, int64_t n_gpu_slots, void *gpu_pool, int32_t n_kv_heads, int32_t head_dim,
                            int32_t *status, cudaStream_t stream);
// the same into an 8-bit pool (head_dim 128): rows are quantised to E4M3 with the append's rule
cudaError_t launch_kv_write8(const void *k, const void *v, const int32_t *token_seq, const int32_t *token_pos, int64_t n_tokens,
                             const int32_t *block_table, int32_t max_blocks, int32_t n_seqs, const int32_t *slot_table,
                             int32_t n_logical, int64_t n_gpu_slots, void *gpu_pool, int32_t n_kv_heads, int32_t dtype,
                             float k_scale, float v_scale, int32_t *status, cudaStream_t stream);

// ---- attention -----------------------------------------------------------------------------------
struct AttnShape {
    int head_dim;      // 64 or 128
    int dtype;         // PIE_F16 / PIE_BF16
    int n_q_heads, n_kv_heads;
    int n_logical;
    int64_t n_gpu_slots;
    int kv_fp8 = 0;    // blocks hold E4M3 bytes (head_dim 128 only)
};

struct AttnScratch {
    int32_t *chunk_off;  // [max_seqs + 1] (used only for batches beyond the in-kernel plan)
    int32_t *counters;   // attn_counter_words(max_seqs, n_kv_heads) int32, zero before the first launch
    float *part_o;       // [max_items][G][D]
    float *part_ml;      // [max_items][G][2]
    float *part_o_more[2] = {nullptr, nullptr};   // optional second and third pair of partial buffers (deferred combine:
    float *part_ml_more[2] = {nullptr, nullptr};  // AttnLaunch::defer_combine; the counters then hold three sets of four words)
    int64_t max_items;   // capacity in items (chunk, kv head)
    int32_t max_seqs;
};

struct AttnLaunch {
    const void *q;
    void *out;
    const int32_t *block_table;
    int32_t max_blocks;
    const int32_t *ctx_lens;
    const int32_t *slot_table;  // this layer's row of the device slot table
    int32_t n_seqs;
    float scale;
    const void *k_new, *v_new;  // optional
    void *gpu_pool;
    int32_t split_tokens;
    int32_t grid;               // persistent CTAs
    int32_t variant;            // kernel variant (0 = default)
    int32_t *status;            // device-visible status word
    uint64_t *stamps = nullptr; // optional, device-visible: [0] start, [1] end of the attention kernel (GPU timer, ns),
                                // [2] ns CTA 0 waited for arriving units, [3] the batch's context tokens
    unsigned long long *done_word = nullptr;  // optional, device memory: the kernel's last CTA stores done_value there
    unsigned long long done_value = 0;        // (the call's compute ticket: copy streams wait for it by value)
    int32_t *tokens_out = nullptr;  // optional, device-visible: receives the batch's context-token count
    const unsigned long long *arrive = nullptr;  // presence wait inside the kernel: wait until *arrive >= arrive_need
    unsigned long long arrive_need = 0;          // (the copy-in stream stores a list's ticket there behind its copies)
    const unsigned long long *inputs_arrive = nullptr;  // the same for the call's q / k_new / v_new where a copy stream brings
    unsigned long long inputs_need = 0;                 // them: no input is read before *inputs_arrive >= inputs_need
    bool dependent_launch = false;  // launch with programmatic stream serialization: only where the kernel before it in
                                    // the stream writes none of this call's lengths and tables
    float k_scale = 1.f, v_scale = 1.f;  // 8-bit pools: a stored byte stands for decode(byte) * scale
    // Deferred combine (needs the scratch's further pairs of partial buffers; ignored without them).  defer_combine: no
    // combine kernel follows this call - the NEXT call must name this call's out as its prev_out, have parity + 1 (the
    // buffers and counter sets are taken in turns of three), follow this call directly in the stream as a dependent
    // launch, and attend the same batch with the same lengths and split; its kernel starts beside this call's tail and
    // merges this call's partials at the end of its own launch, so this call's out is complete when the next call's
    // kernel is.  Whoever defers must see to it that the next call happens (or launch_combine with this call's parity).
    bool defer_combine = false;
    void *prev_out = nullptr;
    int parity = 0;
};

// Build the TMA descriptors of the HBM pool: map3d covers a whole K+V tile in one copy
// (dims {64, rows, D/64}); map2d is the fallback with one copy per 128-byte half.  Returns which
// is usable in *use3d.
cudaError_t make_pool_tensor_maps(void *gpu_pool, int64_t n_gpu_slots, int n_kv_heads, int head_dim, CUtensorMap *map3d,
                                  CUtensorMap *map2d, int *use3d);
int attn_smem_bytes(int head_dim);
int64_t attn_counter_words(int32_t max_seqs, int32_t n_kv_heads);
cudaError_t attn_configure(int head_dim, int dtype, int variant, int *ctas_per_sm, int kv_fp8 = 0);
cudaError_t make_pool_tensor_map_fp8(void *gpu_pool, int64_t n_gpu_slots, int n_kv_heads, CUtensorMap *map2d);
cudaError_t launch_attention(const AttnShape &sh, const AttnScratch &sc, const AttnLaunch &a, const CUtensorMap &map,
                             int use3d, cudaStream_t stream);
// the combine kernel by itself (what launch_attention launches behind a call that does not defer its merge)
cudaError_t launch_combine(const AttnShape &sh, const AttnScratch &sc, void *out, int32_t n_seqs, int32_t max_blocks,
                           int32_t split_tokens, int parity, cudaStream_t stream);

// ---- chunked-prefill attention (tcgen05 / TMEM) ----------------------------------------------------------------
struct PrefillLaunch {
    const void *q;               // [n_tokens][Hq][D], the chunks of all sequences one after the other
    void *out;                   // same shape
    const int32_t *block_table;  // device [n_seqs][max_blocks]
    int32_t max_blocks;
    const int32_t *ctx_lens;     // device [n_seqs]: context length including the chunk
    const int32_t *q_offsets;    // device [n_seqs + 1]: first token of each sequence's chunk
    const int32_t *tile_off;     // device [n_seqs + 1]: first 128-row tile of each sequence (a tile holds 128 / G tokens)
    const int32_t *slot_table;   // this layer's row of the device slot table
    int32_t n_seqs;
    int32_t n_tiles;             // tile_off[n_seqs]
    float scale;
    int32_t *status;
};
// the pool's K and V rows as 16-row TMA tiles (box 64 elements x 16 rows, 128-byte swizzle)
cudaError_t make_prefill_tensor_map(void *gpu_pool, int64_t n_gpu_slots, int n_kv_heads, int head_dim, CUtensorMap *map);
cudaError_t prefill_configure(int head_dim, int dtype);
cudaError_t launch_prefill_attention(const AttnShape &sh, const PrefillLaunch &a, const CUtensorMap &map, cudaStream_t stream);

}  // namespace pie
