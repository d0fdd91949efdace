/*
 * pie.h - C ABI of the B200-native KV-block swapping + paged decode-attention library.
 *
 * The library implements the hot path of performance-transparent swapping (Pie, arXiv 2411.09317,
 * Section 3): paged KV-cache blocks live in an HBM block pool or in a pinned host pool; a mapping table
 * (Section 3.2) says where each (layer, logical block) unit is; background copies move units between
 * the pools while the paged decode attention of the current layer runs, and an adaptive controller
 * (Section 3.4.2) sizes the host-resident share so that copies stay hidden behind compute.
 *
 * Conventions
 *   - every call returns a pie_status (0 = PIE_OK, negative = error); nothing aborts, traps or throws.
 *   - argument errors are found before anything is enqueued: a failed call enqueues nothing and leaves
 *     the mapping table as it was.  Asynchronous CUDA errors surface at a later call as PIE_ERR_CUDA.
 *   - "host" pointers are read during the call and may be freed at return.  "device" pointers must stay
 *     valid until the pool's compute stream has passed the call.
 *   - one host thread per pool.  The library never calls the batched-memcpy runtime entry points.
 *   - slot layout: one slot holds one layer's K and V of one 16-token block as 16-bit elements
 *     [n_kv_heads][2 (K, V)][16 tokens][head_dim]; slot s starts at byte s * block_bytes of its pool.
 *     The paper states no layout; this one makes a head's K+V tile of a block one contiguous piece.
 */
#ifndef PIE_H
#define PIE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum pie_status {
    PIE_OK = 0,
    PIE_ERR_INVALID = -1,      /* null pointer, bad shape or dtype, duplicate id, unallocated block */
    PIE_ERR_RANGE = -2,        /* layer, block or slot id out of range */
    PIE_ERR_NOMEM = -3,        /* no free slot on the destination side / allocation failed */
    PIE_ERR_BUSY = -4,         /* a copy on the unit is still in flight (block free / read / write) */
    PIE_ERR_NOT_RESIDENT = -5, /* attention needs a unit that is neither on the GPU nor arriving */
    PIE_ERR_TIMEOUT = -6,      /* a bounded wait ran out */
    PIE_ERR_CUDA = -7,         /* a CUDA call failed: see pie_last_cuda_error */
    PIE_ERR_UNSUPPORTED = -8   /* head_dim / group size / block size outside the built set */
} pie_status;

enum { PIE_F16 = 0, PIE_BF16 = 1 };
enum { PIE_MODE_AUTO = 0, PIE_MODE_KERNEL = 1, PIE_MODE_COPY_ENGINE = 2, PIE_MODE_KERNEL_BULK = 3 };
enum { PIE_H2D = 0, PIE_D2H = 1 };
/* unit states of the two-phase mapping table (Section 3.2) */
enum { PIE_FREE = 0, PIE_GPU = 1, PIE_TO_HOST = 2, PIE_HOST = 3, PIE_TO_GPU = 4 };
/* copy queues: tickets of one queue complete in order */
enum { PIE_Q_NONE = 0, PIE_Q_IN = 1, PIE_Q_OUT = 2, PIE_Q_COMPUTE = 3 };

typedef struct pie_pool pie_pool;
typedef struct pie_table pie_table;
typedef struct pie_fifo pie_fifo;
typedef struct pie_governor pie_governor;

/* 8-bit blocks: see pie_set_kv_scales */
enum { PIE_KV_16BIT = 0, PIE_KV_E4M3 = 1 };

/* Both structs start with their own size as the caller compiled it: the library reads (pie_pool_config) or writes
 * (pie_stats) that many bytes at most, so a caller built against an older header keeps working when fields are added at
 * the end; fields the caller's struct does not have read as 0.  A size smaller than the first release's struct is
 * PIE_ERR_INVALID. */
typedef struct pie_pool_config {
    uint32_t struct_size;      /* sizeof(pie_pool_config) */
    int32_t n_layers;
    int32_t n_q_heads;
    int32_t n_kv_heads;        /* divides n_q_heads; n_q_heads / n_kv_heads <= 8 */
    int32_t head_dim;          /* 64 or 128 */
    int32_t block_tokens;      /* 16 */
    int32_t dtype;             /* PIE_F16 or PIE_BF16 */
    int32_t n_logical_blocks;  /* logical block ids 0 .. n-1, shared by all layers */
    int32_t max_seqs;          /* largest batch pie_decode_attention will see (scratch sizing) */
    int32_t own_streams;       /* 1: the library creates three non-blocking streams */
    int64_t n_gpu_slots;
    int64_t n_host_slots;
    void *gpu_base;            /* device memory of n_gpu_slots * block_bytes, 128-byte aligned, or NULL:
                                  the library allocates and owns it */
    void *host_base;           /* pinned host memory of n_host_slots * block_bytes, or NULL: the library
                                  allocates (cudaHostAlloc) and owns it */
    void *compute_stream;      /* cudaStream_t values; used only when own_streams == 0 */
    void *copy_in_stream;
    void *copy_out_stream;
    int32_t split_tokens;      /* split-K chunk in tokens, multiple of 16; 0 = the library chooses: 512 (1024 where the pool
                                * is laid out for long sequences: n_logical_blocks * 16 / max_seqs >= 6144) for single
                                * calls and for pie_decode_layer (whose caller puts its own kernels between the layers),
                                * and inside pie_decode_step / pie_decode_step_host, whose launches overlap at their
                                * ends, up to 2048 while every CTA still gets a work item */
    int32_t swap_ctas;         /* CTAs of the swap kernel; 0 = default (16) */
    int32_t attn_ctas_per_sm;  /* 0 = as many as fit */
    int32_t timing;            /* 1: per-layer timing for pie_controller_tick / pie_get_stats (the attention kernel notes
                                *    the GPU's timer in device memory, one copy per step brings the notes to the host;
                                *    timing events only on the copy streams);
                                * 2: also keep the per-layer timeline for pie_get_step_timeline */
    int32_t attn_variant;      /* attention kernel variant, for tuning (0 = default) */
    int32_t visible_blocks;    /* per-layer size visible to allocation at creation, in blocks (0 = n_logical_blocks;
                                * see pie_resize_begin) */
    int32_t kv_format;         /* PIE_KV_16BIT, or PIE_KV_E4M3: the blocks hold K and V as FP8 E4M3 bytes (see
                                * pie_set_kv_scales): head_dim 128 and variants 0 - 2 only (PIE_ERR_UNSUPPORTED
                                * otherwise), block_bytes halves */
    int32_t reserved[5];       /* 0 */
} pie_pool_config;

typedef struct pie_stats {
    uint32_t struct_size;                  /* sizeof(pie_stats): set it before pie_get_stats */
    uint32_t governor_state;               /* the throughput governor's state (pie_governor_state numbering) */
    double bytes_in, bytes_out;            /* swapped so far, per direction */
    double calls_kernel, calls_copy_engine;
    double last_step_compute_ms;           /* sum over layers: end of the previous layer's attention kernel to the end
                                            * of this one's (append, combine and launch gap included), minus the stall */
    double last_step_stall_ms;             /* sum over layers: what the layer's attention kernel (or, for lists an SM
                                            * kernel moved, the stream before it) waited for arriving units: the
                                            * presence wait */
    double last_step_swap_in_ms, last_step_swap_out_ms;   /* the copy streams' busy time: lists of a group count once */
    double last_step_ms;                   /* first layer's start to last layer's end */
    double ratio;                          /* current extension ratio */
    int64_t n_units_gpu, n_units_host, n_units_in_flight;
    int64_t steps_measured;
    double last_step_slowdown_ms;          /* what the step's layers took above its undisturbed ones (hidden copies share
                                            * HBM with the attention kernel); the controller counts it as waiting */
    double ratio_floor;                    /* the smallest extension ratio the GPU pool's size allows with the blocks
                                            * allocated now (the controller never goes below it) */
    double bytes_out_elided;               /* swap-out traffic elided so far (pie_set_retention) */
    double patch_kernel_launches;          /* table-patch kernels launched after copy-engine lists (lists of few id runs
                                            * patch the table by copy and launch none) */
    double governor_cap;                   /* the governor's cap on the ratio (1 = none; 0 before the first
                                            * pie_report_throughput) */
    int64_t prefetch_lists;                /* swap-in lists the decode loop has started so far, and how many of them were for */
    int64_t prefetch_violations;           /* layers of the NEXT token (Section 3.4.2's allowed rule violation) */
    double last_step_violation_ratio;      /* the two, over the last evaluated step */
    double copy_engine_copies;             /* data copies given to the copy engines so far (one per run of consecutive slots) */
    double reserved[3];                    /* 0 */
} pie_stats;

/* ---- pool (Section 3.1: the physical pools; Section 3.2: the mapping table) --------------------- */

/* Create a pool.  Validates the configuration (PIE_ERR_INVALID / PIE_ERR_UNSUPPORTED), allocates what
 * the caller did not supply (PIE_ERR_NOMEM), builds the free lists, the per-layer device slot tables
 * and the TMA descriptor of the HBM pool.  Needs a CUDA device: without one it fails with
 * PIE_ERR_CUDA - there is no CPU path.  *out is written only on success. */
int pie_pool_create(const pie_pool_config *cfg, pie_pool **out);
/* Drain the streams (bounded: 10 s, then PIE_ERR_TIMEOUT is returned but the pool is still freed) and
 * free what the library owns.  NULL is accepted. */
int pie_pool_destroy(pie_pool *pool);
size_t pie_block_bytes(const pie_pool *pool);

/* Allocate n logical blocks (one unit per layer each).  on_host (host, n bytes, may be NULL): non-zero
 * puts every unit of that block in the host pool; zero / NULL puts units on the GPU while slots are
 * available, else on the host (Section 4.1: the block manager hands out blocks).  ids_out (host, n)
 * receives the ids.  All or nothing: PIE_ERR_NOMEM allocates none. */
int pie_block_alloc(pie_pool *pool, int64_t n, const uint8_t *on_host, int32_t *ids_out);
/* Give n blocks back.  PIE_ERR_BUSY if a copy on any unit is still in flight (call pie_sync first). */
int pie_block_free(pie_pool *pool, const int32_t *ids, int64_t n);
/* Synchronous access to one unit wherever it lives (test set-up, read-back).  host_buf holds
 * block_bytes.  These wait for the unit's copies and use plain cudaMemcpy, not the swap path. */
int pie_block_write(pie_pool *pool, int32_t layer, int32_t block, const void *host_buf);
int pie_block_read(pie_pool *pool, int32_t layer, int32_t block, void *host_buf);
/* Table look-up: state (PIE_GPU ...), slots (-1 if none).  Any out pointer may be NULL. */
int pie_block_state(pie_pool *pool, int32_t layer, int32_t block, int32_t *state, int32_t *gpu_slot,
                    int32_t *host_slot);
/* Bulk look-up: side[L*NB] (PIE_FREE / PIE_GPU / PIE_HOST: where the unit is or is heading) and
 * slot[L*NB]; host arrays. */
int pie_get_placement(pie_pool *pool, int32_t *side, int32_t *slot);

/* ---- swapping (Section 3.2 two-phase update; Section 3.3 protocol; Section 4 swap kernel) -------- */

/* Make these logical blocks of `layer` host resident.  Phase 1 (during the call): host slots are
 * chosen and recorded, the copy is enqueued on the copy-out stream behind the layer's last attention
 * call, and the GPU slots are released tagged with this copy's ticket.  Phase 2: once the copy is
 * known complete (observed with cudaEventQuery at any later call) the units read PIE_HOST.
 * Blocks already on, or heading to, the host are skipped.  block_ids: host, n entries, distinct.
 * mode: PIE_MODE_KERNEL = gather/scatter kernel (16-byte loads and stores), PIE_MODE_KERNEL_BULK = the same lists
 * moved by bulk (TMA) copies through small shared-memory stages, PIE_MODE_COPY_ENGINE = one cudaMemcpyAsync per run of
 * consecutive slots, PIE_MODE_AUTO = copy engine when the list is at most 8 runs or its runs average 1 MiB, else
 * the bulk-copy kernel (measured: the copy engine reaches the link rate from
 * ~16 MB and disturbs a concurrent attention kernel several times less than SM-issued host traffic, but one call
 * per scattered 64 KiB block tops out near 12 GB/s; both kernels reach 0.92 of the link on scattered lists, the
 * bulk-copy one at a third of the load/store kernel's cost to the attention).  The slot table follows the data in stream order: written by
 * the kernel, or by one small copy per run of consecutive block ids (a patch kernel beyond 16 such runs). */
int pie_swap_out(pie_pool *pool, int32_t layer, const int32_t *block_ids, int64_t n, int32_t mode);
/* The mirror image on the copy-in stream.  The layer's next pie_decode_attention waits for it
 * (Section 3.2: presence check). */
int pie_swap_in(pie_pool *pool, int32_t layer, const int32_t *block_ids, int64_t n, int32_t mode);
/* The mechanism under both: copy n whole slots between the pools by PHYSICAL slot id, no table change.
 * dir PIE_H2D: src = host slots, dst = GPU slots; PIE_D2H the reverse.  dst ids must be distinct.
 * stream: a cudaStream_t, or NULL for the direction's copy stream.  For the swap microbenchmark and for
 * byte-exact checks. */
int pie_swap_raw(pie_pool *pool, int32_t dir, const int32_t *src_slots, const int32_t *dst_slots, int64_t n,
                 int32_t mode, void *stream);

/* ---- paged decode attention (Section 2.1 decode stage; Section 2.3 paged KV; Section 3.2) --------- */

/* One layer's decode attention for n_seqs sequences, enqueued on the compute stream:
 *   wait for the layer's arriving units -> [append k_new/v_new at position ctx_len-1] -> split-K paged
 *   attention -> combine -> out.
 * q, out: device [n_seqs][n_q_heads][head_dim] in the pool dtype.  k_new, v_new: device
 * [n_seqs][n_kv_heads][head_dim] or NULL (no append).  block_table_dev: device int32
 * [n_seqs][max_blocks_per_seq] of LOGICAL block ids - the kernel resolves them through the layer's slot
 * table, so callers pass the same table whether or not blocks were swapped (Section 4.1: base pointer
 * from the mapping table, offsets unchanged).  ctx_lens_dev: device int32 [n_seqs], context length
 * INCLUDING the appended token; 0 gives a zero output row.
 * block_table_host / ctx_lens_host (host, optional): when given, residency of every referenced unit is
 * checked before anything is enqueued (PIE_ERR_NOT_RESIDENT) and lengths beyond the table are rejected
 * (PIE_ERR_INVALID).  Without them a missing unit makes the kernel skip the tile, set a device status
 * word, and the NEXT call returns PIE_ERR_NOT_RESIDENT.
 * scale multiplies q.k (pass 1/sqrt(head_dim)). */
int pie_decode_attention(pie_pool *pool, int32_t layer, const void *q, void *out, const int32_t *block_table_dev,
                         int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, const int32_t *block_table_host,
                         const int32_t *ctx_lens_host, int32_t n_seqs, float scale, const void *k_new,
                         const void *v_new);

/* One decode step: for every layer, run its attention; by groups of layers (pie_set_lookahead) prefetch the next group's
 * host-resident units when a group starts (wrapping to the first layers of the next token, Section 3.4.2) and push the
 * group's share back out when it has computed (Section 3.3: the layer that just finished is the coldest).  Nothing but
 * the layers' kernels is enqueued on the compute stream: a layer's kernel waits for its arriving units itself (a device
 * word the copy-in stream sets behind each list), the copy streams wait for the kernels by value, and from the second
 * layer on each attention kernel is launched as a programmatic dependent of the one before it (the layers' q / k_new /
 * v_new must therefore all be ready when the call is made - they are: the arrays hold every layer).  The call returns once
 * the step is enqueued; it does not start while the GPU is more than two steps behind (pie_step_begin, pie_set_run_ahead).  A share the GPU pool has no room for when its group is prefetched is fetched at its
 * layer's turn; if there is no room even then the call returns PIE_ERR_NOMEM with the layers before it enqueued and nothing
 * of that layer.  q_all/out_all: device [n_layers][n_seqs][Hq][D]; k_new_all/v_new_all: device [n_layers][n_seqs][Hkv][D]
 * or NULL.  Runs pie_controller_tick at the end. */
int pie_decode_step(pie_pool *pool, const void *q_all, void *out_all, const int32_t *block_table_dev,
                    int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, int32_t n_seqs, float scale,
                    const void *k_new_all, const void *v_new_all, int32_t mode);
/* One layer of pie_decode_step by itself, for callers that run other work between the layers (Section 4.2: supporting
 * a model means adding this control loop to its forward pass): fetches whatever the layer still lacks, starts the
 * prefetch of layer (layer+1) mod n_layers, runs the attention (and the append, if k_new / v_new are given) and
 * pushes this layer's host-resident share out behind it (by groups of layers, as pie_decode_step does: a group left open
 * is closed by pie_controller_tick, pie_step_begin or pie_sync).  q / out / k_new / v_new are this layer's device arrays
 * ([n_seqs][n_q_heads][head_dim], [n_seqs][n_kv_heads][head_dim]).  Call pie_step_begin before layer 0 and
 * pie_controller_tick after the last layer when timing is on.  PIE_ERR_UNSUPPORTED under pie_set_layer_policy. */
int pie_decode_layer(pie_pool *pool, int32_t layer, const void *q, void *out, const int32_t *block_table_dev,
                     int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, int32_t n_seqs, float scale, const void *k_new,
                     const void *v_new, int32_t mode);
/* The same with q / k_new / v_new / out in HOST memory (pinned for full speed): copies the inputs in,
 * runs the step, copies out_all back and waits for it.  ctx_lens_host/block_table_host are uploaded too.
 * Inputs and results move in groups of four layers on two streams of the library's own, so that a group's
 * upload and download overlap the other groups' attention; when the call returns nothing is in flight. */
int pie_decode_step_host(pie_pool *pool, const void *q_all_host, void *out_all_host, const int32_t *block_table_host,
                         int32_t max_blocks_per_seq, const int32_t *ctx_lens_host, int32_t n_seqs, float scale,
                         const void *k_new_all_host, const void *v_new_all_host, int32_t mode);
/* The paper's whole-layer protocol on the GPU (Section 3.3), as a variant of the block-granular plan.  After this
 * call pie_decode_step moves whole layers: when layer k starts, confirmed completions are applied, the coldest
 * GPU layer is swapped out unless every CPU layer is colder or no CPU region is free, and the hottest CPU layer is
 * swapped in unless no GPU region is free; one swap in flight per direction; a layer that is still on the CPU when
 * its turn comes is waited for.  The host keeps step with the device, layer by layer (it waits for the previous
 * layer's attention before deciding), as the paper's per-layer control loop does.  A region is one layer's units.
 * Every layer must be wholly on one side (PIE_ERR_INVALID otherwise); gpu_regions + cpu_regions >= n_layers;
 * the pools must hold that many layers' units.  gpu_regions <= 0 and cpu_regions <= 0: back to the block plan. */
int pie_set_layer_policy(pie_pool *pool, int32_t gpu_regions, int32_t cpu_regions);
/* Adaptive expansion in whole layers (Section 3.4.2 as the paper states it): with the whole-layer protocol set AND the
 * ratio handed to the controller (pie_set_extension_ratio < 0), every pie_decode_step ends by deciding how many layers m
 * live on the CPU from the next token on (pie_layer_controller_decide: one more when no swap-in was needed or the share
 * of swap-ins that fetched a layer of the NEXT token reached the trigger; one fewer when the computation waited) and, if
 * m changed, by moving whole layers until n - m GPU regions and m + 2 CPU regions hold them (the pools must be sized for
 * the values m may take).  share: the trigger, in [0, 1]; 0 = the rule's default (0.3).  pie_stats counts the swap-in
 * lists started and those for the next token in both modes (with equal shares of every layer on the host, the block
 * plan's default, the share is one group of layers in n and says nothing: the trigger acts in whole-layer mode only). */
int pie_set_violation_trigger(pie_pool *pool, double share);
/* The decisions taken so far in whole-layer mode: int32 quadruples {step, layer starting, layer whose swap-out
 * started or -1, layer whose swap-in started or -1}.  log may be NULL to ask for the count only. */
int pie_get_layer_log(pie_pool *pool, int32_t *log, int64_t capacity, int64_t *n_entries);
/* Marks a step boundary (pie_decode_step calls it itself): the per-step timing sets turn over, and the host thread waits
 * here until the GPU has finished the step three before the one that begins - the host enqueues up to two steps beyond
 * the one the GPU is working on, and no further (pie_set_run_ahead).  (Slots freed by a step's swap lists are only known
 * free once their copies have completed; a host many steps ahead would be handed slots still in flight, in the order they
 * were released, and its lists would break into many short copies.) */
int pie_step_begin(pie_pool *pool);

/* ---- policy and controller (Section 3.3, Section 3.4.2) ------------------------------------------ */

/* r in [0,1]: target fraction of each layer's allocated units kept host resident between uses
 * (expansion X = 1/(1-r), Section 3.1).  r < 0: adaptive - the controller owns the ratio, starting from
 * the current one.  Until the first call the host-resident sets are whatever the caller established. */
int pie_set_extension_ratio(pie_pool *pool, float r);
int pie_get_extension_ratio(pie_pool *pool, float *r);
/* Controller constants (the paper gives none): step = ratio change per adjustment (default 1 / n_layers,
 * "one layer"), eps = stall / compute above which a step counts as stalled (0.02), u_hi = link-busy /
 * compute below which the ratio may grow (0.9).  A value <= 0 keeps the current setting.
 * What counts as "stall" is the wait for arriving units plus the attention's slow-down: what the step's layers took above
 * its own undisturbed ones (copies that are hidden can still slow the attention down through shared HBM bandwidth; every
 * layer of a step attends the same batch, and the lists of a group of layers are in flight during the first part of the
 * group only, so the step is its own yardstick and clock drift between steps does not read as a slow-down). */
int pie_set_controller(pie_pool *pool, double step, double eps, double u_hi);
/* Group size of the decode loop (pie_decode_step / pie_decode_layer): the loop issues swap lists for `layers`
 * consecutive layers at a time - while a group computes, the next group's host-resident shares are on their way (wrapping
 * into the next token) and the previous group's are going back.  1 is the paper's per-layer look-ahead (Section 3.4.2).
 * A larger group gives each copy several layers' time to arrive, lets the copies of the group go as one (its blocks in as
 * few copies as their slots allow, its table entries in one strided copy) and costs the compute stream nothing per layer;
 * the price is GPU staging: three groups' shares are on the GPU at a time.  0 (the default): chosen per group from the
 * slots the GPU pool can spare, at most 8 and at most a quarter of the layers.  0 <= layers <= 8 (PIE_ERR_INVALID
 * otherwise); an explicit value is capped at half the layers. */
int pie_set_lookahead(pie_pool *pool, int32_t layers);
/* How many decode steps the host may be ahead of the GPU when pie_step_begin returns: 1 to 3, 2 by default.  With 1
 * the host enqueues a step while the one before it runs and the GPU pool needs the least spare room for whole swap lists
 * (about two steps' host-resident shares), but any delay of the host thread longer than the rest of the running step
 * leaves the GPU idle; each further step absorbs that much more delay and asks for one more step's shares of spare
 * slots (without them swap lists break into short copies: the slots they are given are still in flight).
 * PIE_ERR_INVALID outside 1..3. */
int pie_set_run_ahead(pie_pool *pool, int32_t steps);

/* ---- 8-bit blocks (a variant beyond the paper, whose blocks are 16-bit: a token costs half the bytes in HBM, in the
 * host pool and on the link, so the same link hides twice the tokens per layer - Section 3.1's condition in bytes) ----
 * A pool created with kv_format = PIE_KV_E4M3 stores a block as [n_kv_heads][K|V][16 tokens][128] bytes of E4M3 (1-4-3 bits,
 * bias 7, no infinities, largest value 448); a stored byte b stands for decode(b) * k_scale (keys) or * v_scale
 * (values), one pair of scales for the pool (default 1, 1).  q, out and the new token's k_new / v_new stay in the pool's
 * 16-bit type.  pie_decode_attention computes attention over the decoded values (scores and sums in fp32 as for 16-bit
 * pools; the key scale enters the softmax scale, the value scale the result); its append stores
 * E4M3(fp32(x) / scale), rounded to nearest (ties to the even code), magnitudes beyond 448 saturating, NaN -> 0x7f, and
 * the step's own attention already sees the stored (rounded) token.  Bytes beyond a sequence's length may hold anything.
 * The products run in fp16 for both 16-bit types (every E4M3 value is an fp16 number); a bf16 query is scaled into
 * fp16's range by a power of two per (sequence, KV head), exactly, so no finite query overflows.  Swapping, the table and the controller are
 * unchanged (they move block_bytes).  pie_kv_write quantises its rows with the append's rule.
 * PIE_ERR_INVALID unless both scales are finite and > 0; PIE_ERR_UNSUPPORTED on a 16-bit pool. */
int pie_set_kv_scales(pie_pool *pool, float k_scale, float v_scale);

/* ---- prefill-side KV write (Section 2.2: the prompt's keys and values enter the cache; the decode path above
 * appends one token per sequence, this call writes any number) ---------------------------------------------
 * k, v: device [n_tokens][n_kv_heads][head_dim] in the pool's 16-bit type.  Token t is position
 * token_pos_dev[t] (0-based) of sequence token_seq_dev[t] (row of block_table_dev, n_seqs rows of
 * max_blocks_per_seq ids): its rows go to row pos % 16 of the K and V halves of every head's tile in the block that
 * holds the position.  Enqueued on the compute stream behind every copy that is still bringing a unit of the layer
 * in; swap-outs of the layer issued afterwards wait for it.  Every unit written must be GPU resident: a token whose
 * block is not (or whose position or sequence is out of range) is skipped and the next call that checks the device
 * status word returns PIE_ERR_NOT_RESIDENT / PIE_ERR_INVALID.  Two tokens of one call must not name the same
 * position.  With kept host copies every block of the layer counts as written. */
int pie_kv_write(pie_pool *pool, int32_t layer, const void *k, const void *v, const int32_t *token_seq_dev,
                 const int32_t *token_pos_dev, int64_t n_tokens, const int32_t *block_table_dev, int32_t max_blocks_per_seq,
                 int32_t n_seqs);

/* ---- chunked-prefill attention (Section 2.1: the prefill stage computes all prompt tokens at once; Section 2.2: over the
 * paged cache; the decode call above handles one query token per sequence, this one a chunk) ----------------------
 * Sequence s contributes the query tokens q_offsets[s] .. q_offsets[s + 1] - 1 of the flat arrays q / out (device
 * [n_tokens][n_q_heads][head_dim] in the pool's 16-bit type; q_offsets[0] = 0).  Its chunk of C tokens sits at the END of
 * its context: ctx_lens[s] counts the chunk in, token i of the chunk is position ctx - C + i and attends to positions
 * 0 .. ctx - C + i (causal inside the chunk, everything before it).  The chunk's own keys and values must be in the cache
 * already: call pie_kv_write first.  Scores and sums in fp32, probabilities in the 16-bit type, out rounded to nearest.
 * ctx_lens_host / q_offsets_host (host, required) size the launch and are checked before anything is enqueued: a chunk
 * longer than its context or a context beyond the table is PIE_ERR_INVALID.  Enqueued on the compute stream behind every
 * copy still bringing a unit of the layer in; every unit read must be GPU resident (a missing one raises the device
 * status word: the next call returns PIE_ERR_NOT_RESIDENT).  The kernel runs on the tcgen05 tensor cores with its
 * accumulators in tensor memory: 128 query rows (128 / group tokens) per CTA, streamed against the context in stages of 64
 * (bf16 pools) or 128 (fp16 pools) tokens.  16-bit pools only (PIE_ERR_UNSUPPORTED). */
int pie_prefill_attention(pie_pool *pool, int32_t layer, const void *q, void *out, const int32_t *block_table_dev,
                          int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, const int32_t *q_offsets_dev,
                          const int32_t *ctx_lens_host, const int32_t *q_offsets_host, int32_t n_seqs, float scale);

/* ---- kept host copies and write-back elision (a variant the paper does not have: Section 3.2 gives the
 * CPU region up once a unit has been swapped in) ---------------------------------------------------------
 * on != 0: a unit that is swapped in keeps its host slot; when it is swapped out again it returns to that slot, and
 * no bytes are copied unless the unit was written on the GPU meanwhile.  In decode only the block that receives
 * the new token is written per sequence, so nearly all of the device-to-host traffic of Section 3.3's protocol
 * disappears; the price is host memory for every unit of the host-resident set even while it is on the GPU.
 * Which blocks an attention call with k_new/v_new writes: derived from block_table_host / ctx_lens_host when the
 * call gets them; otherwise the ids given to pie_declare_append_blocks (host, n ids; valid until replaced; the
 * caller vouches for them - a block that is written but not listed would leave a stale host copy); with
 * neither (n < 0 or never declared), every block of the layer counts as written and nothing is elided.
 * Switching off takes effect unit by unit at its next swap-in.  pie_stats.bytes_out_elided counts the bytes elided. */
int pie_set_retention(pie_pool *pool, int32_t on);
int pie_declare_append_blocks(pie_pool *pool, const int32_t *ids, int64_t n);

/* ---- run-time resize of the per-layer cache size (Section 4.1) -----------------------------------
 * n_logical_blocks is the physical width of the per-layer tables; the size visible to allocation is
 * visible_blocks of the configuration at creation (0: the full width) and changes in two phases:
 *   grow:   pie_resize_begin(new) starts it; ids in [old, new) become allocatable only after every layer has
 *           gone through a swap pass (pie_plan_layer / pie_decode_step on that layer, or a swap call on it) -
 *           the space is prepared first and made visible afterwards;
 *   shrink: ids >= new are not handed out from the moment of the call; blocks still in use up there stay
 *           accessible; the new size takes effect once every layer has passed, and freed ids beyond it are
 *           never handed out again.
 * Slots come from the shared pools, so no region is physically moved: what the paper re-allocates per layer
 * is here the layer's row of the slot table, which already has the full width.
 * PIE_ERR_RANGE: new_blocks <= 0 or > n_logical_blocks; PIE_ERR_BUSY: a resize is in progress. */
int pie_resize_begin(pie_pool *pool, int32_t new_blocks);
/* Any pointer may be NULL.  target = -1 when no resize is in progress. */
int pie_resize_status(pie_pool *pool, int32_t *visible, int32_t *alloc_limit, int32_t *target, int32_t *layers_moved);

/* The per-layer plan at the start of layer `layer`: in_ids = units of layer (layer+1) mod L to bring in
 * (ascending id, as many as the GPU pool can take), out_ids = units of `layer` to push out once it has
 * computed.  Arrays are host, capacity n_logical_blocks each. */
int pie_plan_layer(pie_pool *pool, int32_t layer, int32_t *in_ids, int64_t *n_in, int32_t *out_ids, int64_t *n_out);
/* Evaluate, in step order, the event sets of earlier steps that have completed (no blocking), update the
 * stats, and in adaptive mode adjust the ratio.  The library keeps 4 steps of events (callers that go layer by layer
 * without pie_step_begin: the oldest step is waited for when the host gets that far ahead of the GPU). */
int pie_controller_tick(pie_pool *pool, int32_t *changed);
int pie_get_stats(pie_pool *pool, pie_stats *out);
/* Per-layer timeline of the most recently evaluated step (timing = 2 in the configuration; timing = 1 keeps the
 * statistics and the controller but not this table): ms[l][7] = {end of the previous layer's attention kernel,
 * start of this layer's - past its presence wait -, its end, swap-in list start, end, swap-out list start, end} in ms from
 * the start of the step's first attention kernel; -1 where nothing was recorded.  Inside pie_decode_step a layer's kernel
 * starts beside the tail of the layer before it (its first CTAs take the SMs the other's CTAs leave), so its start may lie
 * some microseconds before the previous layer's end.  The lists of a group of layers that went
 * as one appear under the group's first layer.  The compute columns are the kernels' own GPU-timer stamps; the copy columns
 * are copy-stream events tied to them through one event recorded just before the step's first kernel (a few us of slack).
 * capacity = floats available (>= 7 * n_layers).  PIE_ERR_INVALID if no step has been evaluated yet.  Shows what
 * overlapped with what. */
int pie_get_step_timeline(pie_pool *pool, float *ms, int64_t capacity);
/* Wait until everything enqueued so far has completed, at most timeout_us (PIE_ERR_TIMEOUT); applies
 * phase-2 updates and reports a pending device status word (PIE_ERR_NOT_RESIDENT ...). */
int pie_sync(pie_pool *pool, int64_t timeout_us);
const char *pie_status_str(int status);
int pie_last_cuda_error(void);
/* Host-link probe: time a pinned cudaMemcpyAsync of `bytes` in direction dir (or both at once when
 * dir == 2) `reps` times; *gbps = best bytes/time per direction. */
int pie_probe_link(int64_t bytes, int32_t dir, int32_t reps, double *gbps);
/* HBM probe: device-to-device copy kernel-free cudaMemcpyAsync of `bytes`; *gbps counts read+write. */
int pie_probe_hbm(int64_t bytes, int32_t reps, double *gbps);

/* ---- for callers that must not allocate ------------------------------------------------------------ */

#define PIE_NOALLOC_SCRATCH_BYTES (16ll << 20) /* fixed device scratch held by every GPU that loads the library */
#define PIE_NOALLOC_MAX_SEQS 4096

/* (No counterpart in the paper: this entry point exists for the library's users.)
 * Paged decode attention of one layer without any allocation.  pie_decode_attention needs a pie_pool, and
 * creating a pool calls cudaMalloc / cudaHostAlloc.  Some callers may not do that: code running while another
 * component owns the device's memory arena, plug-ins that receive fixed buffers and a stream, loops that
 * cannot afford the device-wide synchronisation an allocation implies.  Here the caller passes everything:
 *   kv_pool     device memory holding n_slots slots in the slot layout above, 128-byte aligned
 *   slot_table  device int32 [n_logical_blocks]: GPU slot of each logical block of this layer, -1 if absent
 *   q, out, block_table_dev, ctx_lens_dev, scale   as for pie_decode_attention (no append)
 *   ctx_lens_host  host copy of the lengths (required: sizes are checked before anything is enqueued)
 *   status_dev  device int32[4], cleared by the caller, or NULL.  The kernels raise (set to 1) word 0 if a referenced
 *               block had no slot (slot_table entry negative or >= n_slots: that tile then reads slot 0 and the output of
 *               its sequence is wrong), word 1 if ctx_lens_dev holds a length beyond the table or more chunks than
 *               ctx_lens_host sized the scratch for (clamped: nothing is computed in the second case), word 2 if a
 *               bounded wait ran out; word 3 receives the batch's context-token count (batches of at most 1024
 *               sequences only).  Nothing clears the words.  With NULL these device-side conditions CANNOT be detected:
 *               the call still returns PIE_OK - pass the words unless the tables are known good
 *   stream      a cudaStream_t
 * The split-K scratch (chunk offsets, fp32 partials) is a static device array of PIE_NOALLOC_SCRATCH_BYTES
 * that every GPU loading the library holds until the process exits.  A call whose partials would not fit
 * (sum over sequences of ceil(ctx / split_tokens), times n_q_heads * (head_dim + 2) * 4 bytes, plus 17 KiB)
 * or with more than PIE_NOALLOC_MAX_SEQS sequences returns PIE_ERR_NOMEM and enqueues nothing; so does every other
 * argument error.  (A CUDA error from the memset or a launch - PIE_ERR_CUDA - may leave the memset enqueued.)
 * All calls on a device share that array and it keeps the previous call's contents: each call clears the
 * counters it needs at zero (a memset on `stream`) and writes every other word before reading it; two calls
 * that overlap on the GPU (different streams, no dependency) race - order them.  The first call on each device looks up the array's device
 * address (cudaGetSymbolAddress) and sets the kernels' shared-memory attribute; make that first call outside
 * any stream capture.  Calls cudaMalloc, cudaFree or any allocating routine: never. */
int pie_decode_attention_noalloc(const void *kv_pool, int64_t n_slots, const int32_t *slot_table,
                                 int32_t n_logical_blocks, const void *q, void *out, const int32_t *block_table_dev,
                                 int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, const int32_t *ctx_lens_host,
                                 int32_t n_seqs, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t dtype,
                                 int32_t split_tokens, float scale, int32_t *status_dev, void *stream);

/* ---- host-only pieces, usable without a GPU ------------------------------------------------------ */

/* The mapping table by itself (what pie_pool uses inside).  Stream-ordered two-phase semantics:
 * pie_table_swap picks destination slots, releases the source slots tagged with the new ticket, and
 * reports the tickets of other queues the copy must wait for; pie_table_confirm is phase 2. */
pie_table *pie_table_create(int32_t n_layers, int32_t n_logical, int64_t n_gpu_slots, int64_t n_host_slots);
void pie_table_destroy(pie_table *t);
int pie_table_alloc(pie_table *t, int32_t block, int32_t on_host);
int pie_table_free(pie_table *t, int32_t block);
/* queue = PIE_Q_IN / PIE_Q_OUT.  Outputs (host): ticket; moved_ids/src_slots/dst_slots with capacity n;
 * n_moved; waits[4] indexed by queue (0 = none). */
int pie_table_swap(pie_table *t, int32_t queue, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket,
                   int32_t *moved_ids, int32_t *src_slots, int32_t *dst_slots, int64_t *n_moved, int64_t *waits);
/* Presence check + compute ticket.  ids may be NULL (n = 0): then no residency check is made and the
 * waits cover every arriving unit of the layer. */
int pie_table_attention(pie_table *t, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket, int64_t *waits);
int pie_table_confirm(pie_table *t, int32_t queue, int64_t ticket);
int pie_table_state(pie_table *t, int32_t layer, int32_t block, int32_t *state, int32_t *gpu_slot, int32_t *host_slot);
/* pie_table_swap with one more output: elided[i] = 1 where pair i needs no bytes moved (see pie_set_retention). */
int pie_table_swap_ex(pie_table *t, int32_t queue, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket,
                      int32_t *moved_ids, int32_t *src_slots, int32_t *dst_slots, uint8_t *elided, int64_t *n_moved,
                      int64_t *waits);
int pie_table_set_retention(pie_table *t, int32_t on);
/* GPU-resident units that hold a kept host copy.  While there are any, a writer has to mark what it writes
 * (pie_table_mark_dirty) even after the switch went off: switching off takes effect unit by unit at the next swap-in. */
int64_t pie_table_kept_copies(const pie_table *t);
int pie_table_mark_dirty(pie_table *t, int32_t layer, const int32_t *ids, int64_t n);
/* A unit that lives on the GPU gives its kept host slot up (no-op otherwise). */
int pie_table_drop_host_copy(pie_table *t, int32_t layer, int32_t block);
/* Run-time resize on the bare table: see pie_resize_begin.  pie_table_init_capacity sets the visible size
 * before anything is allocated; pie_table_layer_pass returns 1 when the call completed a resize, else 0
 * (pie_table_swap makes the same mark for its layer). */
int pie_table_init_capacity(pie_table *t, int32_t size);
int pie_table_resize_begin(pie_table *t, int32_t new_size);
int pie_table_layer_pass(pie_table *t, int32_t layer);
int pie_table_capacity(pie_table *t, int32_t *visible, int32_t *alloc_limit, int32_t *target, int32_t *layers_moved);

/* The whole-layer swap protocol of Section 3.3 as a scheduler object.  on_cpu: n_layers flags. */
pie_fifo *pie_fifo_create(int32_t n_layers, int32_t gpu_regions, int32_t cpu_regions, const uint8_t *on_cpu);
void pie_fifo_destroy(pie_fifo *f);
/* A swap in direction dir (PIE_Q_IN / PIE_Q_OUT) has been confirmed complete. */
int pie_fifo_complete(pie_fifo *f, int32_t dir);
/* Layer k (0-based) starts computing: *start_out / *start_in receive the layer to swap out / in now, or
 * -1.  The caller starts those copies and later reports them with pie_fifo_complete. */
int pie_fifo_layer_start(pie_fifo *f, int32_t k, int32_t *start_out, int32_t *start_in);
/* 0 GPU, 1 CPU, 2 in transit to the CPU, 3 in transit to the GPU */
int pie_fifo_location(pie_fifo *f, int32_t layer);
/* Swap-ins started so far, and how many of them fetched a layer that only the NEXT token needs (a layer below the one
 * starting): Section 3.4.2 allows that violation of "swap what the current token needs" to prevent waiting at the
 * first layers, and takes its frequency as the sign that the expansion is too small.  Either pointer may be NULL. */
int pie_fifo_counters(const pie_fifo *f, int64_t *in_starts, int64_t *violations);
/* Section 3.4.2's rule for the number m of layers kept on the CPU, from one window's measurements (a token or several):
 * the computation waited (stall > eps * compute) -> m - 1, and that m is left alone for a while (4 windows, twice as
 * long after every failed return, at most 96); otherwise, if no swap-in was started at all or the share of swap-ins that
 * were for the next token has reached v_trigger -> m + 1 (at most m_max); else m.  The link is busy the whole time under
 * the whole-layer protocol, whatever m is, so link slack cannot be the signal here.  state: 4 doubles owned by the
 * caller, zero-initialised.  Constants are this build's (the paper gives none): v_trigger <= 0 -> 0.3, eps <= 0 ->
 * 0.02.  With m CPU layers the protocol runs with n - m GPU regions and m + 2 CPU regions (Section 3.3). */
int32_t pie_layer_controller_decide(double *state, int32_t m, int32_t m_max, double stall, double compute, int64_t in_starts,
                                    int64_t violations, double v_trigger, double eps);

/* The controller's decision rule by itself.  state: 16 doubles owned by the caller, zero-initialised
 * (history in [0..4]; [5] = stall tolerance eps, [6] = link-busy ceiling u_hi, 0 = defaults 0.02 / 0.9; [7..11] the
 * cooldown and the performance record: the lowest ratio known to stall and how long to leave it alone, which doubles
 * with every failed probe).  Returns the new ratio for one decode step's measurements (same unit for all three). */
double pie_controller_decide(double *state, double ratio, double step, double stall, double compute,
                             double swap_busy);

/* ---- performance records against throughput (Section 3.4.2, last paragraph) ------------------------------
 * The stall-driven controller above cannot see whether a larger host-resident share buys anything: that shows only
 * in the serving system's throughput.  The governor takes one report per window - the throughput seen at the ratio
 * then in force, any unit - keeps the newest report per ratio (in units of `step`) and answers with a cap on the ratio
 * (1.0 = none), which the controller respects.  NORMAL: no cap, until a report shows no gain (within tol) over the record
 * one step below: the workload has stopped scaling with expansion, so stop increasing and test one step lower.
 * TEST_DOWN: a report at the lowered cap that is not worse than the reference (within tol) keeps it and tries lower
 * still; a worse one goes one step back up -> HOLD.  HOLD: every `period` reports, probe one step up.  PROBE_UP: better
 * than the reference by more than tol -> NORMAL again; else back down -> HOLD.  Reports at a ratio other than the cap only
 * update the records; `patience` of them in a row end a test at the ratio reported.
 * Constants are this build's (the paper gives none): tol 0.02, period 8, patience 6 where the argument is <= 0.
 * Host only, no CUDA.  pie_governor_state: *state 0 NORMAL, 1 TEST_DOWN, 2 HOLD, 3 PROBE_UP; *cap_steps -1 = no cap. */
pie_governor *pie_governor_create(double step, double tol, int32_t period, int32_t patience);
void pie_governor_destroy(pie_governor *g);
double pie_governor_report(pie_governor *g, double ratio, double throughput);
int pie_governor_state(const pie_governor *g, int32_t *state, int32_t *cap_steps);
/* The same inside a pool in adaptive mode: report the window's throughput (e.g. tokens per second); the pool's ratio is
 * held at or below the governor's cap from the next controller tick on (and never below what the GPU pool's size
 * allows).  The governor's step is the controller's (pie_set_controller).  pie_stats.governor_cap = the cap (1 = none),
 * governor_state = the governor's state.  PIE_ERR_INVALID for a throughput that is not finite or negative. */
int pie_report_throughput(pie_pool *pool, double throughput);

#ifdef __cplusplus
}
#endif
#endif /* PIE_H */
