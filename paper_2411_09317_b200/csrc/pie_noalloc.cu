// pie_decode_attention_noalloc: paged decode attention for callers that must not allocate.
//
// Some callers cannot call cudaMalloc (or anything that does so underneath): code that runs while another
// component owns the whole device arena, plug-ins that are handed fixed buffers and a stream, latency-critical
// loops where an allocation's implicit device synchronisation is not acceptable.  The regular entry point needs
// a pie_pool, and creating a pool allocates.  This one needs no pool: the caller passes the KV block memory, the
// slot table, the inputs and the output; the split-K scratch (chunk offsets and fp32 partials) lives in a
// file-scope device array of fixed size that every GPU loading this library holds until the process exits.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "../../include/pie.h"
#include "pie_kernels.h"

namespace {

constexpr int64_t NOALLOC_SCRATCH_BYTES = PIE_NOALLOC_SCRATCH_BYTES;  // 16 MiB
constexpr int32_t NOALLOC_MAX_SEQS = PIE_NOALLOC_MAX_SEQS;            // 4096
constexpr int64_t OFF_STATUS = 0;                                     // 4 status words (used when the caller gives none)
constexpr int64_t OFF_CHUNK = 256;                                    // int32 [MAX_SEQS + 1]
constexpr int64_t OFF_PART = 256 + ((int64_t)(NOALLOC_MAX_SEQS + 1) * 4 + 255) / 256 * 256;

// Shared by every call on this device; it keeps the last call's contents.
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

struct DeviceSetup {
    bool ready = false;
    unsigned char *scratch = nullptr;  // DEVICE address of g_noalloc_scratch on this device
    int n_sms = 0;
    int ctas_per_sm[2][2] = {{0, 0}, {0, 0}};  // [head_dim == 128][dtype]
};
constexpr int MAX_DEVICES = 64;
DeviceSetup g_setup[MAX_DEVICES];
std::mutex g_setup_mutex;

// Once per device, with that device current.  In host code the array's name is only a host-side stand-in: the
// address a kernel may use comes from cudaGetSymbolAddress.
int setup_device(int dev, DeviceSetup **out) {
    if (dev < 0 || dev >= MAX_DEVICES) return PIE_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup &s = g_setup[dev];
    if (!s.ready) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess || ptr == nullptr) return PIE_ERR_CUDA;
        if (cudaDeviceGetAttribute(&s.n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return PIE_ERR_CUDA;
        for (int d128 = 0; d128 < 2; ++d128)
            for (int dt = 0; dt < 2; ++dt)
                if (pie::attn_configure(d128 ? 128 : 64, dt, 0, &s.ctas_per_sm[d128][dt]) != cudaSuccess) return PIE_ERR_CUDA;
        s.scratch = static_cast<unsigned char *>(ptr);
        s.ready = true;
    }
    *out = &s;
    return PIE_OK;
}

}  // namespace

extern "C" int pie_decode_attention_noalloc(const void *kv_pool, int64_t n_slots, const int32_t *slot_table,
                                            int32_t n_logical_blocks, const void *q, void *out,
                                            const int32_t *block_table_dev, int32_t max_blocks_per_seq,
                                            const int32_t *ctx_lens_dev, const int32_t *ctx_lens_host, int32_t n_seqs,
                                            int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t dtype,
                                            int32_t split_tokens, float scale, int32_t *status_dev, void *stream) {
    if (!kv_pool || !slot_table || !q || !out || !block_table_dev || !ctx_lens_dev || !ctx_lens_host) return PIE_ERR_INVALID;
    if (n_slots <= 0 || n_logical_blocks <= 0 || n_seqs < 0 || max_blocks_per_seq <= 0) return PIE_ERR_INVALID;
    if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0) return PIE_ERR_INVALID;
    if (dtype != PIE_F16 && dtype != PIE_BF16) return PIE_ERR_INVALID;
    if ((head_dim != 64 && head_dim != 128) || n_q_heads / n_kv_heads > 8) return PIE_ERR_UNSUPPORTED;
    if (split_tokens == 0) split_tokens = 512;
    if (split_tokens < 0 || split_tokens % 16 != 0) return PIE_ERR_INVALID;
    if (((uintptr_t)kv_pool & 127) != 0) return PIE_ERR_INVALID;
    if ((uint64_t)n_slots * (uint64_t)n_kv_heads * 32u > 0x7fffffffull) return PIE_ERR_UNSUPPORTED;
    if (n_seqs > NOALLOC_MAX_SEQS) return PIE_ERR_NOMEM;  // beyond the fixed scratch: use the pool entry point
    if (n_seqs == 0) return PIE_OK;

    // the scratch must hold one fp32 partial (+ m, l) per (chunk, KV head, query head of the group)
    const int group = n_q_heads / n_kv_heads;
    int64_t chunks = 0;
    for (int32_t s = 0; s < n_seqs; ++s) {
        const int32_t ctx = ctx_lens_host[s];
        if (ctx < 0 || ctx > max_blocks_per_seq * 16) return PIE_ERR_INVALID;
        chunks += (ctx + split_tokens - 1) / split_tokens;
    }
    const int64_t items = chunks * n_kv_heads;
    const int64_t cnt_bytes = (pie::attn_counter_words(n_seqs, n_kv_heads) * 4 + 255) / 256 * 256;
    const int64_t ml_bytes = (items * group * 2 * 4 + 255) / 256 * 256;
    const int64_t o_bytes = items * group * head_dim * 4;
    if (OFF_PART + cnt_bytes + ml_bytes + o_bytes > NOALLOC_SCRATCH_BYTES) return PIE_ERR_NOMEM;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PIE_ERR_CUDA;
    DeviceSetup *setup = nullptr;
    int st = setup_device(dev, &setup);
    if (st != PIE_OK) return st;

    CUtensorMap map3d, map2d;
    int use3d = 0;
    if (pie::make_pool_tensor_maps(const_cast<void *>(kv_pool), n_slots, n_kv_heads, head_dim, &map3d, &map2d, &use3d) !=
        cudaSuccess)
        return PIE_ERR_CUDA;

    pie::AttnShape sh{head_dim, dtype, n_q_heads, n_kv_heads, n_logical_blocks, n_slots};
    pie::AttnScratch sc{};
    sc.chunk_off = reinterpret_cast<int32_t *>(setup->scratch + OFF_CHUNK);
    sc.counters = reinterpret_cast<int32_t *>(setup->scratch + OFF_PART);
    sc.part_ml = reinterpret_cast<float *>(setup->scratch + OFF_PART + cnt_bytes);
    sc.part_o = reinterpret_cast<float *>(setup->scratch + OFF_PART + cnt_bytes + ml_bytes);
    const int32_t grid = setup->ctas_per_sm[head_dim == 128][dtype] * setup->n_sms;
    if (grid <= 0) return PIE_ERR_UNSUPPORTED;   // nothing has been enqueued yet
    // the array keeps the last call's contents: the work and completion counters must start at zero
    if (cudaMemsetAsync(sc.counters, 0, (size_t)cnt_bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess) return PIE_ERR_CUDA;
    sc.max_items = items;
    sc.max_seqs = NOALLOC_MAX_SEQS;
    pie::AttnLaunch a{};
    a.q = q;
    a.out = out;
    a.block_table = block_table_dev;
    a.max_blocks = max_blocks_per_seq;
    a.ctx_lens = ctx_lens_dev;
    a.slot_table = slot_table;
    a.n_seqs = n_seqs;
    a.scale = scale;
    a.k_new = nullptr;
    a.v_new = nullptr;
    a.gpu_pool = const_cast<void *>(kv_pool);
    a.split_tokens = split_tokens;
    a.variant = 0;
    a.grid = grid;
    // without status words of the caller's the kernels' flags land in the shared scratch, where nobody reads them
    a.status = status_dev ? status_dev : reinterpret_cast<int32_t *>(setup->scratch + OFF_STATUS);
    a.tokens_out = a.status + 3;
    if (pie::launch_attention(sh, sc, a, use3d ? map3d : map2d, use3d, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return PIE_ERR_CUDA;
    return PIE_OK;
}
