// Seeded input generator on the GPU: the same counter-based generator as synth.py, bit for bit
// (SplitMix64 finaliser -> twelve 16-bit uniforms -> centred sum * 2^-16 -> fp16/bf16, nearest even).
// It fills pool slots and dense tensors for benchmarks whose inputs are too large to build on the host.
// It holds none of the method's arithmetic and is not part of libpie.so.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#define PIE_SYNTH_API extern "C"

namespace {

constexpr uint64_t GOLDEN = 0x9E3779B97F4A7C15ull;

__device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ __forceinline__ uint16_t draw(uint64_t base, uint64_t idx, int dtype, float gain) {
    int32_t acc = 0;
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        const uint64_t h = mix64(base + GOLDEN * (idx * 3ull + (uint64_t)(j + 1)));
        acc += (int32_t)(h & 0xFFFF) + (int32_t)((h >> 16) & 0xFFFF) + (int32_t)((h >> 32) & 0xFFFF) + (int32_t)(h >> 48);
    }
    float v = __fmul_rn((float)(acc - 393210), 1.52587890625e-05f);
    v = __fmul_rn(v, gain);
    if (dtype == 0) return __half_as_ushort(__float2half_rn(v));
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));
}

// slot s holds unit slot_unit[s] (or nothing if < 0); element e of the unit has index unit * elems + e
__global__ void fill_slots_kernel(uint16_t *pool, const int64_t *__restrict__ slot_unit, int64_t n_slots, int64_t elems,
                                  uint64_t base, int dtype, float gain) {
    const int64_t vec_per_slot = elems / 8;
    const int64_t total = n_slots * vec_per_slot;
    for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < total; v += (int64_t)gridDim.x * blockDim.x) {
        const int64_t slot = v / vec_per_slot;
        const int64_t unit = slot_unit[slot];
        if (unit < 0) continue;
        const int64_t e0 = (v - slot * vec_per_slot) * 8;
        uint16_t r[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) r[k] = draw(base, (uint64_t)(unit * elems + e0 + k), dtype, gain);
        uint4 w;
        w.x = r[0] | ((uint32_t)r[1] << 16);
        w.y = r[2] | ((uint32_t)r[3] << 16);
        w.z = r[4] | ((uint32_t)r[5] << 16);
        w.w = r[6] | ((uint32_t)r[7] << 16);
        *reinterpret_cast<uint4 *>(pool + slot * elems + e0) = w;
    }
}

// 8-bit pools: a byte with a random sign and mantissa and an exponent field of 3 .. 10 (never the all-ones one)
__device__ __forceinline__ uint8_t draw_byte(uint64_t base, uint64_t idx) {
    const uint64_t h = mix64(base + GOLDEN * (idx + 1ull));
    return (uint8_t)(((h >> 32) & 0x87u) | ((((h >> 40) & 7u) + 3u) << 3));
}

__global__ void fill_slots_bytes_kernel(uint8_t *pool, const int64_t *__restrict__ slot_unit, int64_t n_slots, int64_t elems,
                                        uint64_t base) {
    const int64_t vec_per_slot = elems / 16;
    const int64_t total = n_slots * vec_per_slot;
    for (int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; v < total; v += (int64_t)gridDim.x * blockDim.x) {
        const int64_t slot = v / vec_per_slot;
        const int64_t unit = slot_unit[slot];
        if (unit < 0) continue;
        const int64_t e0 = (v - slot * vec_per_slot) * 16;
        uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
        for (int k = 0; k < 16; ++k) w[k >> 2] |= (uint32_t)draw_byte(base, (uint64_t)(unit * elems + e0 + k)) << (8 * (k & 3));
        *reinterpret_cast<uint4 *>(pool + slot * elems + e0) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

__global__ void fill_tensor_kernel(uint16_t *dst, int64_t n, uint64_t base, uint64_t offset, int dtype, float gain) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = draw(base, offset + (uint64_t)i, dtype, gain);
}

// row r of dst (row_elems values) = the generator's values at indices row_offset[r] .. + row_elems
__global__ void fill_rows_kernel(uint16_t *dst, const int64_t *__restrict__ row_offset, int64_t n_rows, int64_t row_elems,
                                 uint64_t base, int dtype, float gain) {
    const int64_t total = n_rows * row_elems;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / row_elems;
        dst[i] = draw(base, (uint64_t)(row_offset[r] + (i - r * row_elems)), dtype, gain);
    }
}

}  // namespace

// pool: device-accessible memory (HBM, or pinned host memory through its device pointer); slot_unit: device
// int64 [n_slots].  Returns the cudaError_t of the launch.
PIE_SYNTH_API int pie_synth_fill_slots(void *pool, const int64_t *slot_unit, int64_t n_slots, int64_t elems_per_slot,
                                       uint64_t base, int dtype, float gain, void *stream) {
    if (n_slots <= 0) return 0;
    if (elems_per_slot % 8 != 0) return (int)cudaErrorInvalidValue;
    const int64_t total = n_slots * (elems_per_slot / 8);
    const int grid = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    fill_slots_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((uint16_t *)pool, slot_unit, n_slots, elems_per_slot, base, dtype, gain);
    return (int)cudaGetLastError();
}

// the same for pools whose elements are bytes (8-bit blocks)
PIE_SYNTH_API int pie_synth_fill_slots_bytes(void *pool, const int64_t *slot_unit, int64_t n_slots, int64_t elems_per_slot,
                                             uint64_t base, void *stream) {
    if (n_slots <= 0) return 0;
    if (elems_per_slot % 16 != 0) return (int)cudaErrorInvalidValue;
    const int64_t total = n_slots * (elems_per_slot / 16);
    const int grid = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    fill_slots_bytes_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((uint8_t *)pool, slot_unit, n_slots, elems_per_slot, base);
    return (int)cudaGetLastError();
}

PIE_SYNTH_API int pie_synth_fill_tensor(void *dst, int64_t n, uint64_t base, uint64_t offset, int dtype, float gain, void *stream) {
    if (n <= 0) return 0;
    const int grid = (int)((n + 255) / 256 < 148 * 16 ? (n + 255) / 256 : 148 * 16);
    fill_tensor_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((uint16_t *)dst, n, base, offset, dtype, gain);
    return (int)cudaGetLastError();
}

// dst: device [n_rows][row_elems] 16-bit; row_offset: device int64 [n_rows]
PIE_SYNTH_API int pie_synth_fill_rows(void *dst, const int64_t *row_offset, int64_t n_rows, int64_t row_elems, uint64_t base,
                                      int dtype, float gain, void *stream) {
    if (n_rows <= 0 || row_elems <= 0) return 0;
    const int64_t total = n_rows * row_elems;
    const int grid = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    fill_rows_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>((uint16_t *)dst, row_offset, n_rows, row_elems, base, dtype, gain);
    return (int)cudaGetLastError();
}
