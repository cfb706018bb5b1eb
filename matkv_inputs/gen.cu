// Device twin of the counter-based bf16 generator in matkv_inputs/__init__.py (same integer recipe,
// so host and device produce identical bytes).  Holds no attention arithmetic.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

__global__ void k_fill_bf16(__nv_bfloat16 *out, uint64_t n, uint64_t seed, uint64_t stream, int shift, uint64_t start) {
    const uint64_t base0 = seed * 0x9E3779B97F4A7C15ull + stream * 0xD1B54A32D192ED03ull;
    const float scale = exp2f((float)(shift - 16));   // a power of two: exact
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t base = base0 + (start + i) * 3ull;
        int32_t acc = 0;
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            const uint64_t h = mix64(base + k);
            acc += (int32_t)(h & 0xFFFF) + (int32_t)((h >> 16) & 0xFFFF) + (int32_t)((h >> 32) & 0xFFFF) + (int32_t)(h >> 48);
        }
        out[i] = __float2bfloat16_rn((float)(acc - 393210) * scale);   // |acc-c| < 2^20: the float is exact
    }
}

extern "C" int matkv_inputs_fill_bf16(void *dev, uint64_t n, uint64_t seed, uint64_t stream, int shift, uint64_t start,
                                      void *cuda_stream) {
    if (n == 0) return 0;
    uint64_t blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    k_fill_bf16<<<(unsigned)blocks, 256, 0, (cudaStream_t)cuda_stream>>>((__nv_bfloat16 *)dev, n, seed, stream, shift, start);
    return (int)cudaGetLastError();
}
