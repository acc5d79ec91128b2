// Device half of the seeded input generator (see synth.py): no arithmetic of the
// attention method lives here.  dst[i] = table[mix64(key + (offset + i) * GOLD) >> 48].
#include <cuda_runtime.h>
#include <stdint.h>

__device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

__global__ void synth_fill_bf16_kernel(uint16_t* __restrict__ dst, int64_t n, uint64_t key,
                                       int64_t offset, const uint16_t* __restrict__ table)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x * 8;
    for (int64_t base = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; base < n; base += stride) {
        uint16_t v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint64_t idx = (uint64_t)(offset + base + j);
            v[j] = __ldg(table + (mix64(key + idx * 0x9E3779B97F4A7C15ull) >> 48));
        }
        if (base + 8 <= n && ((reinterpret_cast<uintptr_t>(dst + base) & 15) == 0)) {
            uint4 pk;
            pk.x = v[0] | ((uint32_t)v[1] << 16);
            pk.y = v[2] | ((uint32_t)v[3] << 16);
            pk.z = v[4] | ((uint32_t)v[5] << 16);
            pk.w = v[6] | ((uint32_t)v[7] << 16);
            *reinterpret_cast<uint4*>(dst + base) = pk;
        } else {
            for (int j = 0; j < 8 && base + j < n; ++j) dst[base + j] = v[j];
        }
    }
}

extern "C" int synth_fill_bf16(void* dst, int64_t n, uint64_t key, int64_t offset, const void* table,
                               void* stream)
{
    if (n <= 0) return 0;
    int64_t groups = (n + 7) / 8;
    int blocks = (int)((groups + 255) / 256);
    if (blocks > 148 * 16) blocks = 148 * 16;
    synth_fill_bf16_kernel<<<blocks, 256, 0, (cudaStream_t)stream>>>(
        (uint16_t*)dst, n, key, offset, (const uint16_t*)table);
    return (int)cudaGetLastError();
}
