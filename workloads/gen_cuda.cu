// CUDA twin of the seeded bf16 normal generator (integer arithmetic only):
// element i of stream `key` from counter idx0 is
//     table[ finalise(key + (idx0 + i + 1) * gamma) >> 48 ]
// with SplitMix64's published finaliser and increment, and `table` the 65 536
// bf16 inverse-normal-CDF values uploaded by the host side.  No attention
// arithmetic lives here.
#include <cuda_runtime.h>
#include <stdint.h>

__global__ void normal_bf16_kernel(uint16_t* dst, uint64_t key, uint64_t idx0, uint64_t count, const uint16_t* __restrict__ table) {
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (uint64_t)gridDim.x * blockDim.x) {
        uint64_t z = key + (idx0 + i + 1) * 0x9E3779B97F4A7C15ull;
        z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
        z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
        z ^= z >> 31;
        dst[i] = table[z >> 48];
    }
}

extern "C" int psgen_normal_bf16(void* dst_dev, uint64_t key, uint64_t idx0, uint64_t count, const void* table_dev, void* stream) {
    if (count == 0) return 0;
    uint64_t blocks = (count + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    normal_bf16_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>((uint16_t*)dst_dev, key, idx0, count, (const uint16_t*)table_dev);
    return (int)cudaGetLastError();
}
