// Test helper: raw Philox4x32-10 blocks from cuRAND's device implementation, for comparison with the oracle.
#include <cstdint>
#include <cuda_runtime.h>
#include <curand_kernel.h>

__global__ void philox_blocks(const uint4* ctr, const uint2* key, uint4* out, int n) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = curand_Philox4x32_10(ctr[i], key[i]);
}

extern "C" int curand_philox_blocks(const void* ctr, const void* key, void* out, int n) {
    philox_blocks<<<(n + 127) / 128, 128>>>((const uint4*)ctr, (const uint2*)key, (uint4*)out, n);
    return (int)cudaDeviceSynchronize();
}
