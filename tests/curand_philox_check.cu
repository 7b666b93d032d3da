// Test-only: runs the CUDA toolkit's own Philox-4x32-10 routine (cuRAND device
// header) on caller-supplied counters and keys, so the library's generator can
// be compared with an independent implementation on the device.
#include <cstdint>
#include <cuda_runtime.h>
#include <curand_philox4x32_x.h>

__global__ void curand_philox_kernel(const uint32_t *ctr, const uint32_t *key, uint32_t *out, uint64_t n)
{
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n;
         k += (uint64_t)gridDim.x * blockDim.x) {
        const uint4 c = make_uint4(ctr[4 * k], ctr[4 * k + 1], ctr[4 * k + 2], ctr[4 * k + 3]);
        const uint2 kk = make_uint2(key[2 * k], key[2 * k + 1]);
        const uint4 o = curand_Philox4x32_10(c, kk);
        out[4 * k] = o.x; out[4 * k + 1] = o.y; out[4 * k + 2] = o.z; out[4 * k + 3] = o.w;
    }
}

extern "C" int curand_philox_check(const uint32_t *ctr_host, const uint32_t *key_host,
                                   uint32_t *out_host, uint64_t n)
{
    uint32_t *c = nullptr, *k = nullptr, *o = nullptr;
    cudaError_t e = cudaMalloc(&c, n * 16);
    if (e == cudaSuccess) e = cudaMalloc(&k, n * 8);
    if (e == cudaSuccess) e = cudaMalloc(&o, n * 16);
    if (e == cudaSuccess) e = cudaMemcpy(c, ctr_host, n * 16, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(k, key_host, n * 8, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        curand_philox_kernel<<<1024, 256>>>(c, k, o, n);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpy(out_host, o, n * 16, cudaMemcpyDeviceToHost);
    cudaFree(c); cudaFree(k); cudaFree(o);
    return (int)e;
}
