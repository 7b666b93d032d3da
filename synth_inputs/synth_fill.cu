// Device twin of synth_inputs.normal_host: fills a device buffer with the same
// pseudo-normal stream, bit for bit.  Input generation only -- none of the
// update's arithmetic lives here.
#include <cstdint>
#include <cuda_runtime.h>

__device__ __forceinline__ uint64_t mix64(uint64_t x)
{
    x += 0x9E3779B97F4A7C15ull;
    uint64_t z = x;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__global__ void synth_fill_kernel(float *dst, uint64_t n, uint64_t coord0, uint64_t key, float scale)
{
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n;
         k += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t h = mix64(key + coord0 + k);
        const int s = (int)((h & 0xFFFFu) + ((h >> 16) & 0xFFFFu) + ((h >> 32) & 0xFFFFu) + (h >> 48)) - 131070;
        dst[k] = __fmul_rn((float)s, scale);
    }
}

// dst_device[0..n) <- stream `key` at coordinates coord0 .. coord0+n-1, times scale.
// Returns 0 or the cudaError_t of the launch.  Asynchronous on `stream`.
extern "C" int synth_fill_normal(float *dst_device, uint64_t n, uint64_t coord0, uint64_t key,
                                 float scale, void *stream)
{
    if (n == 0) return 0;
    uint64_t blocks = (n + 255) / 256;
    if (blocks > 148ull * 32) blocks = 148ull * 32;
    synth_fill_kernel<<<(int)blocks, 256, 0, (cudaStream_t)stream>>>(dst_device, n, coord0, key, scale);
    return (int)cudaGetLastError();
}
