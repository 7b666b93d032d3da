// Test-only probe of the memory system: what sparse 16-byte updates of a large array
// cost, by access form.  A warp walks the array 128 entries (of 16 bytes) at a time,
// a lane owns 4 consecutive entries, each entry is selected with probability p (a hash):
// the access pattern of the EMA state d in the step kernels.  Forms:
//   0 nothing (loop and hash only)      1 read the 16 bytes
//   2 store 16 bytes (half a sector)    3 store the aligned 32-byte sector
//   4 as 2, but the warp first compacts the selected entries so that lanes 0..n-1 store
//   5 as 3, compacted the same way
#include <cstdint>
#include <cuda_runtime.h>

namespace {

__device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__device__ __forceinline__ void store_form(float *D, uint64_t entry, int wide, float v)
{
    if (wide) {
        float *p = D + (entry & ~(uint64_t)1) * 4;
        asm volatile("st.global.v8.f32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1};" ::"l"(p), "f"(v) : "memory");
    } else {
        *reinterpret_cast<float4 *>(D + entry * 4) = make_float4(v, v, v, v);
    }
}

template <int FORM>
__global__ void probe_kernel(float *D, uint64_t n_entries, uint32_t thresh, float *sink)
{
    __shared__ uint32_t list[8][128];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint64_t n_warps = (uint64_t)gridDim.x * (blockDim.x / 32);
    float acc = 0.f;
    for (uint64_t g = (uint64_t)blockIdx.x * (blockDim.x / 32) + warp; g < n_entries / 128; g += n_warps) {
        const uint64_t first = g * 128 + (uint64_t)lane * 4;
        const uint64_t h = mix64(first);
        uint32_t m = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if ((uint32_t)(h >> (16 * j)) % 65536u < thresh) m |= 1u << j;
        if (FORM == 0) {
            acc += (float)m;
        } else if (FORM <= 3) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if ((m >> j) & 1u) {
                    if (FORM == 1) acc += reinterpret_cast<const float4 *>(D)[first + j].x;
                    else store_form(D, first + j, FORM == 3, (float)lane);
                }
            }
        } else {
            uint32_t run = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t b = __ballot_sync(0xFFFFFFFFu, (m >> j) & 1u);
                if ((m >> j) & 1u) list[warp][run + __popc(b & ((1u << lane) - 1u))] = (uint32_t)(4 * lane + j);
                run += __popc(b);
            }
            __syncwarp();
            for (uint32_t e = lane; e < run; e += 32) store_form(D, g * 128 + list[warp][e], FORM == 5, (float)e);
            __syncwarp();
        }
    }
    if (acc == 1234.5f) *sink = acc;
}

}  // namespace

// ms_out[6]: best-of-3 device time of each form; returns the CUDA error code.
extern "C" int sparse_store_probe(unsigned long long n_entries, double p, float *ms_out)
{
    float *D = nullptr, *sink = nullptr;
    cudaError_t e = cudaMalloc(&D, n_entries * 16);
    if (e == cudaSuccess) e = cudaMalloc(&sink, 16);
    if (e == cudaSuccess) e = cudaMemset(D, 0, n_entries * 16);
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    const uint32_t thresh = (uint32_t)(p * 65536.0);
    for (int form = 0; form < 6 && e == cudaSuccess; ++form) {
        float best = 1e30f;
        for (int rep = 0; rep < 3; ++rep) {
            cudaEventRecord(e0);
            switch (form) {
            case 0: probe_kernel<0><<<148 * 8, 256>>>(D, n_entries, thresh, sink); break;
            case 1: probe_kernel<1><<<148 * 8, 256>>>(D, n_entries, thresh, sink); break;
            case 2: probe_kernel<2><<<148 * 8, 256>>>(D, n_entries, thresh, sink); break;
            case 3: probe_kernel<3><<<148 * 8, 256>>>(D, n_entries, thresh, sink); break;
            case 4: probe_kernel<4><<<148 * 8, 256>>>(D, n_entries, thresh, sink); break;
            default: probe_kernel<5><<<148 * 8, 256>>>(D, n_entries, thresh, sink);
            }
            cudaEventRecord(e1);
            e = cudaEventSynchronize(e1);
            if (e != cudaSuccess) break;
            float ms = 0.f;
            cudaEventElapsedTime(&ms, e0, e1);
            best = ms < best ? ms : best;
        }
        ms_out[form] = best;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(D);
    cudaFree(sink);
    return (int)e;
}
