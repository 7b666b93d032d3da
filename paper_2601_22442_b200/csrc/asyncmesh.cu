// C ABI of the AsyncMesh step library (see include/asyncmesh.h for the contract
// of every entry point).  Host logic only: argument checks, memory layout, the
// per-step scalars, kernel dispatch.  All arithmetic of the method runs in the
// kernels of step_kernel.cuh and in the small kernels below.
#include "../../include/asyncmesh.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include <cuda_runtime.h>

#include "step_kernel.cuh"
#include "kernel_table.cuh"

using namespace amk;

// ---------------------------------------------------------------------------
// errors
// ---------------------------------------------------------------------------

static thread_local char g_err[512] = "";

static int fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

#define CU_TRY(expr)                                                              \
    do {                                                                          \
        cudaError_t e_ = (expr);                                                  \
        if (e_ != cudaSuccess)                                                    \
            return fail(ASYNCMESH_ERR_CUDA, "%s failed: %s", #expr,               \
                        cudaGetErrorString(e_));                                  \
    } while (0)

extern "C" const char *asyncmesh_last_error(void) { return g_err; }

namespace {

struct DeviceScope {   // make the handle's device current for the call
    int prev = -1;
    bool ok = false;
    explicit DeviceScope(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceScope()
    {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

}  // namespace

// ---------------------------------------------------------------------------
// the handle
// ---------------------------------------------------------------------------

struct asyncmesh {
    uint32_t R = 0, S = 0, tau = 0;
    uint32_t wire = 0;                // 0 fp32, 1 ASYNCMESH_FLAG_BF16_EXCHANGE, 2 ASYNCMESH_FLAG_FP8_EXCHANGE
    uint32_t correction = 0;          // ASYNCMESH_CORRECTION_*
    uint32_t optimizer = 0;           // ASYNCMESH_OPT_*
    double momentum_decay = 4e-3, mu_product = 1.0;   // NAdamW's momentum schedule
    uint32_t K = 1;                   // averaging interval in steps; tau is a multiple of it
    uint32_t lag = 0;                 // tau / K: averaging rounds between launch and arrival
    double p = 0, ema_beta = 0, lr = 0, beta1 = 0, beta2 = 0, eps = 0, wd = 0;
    uint64_t seed = 0;
    int device = 0;
    cudaStream_t stream = nullptr;
    asyncmesh_alloc_fn alloc = nullptr;
    asyncmesh_free_fn dealloc = nullptr;
    void *alloc_ctx = nullptr;

    std::vector<uint64_t> numel, stride;
    std::vector<uint32_t> delay;
    std::vector<StageDesc> sd;        // host copy of the stage table
    std::vector<float *> gstage;      // staging gradients for asyncmesh_step_host
    std::vector<float *> wprev;       // w^{t-1} per stage (ASYNCMESH_FLAG_KEEP_PREVIOUS)
    std::vector<float *> lookx;       // look-ahead at a delay asked for after the fact, per stage
    std::vector<void *> owned;        // everything obtained from the allocator

    StageDesc *sd_dev = nullptr;
    StageDesc *sd_single_dev = nullptr;   // the same table with chunk_begin = 0: one-stage launches
    cudaStream_t copy_stream = nullptr;   // asyncmesh_step_host: gradient copies, overlapping the kernels
    std::vector<cudaEvent_t> ev_ready, ev_done;   // per stage: gradients copied / kernel done with them
    std::vector<char> done_recorded;
    unsigned int *cursors = nullptr;  // [n_slots][S]
    int *status = nullptr;
    double *scratch = nullptr;        // a few doubles for reductions
    double *diag = nullptr;           // [S] consensus error accumulated by the last step (tracking kernels)
    bool tracking = false;
    uint64_t diag_step = 0;           // the step diag belongs to

    int mode = kSync;
    int pipelined = 0;
    bool general = false;             // the kernels' general form (E4M3 exchange, eager estimate, NAdamW)
    bool nadam_form = false;          // the owner kernel's common form with NAdamW fixed at compile time
    KernelChoice kernel;
    uint32_t n_slots = 0;
    uint32_t total_chunks = 0;
    int grid = 0;
    SubsetRule rule{};
    uint64_t t = 0;
    uint64_t last_bytes = 0;
};

static void *dev_alloc(asyncmesh *h, size_t bytes)
{
    if (bytes == 0) bytes = 256;
    void *ptr = nullptr;
    if (h->alloc) {
        ptr = h->alloc(h->alloc_ctx, bytes);
    } else if (cudaMalloc(&ptr, bytes) != cudaSuccess) {
        cudaGetLastError();
        ptr = nullptr;
    }
    if (ptr) h->owned.push_back(ptr);
    return ptr;
}

static void dev_free(asyncmesh *h, void *ptr)
{
    if (!ptr) return;
    for (size_t k = 0; k < h->owned.size(); ++k)
        if (h->owned[k] == ptr) {
            h->owned.erase(h->owned.begin() + k);
            break;
        }
    if (h->dealloc) h->dealloc(h->alloc_ctx, ptr);
    else cudaFree(ptr);
}

static void release_all(asyncmesh *h)
{
    while (!h->owned.empty()) dev_free(h, h->owned.back());
}

// ---------------------------------------------------------------------------
// small kernels
// ---------------------------------------------------------------------------

__global__ void subset_bitmap_kernel(SubsetRule rule, uint32_t stage, uint32_t step, uint64_t N,
                                     uint32_t quad_base, uint8_t *bitmap)
{
    const uint64_t nbytes = (N + 7) / 8;
    for (uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nbytes;
         b += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t mu = b * 8;
        uint32_t bits = subset_bits(rule, stage, step, quad_base + (uint32_t)(mu >> 2));
        if (mu + 4 < N) bits |= subset_bits(rule, stage, step, quad_base + (uint32_t)((mu + 4) >> 2)) << 4;
        const uint64_t left = N - mu;
        if (left < 8) bits &= (1u << (uint32_t)left) - 1u;
        bitmap[b] = (uint8_t)bits;
    }
}

// dst[k] = D[first + k][i]   (D is coordinate-major)
__global__ void gather_column_kernel(const float *D, uint32_t R, uint32_t i, uint64_t first,
                                     uint64_t count, float *dst)
{
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < count;
         k += (uint64_t)gridDim.x * blockDim.x)
        dst[k] = D[(first + k) * R + i];
}

// Replica mean in replica order, one division by (float) R.
__global__ void mean_rows_kernel(const float *W, uint32_t R, uint64_t stride, uint64_t N, float Rf,
                                 float *dst)
{
    for (uint64_t mu = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; mu < N;
         mu += (uint64_t)gridDim.x * blockDim.x) {
        float a = W[mu];
        for (uint32_t i = 1; i < R; ++i) a = __fadd_rn(a, W[(uint64_t)i * stride + mu]);
        dst[mu] = __fdiv_rn(a, Rf);
    }
}

// Block-wide sum of a double into *out (one atomicAdd per block).
__device__ __forceinline__ void block_sum_to(double acc, double *out)
{
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
    __shared__ double part[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) part[warp] = acc;
    __syncthreads();
    if (warp == 0) {
        acc = lane < (int)(blockDim.x >> 5) ? part[lane] : 0.0;
        for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
        if (lane == 0) atomicAdd(out, acc);
    }
}

// sum over coordinates and replicas of (w_i - mean)^2, in double.  A thread takes four
// consecutive coordinates (one 16-byte load per replica row; rows are padded to 32
// floats and 16-byte aligned) and keeps the R x 4 values in registers between the two
// passes, so every byte is read once: a read-only stream.
template <int R>
__global__ void consensus_kernel(const float *W, uint64_t stride, uint64_t N, double *out)
{
    double acc = 0.0;
    const uint64_t n4 = (N + 3) / 4;
    for (uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n4;
         q += (uint64_t)gridDim.x * blockDim.x) {
        float4 x[R];
#pragma unroll
        for (int i = 0; i < R; ++i) x[i] = __ldcs(reinterpret_cast<const float4 *>(W + (uint64_t)i * stride) + q);
        const uint64_t left = N - 4 * q;   // coordinates of this group that exist (1..4 at the tail)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if ((uint64_t)c < left) {
                double mean = 0.0;
#pragma unroll
                for (int i = 0; i < R; ++i) mean += (double)reinterpret_cast<const float *>(&x[i])[c];
                mean /= (double)R;
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const double e = (double)reinterpret_cast<const float *>(&x[i])[c] - mean;
                    acc += e * e;
                }
            }
        }
    }
    block_sum_to(acc, out);
}

typedef void (*consensus_fn)(const float *, uint64_t, uint64_t, double *);
static consensus_fn consensus_for(uint32_t R)
{
    switch (R) {
    case 1: return consensus_kernel<1>;   case 2: return consensus_kernel<2>;
    case 3: return consensus_kernel<3>;   case 4: return consensus_kernel<4>;
    case 5: return consensus_kernel<5>;   case 6: return consensus_kernel<6>;
    case 7: return consensus_kernel<7>;   case 8: return consensus_kernel<8>;
    case 9: return consensus_kernel<9>;   case 10: return consensus_kernel<10>;
    case 11: return consensus_kernel<11>; case 12: return consensus_kernel<12>;
    case 13: return consensus_kernel<13>; case 14: return consensus_kernel<14>;
    case 15: return consensus_kernel<15>; default: return consensus_kernel<16>;
    }
}

// look = w + delay (w - w_prev) (Section 2.2), float4 at a time (rows are padded to 32 floats).
__global__ void extrapolate_kernel(const float *W, const float *Wprev, float *out, float delay,
                                   uint64_t n4)
{
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n4;
         k += (uint64_t)gridDim.x * blockDim.x) {
        const float4 w = reinterpret_cast<const float4 *>(W)[k];
        const float4 q = reinterpret_cast<const float4 *>(Wprev)[k];
        float4 o;
        o.x = __fadd_rn(w.x, __fmul_rn(delay, __fsub_rn(w.x, q.x)));
        o.y = __fadd_rn(w.y, __fmul_rn(delay, __fsub_rn(w.y, q.y)));
        o.z = __fadd_rn(w.z, __fmul_rn(delay, __fsub_rn(w.z, q.z)));
        o.w = __fadd_rn(w.w, __fmul_rn(delay, __fsub_rn(w.w, q.w)));
        reinterpret_cast<float4 *>(out)[k] = o;
    }
}

// Per coordinate the population variance of d over the replicas, in double;
// out[0] accumulates the sum over coordinates, out[1] the maximum (variances are
// non-negative, so their bit patterns order like unsigned integers).
// MAJOR 0: d is coordinate-major [stride][R], a thread takes one coordinate's R
// contiguous floats (vector loads); MAJOR 1: replica-major [R][stride] (dense ring),
// a thread takes four consecutive coordinates, one 16-byte load per row.  Either way
// every byte is read once: a read-only stream.
template <int R, int MAJOR>
__global__ void spread_kernel(const float *D, uint64_t stride, uint64_t N, double *out)
{
    double acc = 0.0, mx = 0.0;
    auto one = [&](const float (&x)[R]) {
        double mean = 0.0;
#pragma unroll
        for (int i = 0; i < R; ++i) mean += (double)x[i];
        mean /= (double)R;
        double var = 0.0;
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const double e = (double)x[i] - mean;
            var += e * e;
        }
        var /= (double)R;
        acc += var;
        mx = var > mx ? var : mx;
    };
    if constexpr (MAJOR == 0) {
        for (uint64_t mu = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; mu < N;
             mu += (uint64_t)gridDim.x * blockDim.x) {
            float x[R];
            load_replicas<R>(D + mu * R, x);
            one(x);
        }
    } else {
        const uint64_t n4 = (N + 3) / 4;
        for (uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; q < n4;
             q += (uint64_t)gridDim.x * blockDim.x) {
            float4 r4[R];
#pragma unroll
            for (int i = 0; i < R; ++i) r4[i] = __ldcs(reinterpret_cast<const float4 *>(D + (uint64_t)i * stride) + q);
            const uint64_t left = N - 4 * q;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                if ((uint64_t)c < left) {
                    float x[R];
#pragma unroll
                    for (int i = 0; i < R; ++i) x[i] = reinterpret_cast<const float *>(&r4[i])[c];
                    one(x);
                }
            }
        }
    }
    for (int d = 16; d > 0; d >>= 1) {
        acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
        const double o = __shfl_down_sync(0xFFFFFFFFu, mx, d);
        mx = o > mx ? o : mx;
    }
    __shared__ double part[32], pmax[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { part[warp] = acc; pmax[warp] = mx; }
    __syncthreads();
    if (warp == 0) {
        const bool have = lane < (int)(blockDim.x >> 5);
        acc = have ? part[lane] : 0.0;
        mx = have ? pmax[lane] : 0.0;
        for (int d = 16; d > 0; d >>= 1) {
            acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
            const double o = __shfl_down_sync(0xFFFFFFFFu, mx, d);
            mx = o > mx ? o : mx;
        }
        if (lane == 0) {
            atomicAdd(out, acc);
            atomicMax(reinterpret_cast<unsigned long long *>(out + 1),
                      (unsigned long long)__double_as_longlong(mx));
        }
    }
}

typedef void (*spread_fn)(const float *, uint64_t, uint64_t, double *);
template <int MAJOR>
static spread_fn spread_for(uint32_t R)
{
    switch (R) {
    case 1: return spread_kernel<1, MAJOR>;   case 2: return spread_kernel<2, MAJOR>;
    case 3: return spread_kernel<3, MAJOR>;   case 4: return spread_kernel<4, MAJOR>;
    case 5: return spread_kernel<5, MAJOR>;   case 6: return spread_kernel<6, MAJOR>;
    case 7: return spread_kernel<7, MAJOR>;   case 8: return spread_kernel<8, MAJOR>;
    case 9: return spread_kernel<9, MAJOR>;   case 10: return spread_kernel<10, MAJOR>;
    case 11: return spread_kernel<11, MAJOR>; case 12: return spread_kernel<12, MAJOR>;
    case 13: return spread_kernel<13, MAJOR>; case 14: return spread_kernel<14, MAJOR>;
    case 15: return spread_kernel<15, MAJOR>; default: return spread_kernel<16, MAJOR>;
    }
}

__global__ void philox_debug_kernel(const uint32_t *ctr, const uint32_t *key, uint32_t *out,
                                    uint64_t n)
{
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n;
         k += (uint64_t)gridDim.x * blockDim.x) {
        const PhiloxOut o = philox4x32_10(ctr[4 * k], ctr[4 * k + 1], ctr[4 * k + 2],
                                          ctr[4 * k + 3], key[2 * k], key[2 * k + 1]);
        for (int j = 0; j < 4; ++j) out[4 * k + j] = o.x[j];
    }
}

static int grid_for(uint64_t items, int threads)
{
    uint64_t blocks = (items + threads - 1) / threads;
    if (blocks < 1) blocks = 1;
    if (blocks > 148ull * 16) blocks = 148ull * 16;
    return (int)blocks;
}

// ---------------------------------------------------------------------------
// kernel dispatch
// ---------------------------------------------------------------------------

// asyncmesh::pipelined for the owner kernel: 4 few, 7 some, 5 many entries fetched ahead; 6 synchronous
static int owner_entries(int pipelined)
{
    return pipelined == 4 ? kOwnerEntriesFew : (pipelined == 7 ? kOwnerEntriesMid : kOwnerEntriesMany);
}

static KernelChoice pick_kernel(uint32_t R, int mode, int pipelined, bool general, uint32_t S)
{
    if (pipelined >= 4) {
        const int entries = owner_entries(pipelined);
        return general ? pick_owner_general(R, mode, entries, S) : pick_owner_common(R, mode, entries, S);
    }
    if (pipelined && R <= 8)
        return general ? pick_pipelined_few_general(R, pipelined, S) : pick_pipelined_few_common(R, pipelined, S);
    if (pipelined)
        return general ? pick_pipelined_many_general(R, pipelined, S) : pick_pipelined_many_common(R, pipelined, S);
    if (mode > kDense) return pick_direct_stored(R, mode, general);
    if (R <= 8) return pick_direct_few(R, mode, general);
    return general ? pick_direct_many_general(R, mode) : pick_direct_many_common(R, mode);
}

// The pipelined kernel stashes the selected coordinates of a sub-iteration
// (union of two subsets); a shape pays off while they fit its stash.  With up to
// four replicas the narrow shape (which then asks for two rounds of selected
// coordinates ahead) overtakes the wide one earlier: 1B layout, p = 0.06: 24.6
// against 25.2 ms, p = 0.07: 25.0 against 26.7 (p = 0.05: 24.1 against 23.6).
template <class SH>
static bool stash_fits(double p, uint32_t R)
{
    const double q = 1.0 - (1.0 - p) * (1.0 - p);
    const double mean = SH::kSubCoords * q, sd = std::sqrt(SH::kSubCoords * q * (1.0 - q));
    const double sigmas = (SH::V == 2 && R <= 4) ? 7.5 : 4.0;
    return mean + sigmas * sd <= (double)SH::CAP;
}

// ---------------------------------------------------------------------------
// create / destroy
// ---------------------------------------------------------------------------

static uint64_t round_up(uint64_t x, uint64_t m) { return (x + m - 1) / m * m; }

extern "C" int asyncmesh_create(const asyncmesh_config *cfg, asyncmesh **out)
{
    if (out) *out = nullptr;
    if (!cfg || !out) return fail(ASYNCMESH_ERR_INVALID_ARG, "create: cfg and out must be non-NULL");
    if (cfg->R < 1 || cfg->R > ASYNCMESH_MAX_REPLICAS)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: R = %u outside 1..%u", cfg->R,
                    ASYNCMESH_MAX_REPLICAS);
    if (cfg->S < 1 || cfg->S > ASYNCMESH_MAX_STAGES)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: S = %u outside 1..%u", cfg->S,
                    ASYNCMESH_MAX_STAGES);
    if (!cfg->stage_numel) return fail(ASYNCMESH_ERR_INVALID_ARG, "create: stage_numel is NULL");
    if (!(cfg->p >= 0.0 && cfg->p <= 1.0))
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: p = %g outside [0, 1]", cfg->p);
    if (cfg->tau > ASYNCMESH_MAX_TAU)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: tau = %u above %u", cfg->tau,
                    ASYNCMESH_MAX_TAU);
    if (!(cfg->ema_beta >= 0.0 && cfg->ema_beta <= 1.0))
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: ema_beta = %g outside [0, 1]", cfg->ema_beta);
    if (!(cfg->lr > 0.0) || !(cfg->eps > 0.0) || !(cfg->weight_decay >= 0.0))
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: need lr > 0, eps > 0, weight_decay >= 0");
    if (!(cfg->beta1 >= 0.0 && cfg->beta1 < 1.0) || !(cfg->beta2 >= 0.0 && cfg->beta2 < 1.0))
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: betas must lie in [0, 1)");
    if ((cfg->flags & ~(ASYNCMESH_FLAG_SMALL_RING | ASYNCMESH_FLAG_DIRECT_KERNEL |
                        ASYNCMESH_FLAG_PIPELINED_KERNEL | ASYNCMESH_FLAG_BF16_EXCHANGE |
                        ASYNCMESH_FLAG_DENSE_RING | ASYNCMESH_FLAG_FP8_EXCHANGE |
                        ASYNCMESH_FLAG_KEEP_PREVIOUS | ASYNCMESH_FLAG_OWNER_KERNEL |
                        ASYNCMESH_FLAG_TRACK_CONSENSUS | ASYNCMESH_FLAG_RING_AS_EXCHANGED)) != 0)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: unknown flags");
    if (cfg->flags & ASYNCMESH_FLAG_RING_AS_EXCHANGED) {
        if (!(cfg->flags & (ASYNCMESH_FLAG_BF16_EXCHANGE | ASYNCMESH_FLAG_FP8_EXCHANGE)) || cfg->tau == 0)
            return fail(ASYNCMESH_ERR_INVALID_ARG,
                        "create: RING_AS_EXCHANGED needs BF16_EXCHANGE or FP8_EXCHANGE and tau > 0");
        if (cfg->flags & (ASYNCMESH_FLAG_SMALL_RING | ASYNCMESH_FLAG_PIPELINED_KERNEL | ASYNCMESH_FLAG_OWNER_KERNEL))
            return fail(ASYNCMESH_ERR_INVALID_ARG,
                        "create: RING_AS_EXCHANGED uses the dense ring and the direct kernel: not together with "
                        "SMALL_RING, PIPELINED_KERNEL or OWNER_KERNEL");
    }
    if ((cfg->flags & ASYNCMESH_FLAG_BF16_EXCHANGE) && (cfg->flags & ASYNCMESH_FLAG_FP8_EXCHANGE))
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: BF16_EXCHANGE and FP8_EXCHANGE exclude each other");
    if (cfg->optimizer > ASYNCMESH_OPT_NADAMW || cfg->correction > ASYNCMESH_CORRECTION_EAGER ||
        !(cfg->momentum_decay >= 0.0))
        return fail(ASYNCMESH_ERR_INVALID_ARG,
                    "create: optimizer must be 0 (AdamW) or 1 (NAdamW), correction 0 (EMA) or 1 (eager), "
                    "momentum_decay >= 0");
    const uint32_t K = cfg->avg_interval < 1 ? 1u : (uint32_t)cfg->avg_interval;
    if (cfg->avg_interval < 0 || cfg->tau % K != 0)
        return fail(ASYNCMESH_ERR_INVALID_ARG,
                    "create: avg_interval = %d must be >= 0 and divide tau = %u", cfg->avg_interval,
                    cfg->tau);
    if ((cfg->alloc == nullptr) != (cfg->free == nullptr))
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: give both alloc and free, or neither");
    for (uint32_t s = 0; s < cfg->S; ++s)
        if (cfg->stage_numel[s] < 1 || cfg->stage_numel[s] > 0xFFFFFFFFull)
            return fail(ASYNCMESH_ERR_INVALID_ARG, "create: stage_numel[%u] outside 1..2^32-1", s);
    if (cfg->coord_base)
        for (uint32_t s = 0; s < cfg->S; ++s)
            if ((cfg->coord_base[s] & 3u) != 0 || cfg->coord_base[s] + cfg->stage_numel[s] > 0x100000000ull)
                return fail(ASYNCMESH_ERR_INVALID_ARG,
                            "create: coord_base[%u] must be a multiple of 4 and coord_base + stage_numel "
                            "at most 2^32", s);

    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev < 1) {
        cudaGetLastError();
        return fail(ASYNCMESH_ERR_CUDA, "create: no CUDA device is usable (there is no CPU path)");
    }
    if (cfg->device < 0 || cfg->device >= ndev)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: device %d outside 0..%d", cfg->device, ndev - 1);

    DeviceScope scope(cfg->device);
    if (!scope.ok) return fail(ASYNCMESH_ERR_CUDA, "create: cudaSetDevice(%d) failed", cfg->device);

    asyncmesh *h = new (std::nothrow) asyncmesh();
    if (!h) return fail(ASYNCMESH_ERR_OOM, "create: host allocation failed");
    h->R = cfg->R; h->S = cfg->S; h->tau = cfg->tau;
    h->K = K; h->lag = cfg->tau / K;
    h->optimizer = cfg->optimizer;
    h->wire = (cfg->flags & ASYNCMESH_FLAG_BF16_EXCHANGE) ? 1u
              : (cfg->flags & ASYNCMESH_FLAG_FP8_EXCHANGE) ? 2u : 0u;
    h->correction = cfg->correction;
    h->momentum_decay = cfg->momentum_decay > 0.0 ? cfg->momentum_decay : 4e-3;
    h->p = cfg->p; h->ema_beta = cfg->ema_beta; h->lr = cfg->lr;
    h->beta1 = cfg->beta1; h->beta2 = cfg->beta2; h->eps = cfg->eps; h->wd = cfg->weight_decay;
    h->seed = cfg->seed; h->device = cfg->device; h->stream = (cudaStream_t)cfg->stream;
    h->alloc = cfg->alloc; h->dealloc = cfg->free; h->alloc_ctx = cfg->alloc_ctx;

    const uint32_t R = h->R, S = h->S;
    h->numel.assign(cfg->stage_numel, cfg->stage_numel + S);
    h->stride.resize(S);
    h->delay.resize(S);
    h->sd.assign(S, StageDesc{});
    h->gstage.assign(S, nullptr);
    h->wprev.assign(S, nullptr);
    h->lookx.assign(S, nullptr);

    // subset rule: floor(p * 2^32) in double
    const double tf = std::floor(cfg->p * 4294967296.0);
    h->rule.key0 = (uint32_t)h->seed;
    h->rule.key1 = (uint32_t)(h->seed >> 32);
    if (tf >= 4294967296.0) { h->rule.mode = 1; h->rule.thresh = 0xFFFFFFFFu; }
    else if (tf <= 0.0) { h->rule.mode = 2; h->rule.thresh = 0; }
    else { h->rule.mode = 0; h->rule.thresh = (uint32_t)tf; }

    // ring layout: compact unless it would not be smaller than dense
    std::vector<uint64_t> cap(S);
    long double compact_total = 0, dense_total = 0;
    uint64_t chunks = 0;
    for (uint32_t s = 0; s < S; ++s) {
        const uint64_t N = h->numel[s];
        h->stride[s] = round_up(N, 32);
        h->delay[s] = cfg->lookahead_delay ? cfg->lookahead_delay[s] : (S - 1 - s);
        const double mean = cfg->p * (double)N;
        const double sd = std::sqrt(mean * (1.0 - cfg->p));
        double c = std::ceil(mean + 8.0 * sd) + 64.0;   // 8 sigma: never reached in practice
        if (c > (double)N) c = (double)N;
        cap[s] = (uint64_t)c;
        if ((cfg->flags & ASYNCMESH_FLAG_SMALL_RING) && h->tau > 0) cap[s] = cap[s] / 8 + 1;
        compact_total += (long double)(h->lag + 1) * cap[s];
        dense_total += (long double)h->lag * h->stride[s];
        h->sd[s].n_chunks = (uint32_t)((N + kWarpChunk - 1) / kWarpChunk);
        h->sd[s].chunk_begin = (uint32_t)chunks;
        chunks += h->sd[s].n_chunks;
    }
    if (chunks > 0xFFFFFFF0ull) {
        delete h;
        return fail(ASYNCMESH_ERR_INVALID_ARG, "create: too many coordinates in total");
    }
    h->total_chunks = (uint32_t)chunks;
    if (h->tau == 0) { h->mode = kSync; h->n_slots = 0; }
    else if (cfg->flags & ASYNCMESH_FLAG_RING_AS_EXCHANGED) {
        h->mode = h->wire == 1u ? kDenseBf16 : kDenseE4m3; h->n_slots = h->lag;
    }
    else if ((cfg->flags & ASYNCMESH_FLAG_DENSE_RING) && !(cfg->flags & ASYNCMESH_FLAG_SMALL_RING)) {
        h->mode = kDense; h->n_slots = h->lag;
    }
    // dense once compaction would save less than a third of the ring: from there on
    // nearly every coordinate is selected and streaming beats per-coordinate work
    else if (dense_total <= 1.5L * compact_total &&
             !(cfg->flags & (ASYNCMESH_FLAG_SMALL_RING | ASYNCMESH_FLAG_PIPELINED_KERNEL |
                               ASYNCMESH_FLAG_OWNER_KERNEL))) {
        h->mode = kDense; h->n_slots = h->lag;
    }
    else { h->mode = kCompact; h->n_slots = h->lag + 1; }

    // the compact ring has two kernels; which one is fixed for the handle's life
    h->pipelined = 0;   // 0 direct, 1 pipelined wide, 2 pipelined narrow, 3 pipelined narrow synchronous,
                        // 4 to 7 owner (below)
    // synchronous mode: the stash route pays while most float4 groups are only partly
    // selected; towards p = 1 the direct kernel writes whole groups and wins
    if (h->mode == kSync && !(cfg->flags & ASYNCMESH_FLAG_DIRECT_KERNEL) &&
        (cfg->p <= 0.8 || (cfg->flags & ASYNCMESH_FLAG_PIPELINED_KERNEL)))
        h->pipelined = 3;
    if (h->mode == kCompact && !(cfg->flags & ASYNCMESH_FLAG_DIRECT_KERNEL)) {
        if (stash_fits<PipeWide>(cfg->p, R)) h->pipelined = 1;
        else if (stash_fits<PipeNarrow>(cfg->p, R) || (cfg->flags & ASYNCMESH_FLAG_PIPELINED_KERNEL))
            h->pipelined = 2;
    }

    // Up to four replicas: the owner kernel (4: few ring / d entries fetched ahead per
    // group, 7: some, 5: many, 6: synchronous) wherever one of the two pipelined shapes would run,
    // unless a flag asks for another kernel.  1B layout, tau = 4, ms per step, pipelined
    // against owner: p = 0.01 21.6 / 20.7, 0.05 23.4 / 22.7, 0.1 26.2 / 23.9, 0.25 30.9 / 25.6,
    // 0.5 37.4 / 29.0; tau = 0: 20.8 to 24.4 / 20.5 to 20.7 at every p.
    // E4M3 exchange, the eager estimate and NAdamW: the kernels' general form.  With the ring the
    // owner kernel loses more to that form than the pipelined kernel does (1B layout, E4M3 exchange:
    // 26.9 against 23.4 ms per step at p = 0.05, 33.6 against 30.4 at p = 0.25), so there the general
    // form stays with the pipelined kernel; for tau = 0 the owner kernel keeps its lead (19.3 against 20.7).
    // (a ring kept as exchanged converts by its slot format, which is a template parameter: common form)
    const bool general = (h->wire == 2u && h->mode <= kDense) || h->correction == ASYNCMESH_CORRECTION_EAGER ||
                         h->optimizer == ASYNCMESH_OPT_NADAMW;
    // NAdamW alone (the optimizer of the paper's asynchronous-pipeline runs) has an owner form of its
    // own, with the optimizer fixed at compile time, and goes where AdamW goes.  1B layout, ms per step,
    // that form against the pipelined kernel's general form: tau = 0 19.1 / 20.9; tau = 4, p = 0.05
    // 22.6 / 23.3, p = 0.25 27.1 / 29.7 (AdamW in the owner kernel: 19.1, 22.5, 25.6).
    const bool nadam_only = h->optimizer == ASYNCMESH_OPT_NADAMW && h->wire != 2u &&
                            h->correction != ASYNCMESH_CORRECTION_EAGER;
    const bool owner_asked = (cfg->flags & ASYNCMESH_FLAG_OWNER_KERNEL) != 0;
    const bool owner_default =
        (!general || nadam_only || h->mode == kSync) && !(cfg->flags & (ASYNCMESH_FLAG_DIRECT_KERNEL | ASYNCMESH_FLAG_PIPELINED_KERNEL)) &&
        (h->mode == kCompact || (h->mode == kSync && cfg->p <= 0.8));
    // (five to eight replicas: for tau = 0 only; 350M layout, p = 0.05: 14.15 against 15.09 ms, while with
    // the ring the pipelined kernel is as fast at p = 0.05 and faster at p = 0.01 and 0.25)
    // Six and eight replicas with the ring: two passes of three and four replicas over each group.  350M
    // layout (R = 8, tau = 4), ms per step, pipelined against that: p = 0.01 14.51 / 14.47, 0.05 15.73 / 15.66,
    // 0.25 20.15 / 18.80, 0.5 21.93 / 21.80; 125M layout (tau = 2): 4.66 / 4.68, 5.03 / 5.06, 6.43 / 6.02.
    // The default where it wins: the subsets that need the many-entries form.
    const bool two_pass = (R == 6 || R == 8) && h->mode == kCompact;
    const double group_mean = 128.0 * kOwnerV * cfg->p;
    const bool few_entries = group_mean + 4.0 * std::sqrt(group_mean * (1.0 - cfg->p)) <= (double)kOwnerEntriesFew;
    if ((R <= 4 || (R <= 8 && h->mode == kSync) || two_pass) && !is_dense(h->mode) &&
        (owner_asked || (owner_default && (!two_pass || !few_entries))))
        h->pipelined = h->mode == kSync ? 6 : few_entries ? 4 : (!two_pass && group_mean <= 96.0) ? 7 : 5;


    auto bail = [&](int code, const char *what) {
        release_all(h);
        delete h;
        return fail(code, "create: %s", what);
    };

    // allocations (all zeroed on the stream)
    auto zalloc = [&](size_t bytes) -> void * {
        void *ptr = dev_alloc(h, bytes);
        if (ptr && cudaMemsetAsync(ptr, 0, bytes ? bytes : 256, h->stream) != cudaSuccess) return nullptr;
        return ptr;
    };
    for (uint32_t s = 0; s < S; ++s) {
        StageDesc &d = h->sd[s];
        const size_t row_bytes = (size_t)R * h->stride[s] * sizeof(float);
        d.N = h->numel[s];
        d.stride = h->stride[s];
        d.stage_id = s;
        d.quad_base = cfg->coord_base ? (uint32_t)(cfg->coord_base[s] >> 2) : 0u;
        d.delta = (float)h->delay[s];
        d.cap = (uint32_t)cap[s];
        d.W = (float *)zalloc(row_bytes);
        d.M = (float *)zalloc(row_bytes);
        d.V = (float *)zalloc(row_bytes);
        d.D = (float *)zalloc(row_bytes);
        if (!d.W || !d.M || !d.V || !d.D) return bail(ASYNCMESH_ERR_OOM, "out of device memory (state)");
        if (cfg->flags & ASYNCMESH_FLAG_KEEP_PREVIOUS) {
            h->wprev[s] = (float *)zalloc(row_bytes);
            if (!h->wprev[s]) return bail(ASYNCMESH_ERR_OOM, "out of device memory (previous weights)");
        }
        d.LOOK = d.W;
        if (h->delay[s] != 0) {
            d.LOOK = (float *)zalloc(row_bytes);
            if (!d.LOOK) return bail(ASYNCMESH_ERR_OOM, "out of device memory (look-ahead)");
        }
        if (h->mode == kCompact) {
            d.slot_floats = round_up(cap[s] * R, 64);
            d.chunk_base = (uint32_t *)zalloc((size_t)h->n_slots * d.n_chunks * sizeof(uint32_t));
            if (!d.chunk_base) return bail(ASYNCMESH_ERR_OOM, "out of device memory (ring index)");
            if (h->pipelined) {
                d.bitmap = (uint32_t *)zalloc((size_t)h->n_slots * d.n_chunks * 32 * sizeof(uint32_t));
                if (!d.bitmap) return bail(ASYNCMESH_ERR_OOM, "out of device memory (subset masks)");
            }
        } else if (is_dense(h->mode)) {
            d.slot_floats = h->stride[s] * R;   // values per slot, ring_value_bytes(mode) each
        }
        if (h->mode != kSync) {
            d.ring = (float *)zalloc((size_t)h->n_slots * d.slot_floats * (size_t)ring_value_bytes(h->mode));
            if (!d.ring) return bail(ASYNCMESH_ERR_OOM, "out of device memory (snapshot ring)");
        }
    }
    h->sd_dev = (StageDesc *)zalloc(S * sizeof(StageDesc));
    h->sd_single_dev = (StageDesc *)zalloc(S * sizeof(StageDesc));
    h->cursors = (unsigned int *)zalloc((size_t)(h->n_slots + 1) * S * sizeof(unsigned int));
    h->status = (int *)zalloc(256);
    h->scratch = (double *)zalloc(256);
    h->diag = (double *)zalloc((size_t)S * sizeof(double));
    if (!h->sd_dev || !h->sd_single_dev || !h->cursors || !h->status || !h->scratch || !h->diag)
        return bail(ASYNCMESH_ERR_OOM, "out of device memory (tables)");
    std::vector<StageDesc> single(h->sd);
    for (StageDesc &d1 : single) d1.chunk_begin = 0;
    if (cudaMemcpyAsync(h->sd_dev, h->sd.data(), S * sizeof(StageDesc), cudaMemcpyHostToDevice,
                        h->stream) != cudaSuccess ||
        cudaMemcpyAsync(h->sd_single_dev, single.data(), S * sizeof(StageDesc), cudaMemcpyHostToDevice,
                        h->stream) != cudaSuccess ||
        cudaStreamSynchronize(h->stream) != cudaSuccess) {
        const char *msg = cudaGetErrorString(cudaGetLastError());
        release_all(h);
        delete h;
        return fail(ASYNCMESH_ERR_CUDA, "create: uploading the stage table failed: %s", msg);
    }

    // persistent grid: every SM filled to the kernel's occupancy
    h->nadam_form = h->pipelined >= 4 && nadam_only;
    h->general = general && !h->nadam_form;
    h->kernel = h->nadam_form
        ? pick_owner_nadamw(R, h->mode, owner_entries(h->pipelined), S)
        : pick_kernel(R, h->mode, h->pipelined, general, S);
    if ((cfg->flags & ASYNCMESH_FLAG_TRACK_CONSENSUS) && h->pipelined >= 4 && !general &&
        (R <= 4 || h->mode == kSync)) {
        h->tracking = true;
        h->kernel = pick_owner_tracking(R, h->mode, owner_entries(h->pipelined), S);
    }
    int sms = 0, per_sm = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->device);
    cudaError_t ke = cudaSuccess;
    if (h->kernel.smem > 48 * 1024)
        ke = cudaFuncSetAttribute((const void *)h->kernel.fn,
                                  cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->kernel.smem);
    if (ke == cudaSuccess)
        ke = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, (const void *)h->kernel.fn,
                                                           h->kernel.threads, h->kernel.smem);
    if (ke != cudaSuccess || per_sm < 1 || sms < 1) {
        const char *msg = cudaGetErrorString(ke != cudaSuccess ? ke : cudaGetLastError());
        release_all(h);
        delete h;
        return fail(ASYNCMESH_ERR_CUDA, "create: the step kernel cannot run on this device: %s", msg);
    }
    if (h->kernel.max_blocks_per_sm > 0 && per_sm > h->kernel.max_blocks_per_sm)
        per_sm = h->kernel.max_blocks_per_sm;
    uint64_t blocks = (uint64_t)sms * per_sm;
    const uint64_t wpb = (uint64_t)h->kernel.threads / 32;
    const uint64_t need = ((uint64_t)h->total_chunks + wpb - 1) / wpb;
    if (blocks > need) blocks = need;
    h->grid = (int)blocks;

    *out = h;
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_destroy(asyncmesh *h)
{
    if (!h) return ASYNCMESH_OK;
    DeviceScope scope(h->device);
    cudaStreamSynchronize(h->stream);
    if (h->copy_stream) {
        cudaStreamSynchronize(h->copy_stream);
        for (cudaEvent_t e : h->ev_ready) cudaEventDestroy(e);
        for (cudaEvent_t e : h->ev_done) cudaEventDestroy(e);
        cudaStreamDestroy(h->copy_stream);
    }
    release_all(h);
    delete h;
    return ASYNCMESH_OK;
}

// ---------------------------------------------------------------------------
// parameters in
// ---------------------------------------------------------------------------

extern "C" int asyncmesh_init_params(asyncmesh *h, uint32_t stage, int32_t replica,
                                     const float *src, uint64_t n, int src_on_device)
{
    if (!h || !src) return fail(ASYNCMESH_ERR_INVALID_ARG, "init_params: NULL argument");
    if (stage >= h->S) return fail(ASYNCMESH_ERR_INVALID_ARG, "init_params: stage %u >= S", stage);
    if (replica < -1 || replica >= (int32_t)h->R)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "init_params: replica %d outside -1..R-1", replica);
    if (n != h->numel[stage])
        return fail(ASYNCMESH_ERR_INVALID_ARG, "init_params: n = %llu, stage holds %llu",
                    (unsigned long long)n, (unsigned long long)h->numel[stage]);
    if (h->t != 0) return fail(ASYNCMESH_ERR_BAD_STATE, "init_params: steps were already taken");
    DeviceScope scope(h->device);
    const StageDesc &d = h->sd[stage];
    const cudaMemcpyKind kind = src_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
    for (uint32_t i = 0; i < h->R; ++i) {
        if (replica >= 0 && (uint32_t)replica != i) continue;
        CU_TRY(cudaMemcpyAsync(d.W + (uint64_t)i * d.stride, src, n * sizeof(float), kind, h->stream));
        if (d.LOOK != d.W)
            CU_TRY(cudaMemcpyAsync(d.LOOK + (uint64_t)i * d.stride, src, n * sizeof(float), kind,
                                   h->stream));
    }
    if (!src_on_device) CU_TRY(cudaStreamSynchronize(h->stream));
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_row_stride(const asyncmesh *h, uint32_t stage, uint64_t *stride)
{
    if (!h || !stride || stage >= h->S)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "row_stride: bad handle, stage or output");
    *stride = h->stride[stage];
    return ASYNCMESH_OK;
}

// ---------------------------------------------------------------------------
// the step
// ---------------------------------------------------------------------------

// stage_ready: NULL, or one event per stage that the stage's gradients wait for; the step then
// runs as one launch per stage, each as soon as its gradients are there.
static int launch_step(asyncmesh *h, const float *const *grads, double ema_beta_t, double lr_t,
                       const cudaEvent_t *stage_ready = nullptr)
{
    if (ema_beta_t > 1.0) return fail(ASYNCMESH_ERR_INVALID_ARG, "step: ema_beta_t = %g above 1", ema_beta_t);
    StepParams P;
    std::memset(&P, 0, sizeof(P));
    for (uint32_t s = 0; s < h->S; ++s) {
        if (!grads[s]) return fail(ASYNCMESH_ERR_INVALID_ARG, "step: grads[%u] is NULL", s);
        if (((uintptr_t)grads[s] & 15u) != 0)
            return fail(ASYNCMESH_ERR_INVALID_ARG, "step: grads[%u] is not 16-byte aligned", s);
        P.G[s] = grads[s];
    }
    const uint64_t t = h->t + 1;
    const double lam = ema_beta_t >= 0.0 ? ema_beta_t : h->ema_beta;
    const double lr = lr_t >= 0.0 ? lr_t : h->lr;

    P.stages = h->sd_dev;
    P.cursors = h->cursors;
    P.status = h->status;
    P.diag = h->diag;
    P.S = h->S;
    P.total_chunks = h->total_chunks;
    P.cursor_S = h->S;
    P.s_base = 0;
    P.step = (uint32_t)t;
    // averaging rounds are the steps K, 2K, ...; in between the step is purely local
    const bool round = (t % h->K) == 0;
    const uint64_t r = t / h->K;   // index of this round
    P.cons_step = (uint32_t)(t - h->tau);
    P.produce = round ? 1u : 0u;
    P.consume = (h->mode != kSync && round && t > h->tau) ? 1u : 0u;
    if (h->mode == kCompact) {
        P.prod_slot = (uint32_t)(r % (h->lag + 1));
        P.cons_slot = (uint32_t)((r - h->lag) % (h->lag + 1));   // unused while t <= tau
    } else if (is_dense(h->mode)) {
        P.prod_slot = P.cons_slot = (uint32_t)(r % h->lag);
    }
    P.rule = h->rule;
    // per-step scalars: double arithmetic, one rounding to fp32 each
    P.b1 = (float)h->beta1;
    P.b2 = (float)h->beta2;
    P.omb1 = (float)(1.0 - h->beta1);
    P.omb2 = (float)(1.0 - h->beta2);
    P.ib1 = (float)(1.0 / (1.0 - std::pow(h->beta1, (double)t)));
    P.ib2 = (float)(1.0 / (1.0 - std::pow(h->beta2, (double)t)));
    P.eps = (float)h->eps;
    P.lr = (float)lr;
    P.lrwd = (float)(lr * h->wd);
    P.lam = (float)lam;
    P.oml = (float)(1.0 - lam);
    P.Rf = (float)h->R;
    P.wire = h->wire;
    P.eager = h->correction == ASYNCMESH_CORRECTION_EAGER ? 1u : 0u;
    P.nesterov = h->optimizer == ASYNCMESH_OPT_NADAMW ? 1u : 0u;
    P.eps_inrange = (P.eps <= 1.152921504606847e18f) ? 1u : 0u;   // 2^60, see rounded_math.cuh
    double mu_product = h->mu_product;
    if (P.nesterov) {   // mu_t, mu_{t+1} and the running product of the momentum schedule
        const double mu_t = h->beta1 * (1.0 - 0.5 * std::pow(0.96, (double)t * h->momentum_decay));
        const double mu_n = h->beta1 * (1.0 - 0.5 * std::pow(0.96, (double)(t + 1) * h->momentum_decay));
        mu_product *= mu_t;
        P.cg = (float)(lr * (1.0 - mu_t) / (1.0 - mu_product));
        P.cm = (float)(lr * mu_n / (1.0 - mu_product * mu_n));
    }

    for (uint32_t s = 0; s < h->S; ++s)   // w^{t-1} for look-aheads asked for after the fact
        if (h->wprev[s])
            CU_TRY(cudaMemcpyAsync(h->wprev[s], h->sd[s].W, (size_t)h->R * h->stride[s] * sizeof(float),
                                   cudaMemcpyDeviceToDevice, h->stream));

    if (h->mode == kCompact && round)   // the producing slot's cursors start this step at zero
        CU_TRY(cudaMemsetAsync(h->cursors + (size_t)P.prod_slot * h->S, 0,
                               h->S * sizeof(unsigned int), h->stream));

    if (h->tracking)   // this step's consensus errors start at zero
        CU_TRY(cudaMemsetAsync(h->diag, 0, (size_t)h->S * sizeof(double), h->stream));
    if (!stage_ready) {
        h->kernel.fn<<<h->grid, h->kernel.threads, h->kernel.smem, h->stream>>>(P);
        CU_TRY(cudaGetLastError());
    } else {
        const uint32_t wpb = (uint32_t)h->kernel.threads / 32;
        for (uint32_t s = 0; s < h->S; ++s) {
            StepParams Q = P;
            Q.stages = h->sd_single_dev + s;
            Q.S = 1;
            Q.s_base = s;
            Q.total_chunks = h->sd[s].n_chunks;
            Q.G[0] = grads[s];
            int grid = (int)((Q.total_chunks + wpb - 1) / wpb);
            if (grid > h->grid) grid = h->grid;
            CU_TRY(cudaStreamWaitEvent(h->stream, stage_ready[s], 0));
            h->kernel.fn<<<grid, h->kernel.threads, h->kernel.smem, h->stream>>>(Q);
            CU_TRY(cudaGetLastError());
            CU_TRY(cudaEventRecord(h->ev_done[s], h->stream));
            h->done_recorded[s] = 1;
        }
    }
    h->t = t;
    h->diag_step = t;
    h->mu_product = mu_product;

    // roofline numerator (see the header): bytes this step could not avoid
    double bytes = 0.0;
    for (uint32_t s = 0; s < h->S; ++s) {
        double per = 28.0 + (h->delay[s] ? 4.0 : 0.0);
        // snapshot written, and on arrival read again with d read and written
        const double rb = h->mode == kSync ? 0.0 : (double)ring_value_bytes(h->mode);
        if (h->mode != kSync && round) per += rb * h->p + (P.consume ? (rb + 8.0) * h->p : 0.0);
        bytes += per * (double)h->R * (double)h->numel[s];
    }
    h->last_bytes = (uint64_t)bytes;
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_step_ex(asyncmesh *h, const float *const *grads, double ema_beta_t,
                                 double lr_t)
{
    if (!h || !grads) return fail(ASYNCMESH_ERR_INVALID_ARG, "step: NULL argument");
    DeviceScope scope(h->device);
    return launch_step(h, grads, ema_beta_t, lr_t);
}

extern "C" int asyncmesh_step(asyncmesh *h, const float *const *grads)
{
    return asyncmesh_step_ex(h, grads, -1.0, -1.0);
}

extern "C" int asyncmesh_step_host_ex(asyncmesh *h, const float *const *grads_host,
                                      double ema_beta_t, double lr_t)
{
    if (!h || !grads_host) return fail(ASYNCMESH_ERR_INVALID_ARG, "step_host: NULL argument");
    DeviceScope scope(h->device);
    for (uint32_t s = 0; s < h->S; ++s)
        if (!grads_host[s]) return fail(ASYNCMESH_ERR_INVALID_ARG, "step_host: grads_host[%u] is NULL", s);
    if (!h->copy_stream) {   // first call: a stream for the copies and the events that tie it to the kernels
        CU_TRY(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
        h->ev_ready.assign(h->S, nullptr);
        h->ev_done.assign(h->S, nullptr);
        h->done_recorded.assign(h->S, 0);
        for (uint32_t s = 0; s < h->S; ++s) {
            CU_TRY(cudaEventCreateWithFlags(&h->ev_ready[s], cudaEventDisableTiming));
            CU_TRY(cudaEventCreateWithFlags(&h->ev_done[s], cudaEventDisableTiming));
        }
    }
    // Stage by stage on the copy stream: wait until the previous step's kernel is done with the
    // stage's staging buffer, copy, signal.  The kernels (one launch per stage, on the handle's
    // stream) start as their gradients arrive, so all but the last stage's compute hides behind
    // the copies of the stages after it.
    for (uint32_t s = 0; s < h->S; ++s) {
        if (!h->gstage[s]) {
            const size_t bytes = (size_t)h->R * h->stride[s] * sizeof(float);
            h->gstage[s] = (float *)dev_alloc(h, bytes);
            if (!h->gstage[s]) return fail(ASYNCMESH_ERR_OOM, "step_host: out of device memory (staging)");
            CU_TRY(cudaMemsetAsync(h->gstage[s], 0, bytes, h->copy_stream));
        }
        if (h->done_recorded[s]) CU_TRY(cudaStreamWaitEvent(h->copy_stream, h->ev_done[s], 0));
        // one copy per replica row (a 2-D copy would cap the row at the device's largest pitch)
        const size_t n = h->numel[s] * sizeof(float);
        for (uint32_t i = 0; i < h->R; ++i)
            CU_TRY(cudaMemcpyAsync(h->gstage[s] + (uint64_t)i * h->stride[s], grads_host[s] + (uint64_t)i * h->numel[s],
                                   n, cudaMemcpyHostToDevice, h->copy_stream));
        CU_TRY(cudaEventRecord(h->ev_ready[s], h->copy_stream));
    }
    return launch_step(h, h->gstage.data(), ema_beta_t, lr_t, h->ev_ready.data());
}

extern "C" int asyncmesh_step_host(asyncmesh *h, const float *const *grads_host)
{
    return asyncmesh_step_host_ex(h, grads_host, -1.0, -1.0);
}

// ---------------------------------------------------------------------------
// results out
// ---------------------------------------------------------------------------

static int check_status(asyncmesh *h, const char *who)
{
    int st = 0;
    CU_TRY(cudaMemcpyAsync(&st, h->status, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
    CU_TRY(cudaStreamSynchronize(h->stream));
    if (st == kStatusRingOverflow)
        return fail(ASYNCMESH_ERR_DEVICE_STATUS,
                    "%s: a snapshot ring slot overflowed its capacity; results are invalid", who);
    if (st != 0) return fail(ASYNCMESH_ERR_DEVICE_STATUS, "%s: device status %d", who, st);
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_status(asyncmesh *h)
{
    if (!h) return fail(ASYNCMESH_ERR_INVALID_ARG, "status: NULL handle");
    DeviceScope scope(h->device);
    return check_status(h, "status");
}

extern "C" int asyncmesh_lookahead_weights(asyncmesh *h, uint32_t stage, uint32_t delay,
                                           const float **out_device, uint64_t *row_stride)
{
    if (!h || !out_device || !row_stride || stage >= h->S)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "lookahead_weights: bad handle, stage or output");
    const StageDesc &d = h->sd[stage];
    if (delay == 0 || h->t == 0) *out_device = d.W;   // before the first step w^{-1} = w^0
    else if (delay == h->delay[stage]) *out_device = d.LOOK;
    else if (h->wprev[stage]) {
        DeviceScope scope(h->device);
        const uint64_t n = (uint64_t)h->R * d.stride;
        if (!h->lookx[stage]) {
            h->lookx[stage] = (float *)dev_alloc(h, n * sizeof(float));
            if (!h->lookx[stage]) return fail(ASYNCMESH_ERR_OOM, "lookahead_weights: out of device memory");
        }
        extrapolate_kernel<<<grid_for(n / 4, 256), 256, 0, h->stream>>>(d.W, h->wprev[stage], h->lookx[stage],
                                                                       (float)delay, n / 4);
        CU_TRY(cudaGetLastError());
        *out_device = h->lookx[stage];
    } else
        return fail(ASYNCMESH_ERR_UNSUPPORTED,
                    "lookahead_weights: stage %u was configured with delay %u, not %u (any delay "
                    "needs ASYNCMESH_FLAG_KEEP_PREVIOUS)", stage, h->delay[stage], delay);
    *row_stride = d.stride;
    return ASYNCMESH_OK;
}

// Copy N floats produced on the device (by `produce`, into a device buffer) to dst.
template <typename Produce>
static int deliver(asyncmesh *h, float *dst, uint64_t n, int dst_on_device, Produce produce)
{
    float *tmp = dst;
    if (!dst_on_device) {
        tmp = (float *)dev_alloc(h, n * sizeof(float));
        if (!tmp) return fail(ASYNCMESH_ERR_OOM, "read: out of device memory (temporary)");
    }
    produce(tmp);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && !dst_on_device)
        e = cudaMemcpyAsync(dst, tmp, n * sizeof(float), cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    if (!dst_on_device) dev_free(h, tmp);
    if (e != cudaSuccess) return fail(ASYNCMESH_ERR_CUDA, "read: %s", cudaGetErrorString(e));
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_read_state_range(asyncmesh *h, uint32_t stage, int which, int32_t replica,
                                          uint64_t first, uint64_t count, float *dst,
                                          int dst_on_device)
{
    if (!h || !dst) return fail(ASYNCMESH_ERR_INVALID_ARG, "read_state: NULL argument");
    if (stage >= h->S) return fail(ASYNCMESH_ERR_INVALID_ARG, "read_state: stage %u >= S", stage);
    if (replica < 0 || replica >= (int32_t)h->R)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "read_state: replica %d outside 0..R-1", replica);
    if (count < 1 || first >= h->numel[stage] || count > h->numel[stage] - first)
        return fail(ASYNCMESH_ERR_INVALID_ARG,
                    "read_state: range [%llu, +%llu) outside the stage's %llu coordinates",
                    (unsigned long long)first, (unsigned long long)count,
                    (unsigned long long)h->numel[stage]);
    DeviceScope scope(h->device);
    int rc = check_status(h, "read_state");
    if (rc != ASYNCMESH_OK) return rc;
    const StageDesc &d = h->sd[stage];
    const float *row = nullptr;
    switch (which) {
    case ASYNCMESH_STATE_W: row = d.W; break;
    case ASYNCMESH_STATE_M: row = d.M; break;
    case ASYNCMESH_STATE_V: row = d.V; break;
    case ASYNCMESH_STATE_LOOK: row = d.LOOK; break;
    case ASYNCMESH_STATE_D: if (is_dense(h->mode)) row = d.D; break;   // replica-major there
    default: return fail(ASYNCMESH_ERR_INVALID_ARG, "read_state: unknown selector %d", which);
    }
    if (row) {
        CU_TRY(cudaMemcpyAsync(dst, row + (uint64_t)replica * d.stride + first, count * sizeof(float),
                               dst_on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost,
                               h->stream));
        CU_TRY(cudaStreamSynchronize(h->stream));
        return ASYNCMESH_OK;
    }
    return deliver(h, dst, count, dst_on_device, [&](float *out) {
        gather_column_kernel<<<grid_for(count, 256), 256, 0, h->stream>>>(d.D, h->R, (uint32_t)replica,
                                                                         first, count, out);
    });
}

extern "C" int asyncmesh_read_state(asyncmesh *h, uint32_t stage, int which, int32_t replica,
                                    float *dst, uint64_t n, int dst_on_device)
{
    if (!h || !dst) return fail(ASYNCMESH_ERR_INVALID_ARG, "read_state: NULL argument");
    if (stage >= h->S) return fail(ASYNCMESH_ERR_INVALID_ARG, "read_state: stage %u >= S", stage);
    if (n != h->numel[stage])
        return fail(ASYNCMESH_ERR_INVALID_ARG, "read_state: n = %llu, stage holds %llu",
                    (unsigned long long)n, (unsigned long long)h->numel[stage]);
    return asyncmesh_read_state_range(h, stage, which, replica, 0, n, dst, dst_on_device);
}

extern "C" int asyncmesh_read_params(asyncmesh *h, uint32_t stage, int32_t replica, float *dst,
                                     uint64_t n, int dst_on_device)
{
    if (!h || !dst) return fail(ASYNCMESH_ERR_INVALID_ARG, "read_params: NULL argument");
    if (replica >= 0) return asyncmesh_read_state(h, stage, ASYNCMESH_STATE_W, replica, dst, n, dst_on_device);
    if (replica != -1) return fail(ASYNCMESH_ERR_INVALID_ARG, "read_params: replica %d outside -1..R-1", replica);
    if (stage >= h->S) return fail(ASYNCMESH_ERR_INVALID_ARG, "read_params: stage %u >= S", stage);
    if (n != h->numel[stage])
        return fail(ASYNCMESH_ERR_INVALID_ARG, "read_params: n = %llu, stage holds %llu",
                    (unsigned long long)n, (unsigned long long)h->numel[stage]);
    DeviceScope scope(h->device);
    int rc = check_status(h, "read_params");
    if (rc != ASYNCMESH_OK) return rc;
    const StageDesc &d = h->sd[stage];
    return deliver(h, dst, n, dst_on_device, [&](float *out) {
        mean_rows_kernel<<<grid_for(n, 256), 256, 0, h->stream>>>(d.W, h->R, d.stride, n, (float)h->R, out);
    });
}

extern "C" int asyncmesh_subset_mask(asyncmesh *h, uint32_t stage, uint64_t step,
                                     uint8_t *bitmap_host)
{
    if (!h || !bitmap_host || stage >= h->S)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "subset_mask: bad handle, stage or output");
    DeviceScope scope(h->device);
    const uint64_t N = h->numel[stage], nbytes = (N + 7) / 8;
    uint8_t *tmp = (uint8_t *)dev_alloc(h, nbytes);
    if (!tmp) return fail(ASYNCMESH_ERR_OOM, "subset_mask: out of device memory (temporary)");
    subset_bitmap_kernel<<<grid_for(nbytes, 256), 256, 0, h->stream>>>(h->rule, stage, (uint32_t)step, N,
                                                                          h->sd[stage].quad_base, tmp);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaMemcpyAsync(bitmap_host, tmp, nbytes, cudaMemcpyDeviceToHost, h->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(h->stream);
    dev_free(h, tmp);
    if (e != cudaSuccess) return fail(ASYNCMESH_ERR_CUDA, "subset_mask: %s", cudaGetErrorString(e));
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_consensus_error(asyncmesh *h, uint32_t stage, double *out_host)
{
    if (!h || !out_host || stage >= h->S)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "consensus_error: bad handle, stage or output");
    DeviceScope scope(h->device);
    int rc = check_status(h, "consensus_error");
    if (rc != ASYNCMESH_OK) return rc;
    const StageDesc &d = h->sd[stage];
    if (h->tracking && h->t > 0 && h->diag_step == h->t) {   // the last step accumulated it on its way
        CU_TRY(cudaMemcpyAsync(out_host, h->diag + stage, sizeof(double), cudaMemcpyDeviceToHost, h->stream));
        CU_TRY(cudaStreamSynchronize(h->stream));
        return ASYNCMESH_OK;
    }
    CU_TRY(cudaMemsetAsync(h->scratch, 0, sizeof(double), h->stream));
    consensus_for(h->R)<<<grid_for((d.N + 3) / 4, 256), 256, 0, h->stream>>>(d.W, d.stride, d.N, h->scratch);
    CU_TRY(cudaGetLastError());
    CU_TRY(cudaMemcpyAsync(out_host, h->scratch, sizeof(double), cudaMemcpyDeviceToHost, h->stream));
    CU_TRY(cudaStreamSynchronize(h->stream));
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_ema_variance(asyncmesh *h, uint32_t stage, double *mean_host,
                                      double *max_host)
{
    if (!h || !mean_host || !max_host || stage >= h->S)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "ema_variance: bad handle, stage or output");
    DeviceScope scope(h->device);
    int rc = check_status(h, "ema_variance");
    if (rc != ASYNCMESH_OK) return rc;
    const StageDesc &d = h->sd[stage];
    // d is coordinate-major [stride][R] except with the dense ring ([R][stride])
    CU_TRY(cudaMemsetAsync(h->scratch, 0, 2 * sizeof(double), h->stream));
    if (is_dense(h->mode))
        spread_for<1>(h->R)<<<grid_for((d.N + 3) / 4, 256), 256, 0, h->stream>>>(d.D, d.stride, d.N, h->scratch);
    else
        spread_for<0>(h->R)<<<grid_for(d.N, 256), 256, 0, h->stream>>>(d.D, d.stride, d.N, h->scratch);
    CU_TRY(cudaGetLastError());
    double out[2];
    CU_TRY(cudaMemcpyAsync(out, h->scratch, sizeof out, cudaMemcpyDeviceToHost, h->stream));
    CU_TRY(cudaStreamSynchronize(h->stream));
    *mean_host = out[0] / (double)d.N;
    *max_host = out[1];
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_step_count(const asyncmesh *h, uint64_t *t)
{
    if (!h || !t) return fail(ASYNCMESH_ERR_INVALID_ARG, "step_count: NULL argument");
    *t = h->t;
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_kernel_name(const asyncmesh *h, char *buf, size_t cap)
{
    if (!h || !buf || cap == 0) return fail(ASYNCMESH_ERR_INVALID_ARG, "kernel_name: NULL argument");
    const char *mode = h->mode == kSync ? "sync" : h->mode == kDense ? "dense" : h->mode == kDenseBf16 ? "dense-bf16"
                       : h->mode == kDenseE4m3 ? "dense-e4m3" : "compact";
    const char *form = h->general ? " general" : h->tracking ? " tracking" : h->nadam_form ? " nadamw" : "";
    switch (h->pipelined) {
    case 0: snprintf(buf, cap, "direct R=%u %s%s", h->R, mode, form); break;
    case 1: snprintf(buf, cap, "pipelined R=%u %s wide%s", h->R, mode, form); break;
    case 2: case 3: snprintf(buf, cap, "pipelined R=%u %s narrow%s", h->R, mode, form); break;
    case 4: snprintf(buf, cap, "owner R=%u %s entries=%d%s", h->R, mode, kOwnerEntriesFew, form); break;
    case 5: snprintf(buf, cap, "owner R=%u %s entries=%d%s", h->R, mode, kOwnerEntriesMany, form); break;
    case 7: snprintf(buf, cap, "owner R=%u %s entries=%d%s", h->R, mode, kOwnerEntriesMid, form); break;
    default: snprintf(buf, cap, "owner R=%u %s%s", h->R, mode, form);
    }
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_min_bytes_last_step(const asyncmesh *h, uint64_t *bytes)
{
    if (!h || !bytes) return fail(ASYNCMESH_ERR_INVALID_ARG, "min_bytes_last_step: NULL argument");
    *bytes = h->last_bytes;
    return ASYNCMESH_OK;
}

extern "C" int asyncmesh_debug_philox(int device, const uint32_t *ctr_host, const uint32_t *key_host,
                                      uint32_t *out_host, uint64_t n)
{
    if (!ctr_host || !key_host || !out_host) return fail(ASYNCMESH_ERR_INVALID_ARG, "debug_philox: NULL argument");
    if (n == 0) return ASYNCMESH_OK;
    DeviceScope scope(device);
    if (!scope.ok) return fail(ASYNCMESH_ERR_CUDA, "debug_philox: cudaSetDevice(%d) failed", device);
    uint32_t *c = nullptr, *k = nullptr, *o = nullptr;
    cudaError_t e = cudaMalloc(&c, n * 16);
    if (e == cudaSuccess) e = cudaMalloc(&k, n * 8);
    if (e == cudaSuccess) e = cudaMalloc(&o, n * 16);
    if (e == cudaSuccess) e = cudaMemcpy(c, ctr_host, n * 16, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(k, key_host, n * 8, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) {
        philox_debug_kernel<<<grid_for(n, 256), 256>>>(c, k, o, n);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpy(out_host, o, n * 16, cudaMemcpyDeviceToHost);
    cudaFree(c); cudaFree(k); cudaFree(o);
    if (e != cudaSuccess) return fail(ASYNCMESH_ERR_CUDA, "debug_philox: %s", cudaGetErrorString(e));
    return ASYNCMESH_OK;
}


// ---------------------------------------------------------------------------
// consensus error without any allocation
// ---------------------------------------------------------------------------
//
// Some callers cannot take an entry point that allocates: a host that has handed
// all of the GPU's memory to its own pool (a raw cudaMalloc would fail or eat
// into a reserve it does not own), a control loop that must not hit the
// device-wide synchronisation an allocation can cause, a monitoring hook that
// runs where the process is not allowed to grow.  For them the reduction's
// scratch lives in the library image itself: a fixed array in device memory that
// every GPU holds from the moment it loads the library until the process exits.

constexpr uint32_t kNoAllocTile = 1u << 16;        // coordinates one block reduces
constexpr uint32_t kNoAllocMaxBlocks = 4096;       // => at most 2^28 coordinates per call
constexpr uint64_t kNoAllocMaxCoords = (uint64_t)kNoAllocTile * kNoAllocMaxBlocks;

// per-block partial sums, then the total in the last slot (33 KB per GPU)
static __device__ __align__(256) double g_noalloc_scratch[kNoAllocMaxBlocks + 1];

// In host code `g_noalloc_scratch` is only a stand-in for the device array; the
// address kernels may use is looked up once per device and kept here.
static double *g_noalloc_ptr[64] = {nullptr};

__global__ void consensus_partial_kernel(const float *W, uint32_t R, uint64_t stride, uint64_t N,
                                         double *partial)
{
    const uint64_t begin = (uint64_t)blockIdx.x * kNoAllocTile;
    const uint64_t end = begin + kNoAllocTile < N ? begin + kNoAllocTile : N;
    double acc = 0.0;
    for (uint64_t mu = begin + threadIdx.x; mu < end; mu += blockDim.x) {
        double mean = 0.0;
        for (uint32_t i = 0; i < R; ++i) mean += (double)W[(uint64_t)i * stride + mu];
        mean /= (double)R;
        for (uint32_t i = 0; i < R; ++i) {
            const double e = (double)W[(uint64_t)i * stride + mu] - mean;
            acc += e * e;
        }
    }
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
    __shared__ double part[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) part[warp] = acc;
    __syncthreads();
    if (warp == 0) {
        acc = lane < (int)(blockDim.x >> 5) ? part[lane] : 0.0;
        for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
        if (lane == 0) partial[blockIdx.x] = acc;   // every slot in use is overwritten: no clearing needed
    }
}

__global__ void consensus_final_kernel(const double *partial, uint32_t n, double *total)
{
    double acc = 0.0;
    for (uint32_t k = threadIdx.x; k < n; k += blockDim.x) acc += partial[k];
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
    __shared__ double part[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) part[warp] = acc;
    __syncthreads();
    if (warp == 0) {
        acc = lane < (int)(blockDim.x >> 5) ? part[lane] : 0.0;
        for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(0xFFFFFFFFu, acc, d);
        if (lane == 0) *total = acc;
    }
}

extern "C" int asyncmesh_consensus_error_noalloc(int device, void *stream, const float *w_device,
                                                 uint32_t R, uint64_t n, uint64_t row_stride,
                                                 double *out_host)
{
    if (!w_device || !out_host)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "consensus_error_noalloc: NULL argument");
    if (R < 1 || n < 1 || row_stride < n)
        return fail(ASYNCMESH_ERR_INVALID_ARG,
                    "consensus_error_noalloc: need R >= 1, n >= 1, row_stride >= n");
    if (n > kNoAllocMaxCoords)
        return fail(ASYNCMESH_ERR_INVALID_ARG,
                    "consensus_error_noalloc: n = %llu exceeds the built-in scratch (at most %llu "
                    "coordinates per call; split the rows and add the results)",
                    (unsigned long long)n, (unsigned long long)kNoAllocMaxCoords);
    if (device < 0 || device >= 64)
        return fail(ASYNCMESH_ERR_INVALID_ARG, "consensus_error_noalloc: device %d outside 0..63", device);
    DeviceScope scope(device);
    if (!scope.ok) return fail(ASYNCMESH_ERR_CUDA, "consensus_error_noalloc: cudaSetDevice(%d) failed", device);
    if (!g_noalloc_ptr[device]) {   // first call on this device: find the array's device address
        double *ptr = nullptr;
        CU_TRY(cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch));
        g_noalloc_ptr[device] = ptr;
    }
    double *scratch = g_noalloc_ptr[device];
    const uint32_t blocks = (uint32_t)((n + kNoAllocTile - 1) / kNoAllocTile);
    cudaStream_t st = (cudaStream_t)stream;
    consensus_partial_kernel<<<blocks, 256, 0, st>>>(w_device, R, row_stride, n, scratch);
    CU_TRY(cudaGetLastError());
    consensus_final_kernel<<<1, 256, 0, st>>>(scratch, blocks, scratch + kNoAllocMaxBlocks);
    CU_TRY(cudaGetLastError());
    CU_TRY(cudaMemcpyAsync(out_host, scratch + kNoAllocMaxBlocks, sizeof(double),
                           cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    return ASYNCMESH_OK;
}
