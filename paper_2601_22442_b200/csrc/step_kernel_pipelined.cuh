// Pipelined variant of the fused step for the compact snapshot ring (the
// paper's main regime: a small subset, tau >= 1).  Same results as the direct
// kernel of step_kernel.cuh, bit for bit; different data movement:
//
//  * Dense streams.  A warp walks its chunk in sub-iterations of V x 128
//    coordinates; per sub-iteration and replica it needs w, g, m, v as V float4
//    per lane and array (one "unit", V x 2 KB).  Units are fetched with
//    per-thread 16-byte asynchronous copies (cp.async) into a ring of shared-
//    memory stages private to the warp, ahead of the arithmetic.  A lane reads
//    back only what it copied itself, so the pipeline needs no barrier, only
//    cp.async.wait_group; the bytes in flight per SM are set by the stage count,
//    not by registers or occupancy.  With V = 2 a lane carries eight independent
//    coordinates through the optimizer arithmetic, which is what keeps the issue
//    slots busy between the long IEEE divide / square-root sequences.
//  * Sparse work is compacted across the warp.  The selected coordinates of a
//    sub-iteration (union of S^t and S^{t-tau}, ~25 of 256 at p = 0.05) are
//    ranked with a warp scan; while the dense arithmetic runs, the owning lanes
//    drop the values those coordinates need (w^ and w^{t-1} per replica) into a
//    small shared-memory stash; afterwards lane q finishes the q-th selected
//    coordinate for all replicas with vector accesses to the ring and to d.
//    (With 5 to 8 replicas the wide shape skips the value stash: the finishing
//    lane reads w^{t-1} from the w rows before they are written and w^ from
//    them afterwards.)
//    Its ring and d loads are issued before the dense arithmetic starts, so
//    their latency hides behind it.  Coordinates beyond the stash capacity
//    (possible only for large p) are handled in place by their owning lane.
//
// Bulk copies (cp.async.bulk with an mbarrier per stage, one lane issuing four
// 1 KB copies per unit) were measured in place of the per-thread copies: 24.4 ms
// against 24.0 ms per step on the 1B workload in the same run; the warp-wide
// hand-over they need costs more than the issue slots they save, so the
// per-thread form stays.
#pragma once
#include <type_traits>

#include "step_kernel.cuh"

namespace amk {

constexpr int kPipeThreads = 128;   // 4 warps per block
constexpr int kPipeBlocksPerSM = 3; // at most: 12 warps per SM.  Measured on the 1B layout: 10 warps 24.9 ms,
                                    // 12 warps 23.6, 14 warps 23.9, 18 warps 25.9; with 8 replicas the wide
                                    // shape takes more registers than three blocks leave and runs 8 warps
                                    // (350M layout 15.8 ms against 16.3 for 12 warps held to 156 registers)
constexpr int kPipeStages = 3;      // units in the shared-memory ring of a warp

// Two shapes of the same kernel.  Wide: 8 coordinates per lane and unit, stash
// for 64 selected coordinates per 256: the small subsets the paper works with.
// Narrow: 4 coordinates per lane and unit, stash for all 128 coordinates of a
// sub-iteration: any larger subset (until the dense ring takes over).
template <int V_, int CAP_>
struct PipeShape {
    static constexpr int V = V_;                        // float4 per lane, array and unit
    static constexpr int CAP = CAP_;                    // selected coordinates a sub-iteration can stash
    static constexpr int kSubCoords = 128 * V;          // coordinates per sub-iteration
    static constexpr int kSubIters = kWarpChunk / kSubCoords;
    static constexpr int kBits = 4 * V;                 // mask bits per lane and sub-iteration
    static constexpr int kUnitBytes = 4 * V * 512;      // w, g, m, v: V float4 per lane each
    static_assert(kSubIters * kBits == 32, "a lane's chunk mask must fill 32 bits");
};
using PipeWide = PipeShape<2, 64>;
using PipeNarrow = PipeShape<1, 128>;

__device__ __forceinline__ void cp_async16(uint32_t smem_addr, const void *gptr)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_addr), "l"(gptr)
                 : "memory");
}
__device__ __forceinline__ void st_keep(float *p, const float (&x)[4])
{
    __stcg(reinterpret_cast<float4 *>(p), make_float4(x[0], x[1], x[2], x[3]));
}
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;\n" ::: "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}

// 32 bytes to a 32-byte aligned address in one request
__device__ __forceinline__ void st_sector(float *p, const float (&x)[8])
{
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]),
                 "f"(x[3]), "f"(x[4]), "f"(x[5]), "f"(x[6]), "f"(x[7])
                 : "memory");
}

template <int R>
__device__ __forceinline__ void store_replicas(float *p, const float (&x)[R])
{
    if constexpr (R % 8 == 0) {   // whole 32-byte sectors (entries of 8 replicas are 32-byte aligned)
#pragma unroll
        for (int q = 0; q < R / 8; ++q) {
            const float s8[8] = {x[8 * q], x[8 * q + 1], x[8 * q + 2], x[8 * q + 3],
                                 x[8 * q + 4], x[8 * q + 5], x[8 * q + 6], x[8 * q + 7]};
            st_sector(p + 8 * q, s8);
        }
    } else if constexpr (R % 4 == 0) {
#pragma unroll
        for (int q = 0; q < R / 4; ++q)
            *reinterpret_cast<float4 *>(p + 4 * q) =
                make_float4(x[4 * q], x[4 * q + 1], x[4 * q + 2], x[4 * q + 3]);
    } else if constexpr (R % 2 == 0) {
#pragma unroll
        for (int q = 0; q < R / 2; ++q)
            *reinterpret_cast<float2 *>(p + 2 * q) = make_float2(x[2 * q], x[2 * q + 1]);
    } else {
#pragma unroll
        for (int i = 0; i < R; ++i) p[i] = x[i];
    }
}

template <int R, class SH>
struct PipeCfg {
    static constexpr int kStash = SH::CAP;
    static constexpr int kStashWords = kStash * (2 * R + 3);   // what, wold, coord, cidx, pidx
    static constexpr int kStashBytes = (kStashWords * 4 + 15) / 16 * 16;
    __host__ __device__ static constexpr int warp_bytes(int stages)
    {
        return stages * SH::kUnitBytes + kStashBytes;
    }
};

// Dynamic shared memory: the stage table (S entries), then one region per warp.
__host__ __device__ constexpr int pipe_table_bytes(uint32_t S)
{
    // a multiple of 128 bytes: the warps' copy stages behind it then start on a 128-byte
    // boundary, and a warp's 512-byte rows of 16-byte copies fall into whole shared-memory lines
    return (int)((S * sizeof(StageDesc) + 127) / 128 * 128);
}

template <class SH>
__device__ __forceinline__ int pipe_sub_iterations(uint64_t N, uint32_t chunk)
{
    const uint64_t rem = N - (uint64_t)chunk * kWarpChunk;
    return rem >= (uint64_t)kWarpChunk ? SH::kSubIters
                                       : (int)((rem + SH::kSubCoords - 1) / SH::kSubCoords);
}

// Walks the warp's units in the order the arithmetic consumes them (chunk by
// grid stride -> sub-iteration k -> replica i) and issues their copies.  The
// stage's pointers live in registers and are refreshed when the chunk changes.
struct UnitCursor {
    const float *W, *G, *M, *V;   // of the current stage
    uint64_t N, stride;
    uint64_t mu0;                 // first coordinate of this lane in the current sub-iteration
    uint32_t gc, s;
    int k, i, kmax;
    bool valid;
};

template <class SH>
__device__ __forceinline__ void cursor_enter_chunk(UnitCursor &c, const StepParams &P,
                                                   const StageDesc *sd, int lane)
{
    c.valid = c.gc < P.total_chunks;
    if (!c.valid) return;
    while (c.s + 1 < P.S && c.gc >= sd[c.s + 1].chunk_begin) ++c.s;
    const StageDesc &st = sd[c.s];
    const uint32_t chunk = c.gc - st.chunk_begin;
    c.W = st.W; c.M = st.M; c.V = st.V; c.G = P.G[c.s];
    c.N = st.N; c.stride = st.stride;
    c.kmax = pipe_sub_iterations<SH>(st.N, chunk);
    c.k = 0;
    c.i = 0;
    c.mu0 = (uint64_t)chunk * kWarpChunk + (uint64_t)lane * 4;
}

template <int R, class SH>
__device__ __forceinline__ void issue_unit(UnitCursor &c, const StepParams &P, const StageDesc *sd,
                                           uint32_t slot_addr, int lane, uint32_t n_warps)
{
    if (c.valid) {
        const uint32_t a = slot_addr + lane * 16;
#pragma unroll
        for (int h = 0; h < SH::V; ++h) {
            const uint64_t mu = c.mu0 + (uint64_t)h * 128;
            if (mu < c.N) {
                const uint64_t off = (uint64_t)c.i * c.stride + mu;
                cp_async16(a + (0 * SH::V + h) * 512, c.W + off);
                cp_async16(a + (1 * SH::V + h) * 512, c.G + off);
                cp_async16(a + (2 * SH::V + h) * 512, c.M + off);
                cp_async16(a + (3 * SH::V + h) * 512, c.V + off);
            }
        }
        if (++c.i == R) {
            c.i = 0;
            c.mu0 += SH::kSubCoords;
            if (++c.k == c.kmax) {
                c.gc += n_warps;
                cursor_enter_chunk<SH>(c, P, sd, lane);
            }
        }
    }
    cp_async_commit();   // always: keeps the group count in step with the unit count
}

// GEN: the general form of the sparse arithmetic (see on_wire), a separate set of
// instantiations.
// MODE is kCompact (tau >= 1: ring, d, bitmap) or kSync (tau = 0, Eq. "sparta": the
// replica mean of the selected coordinates is formed from the stash itself; needs
// a stash that holds a whole sub-iteration, i.e. the narrow shape).
template <int R, int NST, class SH, int MODE, bool GEN>
__global__ void __launch_bounds__(kPipeThreads, 2)
asyncmesh_step_kernel_pipelined(const __grid_constant__ StepParams P)
{
    static_assert(MODE == kCompact || (MODE == kSync && SH::CAP >= SH::kSubCoords),
                  "the synchronous mode cannot fall back to in-place work");
    using Cfg = PipeCfg<R, SH>;
    constexpr int CAP = Cfg::kStash;
    constexpr int V = SH::V;
    constexpr int NB = SH::kBits;   // mask bits per lane and sub-iteration
    constexpr int kUnitBytes = SH::kUnitBytes;
    constexpr int kPipeSubCoords = SH::kSubCoords;
    // Wide shape, 5 to 8 replicas: the sparse phase takes w^ back from the w row the dense
    // phase has just written (an L2 hit) and w^{t-1} from the same row before it is
    // written, instead of from the stash that predicated stores in the dense loop fill.
    // Measured on the 350M layout (R = 8): 16.5 against 17.1 ms per step at p = 0.05, 15.86
    // against 15.77 at p = 0.01; no difference at R = 4 (1B layout); beyond 8 replicas the
    // registers for w^{t-1} (CAP / 32 entries per lane) are not there.
    constexpr bool kReload = (MODE == kCompact) && R > 4 && R <= 8 && CAP <= 64;
    constexpr int kRounds = (CAP + 31) / 32;
    // rounds of the sparse phase whose ring and d loads go out before the dense loop; the
    // narrow shape serves subsets for which a second round is the rule, not the exception
    // (1B layout, R = 4, p = 0.25: 31.1 -> 29.9 ms; with 8 replicas the registers this
    // takes cost more than it saves: 20.4 -> 21.1 ms on the 350M layout)
    constexpr int kPre = (V == 1 && MODE == kCompact && R <= 4) ? 2 : 1;
    extern __shared__ __align__(16) unsigned char dyn_smem_all[];
    StageDesc *sd = reinterpret_cast<StageDesc *>(dyn_smem_all);
    unsigned char *dyn_smem = dyn_smem_all + pipe_table_bytes(P.S);
    {
        const uint32_t words = P.S * (uint32_t)(sizeof(StageDesc) / 4);
        const uint32_t *src = reinterpret_cast<const uint32_t *>(P.stages);
        uint32_t *dst = reinterpret_cast<uint32_t *>(sd);
        for (uint32_t x = threadIdx.x; x < words; x += blockDim.x) dst[x] = src[x];
    }
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    constexpr uint32_t wpb = kPipeThreads / 32;
    const uint32_t n_warps = gridDim.x * wpb;

    unsigned char *my = dyn_smem + (size_t)warp * Cfg::warp_bytes(NST);
    const uint32_t stage_base = (uint32_t)__cvta_generic_to_shared(my);
    // stash of the current sub-iteration's selected coordinates
    float *st_what = reinterpret_cast<float *>(my + NST * kUnitBytes);   // [CAP][R]
    float *st_wold = st_what + CAP * R;                                  // [CAP][R]
    uint32_t *st_coord = reinterpret_cast<uint32_t *>(st_wold + CAP * R);
    uint32_t *st_cidx = st_coord + CAP;
    uint32_t *st_pidx = st_cidx + CAP;

    // ---- start the copy pipeline: NST - 1 units ahead --------------------------
    UnitCursor pf;
    pf.gc = blockIdx.x * wpb + warp;
    pf.s = 0;
    cursor_enter_chunk<SH>(pf, P, sd, lane);
#pragma unroll
    for (int q = 0; q < NST - 1; ++q)
        issue_unit<R, SH>(pf, P, sd, stage_base + q * kUnitBytes, lane, n_warps);
    uint32_t rd = 0, wr = NST - 1;   // ring slot being consumed / being filled

    const bool consume = (MODE == kCompact) && P.consume != 0u;
    uint32_t s = 0;
    for (uint32_t gc = blockIdx.x * wpb + warp; gc < P.total_chunks; gc += n_warps) {
        while (s + 1 < P.S && gc >= sd[s + 1].chunk_begin) ++s;
        const StageDesc &st = sd[s];
        const uint32_t chunk = gc - st.chunk_begin;
        const uint64_t N = st.N, stride = st.stride;
        const uint64_t c0 = (uint64_t)chunk * kWarpChunk + (uint64_t)lane * 4;
        const int kmax = pipe_sub_iterations<SH>(N, chunk);

        // position of this chunk in the consumed slot and the membership mask stored
        // when that slot was produced: ask early, use late
        uint32_t cbase = 0, cmask = 0;
        const uint64_t word = (uint64_t)chunk * 32 + lane;
        if (consume) {
            cbase = st.chunk_base[(uint64_t)P.cons_slot * st.n_chunks + chunk];
            cmask = st.bitmap[(uint64_t)P.cons_slot * st.n_chunks * 32 + word];
        }

        // ---- membership of this lane's 32 coordinates in S^t (S^{t-tau} was read
        // above: the generator runs once per coordinate and step) ----
        // bit 4b + c  <->  coordinate c0 + 128 b + c; sub-iteration k owns bits NB*k ..
        uint32_t pmask = 0;
        const uint32_t quad0 = st.quad_base + (uint32_t)(c0 >> 2);   // global index / 4 of the lane's first quad
#pragma unroll 2
        for (int b = 0; b < 8; ++b) {   // 8 quads per lane and chunk
            const uint64_t mu = c0 + (uint64_t)b * 128;
            if (mu < N) {
                const uint64_t left = N - mu;
                const uint32_t valid = left >= 4 ? 0xFu : ((1u << (uint32_t)left) - 1u);
                const uint32_t quad = quad0 + (uint32_t)b * 32u;
                if (P.produce)
                    pmask |= (subset_bits(P.rule, st.stage_id, P.step, quad) & valid) << (4 * b);
            }
        }

        // ---- room in the producing slot -----------------------------------------
        uint32_t pbase = 0, cexcl = 0, pexcl = 0;
        if constexpr (MODE == kCompact) {
        uint32_t total;
        pexcl = warp_exclusive_sum(__popc(pmask), lane, total);
        if (lane == 0) {
            uint32_t b = 0;
            if (total) {
                b = atomicAdd(&P.cursors[P.prod_slot * P.cursor_S + P.s_base + s], total);
                if (b > st.cap || total > st.cap - b) {   // slot full: drop loudly
                    b = kInvalidBase;
                    atomicExch(P.status, kStatusRingOverflow);
                }
            }
            if (P.produce) st.chunk_base[(uint64_t)P.prod_slot * st.n_chunks + chunk] = b;
            pbase = b;
        }
        if (consume) {
            if (cbase == kInvalidBase) cmask = 0;
            uint32_t ctotal;
            cexcl = warp_exclusive_sum(__popc(cmask), lane, ctotal);
        }
        pbase = __shfl_sync(kFullMask, pbase, 0);
        if (pbase == kInvalidBase) pmask = 0;
        if (P.produce)   // kept for step t + tau
            st.bitmap[(uint64_t)P.prod_slot * st.n_chunks * 32 + word] = pmask;
        }
        const float *ring_cons = st.ring + (uint64_t)P.cons_slot * st.slot_floats;
        float *ring_prod = st.ring + (uint64_t)P.prod_slot * st.slot_floats;
        const float delta = st.delta;
        const bool has_look = st.delta != 0.0f;

#pragma unroll 1
        for (int k = 0; k < kmax; ++k) {
            const uint64_t mu0 = c0 + (uint64_t)k * kPipeSubCoords;   // h = 0; h adds 128
            constexpr uint32_t kSubMask = (NB == 32) ? 0xFFFFFFFFu : ((1u << (NB % 32)) - 1u);
            const uint32_t lowbits = (k == 0) ? 0u : ((1u << ((NB * k) % 32)) - 1u);
            const uint32_t pm = (pmask >> (NB * k)) & kSubMask;
            const uint32_t cm = (cmask >> (NB * k)) & kSubMask;
            const uint32_t um = pm | cm;

            // ---- rank the selected coordinates of this sub-iteration ------------
            uint32_t n_u;
            const uint32_t uexcl = warp_exclusive_sum(__popc(um), lane, n_u);
            const uint32_t cfirst = cbase + cexcl + __popc(cmask & lowbits);
            const uint32_t pfirst = pbase + pexcl + __popc(pmask & lowbits);
            uint32_t sm = 0;   // bits of um that fit the stash
            if (um) {
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    if ((um >> j) & 1u) {
                        const uint32_t below = (1u << j) - 1u;
                        const uint32_t r = uexcl + __popc(um & below);
                        if (r < (uint32_t)CAP) {
                            sm |= 1u << j;
                            st_coord[r] = (uint32_t)(mu0 + (uint64_t)(j >> 2) * 128 + (j & 3));
                            st_cidx[r] = ((cm >> j) & 1u) ? cfirst + __popc(cm & below) : kInvalidBase;
                            st_pidx[r] = ((pm >> j) & 1u) ? pfirst + __popc(pm & below) : kInvalidBase;
                        }
                    }
                }
            }
            const uint32_t om = um & ~sm;   // handled in place (only when the stash is full)
            __syncwarp();

            // ---- lane q adopts the q-th selected coordinate; its loads go out now
            const uint32_t n_s = n_u < (uint32_t)CAP ? n_u : (uint32_t)CAP;
            uint32_t e_coord = 0, e_c = kInvalidBase, e_p = kInvalidBase;
            float s_old[R], s_dd[R];
#pragma unroll
            for (int i = 0; i < R; ++i) { s_old[i] = 0.f; s_dd[i] = 0.f; }
            if ((uint32_t)lane < n_s) {
                e_coord = st_coord[lane];
                e_c = st_cidx[lane];
                e_p = st_pidx[lane];
                if (e_c != kInvalidBase) {
                    load_replicas<R>(ring_cons + (uint64_t)e_c * R, s_old);
                    load_replicas<R>(st.D + (uint64_t)e_coord * R, s_dd);
                }
            }
            // a second entry per lane when the subset is large
            uint32_t e1_coord = 0, e1_c = kInvalidBase, e1_p = kInvalidBase;
            float s1_old[kPre > 1 ? R : 1], s1_dd[kPre > 1 ? R : 1];
            if constexpr (kPre > 1) {
#pragma unroll
                for (int i = 0; i < R; ++i) { s1_old[i] = 0.f; s1_dd[i] = 0.f; }
                if (32u + (uint32_t)lane < n_s) {
                    e1_coord = st_coord[32 + lane];
                    e1_c = st_cidx[32 + lane];
                    e1_p = st_pidx[32 + lane];
                    if (e1_c != kInvalidBase) {
                        load_replicas<R>(ring_cons + (uint64_t)e1_c * R, s1_old);
                        load_replicas<R>(st.D + (uint64_t)e1_coord * R, s1_dd);
                    }
                }
            }
            // w^{t-1} of the adopted entries (only consumed ones need it), straight from
            // the w rows, which still hold it at this point
            float wprev[kReload ? kRounds : 1][R];
            if constexpr (kReload) {
#pragma unroll
                for (int rr = 0; rr < kRounds; ++rr) {
                    const uint32_t q = rr * 32 + lane;
#pragma unroll
                    for (int i = 0; i < R; ++i) wprev[rr][i] = 0.f;
                    if (q < n_s && (rr == 0 || n_s > 32u)) {
                        const uint32_t cc = rr == 0 ? e_coord : st_coord[q];
                        const uint32_t ci = rr == 0 ? e_c : st_cidx[q];
                        if (ci != kInvalidBase) {
#pragma unroll
                            for (int i = 0; i < R; ++i)
                                wprev[rr][i] = __ldcg(st.W + (uint64_t)i * stride + cc);
                        }
                    }
                }
                // every lane has read w^{t-1} of the coordinate it adopted (another lane's)
                // before any lane overwrites that row in the dense loop below
                __syncwarp();
            }

            // ---- dense arithmetic, one replica (= one pipeline unit) at a time ----
            // (unrolled only for few replicas: beyond that the loop body no longer
            // fits the instruction cache and fetch stalls cost more than the
            // loop overhead saves)
            // Two copies of the loop: the one that runs (no selected coordinate beyond the
            // stash) carries no code for the in-place work, which otherwise sits, never
            // executed, in the middle of the hottest instructions.
            auto dense = [&](auto in_place_tag) {
            constexpr bool kInPlace = decltype(in_place_tag)::value;
            constexpr int kUnroll = R <= 4 ? R : 1;
#pragma unroll(kUnroll)
            for (int i = 0; i < R; ++i) {
                cp_async_wait<NST - 2>();
                issue_unit<R, SH>(pf, P, sd, stage_base + wr * kUnitBytes, lane, n_warps);
                const unsigned char *slot = my + rd * kUnitBytes + lane * 16;
                rd = (rd + 1 == NST) ? 0 : rd + 1;
                wr = (wr + 1 == NST) ? 0 : wr + 1;
                // (lanes past the end of the stage compute on whatever their slot
                // holds: nothing of it is stored, stashed or selected)
                float wn[V * 4], wo[V * 4];
                {
                    float g[V * 4], m[V * 4], v[V * 4];
#pragma unroll
                    for (int h = 0; h < V; ++h) {
                        const float4 w4 = *reinterpret_cast<const float4 *>(slot + (0 * V + h) * 512);
                        const float4 g4 = *reinterpret_cast<const float4 *>(slot + (1 * V + h) * 512);
                        const float4 m4 = *reinterpret_cast<const float4 *>(slot + (2 * V + h) * 512);
                        const float4 v4 = *reinterpret_cast<const float4 *>(slot + (3 * V + h) * 512);
                        wo[4 * h] = w4.x; wo[4 * h + 1] = w4.y; wo[4 * h + 2] = w4.z; wo[4 * h + 3] = w4.w;
                        g[4 * h] = g4.x; g[4 * h + 1] = g4.y; g[4 * h + 2] = g4.z; g[4 * h + 3] = g4.w;
                        m[4 * h] = m4.x; m[4 * h + 1] = m4.y; m[4 * h + 2] = m4.z; m[4 * h + 3] = m4.w;
                        v[4 * h] = v4.x; v[4 * h + 1] = v4.y; v[4 * h + 2] = v4.z; v[4 * h + 3] = v4.w;
                    }
                    adamw_group<GEN, V * 4>(P, wo, g, m, v, wn);
#pragma unroll
                    for (int h = 0; h < V; ++h) {
                        const uint64_t mu = mu0 + (uint64_t)h * 128;
                        if (mu < N) {
                            const uint64_t off = (uint64_t)i * stride + mu;
                            __stcs(reinterpret_cast<float4 *>(st.M + off),
                                   make_float4(m[4 * h], m[4 * h + 1], m[4 * h + 2], m[4 * h + 3]));
                            __stcs(reinterpret_cast<float4 *>(st.V + off),
                                   make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]));
                        }
                    }
                }

                if (!kReload && sm) {   // hand w^ and w^{t-1} of selected coordinates to the stash
#pragma unroll
                    for (int j = 0; j < NB; ++j) {
                        if ((sm >> j) & 1u) {
                            const uint32_t r = uexcl + __popc(um & ((1u << j) - 1u));
                            st_what[r * R + i] = wn[j];
                            st_wold[r * R + i] = wo[j];
                        }
                    }
                }
                if (kInPlace && om) {   // stash full: this lane does the sparse work itself
#pragma unroll
                    for (int j = 0; j < NB; ++j) {
                        if ((om >> j) & 1u) {
                            const uint32_t below = (1u << j) - 1u;
                            const float whj = wn[j];
                            if ((cm >> j) & 1u) {
                                const uint64_t ce = (uint64_t)(cfirst + __popc(cm & below)) * R;
                                float old[R];
                                load_replicas<R>(ring_cons + ce, old);
                                float a = on_wire<GEN>(P, old[0]);
#pragma unroll
                                for (int q = 1; q < R; ++q) a = __fadd_rn(a, on_wire<GEN>(P, old[q]));
                                const float abar = __fdiv_rn(a, P.Rf);
                                float *dp = st.D + (mu0 + (uint64_t)(j >> 2) * 128 + (j & 3)) * R + i;
                                float old_i = old[0];
#pragma unroll
                                for (int q = 1; q < R; ++q) old_i = (q == i) ? old[q] : old_i;
                                const float diff = __fsub_rn(whj, old_i);
                                const float dn = staleness<GEN>(P, *dp, diff);
                                *dp = dn;
                                wn[j] = __fadd_rn(abar, dn);
                            }
                            if ((pm >> j) & 1u)
                                ring_prod[(uint64_t)(pfirst + __popc(pm & below)) * R + i] = whj;
                        }
                    }
                }

#pragma unroll
                for (int h = 0; h < V; ++h) {
                    const uint64_t mu = mu0 + (uint64_t)h * 128;
                    if (mu < N) {
                        const uint64_t off = (uint64_t)i * stride + mu;
                        // w and the look-ahead stay in L2 with normal priority: the few
                        // selected coordinates of these lines are patched a moment later
                        __stcg(reinterpret_cast<float4 *>(st.W + off),
                               make_float4(wn[4 * h], wn[4 * h + 1], wn[4 * h + 2], wn[4 * h + 3]));
                        if (has_look) {   // Section 2.2: extrapolate the last update direction
                            float lk[4];
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                lk[c] = __fadd_rn(wn[4 * h + c],
                                                  __fmul_rn(delta, __fsub_rn(wn[4 * h + c], wo[4 * h + c])));
                            st_keep(st.LOOK + off, lk);
                        }
                    }
                }
            }
            };
            if (CAP < kPipeSubCoords && n_u > (uint32_t)CAP) dense(std::true_type{});
            else dense(std::false_type{});
            __syncwarp();   // stash complete; dense stores ordered before the fix-ups below

            // ---- sparse phase: lane q finishes the q-th selected coordinate -------
#pragma unroll
            for (int rr = 0; rr < kRounds; ++rr) {
                const uint32_t r0 = rr * 32;
                if (r0 >= n_s) break;
                const uint32_t q = r0 + lane;
                if (q < n_s) {
                    if (kPre > 1 && rr == 1) {   // second round: asked for ahead as well
                        e_coord = e1_coord;
                        e_c = e1_c;
                        e_p = e1_p;
#pragma unroll
                        for (int i = 0; i < R; ++i) { s_old[i] = s1_old[i]; s_dd[i] = s1_dd[i]; }
                    } else if (r0 != 0) {   // later rounds: loads were not issued ahead
                        e_coord = st_coord[q];
                        e_c = st_cidx[q];
                        e_p = st_pidx[q];
                        if (e_c != kInvalidBase) {
                            load_replicas<R>(ring_cons + (uint64_t)e_c * R, s_old);
                            load_replicas<R>(st.D + (uint64_t)e_coord * R, s_dd);
                        }
                    }
                    float wh[R];
                    if constexpr (kReload) {
#pragma unroll
                        for (int i = 0; i < R; ++i) wh[i] = __ldcg(st.W + (uint64_t)i * stride + e_coord);
                    } else {
                        load_replicas<R>(st_what + q * R, wh);
                    }
                    if constexpr (MODE == kSync) {
                        // Eq. "sparta": the selected coordinate takes the replica mean; the
                        // EMA state stays exactly zero (its sample is w^ - w^), hence mean + 0
                        float wold[R];
                        load_replicas<R>(st_wold + q * R, wold);
                        float a = on_wire<GEN>(P, wh[0]);
#pragma unroll
                        for (int i = 1; i < R; ++i) a = __fadd_rn(a, on_wire<GEN>(P, wh[i]));
                        const float wnew = __fadd_rn(__fdiv_rn(a, P.Rf), 0.0f);
#pragma unroll
                        for (int i = 0; i < R; ++i) {
                            const uint64_t o1 = (uint64_t)i * stride + e_coord;
                            st.W[o1] = wnew;
                            if (has_look)
                                st.LOOK[o1] = __fadd_rn(wnew, __fmul_rn(delta, __fsub_rn(wnew, wold[i])));
                        }
                    } else if (e_c != kInvalidBase) {
                        // Eq. "ema" + corrected averaging on S^{t-tau}
                        float wold[R];
                        if constexpr (kReload) {
#pragma unroll
                            for (int i = 0; i < R; ++i) wold[i] = wprev[rr][i];
                        } else {
                            load_replicas<R>(st_wold + q * R, wold);
                        }
                        float a = on_wire<GEN>(P, s_old[0]);
#pragma unroll
                        for (int i = 1; i < R; ++i) a = __fadd_rn(a, on_wire<GEN>(P, s_old[i]));
                        const float abar = __fdiv_rn(a, P.Rf);
#pragma unroll
                        for (int i = 0; i < R; ++i) {
                            const float diff = __fsub_rn(wh[i], s_old[i]);
                            const float dn = staleness<GEN>(P, s_dd[i], diff);
                            s_dd[i] = dn;
                            const float wnew = __fadd_rn(abar, dn);
                            const uint64_t o1 = (uint64_t)i * stride + e_coord;
                            st.W[o1] = wnew;
                            if (has_look)
                                st.LOOK[o1] = __fadd_rn(wnew, __fmul_rn(delta, __fsub_rn(wnew, wold[i])));
                        }
                        store_replicas<R>(st.D + (uint64_t)e_coord * R, s_dd);
                    }
                    if (MODE == kCompact && e_p != kInvalidBase)   // snapshot of the local iterate on S^t
                        store_replicas<R>(ring_prod + (uint64_t)e_p * R, wh);
                }
            }
            __syncwarp();   // the stash may be overwritten by the next sub-iteration
        }
    }
    cp_async_wait<0>();
}

}  // namespace amk
