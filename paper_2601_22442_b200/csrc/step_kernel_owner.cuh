// Third form of the fused step, for few replicas (up to four; up to eight for tau = 0; six and
// eight with the ring as two passes of three and four, see NH below):
// the lane that owns a coordinate does all of its work, sparse part included, and
// nothing is handed from lane to lane.  Same results as the other two kernels, bit
// for bit.
//
//  * A lane owns 4 V coordinates of a group of 128 V (V float4 per array row) and
//    keeps the R replica values of each in registers: the stale replica average
//    (Eq. "asparta"), the EMA correction (Eq. "ema") and, with tau = 0, the
//    synchronous mean (Eq. "sparta") are plain register arithmetic of that lane.
//  * A group arrives as R / RU pipeline units of RU replica rows of w, g, m, v each,
//    fetched with per-thread 16-byte cp.async into a ring of shared-memory stages
//    private to the warp, as in the pipelined kernel.
//  * The ring entry and the d entry of a coordinate that consumes an average this
//    step (R floats each, contiguous) ride in the same cp.async group as the first
//    unit of the coordinate group they belong to, into a small area of their own;
//    they are asked for as far ahead as the dense data, so their latency is hidden
//    the same way and no lane ever waits on a scattered load.
//  * Final weights are known before the one dense store of w and of the look-ahead:
//    no second pass, no 4-byte patches, no stash.
//  * Ring positions come from warp votes: inside a 1024-coordinate chunk the selected
//    coordinates are ordered by (group, bit position within the lane's 4 V, lane).  The
//    same votes give a coordinate its place in the sparse area.  Producer and consumer
//    use the same order; there is no scan.
//  * With four replicas a coordinate's d entry is half a 32-byte sector and the other
//    half belongs to a coordinate of the same lane, so d travels in whole sectors
//    (pairs of coordinates): a scattered store of half a sector costs this memory
//    system more than a store of the whole sector, which needs no fill (measured by
//    tests/sparse_store_probe.cu: 0.36 against 0.26 ms for 13.4 M scattered stores).
#pragma once
#include "step_kernel_pipelined.cuh"

namespace amk {

constexpr int kOwnerThreads = 128;
constexpr int kOwnerBlocksPerSM = 3;   // the register budget up to four replicas (12 warps per SM; with more
                                       // replicas the kernel is compiled for two blocks)

// R contiguous floats, global -> shared, asynchronously
template <int R>
__device__ __forceinline__ void cp_async_replicas(uint32_t smem_addr, const float *g)
{
    if constexpr (R % 4 == 0) {
#pragma unroll
        for (int q = 0; q < R / 4; ++q) cp_async16(smem_addr + 16 * q, g + 4 * q);
    } else if constexpr (R % 2 == 0) {
#pragma unroll
        for (int q = 0; q < R / 2; ++q)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(smem_addr + 8 * q), "l"(g + 2 * q)
                         : "memory");
    } else {
#pragma unroll
        for (int q = 0; q < R; ++q)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(smem_addr + 4 * q), "l"(g + q)
                         : "memory");
    }
}

// RU: replica rows per pipeline unit (divides R); V: float4 per lane, array row and unit;
// E: coordinates per group whose ring and d entries are fetched ahead (further ones,
// possible only when p is large for the E chosen, are read in place).
// NH: passes over a group.  A lane holds R replicas at a time; with NH > 1 the stage has R NH replicas
// and a group is walked NH times, R replica rows per pass (the ring entry carries all of them for the
// mean, d and the snapshot move in the pass's own part).
template <int R, int RU, int V, int E, int NH = 1>
struct OwnerCfg {
    static_assert(R % RU == 0, "a unit holds whole replica rows");
    static constexpr int kTotal = R * NH;                            // replicas of the stage
    static constexpr int kUnitsPerGroup = R / RU;                    // per pass
    static constexpr int kBits = 4 * V;                              // mask bits per lane and group
    static constexpr int kGroupCoords = 128 * V;
    static constexpr int kGroups = kWarpChunk / kGroupCoords;
    static constexpr int kUnitBytes = 4 * RU * V * 512;              // w, g, m, v
    static constexpr bool kPair = (R == 4 && NH == 1);               // d moves as 32-byte pairs
    static constexpr int kOldFloats = (kTotal + 3) / 4 * 4;          // ring entry, padded to 16 bytes
    static constexpr int kDFloats = kPair ? 8 : (R + 3) / 4 * 4;     // d of the pass's replicas
    static constexpr int kEntryFloats = kOldFloats + kDFloats;
    static constexpr int kSparseBytes = E * kEntryFloats * 4;
    __host__ __device__ static constexpr int sparse_areas(int stages)
    {
        // groups whose sparse data can be in shared memory at a time: the one being finished, the
        // next, and those the copy side has entered beyond it (it runs stages - 1 units ahead of
        // the next group's first unit, which is fetched before the finished group's sparse work)
        return 2 + (stages - 1) / kUnitsPerGroup;
    }
    __host__ __device__ static constexpr int warp_bytes(int stages)
    {
        return stages * kUnitBytes + sparse_areas(stages) * kSparseBytes;
    }
};

// The copy side of the pipeline: walks the warp's units in the order the arithmetic
// consumes them (chunk by grid stride -> group g -> unit u).
struct OwnerCursor {
    uint64_t mu;                 // first coordinate of this lane in the current group
    uint32_t gc, s;
    int g, gmax;                 // passes over groups done in this chunk / in all (groups x NH)
    uint32_t h;                  // pass over the current group
    bool valid;
    uint32_t cmask, cbase, crun; // consumed coordinates of the chunk: lane's mask, slot base, count before group g
    uint32_t nx_cmask, nx_cbase; // the same two for the warp's next chunk, asked for one chunk ahead
    uint32_t sp;                 // sparse area of the current group
};

__device__ __forceinline__ void owner_peek(const StepParams &P, const StageDesc *sd, uint32_t gc,
                                           uint32_t s, int lane, uint32_t &cbase, uint32_t &cmask)
{
    cbase = 0;
    cmask = 0;
    if (gc < P.total_chunks) {
        while (s + 1 < P.S && gc >= sd[s + 1].chunk_begin) ++s;
        const StageDesc &st = sd[s];
        const uint32_t chunk = gc - st.chunk_begin;
        cbase = st.chunk_base[(uint64_t)P.cons_slot * st.n_chunks + chunk];
        cmask = st.bitmap[((uint64_t)P.cons_slot * st.n_chunks + chunk) * 32 + lane];
    }
}

template <int GC>
__device__ __forceinline__ int owner_groups(uint64_t N, uint32_t chunk)
{
    const uint64_t rem = N - (uint64_t)chunk * kWarpChunk;
    return rem >= (uint64_t)kWarpChunk ? kWarpChunk / GC : (int)((rem + GC - 1) / GC);
}

template <int GC, int NH = 1>
__device__ __forceinline__ void owner_enter_chunk(OwnerCursor &c, const StepParams &P,
                                                  const StageDesc *sd, int lane, uint32_t n_warps,
                                                  bool consume)
{
    c.valid = c.gc < P.total_chunks;
    if (!c.valid) return;
    while (c.s + 1 < P.S && c.gc >= sd[c.s + 1].chunk_begin) ++c.s;
    const StageDesc &st = sd[c.s];
    const uint32_t chunk = c.gc - st.chunk_begin;
    c.gmax = owner_groups<GC>(st.N, chunk) * NH;
    c.g = 0;
    c.h = 0;
    c.mu = (uint64_t)chunk * kWarpChunk + (uint64_t)lane * 4;
    if (consume) {
        c.cbase = c.nx_cbase;
        c.cmask = c.nx_cbase == kInvalidBase ? 0u : c.nx_cmask;
        c.crun = 0;
        owner_peek(P, sd, c.gc + n_warps, c.s, lane, c.nx_cbase, c.nx_cmask);
    }
}

// Within-group ranks from votes: e[j] = number of selected coordinates of this group that
// come before (bit j, this lane) in (bit, lane) order; returns the group's total.
template <int NB>
__device__ __forceinline__ uint32_t owner_ranks(uint32_t m, uint32_t lt, uint32_t (&e)[NB])
{
    uint32_t run = 0;
#pragma unroll
    for (int j = 0; j < NB; ++j) {
        const uint32_t b = __ballot_sync(kFullMask, (m >> j) & 1u);
        e[j] = run + __popc(b & lt);
        run += __popc(b);
    }
    return run;
}

// CU: which unit of its group the cursor is at.  The cursor runs a fixed NST - 1 units
// ahead of the arithmetic, whose unit loop is unrolled, so CU is known at compile time
// and the code that only a group's first or last unit needs exists once.
template <int R, int RU, int V, int E, int NST, int CU, int NH = 1>
__device__ __forceinline__ void owner_issue_unit(OwnerCursor &c, const StepParams &P,
                                                 const StageDesc *sd, uint32_t stage_addr,
                                                 uint32_t sparse_base, int lane, uint32_t lt,
                                                 uint32_t n_warps, bool consume)
{
    using Cfg = OwnerCfg<R, RU, V, E, NH>;
    constexpr int NB = Cfg::kBits;
    constexpr int RT = Cfg::kTotal;
    if (c.valid) {
        const StageDesc &st = sd[c.s];
        const uint32_t a = stage_addr + lane * 16;
        const float *G = P.G[c.s];
#pragma unroll
        for (int h = 0; h < V; ++h) {
            const uint64_t mu = c.mu + (uint64_t)h * 128;
            if (mu < st.N) {
#pragma unroll
                for (int ii = 0; ii < RU; ++ii) {
                    const uint64_t off = (uint64_t)(c.h * R + CU * RU + ii) * st.stride + mu;
                    cp_async16(a + ((0 * RU + ii) * V + h) * 512, st.W + off);
                    cp_async16(a + ((1 * RU + ii) * V + h) * 512, G + off);
                    cp_async16(a + ((2 * RU + ii) * V + h) * 512, st.M + off);
                    cp_async16(a + ((3 * RU + ii) * V + h) * 512, st.V + off);
                }
            }
        }
        if (CU == 0 && consume) {   // the group's ring and d entries ride with its first unit
            constexpr uint32_t kGroupMask = NB == 32 ? 0xFFFFFFFFu : ((1u << (NB % 32)) - 1u);
            const uint32_t cm = (c.cmask >> (NB * (c.g / NH))) & kGroupMask;
            uint32_t e[NB];
            const uint32_t total = owner_ranks<NB>(cm, lt, e);
            if (cm) {
                const float *ring_cons = st.ring + (uint64_t)P.cons_slot * st.slot_floats;
                const uint32_t sp = sparse_base + c.sp * Cfg::kSparseBytes;
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    if (((cm >> j) & 1u) && e[j] < (uint32_t)E) {
                        const uint32_t dst = sp + e[j] * (Cfg::kEntryFloats * 4);
                        const uint64_t coord = c.mu + (uint64_t)(j >> 2) * 128 + (j & 3);
                        cp_async_replicas<RT>(dst, ring_cons + (uint64_t)(c.cbase + c.crun + e[j]) * RT);
                        if constexpr (Cfg::kPair)   // the whole sector: this coordinate's d and its pair's
                            cp_async_replicas<8>(dst + Cfg::kOldFloats * 4, st.D + (coord & ~(uint64_t)1) * R);
                        else
                            cp_async_replicas<R>(dst + Cfg::kOldFloats * 4, st.D + coord * RT + c.h * R);
                    }
                }
            }
            if (NH == 1 || c.h == NH - 1) c.crun += total;
        }
        if constexpr (CU == Cfg::kUnitsPerGroup - 1) {
            if (NH == 1 || ++c.h == NH) {   // the group's last pass
                c.h = 0;
                c.mu += Cfg::kGroupCoords;
            }
            c.sp = (c.sp + 1 == (uint32_t)Cfg::sparse_areas(NST)) ? 0u : c.sp + 1;
            if (++c.g == c.gmax) {
                c.gc += n_warps;
                owner_enter_chunk<Cfg::kGroupCoords, NH>(c, P, sd, lane, n_warps, consume);
            }
        }
    }
    cp_async_commit();   // always: keeps the group count in step with the unit count
}

// x / R in replica-count arithmetic: a power of two divides exactly like the
// multiplication by its reciprocal (both round the same real number once).
template <int R>
__device__ __forceinline__ float div_by_replicas(const StepParams &P, float a)
{
    if constexpr ((R & (R - 1)) == 0) return __fmul_rn(a, 1.0f / (float)R);
    else return __fdiv_rn(a, P.Rf);
}

// MODE kCompact (tau >= 1) or kSync (tau = 0).
// DIAG: the pass also accumulates the consensus error sum_i ||w_i - wbar||^2 of every stage (Section 3.3)
// from the final weights it holds in registers anyway: no extra memory traffic, fp64 arithmetic per
// coordinate, one atomicAdd per warp and stage.  A separate set of instantiations.
// NADAM: the common form with NAdamW in the place of AdamW (not together with GEN or DIAG).
// NH: the stage has R NH replicas, a group is walked NH times (see OwnerCfg; compact ring only).
template <int R, int RU, int V, int NST, int E, int MODE, bool GEN, bool DIAG = false, bool NADAM = false,
          int NH = 1>
__global__ void __launch_bounds__(kOwnerThreads, R <= 4 ? kOwnerBlocksPerSM : 2)
asyncmesh_step_kernel_owner(const __grid_constant__ StepParams P)
{
    static_assert(MODE == kCompact || MODE == kSync, "compact ring or synchronous");
    static_assert(NH == 1 || (MODE == kCompact && !DIAG), "several passes: the mean comes from the ring entry");
    using Cfg = OwnerCfg<R, RU, V, E, NH>;
    constexpr int RT = Cfg::kTotal;
    constexpr int NB = Cfg::kBits;
    constexpr int UPG = Cfg::kUnitsPerGroup;
    constexpr int kUnitBytes = Cfg::kUnitBytes;
    constexpr uint32_t kGroupMask = NB == 32 ? 0xFFFFFFFFu : ((1u << (NB % 32)) - 1u);
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
    const uint32_t lt = (1u << lane) - 1u;
    constexpr uint32_t wpb = kOwnerThreads / 32;
    const uint32_t n_warps = gridDim.x * wpb;
    const bool consume = (MODE == kCompact) && P.consume != 0u;

    unsigned char *my = dyn_smem + (size_t)warp * Cfg::warp_bytes(NST);
    const uint32_t stage_base = (uint32_t)__cvta_generic_to_shared(my);
    unsigned char *my_sparse = my + NST * kUnitBytes;
    const uint32_t sparse_base = stage_base + NST * kUnitBytes;

    // ---- start the copy pipeline: NST - 1 units ahead --------------------------
    OwnerCursor pf;
    pf.gc = blockIdx.x * wpb + warp;
    pf.s = 0;
    pf.nx_cbase = 0;
    pf.nx_cmask = 0;
    pf.cmask = pf.cbase = pf.crun = 0;
    pf.sp = 0;
    if (consume) owner_peek(P, sd, pf.gc, 0u, lane, pf.nx_cbase, pf.nx_cmask);
    owner_enter_chunk<Cfg::kGroupCoords, NH>(pf, P, sd, lane, n_warps, consume);
    static_assert(NST == 2 || NST == 3 || NST == 4, "the prologue below issues one to three units");
    owner_issue_unit<R, RU, V, E, NST, 0, NH>(pf, P, sd, stage_base, sparse_base, lane, lt, n_warps, consume);
    if constexpr (NST >= 3)
        owner_issue_unit<R, RU, V, E, NST, 1 % UPG, NH>(pf, P, sd, stage_base + kUnitBytes, sparse_base, lane, lt,
                                                    n_warps, consume);
    if constexpr (NST >= 4)
        owner_issue_unit<R, RU, V, E, NST, 2 % UPG, NH>(pf, P, sd, stage_base + 2 * kUnitBytes, sparse_base, lane,
                                                    lt, n_warps, consume);
    uint32_t rd = 0, wr = NST - 1;   // stage being consumed / being filled
    uint32_t sp_rd = 0;              // sparse area of the group being computed
    // Moves the pipeline on by one unit: waits for the next unit's data, asks for the unit NST - 1 further on
    // (CU: that unit's place in its group) and returns where this lane's part of the arrived unit is.
    auto advance = [&](auto cu_tag) -> const unsigned char * {
        constexpr int CU = decltype(cu_tag)::value;
        cp_async_wait<NST - 2>();
        owner_issue_unit<R, RU, V, E, NST, CU, NH>(pf, P, sd, stage_base + wr * kUnitBytes, sparse_base, lane, lt,
                                               n_warps, consume);
        const unsigned char *slot = my + rd * kUnitBytes + lane * 16;
        rd = (rd + 1 == NST) ? 0 : rd + 1;
        wr = (wr + 1 == NST) ? 0 : wr + 1;
        return slot;
    };
    // A group's first unit is fetched BEFORE the sparse work of the group before it, so that the copies keep
    // flowing while that work runs; this is the very first one.
    const unsigned char *first_slot = advance(std::integral_constant<int, (NST - 1) % UPG>{});

    double diag_acc = 0.0;       // DIAG: this lane's share of the current stage's consensus error
    uint32_t diag_stage = 0;
    auto diag_flush = [&]() {
        for (int d = 16; d > 0; d >>= 1) diag_acc += __shfl_down_sync(kFullMask, diag_acc, d);
        if (lane == 0 && diag_acc != 0.0) atomicAdd(P.diag + P.s_base + diag_stage, diag_acc);
        diag_acc = 0.0;
    };
    uint32_t s = 0;
    for (uint32_t gc = blockIdx.x * wpb + warp; gc < P.total_chunks; gc += n_warps) {
        while (s + 1 < P.S && gc >= sd[s + 1].chunk_begin) ++s;
        if constexpr (DIAG) {
            if (s != diag_stage) {   // warp-uniform: the walk has entered another stage
                diag_flush();
                diag_stage = s;
            }
        }
        const StageDesc &st = sd[s];
        const uint32_t chunk = gc - st.chunk_begin;
        const uint64_t N = st.N, stride = st.stride;
        const uint64_t c0 = (uint64_t)chunk * kWarpChunk + (uint64_t)lane * 4;
        const int gmax = owner_groups<Cfg::kGroupCoords>(N, chunk);

        // what the copy side saw for this chunk (the same two words, by now cached)
        uint32_t cbase = 0, cmask = 0;
        const uint64_t word = (uint64_t)chunk * 32 + lane;
        if (consume) {
            cbase = st.chunk_base[(uint64_t)P.cons_slot * st.n_chunks + chunk];
            cmask = st.bitmap[(uint64_t)P.cons_slot * st.n_chunks * 32 + word];
        }

        // ---- membership of this lane's 32 coordinates in S^t --------------------
        // bit 4b + c  <->  coordinate c0 + 128 b + c; group g owns bits NB g .. NB g + NB - 1
        uint32_t pmask = 0;
        if (P.produce) {
            const uint32_t quad0 = st.quad_base + (uint32_t)(c0 >> 2);
#pragma unroll 2
            for (int b = 0; b < 8; ++b) {
                const uint64_t mu = c0 + (uint64_t)b * 128;
                if (mu < N) {
                    const uint64_t left = N - mu;
                    const uint32_t valid = left >= 4 ? 0xFu : ((1u << (uint32_t)left) - 1u);
                    pmask |= (subset_bits(P.rule, st.stage_id, P.step, quad0 + (uint32_t)b * 32u) & valid)
                             << (4 * b);
                }
            }
        }

        // ---- room in the producing slot -----------------------------------------
        uint32_t pbase = 0;
        if constexpr (MODE == kCompact) {
            const uint32_t total = __reduce_add_sync(kFullMask, (uint32_t)__popc(pmask));
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
            pbase = __shfl_sync(kFullMask, pbase, 0);
            if (pbase == kInvalidBase) pmask = 0;
            if (P.produce)   // kept for step t + tau
                st.bitmap[(uint64_t)P.prod_slot * st.n_chunks * 32 + word] = pmask;
            if (cbase == kInvalidBase) cmask = 0;
        }
        const float *ring_cons = st.ring + (uint64_t)P.cons_slot * st.slot_floats;
        float *ring_prod = st.ring + (uint64_t)P.prod_slot * st.slot_floats;
        const float delta = st.delta;
        const bool has_look = st.delta != 0.0f;
        uint32_t crun = 0, prun = 0;

#pragma unroll 1
        for (int vg = 0; vg < gmax * NH; ++vg) {
            const int g = vg / NH;                         // the group, and which R of its replica rows
            const uint32_t row0 = (uint32_t)(vg % NH) * R;
            const bool last_pass = NH == 1 || (vg % NH) == NH - 1;
            const uint64_t mu0 = c0 + (uint64_t)g * Cfg::kGroupCoords;   // h = 0; h adds 128
            const uint32_t pm = (pmask >> (NB * g)) & kGroupMask;
            const uint32_t cm = (cmask >> (NB * g)) & kGroupMask;

            // ---- local optimizer step of every replica (lanes past the end of the stage
            // compute on whatever their slot holds: nothing of it is stored or selected)
            float wn[R][NB], wo[R][NB];
            auto unit = [&](auto u_tag) {
                constexpr int u = decltype(u_tag)::value;
                const unsigned char *slot =
                    u == 0 ? first_slot : advance(std::integral_constant<int, (u + NST - 1) % UPG>{});
#pragma unroll
                for (int ii = 0; ii < RU; ++ii) {
                    const int i = u * RU + ii;
                    float gg[NB], m[NB], v[NB];
#pragma unroll
                    for (int h = 0; h < V; ++h) {
                        const float4 w4 = *reinterpret_cast<const float4 *>(slot + ((0 * RU + ii) * V + h) * 512);
                        const float4 g4 = *reinterpret_cast<const float4 *>(slot + ((1 * RU + ii) * V + h) * 512);
                        const float4 m4 = *reinterpret_cast<const float4 *>(slot + ((2 * RU + ii) * V + h) * 512);
                        const float4 v4 = *reinterpret_cast<const float4 *>(slot + ((3 * RU + ii) * V + h) * 512);
                        wo[i][4 * h] = w4.x; wo[i][4 * h + 1] = w4.y; wo[i][4 * h + 2] = w4.z; wo[i][4 * h + 3] = w4.w;
                        gg[4 * h] = g4.x; gg[4 * h + 1] = g4.y; gg[4 * h + 2] = g4.z; gg[4 * h + 3] = g4.w;
                        m[4 * h] = m4.x; m[4 * h + 1] = m4.y; m[4 * h + 2] = m4.z; m[4 * h + 3] = m4.w;
                        v[4 * h] = v4.x; v[4 * h + 1] = v4.y; v[4 * h + 2] = v4.z; v[4 * h + 3] = v4.w;
                    }
                    adamw_group<GEN, NB, NADAM>(P, wo[i], gg, m, v, wn[i]);
#pragma unroll
                    for (int h = 0; h < V; ++h) {
                        const uint64_t mu = mu0 + (uint64_t)h * 128;
                        if (mu < N) {
                            const uint64_t off = (uint64_t)(row0 + i) * stride + mu;
                            __stcs(reinterpret_cast<float4 *>(st.M + off),
                                   make_float4(m[4 * h], m[4 * h + 1], m[4 * h + 2], m[4 * h + 3]));
                            __stcs(reinterpret_cast<float4 *>(st.V + off),
                                   make_float4(v[4 * h], v[4 * h + 1], v[4 * h + 2], v[4 * h + 3]));
                        }
                    }
                }
            };
            unit(std::integral_constant<int, 0>{});
            if constexpr (UPG > 1) unit(std::integral_constant<int, 1>{});
            if constexpr (UPG > 2) unit(std::integral_constant<int, 2>{});
            if constexpr (UPG > 3) unit(std::integral_constant<int, 3>{});
            if constexpr (UPG > 4) unit(std::integral_constant<int, 4>{});
            if constexpr (UPG > 5) unit(std::integral_constant<int, 5>{});
            if constexpr (UPG > 6) unit(std::integral_constant<int, 6>{});
            static_assert(UPG <= 7, "at most seven units per group");
            first_slot = advance(std::integral_constant<int, (NST - 1) % UPG>{});   // the next group's, see above

            if constexpr (MODE == kCompact) {
                // ---- snapshot of the local iterate on S^t (Section 3.1) ------------------
                {
                    uint32_t e[NB];
                    const uint32_t total = owner_ranks<NB>(pm, lt, e);
                    if (pm) {
                        // A scattered store instruction costs the memory pipeline about the same
                        // with one lane taking part as with all of them, and most lanes have at
                        // most one entry per group: a lane holds its first entry back, so that one
                        // store instruction at the end serves the first entries of all lanes.
                        float *ring_at = ring_prod + (uint64_t)(pbase + prun) * RT + row0;
                        float held[R];
                        uint32_t held_e = kInvalidBase;
#pragma unroll
                        for (int j = 0; j < NB; ++j) {
                            if ((pm >> j) & 1u) {
                                float x[R];
#pragma unroll
                                for (int i = 0; i < R; ++i) x[i] = wn[i][j];
                                if (held_e == kInvalidBase) {
                                    held_e = e[j];
#pragma unroll
                                    for (int i = 0; i < R; ++i) held[i] = x[i];
                                } else {
                                    store_replicas<R>(ring_at + (uint64_t)e[j] * RT, x);
                                }
                            }
                        }
                        store_replicas<R>(ring_at + (uint64_t)held_e * RT, held);
                    }
                    if (last_pass) prun += total;
                }
                // ---- Eq. "asparta" / Eq. "ema" + corrected averaging on S^{t-tau} --------
                if (consume) {
                    uint32_t e[NB];
                    const uint32_t total = owner_ranks<NB>(cm, lt, e);
                    if (cm) {
                        const float *sp = reinterpret_cast<const float *>(my_sparse + sp_rd * Cfg::kSparseBytes);
                        // one consumed coordinate: stale average from the ring entry, new d, final w
                        // (all: the ring entry, every replica of the stage; old: the values of this pass's replicas)
                        auto consume_one = [&](int j, const float (&all)[RT], const float (&old)[R], float (&dd)[R]) {
                            float a = on_wire<GEN>(P, all[0]);
#pragma unroll
                            for (int i = 1; i < RT; ++i) a = __fadd_rn(a, on_wire<GEN>(P, all[i]));
                            const float abar = div_by_replicas<RT>(P, a);
#pragma unroll
                            for (int i = 0; i < R; ++i) {
                                const float diff = __fsub_rn(wn[i][j], old[i]);
                                dd[i] = staleness<GEN>(P, dd[i], diff);
                                wn[i][j] = __fadd_rn(abar, dd[i]);
                            }
                        };
                        if constexpr (Cfg::kPair) {
                            float held_d[8];
                            float *held_dp = nullptr;
#pragma unroll
                            for (int q = 0; q < NB / 2; ++q) {   // pairs of coordinates = sectors of d
                                const uint32_t pc = (cm >> (2 * q)) & 3u;
                                if (pc) {
                                    const uint64_t coord = mu0 + (uint64_t)(q >> 1) * 128 + 2 * (q & 1);
                                    float *dp = st.D + coord * R;
                                    const uint32_t e0 = (pc & 1u) ? e[2 * q] : e[2 * q + 1];
                                    float dpair[8];
                                    if (e0 < (uint32_t)E) load_replicas<8>(sp + e0 * Cfg::kEntryFloats + Cfg::kOldFloats, dpair);
                                    else load_replicas<8>(dp, dpair);   // beyond what was fetched ahead
#pragma unroll
                                    for (int c = 0; c < 2; ++c) {
                                        if ((pc >> c) & 1u) {
                                            const int j = 2 * q + c;
                                            float old[R], dd[R];
                                            if (e[j] < (uint32_t)E) load_replicas<R>(sp + e[j] * Cfg::kEntryFloats, old);
                                            else load_replicas<R>(ring_cons + (uint64_t)(cbase + crun + e[j]) * R, old);
#pragma unroll
                                            for (int i = 0; i < R; ++i) dd[i] = dpair[R * c + i];
                                            if constexpr (NH == 1) consume_one(j, old, old, dd);
#pragma unroll
                                            for (int i = 0; i < R; ++i) dpair[R * c + i] = dd[i];
                                        }
                                    }
                                    if (held_dp == nullptr) {   // held back, as for the ring entries above
                                        held_dp = dp;
#pragma unroll
                                        for (int x = 0; x < 8; ++x) held_d[x] = dpair[x];
                                    } else {
                                        st_sector(dp, dpair);
                                    }
                                }
                            }
                            st_sector(held_dp, held_d);
                        } else {
#pragma unroll
                            for (int j = 0; j < NB; ++j) {
                                if ((cm >> j) & 1u) {
                                    float all[RT], old[NH == 1 ? 1 : R], dd[R];
                                    float *dp = st.D + (mu0 + (uint64_t)(j >> 2) * 128 + (j & 3)) * RT + row0;
                                    if (e[j] < (uint32_t)E) {
                                        const float *entry = sp + e[j] * Cfg::kEntryFloats;
                                        load_replicas<RT>(entry, all);
                                        if constexpr (NH > 1) load_replicas<R>(entry + row0, old);
                                        load_replicas<R>(entry + Cfg::kOldFloats, dd);
                                    } else {   // beyond what was fetched ahead
                                        const float *entry = ring_cons + (uint64_t)(cbase + crun + e[j]) * RT;
                                        load_replicas<RT>(entry, all);
                                        if constexpr (NH > 1) load_replicas<R>(entry + row0, old);
                                        load_replicas<R>(dp, dd);
                                    }
                                    if constexpr (NH == 1) consume_one(j, all, all, dd);
                                    else consume_one(j, all, old, dd);
                                    store_replicas<R>(dp, dd);
                                }
                            }
                        }
                    }
                    if (last_pass) crun += total;
                    sp_rd = (sp_rd + 1 == (uint32_t)Cfg::sparse_areas(NST)) ? 0u : sp_rd + 1;
                }
            } else {
                // ---- Eq. "sparta": coordinates of S^t take the replica mean; the EMA state
                // stays exactly zero when tau = 0 (its sample is w^ - w^), hence mean + 0
                if (pm) {
#pragma unroll
                    for (int j = 0; j < NB; ++j) {
                        if ((pm >> j) & 1u) {
                            float a = on_wire<GEN>(P, wn[0][j]);
#pragma unroll
                            for (int i = 1; i < R; ++i) a = __fadd_rn(a, on_wire<GEN>(P, wn[i][j]));
                            const float wnew = __fadd_rn(div_by_replicas<R>(P, a), 0.0f);
#pragma unroll
                            for (int i = 0; i < R; ++i) wn[i][j] = wnew;
                        }
                    }
                }
            }

            if constexpr (DIAG) {   // consensus error of the final weights (Section 3.3), in double
#pragma unroll
                for (int j = 0; j < NB; ++j) {
                    if (mu0 + (uint64_t)(j >> 2) * 128 + (j & 3) < N) {
                        double mean = 0.0;
#pragma unroll
                        for (int i = 0; i < R; ++i) mean += (double)wn[i][j];
                        mean /= (double)R;
#pragma unroll
                        for (int i = 0; i < R; ++i) {
                            const double e = (double)wn[i][j] - mean;
                            diag_acc += e * e;
                        }
                    }
                }
            }
            // ---- the one store of w and of the look-ahead (Section 2.2) ----------------
#pragma unroll
            for (int h = 0; h < V; ++h) {
                const uint64_t mu = mu0 + (uint64_t)h * 128;
                if (mu < N) {
#pragma unroll
                    for (int i = 0; i < R; ++i) {
                        const uint64_t off = (uint64_t)(row0 + i) * stride + mu;
                        __stcs(reinterpret_cast<float4 *>(st.W + off),
                               make_float4(wn[i][4 * h], wn[i][4 * h + 1], wn[i][4 * h + 2], wn[i][4 * h + 3]));
                        if (has_look) {
                            float lk[4];
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                lk[c] = __fadd_rn(wn[i][4 * h + c],
                                                  __fmul_rn(delta, __fsub_rn(wn[i][4 * h + c], wo[i][4 * h + c])));
                            st_stream(st.LOOK + off, lk);
                        }
                    }
                }
            }
        }
    }
    if constexpr (DIAG) diag_flush();
    cp_async_wait<0>();
}

}  // namespace amk
