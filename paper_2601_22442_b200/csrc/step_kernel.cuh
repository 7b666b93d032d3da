// The fused AsyncMesh step for sm_100a: one launch advances every stage of the
// mesh by one step.  HBM-bound streaming kernel: per replica-coordinate it reads
// w, g, m, v once (128-bit loads) and writes w, m, v (and the look-ahead) once;
// the sparse parts (snapshot ring, EMA state d) are touched only at selected
// coordinates.  No tensor cores: there is no contraction on this path.
//
// Work decomposition.  A stage's coordinates are cut into warp chunks of 1024
// (8 sub-iterations x 32 lanes x 4 coordinates).  A warp owns a chunk, so a
// lane sees, per sub-iteration, one float4 of every array row of every replica.
// All chunks of all stages form one list that the grid's warps walk with a
// grid-sized stride, so neighbouring warps stream neighbouring 4 KB pieces.
//
// Snapshot ring (Section 3.1: the average of step t is consumed at t + tau; the
// paper's own experiments buffer it).  A slot holds, for one step u, the local
// iterates w^_i^u of the coordinates in S^u, coordinate-major: R floats per
// selected coordinate.  Two layouts:
//   compact  slot = [cap][R]; a warp reserves room for its chunk's selected
//            coordinates with one atomicAdd on the slot's cursor and records the
//            base in chunk_base[slot][chunk]; tau steps later the consumer finds
//            the data through that table and finds membership and rank again
//            (this kernel from Philox, the pipelined one from the mask it stored
//            with the slot), so no index list is stored.  tau / K + 1 slots
//            (K: the averaging interval).
//   dense    slot = [R][row_stride], replica-major like w, coordinate mu at position
//            mu; used when the subset is so large that compaction saves nothing
//            (d is replica-major too in this mode).  tau / K slots; the consumer and
//            producer of a step share a slot and a thread reads a position
//            before it overwrites it.
// With tau = 0 (synchronous sparse averaging, Eq. "sparta") there is no ring:
// the average is formed from the registers of the lane that owns the coordinate.
//
// Arithmetic is written with the round-to-nearest intrinsics, one IEEE
// operation per paper operation, so that no contraction into FMA can change a
// result; the same operation order is what the CPU check uses.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include "philox.cuh"
#include "rounded_math.cuh"

namespace amk {

constexpr int kWarpChunk = 1024;   // coordinates a warp owns at a time
constexpr int kSubIters = 8;       // 8 x (32 lanes x 4 coordinates)
constexpr int kBlockThreads = 256;
constexpr uint32_t kInvalidBase = 0xFFFFFFFFu;
constexpr unsigned kFullMask = 0xFFFFFFFFu;
constexpr int kMaxStages = 64;

// kDenseBf16 / kDenseE4m3: the dense ring holding the snapshot only as exchanged
// (2 or 1 bytes per value; the staleness sample is taken against that rounded value)
enum RingMode : int { kSync = 0, kCompact = 1, kDense = 2, kDenseBf16 = 3, kDenseE4m3 = 4 };
constexpr bool is_dense(int mode) { return mode >= kDense; }
constexpr int ring_value_bytes(int mode) { return mode == kDenseBf16 ? 2 : (mode == kDenseE4m3 ? 1 : 4); }

constexpr int kStatusRingOverflow = 1;

struct StageDesc {
    float *W, *M, *V;       // [R][stride]
    float *D;               // [stride][R]; [R][stride] with the dense ring
    float *LOOK;            // [R][stride]; == W when delta == 0
    float *ring;            // [n_slots][slot_floats]
    uint32_t *chunk_base;   // [n_slots][n_chunks]           (compact only)
    uint32_t *bitmap;       // [n_slots][n_chunks][32] subset masks, lane-major (pipelined kernel only)
    uint64_t N, stride, slot_floats;
    uint32_t n_chunks;      // ceil(N / 1024)
    uint32_t chunk_begin;   // first chunk of this stage in the global list
    uint32_t cap;           // selected coordinates a compact slot can hold
    uint32_t stage_id;
    float delta;            // look-ahead delay as a float; != 0: LOOK is a buffer of its own
    uint32_t quad_base;     // (global index of local coordinate 0) / 4: a handle may hold a
                            // coordinate range of a larger stage (one shard per GPU)
};

struct StepParams {
    const StageDesc *stages;     // device [S]
    unsigned int *cursors;       // device [n_slots][S]            (compact only)
    int *status;                 // device status word
    double *diag;                // device [S]: consensus error per stage, accumulated by the tracking kernels
    const float *G[kMaxStages];  // gradients, [R][stride] each
    uint32_t S, total_chunks;    // stages and warp chunks of THIS launch
    uint32_t cursor_S, s_base;   // stages of the handle and the handle's index of this launch's stage 0:
                                 // a launch may cover one stage only (host gradients arriving stage by stage)
    uint32_t step, cons_step;    // t and t - tau
    uint32_t produce;            // this step is an averaging round: S^t is snapshotted
    uint32_t consume;            // ... and the average launched at t - tau has arrived
    uint32_t prod_slot, cons_slot;
    SubsetRule rule;
    float b1, b2, omb1, omb2, ib1, ib2, eps, lr, lrwd, lam, oml, Rf;
    uint32_t wire;               // snapshots enter the average as fp32 (0), rounded to bfloat16 (1)
                                 // or to 8-bit floating point E4M3 (2)
    uint32_t eager;              // staleness estimate: 0 Eq. "ema", 1 d = (w^ - w^_old) / R
    uint32_t nesterov;           // 0: AdamW, 1: NAdamW (general form only)
    uint32_t eps_inrange;        // eps is at most 2^60: sqrt(v^) + eps then stays in the range of the
                                 // straight-line division whenever v^ is in the square root's
    float cg, cm;                // NAdamW: weights of the gradient and momentum parts
};

__device__ __forceinline__ float4 ld_stream(const float *p)
{
    return __ldcs(reinterpret_cast<const float4 *>(p));
}
__device__ __forceinline__ void st_stream(float *p, const float (&x)[4])
{
    __stcs(reinterpret_cast<float4 *>(p), make_float4(x[0], x[1], x[2], x[3]));
}

// A snapshot value as the other replicas see it: unchanged, or rounded to
// bfloat16 or to E4M3 (round to nearest even; E4M3 clamps at its largest finite
// value 448) when the subset is exchanged in reduced precision (the paper's
// quantisation study).  The average is formed in fp32; a replica's own
// staleness sample keeps using its own unrounded value.
// GEN selects the general form (also E4M3, also the eager estimate below); the
// kernels of the common configurations are compiled without it, as instantiations
// of their own: the pipelined kernel's run time moves by several percent with a
// handful of extra instructions in its sparse phase (measured: +7 % inline, +2 %
// as out-of-line calls, although they never run in those configurations).
template <bool GEN>
__device__ __forceinline__ float on_wire(const StepParams &P, float x)
{
    if constexpr (GEN) {
        if (P.wire == 2u) {
            const __nv_fp8_storage_t q = __nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3);
            return __half2float(__half(__nv_cvt_fp8_to_halfraw(q, __NV_E4M3)));
        }
    }
    return P.wire ? __bfloat162float(__float2bfloat16_rn(x)) : x;
}

// The staleness estimate of a consumed coordinate (Section 3.2): Eq. "ema", or the
// eager estimate the section's last paragraph names as a special case.
template <bool GEN>
__device__ __forceinline__ float staleness(const StepParams &P, float d, float diff)
{
    if constexpr (GEN) {
        if (P.eager) return __fdiv_rn(diff, P.Rf);
    }
    return __fadd_rn(__fmul_rn(P.oml, d), __fmul_rn(P.lam, diff));
}

// u = m^ / (sqrt(v^) + eps) with the toolkit's correctly rounded routines: the route
// of a coordinate group with an operand outside the range of the straight-line
// forms (zero or subnormal moments, huge gradients, Inf, NaN).  Out of line, so that
// the common route carries none of its code.
static __device__ __noinline__ float adam_quotient_anyrange(float mh, float vh, float eps)
{
    return __fdiv_rn(mh, __fadd_rn(__fsqrt_rn(vh), eps));
}

// The local optimizer step (first line of Eq. "sparta") for NC coordinates of one
// replica, one rounding per written operation: AdamW with decoupled weight decay and
// bias correction; in the general form (GEN) also NAdamW.
// AdamW's square root and division are the straight-line forms of rounded_math.cuh
// when every operand of the group lies in their range (one test per group; eps is
// tested by the host: P.eps_inrange), else the toolkit's routines: the same bits
// either way.
// NAdamW (Appendix B.1) from the moments of this step: gradient part and (uncorrected)
// momentum part over the same denominator, weighted by the momentum schedule's cg and cm.
template <int NC>
__device__ __forceinline__ void nadamw_finish(const StepParams &P, const float (&w)[NC], const float (&g)[NC],
                                              const float (&m)[NC], const float (&vh)[NC], float (&what)[NC])
{
    float vlo = vh[0], vhi = vh[0], alo = fminf(fabsf(g[0]), fabsf(m[0])),
          ahi = fmaxf(fabsf(g[0]), fabsf(m[0]));
#pragma unroll
    for (int c = 1; c < NC; ++c) {
        vlo = fminf(vlo, vh[c]);
        vhi = fmaxf(vhi, vh[c]);
        alo = fminf(alo, fminf(fabsf(g[c]), fabsf(m[c])));
        ahi = fmaxf(ahi, fmaxf(fabsf(g[c]), fabsf(m[c])));
    }
    const bool inrange = P.eps_inrange != 0u && vlo >= kSqrtLo && vhi <= kSqrtHi &&
                         alo >= kDivNumLo && ahi <= kDivNumHi;
    float ug[NC], um[NC];
    if (inrange) {   // one branch for the group: the chains of its coordinates interleave
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const float den = __fadd_rn(sqrt_rn_inrange(vh[c]), P.eps);
            ug[c] = div_rn_inrange(g[c], den);
            um[c] = div_rn_inrange(m[c], den);
        }
    } else {
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            ug[c] = adam_quotient_anyrange(g[c], vh[c], P.eps);
            um[c] = adam_quotient_anyrange(m[c], vh[c], P.eps);
        }
    }
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const float decayed = __fsub_rn(w[c], __fmul_rn(P.lrwd, w[c]));
        what[c] = __fsub_rn(__fsub_rn(decayed, __fmul_rn(P.cg, ug[c])), __fmul_rn(P.cm, um[c]));
    }
}

// NADAM: NAdamW and nothing else, decided at compile time (the owner kernel's form for the
// paper's asynchronous-pipeline optimizer); GEN: either optimizer, decided by P.nesterov.
template <bool GEN, int NC, bool NADAM = false>
__device__ __forceinline__ void adamw_group(const StepParams &P, const float (&w)[NC],
                                            const float (&g)[NC], float (&m)[NC], float (&v)[NC],
                                            float (&what)[NC])
{
    float mh[NC], vh[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        m[c] = __fadd_rn(__fmul_rn(P.b1, m[c]), __fmul_rn(P.omb1, g[c]));
        v[c] = __fadd_rn(__fmul_rn(P.b2, v[c]), __fmul_rn(P.omb2, __fmul_rn(g[c], g[c])));
        mh[c] = __fmul_rn(m[c], P.ib1);
        vh[c] = __fmul_rn(v[c], P.ib2);
    }
    if constexpr (NADAM) {
        nadamw_finish<NC>(P, w, g, m, vh, what);
        return;
    } else if constexpr (GEN) {
        if (P.nesterov != 0u) {
            nadamw_finish<NC>(P, w, g, m, vh, what);
            return;
        }
    }
    float u[NC];
    // (min / max drop a NaN operand: a NaN then takes the straight-line route and
    // comes out as a NaN there too)
    float vlo = vh[0], vhi = vh[0], alo = fabsf(mh[0]), ahi = fabsf(mh[0]);
#pragma unroll
    for (int c = 1; c < NC; ++c) {
        vlo = fminf(vlo, vh[c]);
        vhi = fmaxf(vhi, vh[c]);
        alo = fminf(alo, fabsf(mh[c]));
        ahi = fmaxf(ahi, fabsf(mh[c]));
    }
    const bool inrange = P.eps_inrange != 0u && vlo >= kSqrtLo && vhi <= kSqrtHi &&
                         alo >= kDivNumLo && ahi <= kDivNumHi;
    if (inrange) {
#pragma unroll
        for (int c = 0; c < NC; ++c)
            u[c] = div_rn_inrange(mh[c], __fadd_rn(sqrt_rn_inrange(vh[c]), P.eps));
    } else {
#pragma unroll
        for (int c = 0; c < NC; ++c) u[c] = adam_quotient_anyrange(mh[c], vh[c], P.eps);
    }
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const float decayed = __fsub_rn(w[c], __fmul_rn(P.lrwd, w[c]));
        what[c] = __fsub_rn(decayed, __fmul_rn(P.lr, u[c]));
    }
}

// Four consecutive values of a dense ring slot, `off` values from the start of the ring
// (a multiple of 4), in the slot's own format; widening bfloat16 or E4M3 to fp32 is exact.
template <int MODE>
__device__ __forceinline__ float4 ring_load4(const float *ring, uint64_t off)
{
    if constexpr (MODE == kDenseBf16) {
        const uint2 u = *reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(ring) + off);
        return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u),
                           __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u));
    } else if constexpr (MODE == kDenseE4m3) {
        const uint32_t u = *reinterpret_cast<const uint32_t *>(reinterpret_cast<const uint8_t *>(ring) + off);
        float x[4];
#pragma unroll
        for (int c = 0; c < 4; ++c)
            x[c] = __half2float(__half(__nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)((u >> (8 * c)) & 0xFFu), __NV_E4M3)));
        return make_float4(x[0], x[1], x[2], x[3]);
    } else {
        return *reinterpret_cast<const float4 *>(ring + off);
    }
}

// ... and the snapshot of four local iterates into it: rounded to nearest even (E4M3
// clamps at its largest finite value 448) where the slot is narrower than fp32.
template <int MODE>
__device__ __forceinline__ void ring_store4(float *ring, uint64_t off, const float (&x)[4])
{
    if constexpr (MODE == kDenseBf16) {
        uint32_t h[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) h[c] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x[c]));
        __stcs(reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(ring) + off),
               make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16)));
    } else if constexpr (MODE == kDenseE4m3) {
        uint32_t u = 0;
#pragma unroll
        for (int c = 0; c < 4; ++c)
            u |= (uint32_t)__nv_cvt_float_to_fp8(x[c], __NV_SATFINITE, __NV_E4M3) << (8 * c);
        __stcs(reinterpret_cast<uint32_t *>(reinterpret_cast<uint8_t *>(ring) + off), u);
    } else {
        st_stream(ring + off, x);
    }
}

template <int R>
__device__ __forceinline__ void load_replicas(const float *p, float (&x)[R])
{
    if constexpr (R % 4 == 0) {
#pragma unroll
        for (int q = 0; q < R / 4; ++q) {
            const float4 t = *reinterpret_cast<const float4 *>(p + 4 * q);
            x[4 * q] = t.x; x[4 * q + 1] = t.y; x[4 * q + 2] = t.z; x[4 * q + 3] = t.w;
        }
    } else if constexpr (R % 2 == 0) {
#pragma unroll
        for (int q = 0; q < R / 2; ++q) {
            const float2 t = *reinterpret_cast<const float2 *>(p + 2 * q);
            x[2 * q] = t.x; x[2 * q + 1] = t.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < R; ++i) x[i] = p[i];
    }
}

__device__ __forceinline__ uint32_t warp_exclusive_sum(uint32_t x, int lane, uint32_t &total)
{
    uint32_t incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t n = __shfl_up_sync(kFullMask, incl, d);
        if (lane >= d) incl += n;
    }
    total = __shfl_sync(kFullMask, incl, 31);
    return incl - x;
}

template <int R, int MODE, bool GEN>
__device__ __forceinline__ void process_chunk(const StepParams &P, const StageDesc &st,
                                              const float *__restrict__ G, uint32_t s,
                                              uint32_t chunk, int lane)
{
    constexpr int RG = (R % 2 == 0) ? 2 : 1;   // replicas loaded together
    const uint64_t N = st.N, stride = st.stride;
    const uint64_t c0 = (uint64_t)chunk * kWarpChunk + (uint64_t)lane * 4;
    const bool consume = (MODE != kSync) && (P.consume != 0u);
    constexpr bool kStored = MODE > kDense;   // the slot holds values already rounded for the exchange

    // ---- membership of this lane's 32 coordinates in S^t and S^{t-tau} --------
    uint32_t pmask = 0, cmask = 0;   // bit 4k+j: coordinate c0 + 128k + j
#pragma unroll 2
    for (int k = 0; k < kSubIters; ++k) {
        const uint64_t mu = c0 + (uint64_t)k * 128;
        if (mu < N) {
            const uint64_t left = N - mu;
            const uint32_t valid = left >= 4 ? 0xFu : ((1u << (uint32_t)left) - 1u);
            const uint32_t quad = st.quad_base + (uint32_t)(mu >> 2);
            if (P.produce)
                pmask |= (subset_bits(P.rule, st.stage_id, P.step, quad) & valid) << (4 * k);
            if (consume)
                cmask |= (subset_bits(P.rule, st.stage_id, P.cons_step, quad) & valid) << (4 * k);
        }
    }

    // ---- where this chunk's selected coordinates live in the ring slots --------
    uint32_t pbase = 0, pexcl = 0, cbase = 0, cexcl = 0;
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
        pbase = __shfl_sync(kFullMask, pbase, 0);
        if (pbase == kInvalidBase) pmask = 0;
        if (consume) {
            cbase = st.chunk_base[(uint64_t)P.cons_slot * st.n_chunks + chunk];
            if (cbase == kInvalidBase) cmask = 0;
            uint32_t ctotal;
            cexcl = warp_exclusive_sum(__popc(cmask), lane, ctotal);
        }
    }
    const uint64_t cons_off = (uint64_t)P.cons_slot * st.slot_floats;   // in ring values
    const uint64_t prod_off = (uint64_t)P.prod_slot * st.slot_floats;
    const float *ring_cons = st.ring + cons_off;
    float *ring_prod = st.ring + prod_off;
    const float delta = st.delta;
    const bool has_look = st.delta != 0.0f;

#pragma unroll 1
    for (int k = 0; k < kSubIters; ++k) {
        const uint64_t mu = c0 + (uint64_t)k * 128;
        if (mu >= N) break;   // no warp-wide operation below this point
        const uint32_t pm = (pmask >> (4 * k)) & 0xFu;
        const uint32_t cm = (cmask >> (4 * k)) & 0xFu;

        if constexpr (MODE >= kDense) {
            // Large subsets: the ring slot and d are replica-major like w, m, v, so the
            // sparse quantities stream as float4 too.  A lane owns its four coordinates
            // in every replica row, reads a ring position before it overwrites it, and
            // writes whole float4: ring positions of unselected coordinates are never
            // read by anyone, and d is rewritten with its old value there.
            // The stale values of all replicas go out first and are summed only after
            // the first group's dense loads have been issued: instructions issue in
            // order, so a sum placed right behind its loads would hold back every
            // load after it for a full memory round trip.
            float4 r4[R];
#pragma unroll
            for (int i = 0; i < R; ++i) {
                r4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (cm) r4[i] = ring_load4<MODE>(st.ring, cons_off + (uint64_t)i * stride + mu);
            }
            float abar[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i0 = 0; i0 < R; i0 += RG) {
                float4 w4[RG], g4[RG], m4[RG], v4[RG], d4[RG];
#pragma unroll
                for (int ii = 0; ii < RG; ++ii) {
                    const uint64_t off = (uint64_t)(i0 + ii) * stride + mu;
                    w4[ii] = ld_stream(st.W + off);
                    g4[ii] = ld_stream(G + off);
                    m4[ii] = ld_stream(st.M + off);
                    v4[ii] = ld_stream(st.V + off);
                    d4[ii] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (cm) d4[ii] = ld_stream(st.D + off);
                }
                if (i0 == 0 && cm) {   // stale average, replica order, one division
                    float a[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int i = 0; i < R; ++i) {
                        const float r[4] = {r4[i].x, r4[i].y, r4[i].z, r4[i].w};
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const float sent = kStored ? r[c] : on_wire<GEN>(P, r[c]);
                            a[c] = (i == 0) ? sent : __fadd_rn(a[c], sent);
                        }
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) abar[c] = __fdiv_rn(a[c], P.Rf);
                }
#pragma unroll
                for (int ii = 0; ii < RG; ++ii) {
                    const uint64_t off = (uint64_t)(i0 + ii) * stride + mu;
                    const float4 o4 = r4[i0 + ii];
                    const float w[4] = {w4[ii].x, w4[ii].y, w4[ii].z, w4[ii].w};
                    const float g[4] = {g4[ii].x, g4[ii].y, g4[ii].z, g4[ii].w};
                    float m[4] = {m4[ii].x, m4[ii].y, m4[ii].z, m4[ii].w};
                    float v[4] = {v4[ii].x, v4[ii].y, v4[ii].z, v4[ii].w};
                    const float old[4] = {o4.x, o4.y, o4.z, o4.w};
                    float dd[4] = {d4[ii].x, d4[ii].y, d4[ii].z, d4[ii].w};
                    float wh[4], wn[4];
                    adamw_group<GEN, 4>(P, w, g, m, v, wh);
#pragma unroll
                    for (int c = 0; c < 4; ++c) wn[c] = wh[c];
                    st_stream(st.M + off, m);
                    st_stream(st.V + off, v);
                    if (cm) {   // Eq. "ema" + corrected averaging on S^{t-tau}
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            if ((cm >> c) & 1u) {
                                const float diff = __fsub_rn(wh[c], old[c]);
                                dd[c] = staleness<GEN>(P, dd[c], diff);
                                wn[c] = __fadd_rn(abar[c], dd[c]);
                            }
                        }
                        st_stream(st.D + off, dd);
                    }
                    if (pm) ring_store4<MODE>(st.ring, prod_off + off, wh);   // snapshot of the local iterate on S^t
                    st_stream(st.W + off, wn);
                    if (has_look) {
                        float lk[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            lk[c] = __fadd_rn(wn[c], __fmul_rn(delta, __fsub_rn(wn[c], w[c])));
                        st_stream(st.LOOK + off, lk);
                    }
                }
            }
            continue;
        }

        // ---- stale average wbar^{t-tau} of the coordinates being consumed -----
        float abar[4] = {0.f, 0.f, 0.f, 0.f};
        uint64_t ce[4] = {0, 0, 0, 0}, pe[4] = {0, 0, 0, 0};   // ring offsets (floats)
        if constexpr (MODE != kSync) {
            if (cm) {
                const uint32_t below = __popc(cmask & ((1u << (4 * k)) - 1u));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if ((cm >> j) & 1u) {
                        const uint64_t idx = (uint64_t)(cbase + cexcl + below + __popc(cm & ((1u << j) - 1u)));
                        ce[j] = idx * R;
                        float old[R];
                        load_replicas<R>(ring_cons + ce[j], old);
                        float a = on_wire<GEN>(P, old[0]);
#pragma unroll
                        for (int i = 1; i < R; ++i) a = __fadd_rn(a, on_wire<GEN>(P, old[i]));
                        abar[j] = __fdiv_rn(a, P.Rf);
                    }
                }
            }
            if (pm) {
                const uint32_t below = __popc(pmask & ((1u << (4 * k)) - 1u));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if ((pm >> j) & 1u) {
                        const uint64_t idx = (uint64_t)(pbase + pexcl + below + __popc(pm & ((1u << j) - 1u)));
                        pe[j] = idx * R;
                    }
                }
            }
        }

        float wold_keep[MODE == kSync ? R : 1][4];
        float acc[4] = {0.f, 0.f, 0.f, 0.f};

#pragma unroll
        for (int i0 = 0; i0 < R; i0 += RG) {
            // -- load phase: everything this group needs, issued back to back --
            float4 w4[RG], g4[RG], m4[RG], v4[RG];
            float old[RG][4], dd[RG][4];
#pragma unroll
            for (int ii = 0; ii < RG; ++ii) {
                const uint64_t off = (uint64_t)(i0 + ii) * stride + mu;
                w4[ii] = ld_stream(st.W + off);
                g4[ii] = ld_stream(G + off);
                m4[ii] = ld_stream(st.M + off);
                v4[ii] = ld_stream(st.V + off);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    old[ii][j] = 0.f;
                    dd[ii][j] = 0.f;
                    if constexpr (MODE != kSync) {
                        if ((cm >> j) & 1u) {
                            old[ii][j] = ring_cons[ce[j] + (i0 + ii)];
                            dd[ii][j] = st.D[(mu + j) * R + (i0 + ii)];
                        }
                    }
                }
            }
            // -- compute and write back, one replica at a time --
#pragma unroll
            for (int ii = 0; ii < RG; ++ii) {
                const int i = i0 + ii;
                const uint64_t off = (uint64_t)i * stride + mu;
                const float w[4] = {w4[ii].x, w4[ii].y, w4[ii].z, w4[ii].w};
                const float g[4] = {g4[ii].x, g4[ii].y, g4[ii].z, g4[ii].w};
                float m[4] = {m4[ii].x, m4[ii].y, m4[ii].z, m4[ii].w};
                float v[4] = {v4[ii].x, v4[ii].y, v4[ii].z, v4[ii].w};
                float wh[4], wn[4];
                adamw_group<GEN, 4>(P, w, g, m, v, wh);
#pragma unroll
                for (int c = 0; c < 4; ++c) wn[c] = wh[c];
                st_stream(st.M + off, m);
                st_stream(st.V + off, v);

                if constexpr (MODE != kSync) {
                    // Eq. "ema" + corrected averaging on S^{t-tau}
                    if (cm) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            if ((cm >> j) & 1u) {
                                const float diff = __fsub_rn(wh[j], old[ii][j]);
                                const float dn = staleness<GEN>(P, dd[ii][j], diff);
                                st.D[(mu + j) * R + i] = dn;
                                wn[j] = __fadd_rn(abar[j], dn);
                            }
                        }
                    }
                    // snapshot of the local iterate on S^t
                    if (pm) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if ((pm >> j) & 1u) ring_prod[pe[j] + i] = wh[j];
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        acc[c] = (i == 0) ? on_wire<GEN>(P, wh[c]) : __fadd_rn(acc[c], on_wire<GEN>(P, wh[c]));
                        wold_keep[i][c] = w[c];
                    }
                }

                // (synchronous mode with all four coordinates selected: the replica
                // mean below writes these float4 in one go, nothing to store yet)
                if (MODE != kSync || pm != 0xFu) {
                    st_stream(st.W + off, wn);
                    if (has_look) {   // Section 2.2: extrapolate the last update direction
                        float lk[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            lk[c] = __fadd_rn(wn[c], __fmul_rn(delta, __fsub_rn(wn[c], w[c])));
                        st_stream(st.LOOK + off, lk);
                    }
                }
            }
        }

        if constexpr (MODE == kSync) {
            // Eq. "sparta": coordinates of S^t take the replica mean.  The EMA
            // state stays exactly zero when tau = 0 (its sample is w^ - w^ = 0),
            // so the corrected value is mean + 0.
            if (pm == 0xFu) {   // whole float4 selected (always so at p = 1): vector stores
                float wnew[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) wnew[c] = __fadd_rn(__fdiv_rn(acc[c], P.Rf), 0.0f);
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const uint64_t off = (uint64_t)i * stride + mu;
                    st_stream(st.W + off, wnew);
                    if (has_look) {
                        float lk[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            lk[c] = __fadd_rn(wnew[c],
                                              __fmul_rn(delta, __fsub_rn(wnew[c], wold_keep[i][c])));
                        st_stream(st.LOOK + off, lk);
                    }
                }
            } else if (pm) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if ((pm >> j) & 1u) {
                        const float wnew = __fadd_rn(__fdiv_rn(acc[j], P.Rf), 0.0f);
#pragma unroll
                        for (int i = 0; i < R; ++i) {
                            const uint64_t o1 = (uint64_t)i * stride + mu + j;
                            st.W[o1] = wnew;
                            if (has_look)
                                st.LOOK[o1] = __fadd_rn(
                                    wnew, __fmul_rn(delta, __fsub_rn(wnew, wold_keep[i][j])));
                        }
                    }
                }
            }
        }
    }
}

template <int R, int MODE, bool GEN>
__global__ void __launch_bounds__(kBlockThreads)
asyncmesh_step_kernel(const __grid_constant__ StepParams P)
{
    __shared__ StageDesc sd[kMaxStages];
    {
        const uint32_t words = P.S * (uint32_t)(sizeof(StageDesc) / 4);
        const uint32_t *src = reinterpret_cast<const uint32_t *>(P.stages);
        uint32_t *dst = reinterpret_cast<uint32_t *>(sd);
        for (uint32_t x = threadIdx.x; x < words; x += blockDim.x) dst[x] = src[x];
    }
    __syncthreads();

    const int lane = threadIdx.x & 31;
    constexpr uint32_t wpb = kBlockThreads / 32;
    const uint32_t n_warps = gridDim.x * wpb;
    uint32_t s = 0;
    for (uint32_t gc = blockIdx.x * wpb + (threadIdx.x >> 5); gc < P.total_chunks;
         gc += n_warps) {
        while (s + 1 < P.S && gc >= sd[s + 1].chunk_begin) ++s;
        process_chunk<R, MODE, GEN>(P, sd[s], P.G[s], s, gc - sd[s].chunk_begin, lane);
    }
}

}  // namespace amk
