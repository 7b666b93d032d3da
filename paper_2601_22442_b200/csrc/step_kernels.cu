// Instantiations of the step kernels.  Compiled twelve times, -DAM_PART=0..11:
// 0 direct kernel R = 1..8; 1 direct kernel R = 9..16, common form; 2 the same,
// general form; 3 / 4 pipelined kernel R = 1..8, common / general form; 5 / 6
// pipelined kernel R = 9..16, common / general form; 7 / 8 / 9 owner kernel R = 1..8,
// common / general / consensus-tracking form; 10 direct kernel with the dense ring kept as
// exchanged (bfloat16 / E4M3 slots), R = 1..16, both forms; 11 owner kernel, common form with NAdamW.
#include "kernel_table.cuh"

#ifndef AM_PART
#error "compile with -DAM_PART=0..11"
#endif

namespace amk {

#if AM_PART == 10   // direct kernel, ring slots in the exchanged precision

template <int R>
static KernelChoice stored(int mode, bool general)
{
    KernelChoice c;
    if (mode == kDenseBf16)
        c.fn = general ? asyncmesh_step_kernel<R, kDenseBf16, true> : asyncmesh_step_kernel<R, kDenseBf16, false>;
    else if (mode == kDenseE4m3)
        c.fn = general ? asyncmesh_step_kernel<R, kDenseE4m3, true> : asyncmesh_step_kernel<R, kDenseE4m3, false>;
    return c;
}

KernelChoice pick_direct_stored(uint32_t R, int mode, bool general)
{
    switch (R) {
    case 1: return stored<1>(mode, general);
    case 2: return stored<2>(mode, general);
    case 3: return stored<3>(mode, general);
    case 4: return stored<4>(mode, general);
    case 5: return stored<5>(mode, general);
    case 6: return stored<6>(mode, general);
    case 7: return stored<7>(mode, general);
    case 8: return stored<8>(mode, general);
    case 9: return stored<9>(mode, general);
    case 10: return stored<10>(mode, general);
    case 11: return stored<11>(mode, general);
    case 12: return stored<12>(mode, general);
    case 13: return stored<13>(mode, general);
    case 14: return stored<14>(mode, general);
    case 15: return stored<15>(mode, general);
    case 16: return stored<16>(mode, general);
    default: return KernelChoice();
    }
}

#elif AM_PART < 3

template <int R, bool GEN>
static KernelChoice direct_as(int mode)
{
    KernelChoice c;
    switch (mode) {
    case kSync: c.fn = asyncmesh_step_kernel<R, kSync, GEN>; break;
    case kDense: c.fn = asyncmesh_step_kernel<R, kDense, GEN>; break;
    default: c.fn = asyncmesh_step_kernel<R, kCompact, GEN>;
    }
    return c;
}

#if AM_PART == 0
template <int R>
static KernelChoice direct(int mode, bool general)
{
    return general ? direct_as<R, true>(mode) : direct_as<R, false>(mode);
}
KernelChoice pick_direct_few(uint32_t R, int mode, bool general)
{
    switch (R) {
    case 1: return direct<1>(mode, general);
    case 2: return direct<2>(mode, general);
    case 3: return direct<3>(mode, general);
    case 4: return direct<4>(mode, general);
    case 5: return direct<5>(mode, general);
    case 6: return direct<6>(mode, general);
    case 7: return direct<7>(mode, general);
    case 8: return direct<8>(mode, general);
    default: return KernelChoice();
    }
}
#else
constexpr bool kGeneral = (AM_PART == 2);
#if AM_PART == 1
KernelChoice pick_direct_many_common(uint32_t R, int mode)
#else
KernelChoice pick_direct_many_general(uint32_t R, int mode)
#endif
{
    switch (R) {
    case 9: return direct_as<9, kGeneral>(mode);
    case 10: return direct_as<10, kGeneral>(mode);
    case 11: return direct_as<11, kGeneral>(mode);
    case 12: return direct_as<12, kGeneral>(mode);
    case 13: return direct_as<13, kGeneral>(mode);
    case 14: return direct_as<14, kGeneral>(mode);
    case 15: return direct_as<15, kGeneral>(mode);
    case 16: return direct_as<16, kGeneral>(mode);
    default: return KernelChoice();
    }
}
#endif

#elif AM_PART >= 7   // owner kernel

constexpr bool kGeneral = (AM_PART == 8);
constexpr bool kTracking = (AM_PART == 9);   // the common form that also accumulates the consensus error
constexpr bool kNadam = (AM_PART == 11);     // the common form with NAdamW as its optimizer

template <int R, int E, int MODE>
static KernelChoice owner_as(uint32_t S)
{
    KernelChoice c;
    c.fn = asyncmesh_step_kernel_owner<R, owner_ru(R), kOwnerV, owner_stages(MODE), E, MODE, kGeneral, kTracking, kNadam>;
    c.threads = kOwnerThreads;
    c.smem = (size_t)pipe_table_bytes(S) +
             (size_t)(kOwnerThreads / 32) * OwnerCfg<R, owner_ru(R), kOwnerV, E>::warp_bytes(owner_stages(MODE));
    return c;
}

// Twice as many replicas as a lane holds: two passes over each group (compact ring; not the tracking form).
template <int RH, int E>
static KernelChoice owner_two_passes_as(uint32_t S)
{
    KernelChoice c;
    if constexpr (!kTracking) {
        c.fn = asyncmesh_step_kernel_owner<RH, owner_ru(RH), kOwnerV, owner_stages(kCompact), E, kCompact, kGeneral,
                                           false, kNadam, 2>;
        c.threads = kOwnerThreads;
        c.smem = (size_t)pipe_table_bytes(S) +
                 (size_t)(kOwnerThreads / 32) *
                     OwnerCfg<RH, owner_ru(RH), kOwnerV, E, 2>::warp_bytes(owner_stages(kCompact));
    }
    return c;
}
template <int RH>
static KernelChoice owner_two_passes(int entries, uint32_t S)
{
    return entries == kOwnerEntriesFew ? owner_two_passes_as<RH, kOwnerEntriesFew>(S)
                                       : owner_two_passes_as<RH, kOwnerEntriesMany>(S);
}

template <int R>
static KernelChoice owner(int mode, int entries, uint32_t S)
{
    if (mode == kSync) return owner_as<R, 1, kSync>(S);
    return entries == kOwnerEntriesFew   ? owner_as<R, kOwnerEntriesFew, kCompact>(S)
           : entries == kOwnerEntriesMid ? owner_as<R, kOwnerEntriesMid, kCompact>(S)
                                         : owner_as<R, kOwnerEntriesMany, kCompact>(S);
}

#if AM_PART == 7
KernelChoice pick_owner_common(uint32_t R, int mode, int entries, uint32_t S)
#elif AM_PART == 8
KernelChoice pick_owner_general(uint32_t R, int mode, int entries, uint32_t S)
#elif AM_PART == 9
KernelChoice pick_owner_tracking(uint32_t R, int mode, int entries, uint32_t S)
#else
KernelChoice pick_owner_nadamw(uint32_t R, int mode, int entries, uint32_t S)
#endif
{
    switch (R) {
    case 1: return owner<1>(mode, entries, S);
    case 2: return owner<2>(mode, entries, S);
    case 3: return owner<3>(mode, entries, S);
    case 4: return owner<4>(mode, entries, S);
    // five to eight replicas: all of them in registers for the synchronous mode only; with the ring, six
    // and eight replicas as two passes of three and four
    case 5: return mode == kSync ? owner_as<5, 1, kSync>(S) : KernelChoice();
    case 6: return mode == kSync ? owner_as<6, 1, kSync>(S) : owner_two_passes<3>(entries, S);
    case 7: return mode == kSync ? owner_as<7, 1, kSync>(S) : KernelChoice();
    case 8: return mode == kSync ? owner_as<8, 1, kSync>(S) : owner_two_passes<4>(entries, S);
    default: return KernelChoice();
    }
}

#else   // pipelined kernel

constexpr bool kGeneral = (AM_PART == 4 || AM_PART == 6);

template <int R, class SH, int MODE>
static KernelChoice pipelined_as(uint32_t S)
{
    KernelChoice c;
    c.fn = asyncmesh_step_kernel_pipelined<R, kPipeStages, SH, MODE, kGeneral>;
    c.threads = kPipeThreads;
    c.max_blocks_per_sm = kPipeBlocksPerSM;
    c.smem = (size_t)pipe_table_bytes(S) +
             (size_t)(kPipeThreads / 32) * PipeCfg<R, SH>::warp_bytes(kPipeStages);
    return c;
}

template <int R>
static KernelChoice pipelined(int shape, uint32_t S)
{
    switch (shape) {
    case 1: return pipelined_as<R, PipeWide, kCompact>(S);
    case 2: return pipelined_as<R, PipeNarrow, kCompact>(S);
    case 3: return pipelined_as<R, PipeNarrow, kSync>(S);
    default: return KernelChoice();
    }
}

#if AM_PART == 3
KernelChoice pick_pipelined_few_common(uint32_t R, int shape, uint32_t S)
#elif AM_PART == 4
KernelChoice pick_pipelined_few_general(uint32_t R, int shape, uint32_t S)
#elif AM_PART == 5
KernelChoice pick_pipelined_many_common(uint32_t R, int shape, uint32_t S)
#else
KernelChoice pick_pipelined_many_general(uint32_t R, int shape, uint32_t S)
#endif
{
    switch (R) {
#if AM_PART <= 4
    case 1: return pipelined<1>(shape, S);
    case 2: return pipelined<2>(shape, S);
    case 3: return pipelined<3>(shape, S);
    case 4: return pipelined<4>(shape, S);
    case 5: return pipelined<5>(shape, S);
    case 6: return pipelined<6>(shape, S);
    case 7: return pipelined<7>(shape, S);
    case 8: return pipelined<8>(shape, S);
#else
    case 9: return pipelined<9>(shape, S);
    case 10: return pipelined<10>(shape, S);
    case 11: return pipelined<11>(shape, S);
    case 12: return pipelined<12>(shape, S);
    case 13: return pipelined<13>(shape, S);
    case 14: return pipelined<14>(shape, S);
    case 15: return pipelined<15>(shape, S);
    case 16: return pipelined<16>(shape, S);
#endif
    default: return KernelChoice();
    }
}

#endif

}  // namespace amk
