// Which step kernel serves which configuration.  The instantiations (every
// replica count 1..16, three ring modes, two pipelined shapes) take minutes to
// compile in one translation unit, so step_kernels.cu is compiled in twelve parts
// side by side; this header is what the host code sees of them.
#pragma once
#include "step_kernel_pipelined.cuh"
#include "step_kernel_owner.cuh"

namespace amk {

typedef void (*step_fn)(const StepParams);

struct KernelChoice {
    step_fn fn = nullptr;
    size_t smem = 0;              // dynamic shared memory per block
    int threads = kBlockThreads;  // block size
    int max_blocks_per_sm = 0;    // 0: as many as fit
};

// general: the form that also knows the E4M3 exchange and the eager staleness
// estimate.  Direct kernel:
KernelChoice pick_direct_few(uint32_t R, int mode, bool general);    // R = 1..8
KernelChoice pick_direct_many_common(uint32_t R, int mode);          // R = 9..16
KernelChoice pick_direct_many_general(uint32_t R, int mode);
KernelChoice pick_direct_stored(uint32_t R, int mode, bool general);  // R = 1..16; kDenseBf16 or kDenseE4m3
// Pipelined kernel.  shape: 1 wide, 2 narrow (both compact ring), 3 narrow synchronous.
KernelChoice pick_pipelined_few_common(uint32_t R, int shape, uint32_t S);     // R = 1..8
KernelChoice pick_pipelined_few_general(uint32_t R, int shape, uint32_t S);
KernelChoice pick_pipelined_many_common(uint32_t R, int shape, uint32_t S);    // R = 9..16
KernelChoice pick_pipelined_many_general(uint32_t R, int shape, uint32_t S);
// Owner kernel (R = 1..4; R = 5..8 for kSync; R = 6 and 8 for kCompact as two passes over each group).  mode: kCompact or kSync; entries: ring / d entries per group
// of 256 coordinates fetched ahead (kOwnerEntriesFew, kOwnerEntriesMid or kOwnerEntriesMany).
// Shape, measured on the 1B layout (R = 4, p = 0.05, ms per step): one replica row per
// unit and 8 coordinates per lane (1 KB contiguous per array row and request) 22.7;
// two rows per unit 23.0; 4 coordinates per lane (512-byte requests) 24.3 to 24.8 whatever
// the rows per unit: the request size is worth 1 ms, also with nothing selected.
// Stages of the copy pipeline: three with the ring; two for tau = 0, where nothing but the dense stream
// is in flight (1B layout, tau = 0: 19.2 against 20.4 ms per step; 350M layout: 13.9 against 14.2; with the
// ring two stages lose: 25.3 against 22.6 at p = 0.05, 23.1 against 20.7 at p = 0.01, also when the sparse
// copies are tracked apart from the dense ones).
constexpr int owner_stages(int mode) { return mode == kSync ? 2 : 3; }
constexpr int kOwnerV = 2;
// Entries fetched ahead per group: 32 keep three blocks per SM with room to spare; 64 still fit three blocks
// (72 KB each) and serve the medium subsets, where half of the groups then read some entries in place; 128 take
// the kernel down to two blocks per SM.  1B layout, tau = 4, ms per step with 64 against 128: p = 0.1 23.85 /
// 24.33, 0.15 24.66 / 25.61, 0.25 26.33 / 26.62, 0.5 30.43 / 30.31 (96: 25.1, 25.8, 26.7, 33.9).  In two passes
// (six and eight replicas) 64 lose to 128 (350M layout, p = 0.25: 19.3 / 18.8), so that form knows two sizes.
constexpr int kOwnerEntriesFew = 32, kOwnerEntriesMid = 64, kOwnerEntriesMany = 128;
// replica rows per unit: one up to four replicas; with more, two where that divides R (8 KB units)
constexpr int owner_ru(int R) { return (R > 4 && R % 2 == 0) ? 2 : 1; }
KernelChoice pick_owner_common(uint32_t R, int mode, int entries, uint32_t S);
KernelChoice pick_owner_general(uint32_t R, int mode, int entries, uint32_t S);
KernelChoice pick_owner_tracking(uint32_t R, int mode, int entries, uint32_t S);   // common form + consensus error
KernelChoice pick_owner_nadamw(uint32_t R, int mode, int entries, uint32_t S);     // common form, NAdamW for AdamW

}  // namespace amk
