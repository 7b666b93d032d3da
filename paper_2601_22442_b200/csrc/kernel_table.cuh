// Which step kernel serves which configuration.  The instantiations (every
// replica count 1..16, three ring modes, two pipelined shapes) take minutes to
// compile in one translation unit, so step_kernels.cu is compiled in seven parts
// side by side; this header is what the host code sees of them.
#pragma once
#include "step_kernel_pipelined.cuh"

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
// Pipelined kernel.  shape: 1 wide, 2 narrow (both compact ring), 3 narrow synchronous.
KernelChoice pick_pipelined_few_common(uint32_t R, int shape, uint32_t S);     // R = 1..8
KernelChoice pick_pipelined_few_general(uint32_t R, int shape, uint32_t S);
KernelChoice pick_pipelined_many_common(uint32_t R, int shape, uint32_t S);    // R = 9..16
KernelChoice pick_pipelined_many_general(uint32_t R, int shape, uint32_t S);

}  // namespace amk
