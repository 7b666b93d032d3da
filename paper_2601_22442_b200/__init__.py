"""B200 (sm_100a) implementation of the AsyncMesh per-step parameter update:
per-replica AdamW, asynchronous sparse averaging with tau-step-stale values,
EMA staleness correction and pipeline look-ahead, fused in one CUDA kernel
behind a C ABI (``include/asyncmesh.h``).  This package is the thin Python
binding of that library plus the workload layouts."""
from .binding import (AsyncMesh, AsyncMeshError, TorchAllocator, asyncmesh_create,  # noqa: F401
                      asyncmesh_destroy, asyncmesh_init_params, asyncmesh_step,
                      asyncmesh_step_ex, asyncmesh_step_host, asyncmesh_step_host_ex,
                      asyncmesh_kernel_name, asyncmesh_lookahead_weights,
                      asyncmesh_read_params, asyncmesh_read_state, asyncmesh_read_state_range,
                      asyncmesh_subset_mask,
                      asyncmesh_consensus_error, asyncmesh_consensus_error_noalloc,
                      asyncmesh_ema_variance,
                      asyncmesh_debug_philox,
                      asyncmesh_last_error, load)
from .layouts import DEFAULT_HP, llama_stage_numel, workloads  # noqa: F401
from .schedules import ema_coefficient, learning_rate  # noqa: F401
