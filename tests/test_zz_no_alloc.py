"""The allocation-free consensus-error entry point against the regular one.

Some users of the library run where nothing may allocate on the GPU (all device
memory belongs to their own pool, or an allocation's implicit synchronisation
is not acceptable).  ``asyncmesh_consensus_error_noalloc`` serves them with a
scratch array that is part of the library image.  This file is collected last,
so a run that stops at the first failure has already run every other test; it
also passes when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import synth_inputs as si
from tests.util import HP

pytestmark = pytest.mark.gpu


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    import paper_2601_22442_b200 as pkg
    R, numel = 4, [300_001, 70_000]
    g = pkg.AsyncMesh(R, numel, p=0.05, tau=1, ema_beta=0.9, **HP)
    for s, n in enumerate(numel):
        for i in range(R):   # replicas apart, so the error is not trivially zero
            g.init_params(s, si.normal_host(si.stream_key(3, si.KIND_INIT, 0, s, i), 0, n, 0.02),
                          replica=i)
    bufs = g.empty_grads()
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):            # second call reuses the scratch the first one left behind
        for s, n in enumerate(numel):
            si.grads_device(bufs[s], 11, call + 1, s, n)
        g.step(bufs)
        for s, n in enumerate(numel):
            want = g.consensus_error(s)
            ptr, stride = g.lookahead_weights(s, 0)
            before = torch.cuda.memory_allocated()
            free_before = torch.cuda.mem_get_info()[0]      # the driver's own count of free bytes
            got = pkg.asyncmesh_consensus_error_noalloc(ptr, R, n, stride, device=0, stream=stream)
            assert torch.cuda.memory_allocated() == before
            if call == 1:   # module loaded, scratch address known: a raw cudaMalloc would show here
                assert torch.cuda.mem_get_info()[0] == free_before
            assert want > 0
            # both reduce in double; only the summation order differs
            assert abs(got - want) <= 1e-9 * want, (call, s, got, want)
    # and against plain numpy, so the two entry points cannot be wrong together
    W = g.get(1, "w").astype(np.float64)
    ref = ((W - W.mean(0)) ** 2).sum()
    ptr, stride = g.lookahead_weights(1, 0)
    got = pkg.asyncmesh_consensus_error_noalloc(ptr, R, numel[1], stride, stream=stream)
    assert abs(got - ref) <= 1e-9 * ref


def test_noalloc_rejects_sizes_beyond_its_scratch():
    import paper_2601_22442_b200 as pkg
    w = torch.zeros(16, device="cuda")
    with pytest.raises(pkg.AsyncMeshError) as e:
        pkg.asyncmesh_consensus_error_noalloc(w.data_ptr(), 1, (1 << 28) + 1, (1 << 28) + 1)
    assert e.value.code == -1 and "exceeds the built-in scratch" in str(e.value)
    with pytest.raises(pkg.AsyncMeshError):
        pkg.asyncmesh_consensus_error_noalloc(0, 1, 16, 16)
