"""Guard words around every device allocation of the library.

The memory checker of the toolkit is not available on the machines these tests run
on, so out-of-range writes are looked for directly: the library gets its memory
through allocator callbacks that put 4 KB of a known pattern in front of and behind
every block.  After the steps every pad must still hold the pattern, and the padding
columns of the state rows (row stride = N rounded up to 32 floats) must still be zero
beyond the last float4 group that holds a coordinate."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from tests.util import HP

pytestmark = pytest.mark.gpu

PAD = 4096
PATTERN = 0xA5


def am():
    import paper_2601_22442_b200 as pkg
    return pkg


def guard_allocator(device=0):
    from paper_2601_22442_b200.binding import TorchAllocator

    class GuardAllocator(TorchAllocator):
        def __init__(self, dev):
            super().__init__(dev)
            self.blocks = {}          # user pointer -> (tensor, nbytes)
            self.violations = []

        def _alloc(self, _ctx, nbytes):
            n = int(nbytes)
            t = torch.empty(n + 2 * PAD, dtype=torch.uint8, device=self._device)
            t[:PAD].fill_(PATTERN)
            t[PAD + n:].fill_(PATTERN)
            torch.cuda.synchronize()
            ptr = t.data_ptr() + PAD
            assert ptr % 256 == 0
            self.blocks[ptr] = (t, n)
            return ptr

        def check(self, ptr):
            t, n = self.blocks[ptr]
            lo = int((t[:PAD] != PATTERN).sum().item())
            hi = int((t[PAD + n:] != PATTERN).sum().item())
            if lo or hi:
                self.violations.append((n, lo, hi))

        def check_all(self):
            torch.cuda.synchronize()
            for ptr in list(self.blocks):
                self.check(ptr)
            return self.violations

        def _free(self, _ctx, ptr):
            torch.cuda.synchronize()
            self.check(int(ptr))
            del self.blocks[int(ptr)]

    return GuardAllocator(device)


def padding_is_clean(alloc, R, numel):
    """Every block of the size of a state array [R][stride] (or d's [stride][R]): zero in
    the padding columns beyond the last float4 group, in one of the two layouts."""
    bad = []
    by_stride = {}
    for N in numel:                       # stages of equal stride share a block size: take the widest
        stride = (N + 31) // 32 * 32
        by_stride[stride] = max(by_stride.get(stride, 0), N)
    for stride, N in by_stride.items():
        n4 = (N + 3) // 4 * 4
        if stride == n4 or stride < 1024:     # (small blocks: the index tables come in the same sizes)
            continue
        for ptr, (t, n) in alloc.blocks.items():
            if n != R * stride * 4:
                continue
            x = t[PAD:PAD + n].view(torch.float32)
            rows = bool((x.view(R, stride)[:, n4:] == 0).all().item())
            tail = bool((x[N * R:] == 0).all().item())
            if not (rows or tail):
                bad.append((N, n))
    return bad


def run(R, numel, p, tau, flags=0, steps=None, expect_overflow=False, **kw):
    alloc = guard_allocator()
    steps = steps if steps is not None else 2 * tau + 3
    g = am().AsyncMesh(R, numel, p=p, tau=tau, ema_beta=0.9, flags=flags, allocator=alloc, **dict(HP, **kw))
    for s, n in enumerate(numel):
        g.init_params(s, si.init_weights_host(0x1217, s, 0, n))
    bufs = g.empty_grads()
    for b in bufs:
        b.zero_()
    for t in range(1, steps + 1):
        for s, n in enumerate(numel):
            si.grads_device(bufs[s], 0x6AD5, t, s, n)
        g.step(bufs)
    torch.cuda.synchronize()
    if expect_overflow:
        with pytest.raises(Exception):
            g.status()
    else:
        g.status()
        for s in range(len(numel)):       # the read paths allocate and free temporaries too
            g.get(s, "d")
            g.read_params(s)
            g.consensus_error(s)
            g.ema_variance(s)
            g.subset_mask(s, steps)
    assert alloc.check_all() == []
    assert padding_is_clean(alloc, R, numel) == []
    g.destroy()
    assert alloc.violations == [] and alloc.blocks == {}


RAGGED = [1, 3, 4, 5, 127, 128, 129, 1023, 1024, 1025, 4099]


@pytest.mark.parametrize("R,p,tau,flags", [
    (2, 0.5, 1, 0), (4, 0.05, 2, 0), (4, 0.3, 2, 0), (3, 0.2, 0, 0), (4, 1.0, 0, 0), (4, 1.0, 2, 0),
    (8, 0.05, 2, 0), (8, 0.3, 1, 0), (5, 0.3, 0, 0), (4, 0.05, 2, 2), (4, 0.4, 2, 4), (4, 0.4, 0, 4),
    (4, 0.3, 2, 32), (1, 0.3, 2, 0), (2, 0.9, 2, 256), (4, 0.9, 3, 256), (3, 0.6, 1, 256),
    (8, 0.05, 2, 256), (6, 0.4, 2, 256), (8, 1.0, 1, 256), (8, 0.3, 1, 4)])
def test_ragged_stage_sizes_keep_inside_their_blocks(R, p, tau, flags):
    run(R, RAGGED, p, tau, flags)


def test_many_stages_many_replicas_long_delay():
    run(3, [517 + 33 * s for s in range(64)], 0.1, 2)          # 64 stages
    run(16, [4099, 130], 0.2, 2)                               # 16 replicas, both kernels
    run(16, [4099, 130], 0.2, 2, flags=2)
    run(12, [4099], 0.05, 1)
    run(2, [4099, 77], 0.1, 64, steps=70)                      # the longest delay
    run(4, [4099, 77], 0.3, 64, steps=70, avg_interval=16)


def test_paths_for_more_selected_coordinates_than_the_fast_route_holds():
    run(8, [9000, 1024 * 3 + 5], 0.9, 2, flags=4)              # pipelined kernel: stash overflow, in place
    run(4, [9000, 1024 * 3 + 5], 0.9, 2, flags=4)
    run(4, [9000, 1024 * 3 + 5], 1.0, 2, flags=256)            # owner kernel: beyond the entries fetched ahead
    run(4, [9000, 1024 * 3 + 5], 0.05, 2, flags=1, expect_overflow=True)    # ring slot too small: dropped, reported
    run(8, [9000, 1024 * 3 + 5], 0.05, 2, flags=1, expect_overflow=True)
    run(8, [9000, 1024 * 3 + 5], 0.05, 2, flags=1 | 256, expect_overflow=True)   # owner kernel in two passes
    run(8, [9000, 1024 * 3 + 5], 1.0, 2, flags=256)                              # ... beyond the entries fetched ahead
    run(4, [9000], 0.3, 2, flags=128)                          # previous weights kept aside


def test_general_forms():
    run(4, [4099, 77], 0.3, 2, flags=64)                       # 8-bit exchange
    run(8, [4099, 77], 0.3, 2, flags=64)
    run(4, [4099, 77], 0.3, 2, flags=16)
    run(4, [4099, 77], 0.3, 2, optimizer="nadamw")
    run(8, [4099, 77], 0.3, 2, correction="eager")


def test_ring_kept_as_exchanged():
    # (delays chosen so that the ring block is not of a state array's size)
    run(4, RAGGED, 0.4, 1, flags=16 | 1024)
    run(8, RAGGED, 1.0, 3, flags=16 | 1024)
    run(3, RAGGED, 0.4, 2, flags=64 | 1024)
    run(16, [4099, 130], 1.0, 1, flags=64 | 1024)
    run(5, [4099, 130], 0.7, 3, flags=64 | 1024, optimizer="nadamw")
