"""GPU parity: the CUDA library, called through its C ABI, against the CPU
oracle on the same seeded inputs.  Bars: the selected coordinate sets are
bit-identical; w, m, v, d and the look-ahead agree within 1e-6 relative error
(|a-b| / max(|a|,|b|)) -- and, because both sides perform the same IEEE
operations in the same order, they are in fact expected to be bit-identical,
which the tests also assert."""
import ctypes
import os

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests.util import HP, STATE_NAMES, DevicePtr, relerr

pytestmark = pytest.mark.gpu

TOL = 1e-6


def am():
    import paper_2601_22442_b200 as pkg
    return pkg


def make_pair(R, numel, p, tau, lam, delays=None, seed=0x5EED, hp=HP, same_init=True,
              init_seed=0x1217, flags=0, avg_interval=1, optimizer="adamw", exchange="fp32",
              correction="ema", snapshot="own-fp32"):
    flags |= {"fp32": 0, "bf16": 16, "fp8": 64}[exchange]
    flags |= {"own-fp32": 0, "as-exchanged": 1024}[snapshot]
    o = oracle.Oracle(R, numel, p=p, tau=tau, ema_beta=lam, seed=seed,
                      lookahead_delay=delays, avg_interval=avg_interval, optimizer=optimizer,
                      exchange=exchange, correction=correction, snapshot=snapshot, **hp)
    g = am().AsyncMesh(R, numel, p=p, tau=tau, ema_beta=lam, seed=seed,
                       lookahead_delay=delays, flags=flags, avg_interval=avg_interval,
                       optimizer=optimizer, correction=correction, **hp)
    for s, n in enumerate(numel):
        if same_init:
            w0 = si.init_weights_host(init_seed, s, 0, n)
            o.init_params(s, w0)
            g.init_params(s, w0)
        else:
            for i in range(R):
                w0 = si.normal_host(si.stream_key(init_seed, si.KIND_INIT, 0, s, i), 0, n, 0.02)
                o.init_params(s, w0, replica=i)
                g.init_params(s, w0, replica=i)
    return o, g


def step_both(o, g, t, grad_seed=0x6AD5, bufs=None, **kw):
    hg = [si.grads_host(grad_seed, t, s, o.R, 0, n) for s, n in enumerate(o.numel)]
    bufs = bufs if bufs is not None else g.empty_grads()
    for s, n in enumerate(o.numel):
        bufs[s][:, :n].copy_(torch.from_numpy(hg[s]))
    if kw:
        o.step(hg, ema_beta_t=kw.get("ema_beta_t", -1.0), lr_t=kw.get("lr_t", -1.0))
        g.step(bufs, ema_beta_t=kw.get("ema_beta_t", -1.0), lr_t=kw.get("lr_t", -1.0))
    else:
        o.step(hg)
        g.step(bufs)
    return bufs


def compare(o, g, exact=True):
    for s in range(o.S):
        for name in STATE_NAMES:
            a, b = o.get(s, name), g.get(s, name)
            err = relerr(a, b)
            assert err <= TOL, (s, name, err)
            if exact:
                assert np.array_equal(a, b), (s, name, "not bit-identical", err)


def run_case(R, numel, p, tau, lam, steps, delays=None, check_masks=(1, 2), **kw):
    o, g = make_pair(R, numel, p, tau, lam, delays=delays, **kw)
    bufs = None
    for t in range(1, steps + 1):
        bufs = step_both(o, g, t, bufs=bufs)
        if t in check_masks:
            for s in range(o.S):
                assert np.array_equal(o.subset_mask(s, t), g.subset_mask(s, t)), (s, t)
    g.status()
    compare(o, g)
    assert g.step_count == steps == o.step_count
    return o, g


# ---- the generator ------------------------------------------------------------------

def test_device_philox_equals_oracle_and_curand():
    rng = np.random.default_rng(1)
    n = 1_000_000
    ctr = rng.integers(0, 1 << 32, size=(n, 4), dtype=np.uint64).astype(np.uint32)
    key = rng.integers(0, 1 << 32, size=(n, 2), dtype=np.uint64).astype(np.uint32)
    ctr[0], key[0] = 0, 0
    ctr[1], key[1] = 0xFFFFFFFF, 0xFFFFFFFF
    dev = am().asyncmesh_debug_philox(ctr, key)
    assert tuple(dev[0]) == (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)
    # CPU oracle on a sample (ctypes call per block is slow)
    for k in list(range(0, 2000)) + list(range(n - 100, n)):
        assert tuple(int(x) for x in dev[k]) == oracle.philox4x32_10(ctr[k].tolist(), key[k].tolist())
    # the CUDA toolkit's own routine, on every pair
    path = os.path.join(os.path.dirname(__file__), "libcurand_philox_check.so")
    if not os.path.exists(path):
        import subprocess
        subprocess.run(["nvcc", "-O2", "-gencode", "arch=compute_100a,code=sm_100a", "-Xcompiler",
                        "-fPIC", "-shared", "-o", path, path.replace("lib", "", 1).replace(".so", ".cu")],
                       check=True)
    L = ctypes.CDLL(path)
    L.curand_philox_check.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_uint64]
    ref = np.empty_like(ctr)
    assert L.curand_philox_check(ctr.ctypes.data, key.ctypes.data, ref.ctypes.data, n) == 0
    assert np.array_equal(dev, ref)


@pytest.mark.parametrize("p", [0.0, 2.0 ** -32, 0.05, 0.25, 1.0])
def test_subset_masks_bit_exact(p):
    numel = [4099, 1 << 16, 5]
    o = oracle.Oracle(2, numel, p=p, tau=1, ema_beta=0.5, seed=0xDEADBEEFCAFE)
    g = am().AsyncMesh(2, numel, p=p, tau=1, ema_beta=0.5, seed=0xDEADBEEFCAFE)
    for s in range(3):
        for step in (1, 7, 1 << 20):
            assert np.array_equal(o.subset_mask(s, step), g.subset_mask(s, step))


def test_synthetic_inputs_device_equals_host():
    n = 100_003
    dst = torch.empty(n, dtype=torch.float32, device="cuda")
    key = si.stream_key(0x6AD5, si.KIND_GRAD, 9, 3, 2)
    si.normal_device(dst, key, 12345, 1e-3)
    assert np.array_equal(dst.cpu().numpy(), si.normal_host(key, 12345, n, 1e-3))


# ---- the step -----------------------------------------------------------------------------

@pytest.mark.parametrize("tau,p", [(1, 0.05), (2, 0.05), (4, 0.25), (0, 0.05), (0, 1.0),
                                   (1, 1.0), (3, 0.9), (2, 0.0)])
def test_modes_small(tau, p):
    # compact ring, dense ring, synchronous; several tiles and a ragged tail
    run_case(4, [5000, 3 * 1024 + 17], p, tau, 0.9, steps=3 * tau + 4)


def kernel_flag(name):
    from paper_2601_22442_b200 import binding
    return {"direct": binding.FLAG_DIRECT_KERNEL, "pipelined": binding.FLAG_PIPELINED_KERNEL,
            "owner": binding.FLAG_OWNER_KERNEL}[name]


@pytest.mark.parametrize("flag", ["direct", "pipelined", "owner"])
@pytest.mark.parametrize("R,p", [(4, 0.05), (8, 0.3), (3, 0.7), (2, 1.0), (5, 0.0), (1, 0.5)])
def test_all_synchronous_kernels(flag, R, p):
    # tau = 0 (Eq. "sparta") through the direct kernel, through the stash route and (up to
    # four replicas; beyond, the flag changes nothing) in the owning lane's registers
    f = kernel_flag(flag)
    run_case(R, [9000, 1024 * 3 + 5, 77], p, 0, 0.9, steps=5, flags=f)
    run_case(R, [5000], p, 0, 0.9, steps=6, flags=f, avg_interval=2, exchange="bf16")


@pytest.mark.parametrize("R", [1, 2, 3, 5, 7, 8, 12, 16])
def test_replica_counts(R):
    run_case(R, [2500], 0.3, 2, 0.9, steps=7)
    run_case(R, [2500], 0.05, 2, 0.9, steps=7)
    run_case(R, [2500], 0.3, 0, 0.9, steps=3)


@pytest.mark.parametrize("flag", ["direct", "pipelined", "owner"])
@pytest.mark.parametrize("R,p", [(4, 0.05), (8, 0.05), (3, 0.1), (4, 0.5), (8, 0.35), (2, 1.0), (5, 0.9),
                                 (1, 0.3), (4, 1.0), (6, 0.05), (6, 0.6), (8, 1.0)])
def test_all_compact_ring_kernels(flag, R, p):
    # the register-load kernel, the shared-memory pipelined kernel and the owner kernel are
    # three routes to the same numbers; large p forces the pipelined kernel through its
    # in-place path (more selected coordinates per sub-iteration than its stash holds) and
    # the owner kernel past the ring / d entries it fetches ahead; with six and eight replicas
    # the owner kernel walks every group twice, half of the replicas per pass (with five, and
    # with seven, the flag changes nothing)
    f = kernel_flag(flag)
    run_case(R, [9000, 1024 * 3 + 5, 77], p, 2, 0.9, steps=7, flags=f)


def test_two_pass_owner_kernel_features():
    from paper_2601_22442_b200 import binding
    f = binding.FLAG_OWNER_KERNEL
    sizes = [1, 3, 4, 5, 127, 128, 129, 1023, 1024, 1025, 4099]
    run_case(8, sizes, 0.4, 3, 0.7, steps=8, flags=f, delays=[k % 3 for k in range(len(sizes))])
    run_case(6, sizes, 0.05, 1, 0.9, steps=5, flags=f)
    run_case(8, [300000], 0.25, 4, 0.9, steps=11, flags=f, same_init=False)
    run_case(8, [6000, 77], 0.3, 2, 0.9, steps=8, flags=f, exchange="bf16")
    run_case(8, [6000, 77], 0.3, 2, 0.9, steps=8, flags=f, exchange="fp8")          # general form
    run_case(6, [6000, 77], 0.3, 2, 0.9, steps=8, flags=f, correction="eager")
    run_case(8, [6000, 77], 0.3, 2, 0.9, steps=8, flags=f, optimizer="nadamw")       # NAdamW form
    run_case(8, [6000, 77], 0.3, 4, 0.9, steps=12, flags=f, avg_interval=2)
    o, g = run_case(8, [20000], 0.3, 2, 0.9, steps=6)                                # the default there
    assert g.kernel_name() == "owner R=8 compact entries=128"
    # consensus tracking is not available in two passes: the flag changes nothing, the value is still right
    o, g = run_case(8, [20000], 0.3, 2, 0.9, steps=6, flags=binding.FLAG_TRACK_CONSENSUS)
    assert g.kernel_name() == "owner R=8 compact entries=128"
    assert abs(g.consensus_error(0) - o.consensus_error(0)) <= 1e-9 * o.consensus_error(0)


def test_ragged_stage_sizes():
    sizes = [1, 3, 4, 5, 127, 128, 129, 1023, 1024, 1025, 4099]
    run_case(2, sizes, 0.5, 1, 0.9, steps=5)
    run_case(3, sizes, 0.2, 2, 0.7, steps=6, delays=[k % 3 for k in range(len(sizes))])
    run_case(2, sizes, 1.0, 2, 0.7, steps=6)
    run_case(4, sizes, 0.4, 0, 0.7, steps=3)


@pytest.mark.parametrize("K,tau,p", [(2, 2, 0.05), (3, 6, 0.3), (2, 0, 0.3), (4, 4, 1.0), (2, 4, 0.7)])
def test_averaging_interval(K, tau, p):
    # subsets exchanged every K-th step only (all ring modes); in between purely local
    from paper_2601_22442_b200 import binding
    run_case(4, [5000, 1024 * 2 + 3], p, tau, 0.9, steps=4 * K + tau + 1, avg_interval=K)
    run_case(3, [5000], p, tau, 0.9, steps=3 * K + tau + 1, avg_interval=K,
             flags=binding.FLAG_DIRECT_KERNEL)
    run_case(8, [5000], p, tau, 0.9, steps=3 * K + tau + 1, avg_interval=K)   # eight replicas: whichever kernel is the default


@pytest.mark.parametrize("tau,p", [(2, 0.05), (0, 0.3), (1, 1.0), (2, 0.4)])
def test_nadamw(tau, p):
    # the paper's own optimizer for asynchronous pipelines (momentum 0.99)
    from paper_2601_22442_b200 import binding
    hp = dict(HP, beta1=0.99, weight_decay=0.01)
    run_case(4, [6000, 1024 + 9], p, tau, 0.9, steps=3 * tau + 6, optimizer="nadamw", hp=hp)
    run_case(3, [6000], p, tau, 0.9, steps=3 * tau + 6, optimizer="nadamw", hp=hp,
             flags=binding.FLAG_DIRECT_KERNEL)
    run_case(6, [6000], p, tau, 0.9, steps=3 * tau + 6, optimizer="nadamw", hp=hp)   # pipelined kernel
    run_case(4, [6000], p, tau, 0.9, steps=3 * tau + 6, optimizer="nadamw", hp=hp,
             flags=binding.FLAG_OWNER_KERNEL)       # owner kernel, NAdamW form (the default where AdamW has the owner kernel)
    run_case(4, [6000, 1024 + 9], p, tau, 0.9, steps=3 * tau + 6, optimizer="nadamw", hp=hp,
             flags=binding.FLAG_PIPELINED_KERNEL)   # pipelined kernel, general form
    run_case(2, [6000], p, tau, 0.9, steps=3 * tau + 6, optimizer="nadamw", hp=hp, correction="eager",
             flags=binding.FLAG_OWNER_KERNEL)       # owner kernel, general form
    if tau == 0:
        run_case(8, [6000, 77], p, tau, 0.9, steps=6, optimizer="nadamw", hp=hp)   # owner, two rows per unit


@pytest.mark.parametrize("tau,p", [(2, 0.05), (0, 0.3), (1, 1.0), (3, 0.4)])
def test_bf16_exchange(tau, p):
    # subsets exchanged in bfloat16: all three ring modes and both compact-ring kernels
    from paper_2601_22442_b200 import binding
    o, g = run_case(4, [6000, 1024 + 9], p, tau, 0.9, steps=3 * tau + 5, exchange="bf16")
    run_case(3, [6000], p, tau, 0.9, steps=3 * tau + 5, exchange="bf16",
             flags=binding.FLAG_DIRECT_KERNEL)
    run_case(4, [6000], p, tau, 0.9, steps=3 * tau + 5, exchange="bf16",
             flags=binding.FLAG_PIPELINED_KERNEL)
    # and it is not the fp32 exchange
    ref = oracle.Oracle(4, [6000, 1024 + 9], p=p, tau=tau, ema_beta=0.9, **HP)
    for s, n in enumerate([6000, 1024 + 9]):
        ref.init_params(s, si.init_weights_host(0x1217, s, 0, n))
    for t in range(1, 3 * tau + 6):
        ref.step([si.grads_host(0x6AD5, t, s, 4, 0, n) for s, n in enumerate([6000, 1024 + 9])])
    assert np.abs(ref.get(0, "w") - g.get(0, "w")).max() > 0


@pytest.mark.parametrize("tau,p", [(2, 0.05), (0, 0.3), (1, 1.0), (3, 0.4)])
def test_fp8_exchange(tau, p):
    # subsets exchanged in 8-bit floating point (E4M3): all ring modes, both compact-ring kernels
    from paper_2601_22442_b200 import binding
    o, g = run_case(4, [6000, 1024 + 9], p, tau, 0.9, steps=3 * tau + 5, exchange="fp8")
    run_case(3, [6000], p, tau, 0.9, steps=3 * tau + 5, exchange="fp8",
             flags=binding.FLAG_DIRECT_KERNEL)
    run_case(4, [6000], p, tau, 0.9, steps=3 * tau + 5, exchange="fp8",
             flags=binding.FLAG_OWNER_KERNEL)
    ref = oracle.Oracle(4, [6000, 1024 + 9], p=p, tau=tau, ema_beta=0.9, exchange="bf16", **HP)
    for s, n in enumerate([6000, 1024 + 9]):
        ref.init_params(s, si.init_weights_host(0x1217, s, 0, n))
    for t in range(1, 3 * tau + 6):
        ref.step([si.grads_host(0x6AD5, t, s, 4, 0, n) for s, n in enumerate([6000, 1024 + 9])])
    assert np.abs(ref.get(0, "w") - g.get(0, "w")).max() > 0    # nor is it the bfloat16 exchange


@pytest.mark.parametrize("exchange", ["bf16", "fp8"])
@pytest.mark.parametrize("R,tau,p,K", [(4, 2, 1.0, 1), (3, 1, 0.3, 1), (8, 3, 0.6, 1), (1, 2, 1.0, 1),
                                       (2, 4, 0.9, 2), (12, 2, 0.5, 1), (16, 1, 1.0, 1)])
def test_ring_kept_as_exchanged(exchange, R, tau, p, K):
    # second reading of the reduced-precision exchange: the ring holds 2- or 1-byte values and
    # the staleness sample is taken against them
    numel = [6000, 1024 + 9, 77]
    o, g = run_case(R, numel, p, tau, 0.9, steps=3 * tau + 5, exchange=exchange, snapshot="as-exchanged",
                    avg_interval=K)
    assert g.kernel_name() == "direct R=%d dense-%s" % (R, {"bf16": "bf16", "fp8": "e4m3"}[exchange])
    # it is not the first reading: d differs
    first = oracle.Oracle(R, numel, p=p, tau=tau, ema_beta=0.9, exchange=exchange, avg_interval=K, **HP)
    for s, n in enumerate(numel):
        first.init_params(s, si.init_weights_host(0x1217, s, 0, n))
    for t in range(1, 3 * tau + 6):
        first.step([si.grads_host(0x6AD5, t, s, R, 0, n) for s, n in enumerate(numel)])
    assert np.abs(first.get(0, "d") - g.get(0, "d")).max() > 0


def test_ring_kept_as_exchanged_general_form_and_schedules():
    run_case(4, [6000, 77], 0.5, 2, 0.9, steps=9, exchange="fp8", snapshot="as-exchanged", optimizer="nadamw")
    run_case(8, [6000, 77], 1.0, 2, 0.9, steps=9, exchange="bf16", snapshot="as-exchanged", correction="eager")
    o, g = make_pair(4, [5000], 0.7, 2, 0.9, exchange="bf16", snapshot="as-exchanged", same_init=False)
    bufs = None
    for t in range(1, 9):
        bufs = step_both(o, g, t, bufs=bufs, ema_beta_t=0.9 * 0.8 ** t, lr_t=3e-4 * (1 - t / 20))
    g.status()
    compare(o, g)


def test_ring_kept_as_exchanged_takes_half_or_a_quarter_of_the_ring_memory():
    from paper_2601_22442_b200 import binding
    from paper_2601_22442_b200.binding import TorchAllocator

    class Counting(TorchAllocator):
        def __init__(self):
            super().__init__(0)
            self.sizes = []

        def _alloc(self, ctx, nbytes):
            self.sizes.append(int(nbytes))
            return super()._alloc(ctx, nbytes)

    R, N, tau = 4, 1 << 20, 6
    ring = {}
    for name, flags in (("fp32", binding.FLAG_DENSE_RING), ("bf16", 16 | 1024), ("e4m3", 64 | 1024)):
        a = Counting()
        g = am().AsyncMesh(R, [N], p=1.0, tau=tau, ema_beta=0.9, flags=flags, allocator=a, **HP)
        g.destroy()
        # the ring is one block of tau slots of R x N values; nothing else is larger than a state array
        want = tau * R * N * {"fp32": 4, "bf16": 2, "e4m3": 1}[name]
        assert a.sizes.count(want) == 1, (name, sorted(a.sizes)[-8:])
        assert all(n <= R * N * 4 for n in a.sizes if n != want)
        ring[name] = sum(a.sizes)
    assert ring["fp32"] - ring["bf16"] == tau * R * N * 2 and ring["fp32"] - ring["e4m3"] == tau * R * N * 3


def test_fp8_conversion_on_the_device_covers_the_whole_format():
    # every E4M3 value, every midpoint between neighbours and its two fp32 neighbours pass
    # through one synchronous averaging step with R = 1 and p = 1: the result is the
    # snapshot as "the others" see it, i.e. the rounded value itself (mean of one, + 0)
    grid = []
    for e in range(16):
        for mant in range(8):
            if not (e == 15 and mant == 7):
                grid.append(mant / 8 * 2.0 ** -6 if e == 0 else (1 + mant / 8) * 2.0 ** (e - 7))
    xs = []
    for k, x in enumerate(grid):
        xs.append(x)
        if k + 1 < len(grid):
            mid = np.float32((x + grid[k + 1]) / 2)
            xs += [float(mid), float(np.nextafter(mid, np.float32(1e9))), float(np.nextafter(mid, np.float32(0)))]
    xs += [460.0, 1e6, 2.0 ** -11, 3e-5]
    xs = np.array(xs + [-v for v in xs], dtype=np.float32)
    hp = dict(HP, lr=1e-30, weight_decay=0.0)      # the optimizer step leaves w unchanged
    o = oracle.Oracle(1, [xs.size], p=1.0, tau=0, ema_beta=0.9, exchange="fp8", **hp)
    g = am().AsyncMesh(1, [xs.size], p=1.0, tau=0, ema_beta=0.9, flags=64, **hp)
    o.init_params(0, xs); g.init_params(0, xs)
    zero = np.zeros((1, xs.size), dtype=np.float32)
    bufs = g.empty_grads()
    bufs[0].zero_()
    o.step([zero]); g.step(bufs)
    want = np.array([oracle.exchanged(float(x), "fp8") for x in xs], dtype=np.float32)
    assert np.array_equal(o.get(0, "w")[0], want)
    assert np.array_equal(g.get(0, "w")[0], want)


@pytest.mark.parametrize("p,tau,K", [(1.0, 2, 2), (1.0, 4, 4), (0.05, 2, 1), (0.3, 3, 3), (0.5, 0, 1)])
def test_eager_staleness_estimate(p, tau, K):
    # d = (w^_i^t - w^_i^{t-tau}) / R instead of Eq. "ema": dense ring (p = 1), both
    # compact-ring kernels, synchronous mode (where the estimate is exactly 0 either way)
    from paper_2601_22442_b200 import binding
    steps = 3 * max(tau, K) + 4
    o, g = run_case(4, [6000, 1024 + 9], p, tau, 0.9, steps=steps, avg_interval=K, correction="eager")
    if tau:
        assert np.abs(g.get(0, "d")).max() > 0
    run_case(3, [7000], p, tau, 0.4, steps=steps, avg_interval=K, correction="eager",
             flags=binding.FLAG_DIRECT_KERNEL)
    run_case(4, [7000], p, tau, 0.4, steps=steps, avg_interval=K, correction="eager",
             flags=binding.FLAG_OWNER_KERNEL)
    if 0 < p < 1 and tau:
        run_case(3, [7000], p, tau, 0.4, steps=steps, avg_interval=K, correction="eager",
                 flags=binding.FLAG_DENSE_RING)


@pytest.mark.parametrize("p,tau,flags", [(0.05, 2, 0), (0.3, 1, 0), (1.0, 2, 0), (0.3, 2, 2), (0.3, 0, 0)])
def test_ema_variance_diagnostic(p, tau, flags):
    o, g = run_case(4, [6000, 1024 + 9], p, tau, 0.5, steps=3 * tau + 6, flags=flags)
    for s in range(2):
        mean_o, max_o = o.ema_variance(s)
        mean_g, max_g = g.ema_variance(s)
        assert max_g == max_o                       # same double operations per coordinate
        assert abs(mean_g - mean_o) <= 1e-12 * max(mean_o, 1e-300)
        if tau:
            assert max_o > 0
        else:
            assert (mean_o, max_o) == (0.0, 0.0)
    again = am().asyncmesh_ema_variance(g, 1)     # (the sum's order is not fixed: last bits may move)
    assert again[1] == max_g and abs(again[0] - mean_g) <= 1e-12 * max(mean_g, 1e-300)


@pytest.mark.parametrize("lam", [0.0, 1.0])
def test_ema_limits(lam):
    o, g = run_case(3, [3000], 0.3, 2, lam, steps=8)
    if lam == 0.0:
        assert not g.get(0, "d").any()


def test_replicas_starting_apart_and_mean_readback():
    o, g = run_case(4, [6000, 2000], 0.1, 1, 0.9, steps=6, same_init=False)
    for s in range(2):
        assert np.array_equal(o.mean_params(s), g.read_params(s, -1))
        assert np.array_equal(o.row(s, "w", 2), g.read_params(s, 2))
        ce_o, ce_g = o.consensus_error(s), g.consensus_error(s)
        assert abs(ce_o - ce_g) <= 1e-9 * ce_o


@pytest.mark.parametrize("R,p,tau,tracked", [(4, 0.1, 1, True), (4, 0.2, 2, True), (3, 0.3, 0, True), (8, 0.3, 0, True),
                                             (2, 1.0, 0, False), (8, 0.1, 2, False), (4, 1.0, 2, False)])
def test_consensus_error_tracked_by_the_step_itself(R, p, tau, tracked):
    # with FLAG_TRACK_CONSENSUS the owner kernel accumulates the consensus error of the final
    # weights on its way (no second pass); where another kernel runs the flag changes nothing
    from paper_2601_22442_b200 import binding
    numel = [6000, 1024 * 2 + 37, 77]
    o, g = make_pair(R, numel, p, tau, 0.9, same_init=False, flags=binding.FLAG_TRACK_CONSENSUS)
    assert g.kernel_name().endswith(" tracking") == tracked
    for s in range(3):
        assert g.consensus_error(s) > 0           # before any step: the stand-alone pass
    bufs = None
    for t in range(1, 2 * tau + 4):
        bufs = step_both(o, g, t, bufs=bufs)
        for s in range(3):
            ce_o, ce_g = o.consensus_error(s), g.consensus_error(s)
            assert abs(ce_o - ce_g) <= 1e-9 * ce_o, (t, s, ce_o, ce_g)
    compare(o, g)
    # through host gradients (one launch per stage) the per-stage sums land in the same places
    hg = [si.grads_host(0x6AD5, 99, s, R, 0, n) for s, n in enumerate(numel)]
    o.step(hg)
    g.step_host(hg)
    for s in range(3):
        ce_o, ce_g = o.consensus_error(s), g.consensus_error(s)
        assert abs(ce_o - ce_g) <= 1e-9 * ce_o, (s, ce_o, ce_g)


def test_per_step_schedules():
    o, g = make_pair(2, [4000], 0.3, 1, 0.5)
    bufs = None
    for t in range(1, 9):
        lam_t = 0.5 if t < 4 else 0.5 * 0.5 ** (t - 3)
        lr_t = 1e-7 + (3e-4 - 1e-7) * t / 8
        bufs = step_both(o, g, t, bufs=bufs, ema_beta_t=lam_t, lr_t=lr_t)
    compare(o, g)


def test_lookahead_pointers_and_default_delays():
    o, g = run_case(2, [1500, 1500, 1500], 0.2, 1, 0.9, steps=4)
    for s in range(3):
        d = 2 - s
        ptr, stride = g.lookahead_weights(s, d)
        view = torch.as_tensor(DevicePtr(ptr, 2, stride), device="cuda")
        assert np.array_equal(view[:, :1500].cpu().numpy(), o.get(s, "look"))
        ptr0, _ = g.lookahead_weights(s, 0)
        view0 = torch.as_tensor(DevicePtr(ptr0, 2, stride), device="cuda")
        assert np.array_equal(view0[:, :1500].cpu().numpy(), o.get(s, "w"))
        if d == 0:
            assert ptr0 == ptr
    with pytest.raises(am().AsyncMeshError) as e:
        g.lookahead_weights(0, 7)
    assert e.value.code == -5


@pytest.mark.parametrize("p,tau", [(0.2, 2), (0.3, 0), (1.0, 1)])
def test_lookahead_for_any_delay_with_kept_previous_weights(p, tau):
    # ASYNCMESH_FLAG_KEEP_PREVIOUS: w^{t-1} is kept, any delay can be asked for afterwards
    from paper_2601_22442_b200 import binding
    numel = [1500, 1024 + 9]
    o, g = make_pair(3, numel, p, tau, 0.9, delays=[2, 0], flags=binding.FLAG_KEEP_PREVIOUS)
    ptr, stride = g.lookahead_weights(0, 5)          # before any step: the weights themselves
    assert ptr == g.lookahead_weights(0, 0)[0]
    bufs = None
    for t in range(1, 2 * tau + 5):
        bufs = step_both(o, g, t, bufs=bufs)
        for s, n in enumerate(numel):
            for delay in (1, 2, 7, 0):
                ptr, stride = g.lookahead_weights(s, delay)
                view = torch.as_tensor(DevicePtr(ptr, 3, stride), device="cuda")
                assert np.array_equal(view[:, :n].cpu().numpy(), o.lookahead(s, delay)), (t, s, delay)
    compare(o, g)                                    # and the step itself is unchanged by the copies
    assert g.lookahead_weights(0, 2)[0] != g.lookahead_weights(0, 7)[0]   # configured delay: the fused buffer


@pytest.mark.parametrize("p,tau,flags", [(0.05, 2, 0), (0.3, 1, 0), (1.0, 1, 0), (0.3, 0, 0), (0.2, 1, 2)])
def test_coordinate_shards_equal_the_unsharded_stage(p, tau, flags):
    # two handles, each with one coordinate range of every stage (what two GPUs would hold),
    # against the oracle of the whole stage: same subsets (global index in the rule), same state
    from paper_2601_22442_b200.layouts import coordinate_shard
    R, numel, steps = 3, [9000, 4096 + 77], 2 * tau + 4
    o = oracle.Oracle(R, numel, p=p, tau=tau, ema_beta=0.9, **HP)
    for s, n in enumerate(numel):
        o.init_params(s, si.init_weights_host(0x1217, s, 0, n))
    shards = []
    for rank in range(2):
        sizes, bases = coordinate_shard(numel, rank, 2)
        g = am().AsyncMesh(R, sizes, p=p, tau=tau, ema_beta=0.9, flags=flags, coord_base=bases,
                           lookahead_delay=[1, 0], **HP)
        for s in range(2):
            g.init_params(s, si.init_weights_host(0x1217, s, bases[s], sizes[s]))
        shards.append((g, sizes, bases, g.empty_grads()))
    o2 = oracle.Oracle(R, numel, p=p, tau=tau, ema_beta=0.9, lookahead_delay=[1, 0], **HP)
    for s, n in enumerate(numel):
        o2.init_params(s, si.init_weights_host(0x1217, s, 0, n))
    for t in range(1, steps + 1):
        o2.step([si.grads_host(0x6AD5, t, s, R, 0, n) for s, n in enumerate(numel)])
        for g, sizes, bases, bufs in shards:
            for s in range(2):
                bufs[s][:, :sizes[s]].copy_(torch.from_numpy(si.grads_host(0x6AD5, t, s, R, bases[s], sizes[s])))
            g.step(bufs)
    for s, n in enumerate(numel):
        for name in STATE_NAMES:
            whole = np.concatenate([g.get(s, name) for g, _, _, _ in shards], axis=1)
            assert np.array_equal(whole, o2.get(s, name)), (s, name)
        mask = np.concatenate([g.subset_mask(s, steps) for g, _, _, _ in shards])
        assert np.array_equal(mask, o2.subset_mask(s, steps))
    with pytest.raises(am().AsyncMeshError):
        am().AsyncMesh(R, [100], p=p, tau=tau, ema_beta=0.9, coord_base=[6], **HP)


@pytest.mark.parametrize("R,p,tau,flags", [(3, 0.2, 1, 0), (4, 0.05, 2, 0), (8, 0.05, 2, 0), (8, 0.3, 0, 0),
                                           (4, 0.3, 2, 2), (4, 1.0, 2, 0), (5, 0.4, 2, 4), (8, 0.3, 2, 0),
                                           (6, 0.05, 1, 256), (4, 0.6, 2, 16 | 1024), (8, 1.0, 1, 64 | 1024)])
def test_step_host_equals_step(R, p, tau, flags):
    # host gradients: copied stage by stage on the library's own stream, one launch per stage as
    # its gradients arrive -- the same state as the single launch on device gradients
    numel = [3000, 1025, 5000]
    a = am().AsyncMesh(R, numel, p=p, tau=tau, ema_beta=0.9, flags=flags, **HP)
    b = am().AsyncMesh(R, numel, p=p, tau=tau, ema_beta=0.9, flags=flags, **HP)
    for s, n in enumerate(numel):
        w0 = si.init_weights_host(1, s, 0, n)
        a.init_params(s, w0); b.init_params(s, w0)
    bufs = a.empty_grads()
    for t in range(1, 2 * tau + 5):
        hg = [si.grads_host(2, t, s, R, 0, n) for s, n in enumerate(numel)]
        for s, n in enumerate(numel):
            bufs[s][:, :n].copy_(torch.from_numpy(hg[s]))
        pinned = [torch.from_numpy(x).pin_memory() for x in hg]
        if t % 2:
            a.step(bufs)
            b.step_host(pinned)
        else:           # the per-step scalars reach the host-gradient form too
            a.step(bufs, ema_beta_t=0.3, lr_t=1e-4)
            b.step_host(pinned, ema_beta_t=0.3, lr_t=1e-4)
        if t == 2:
            b.status()
    b.status()
    for s in range(len(numel)):
        for name in STATE_NAMES:
            assert np.array_equal(a.get(s, name), b.get(s, name)), (s, name)
        assert np.array_equal(a.subset_mask(s, 3), b.subset_mask(s, 3))


def test_kernel_name_tells_which_kernel_runs():
    from paper_2601_22442_b200 import binding
    mk = lambda R, p, tau, flags=0, **kw: am().AsyncMesh(R, [5000], p=p, tau=tau, ema_beta=0.9, flags=flags,
                                                          **dict(HP, **kw)).kernel_name()
    assert mk(4, 0.05, 2) == "owner R=4 compact entries=32"
    assert mk(4, 0.3, 2) == "owner R=4 compact entries=64" and mk(4, 0.1, 2) == "owner R=4 compact entries=64"
    assert mk(4, 0.4, 4) == "owner R=4 compact entries=128" and mk(3, 0.36, 2) == "owner R=3 compact entries=64"
    assert mk(3, 0.3, 0) == "owner R=3 sync"
    assert mk(8, 0.3, 0) == "owner R=8 sync" and mk(7, 0.05, 0) == "owner R=7 sync"
    assert mk(9, 0.3, 0) == "pipelined R=9 sync narrow"
    assert mk(8, 0.05, 2) == "pipelined R=8 compact wide"
    assert mk(8, 0.3, 2) == "owner R=8 compact entries=128" and mk(6, 0.3, 2) == "owner R=6 compact entries=128"
    assert mk(7, 0.3, 2) == "pipelined R=7 compact narrow"
    assert mk(8, 0.3, 2, binding.FLAG_PIPELINED_KERNEL) == "pipelined R=8 compact narrow"
    assert mk(8, 0.05, 2, binding.FLAG_OWNER_KERNEL) == "owner R=8 compact entries=32"
    assert mk(4, 0.05, 2, binding.FLAG_PIPELINED_KERNEL) == "pipelined R=4 compact wide"
    assert mk(4, 0.05, 2, binding.FLAG_DIRECT_KERNEL) == "direct R=4 compact"
    assert mk(4, 1.0, 2) == "direct R=4 dense"
    assert mk(4, 1.0, 0) == "direct R=4 sync"
    assert mk(4, 0.05, 2, optimizer="nadamw") == "owner R=4 compact entries=32 nadamw"
    assert mk(4, 0.3, 2, optimizer="nadamw") == "owner R=4 compact entries=64 nadamw"
    assert mk(4, 0.05, 0, optimizer="nadamw") == "owner R=4 sync nadamw"
    assert mk(8, 0.05, 0, optimizer="nadamw") == "owner R=8 sync nadamw"
    assert mk(4, 0.3, 0, binding.FLAG_FP8_EXCHANGE) == "owner R=4 sync general"
    assert mk(6, 0.3, 0, correction="eager") == "owner R=6 sync general"
    assert mk(4, 0.05, 2, binding.FLAG_FP8_EXCHANGE) == "pipelined R=4 compact wide general"
    assert mk(8, 0.05, 2, optimizer="nadamw") == "pipelined R=8 compact wide general"
    assert mk(4, 0.05, 2, binding.FLAG_PIPELINED_KERNEL, optimizer="nadamw") == "pipelined R=4 compact wide general"
    assert mk(4, 0.05, 2, optimizer="nadamw", correction="eager") == "pipelined R=4 compact wide general"
    assert mk(4, 0.05, 2, binding.FLAG_OWNER_KERNEL, correction="eager") == "owner R=4 compact entries=32 general"
    assert mk(4, 0.05, 0, binding.FLAG_BF16_EXCHANGE, optimizer="nadamw") == "owner R=4 sync nadamw"


def test_init_from_device_tensor_and_bad_state():
    g = am().AsyncMesh(2, [1000], p=0.1, tau=1, ema_beta=0.9, **HP)
    w0 = torch.randn(1000, device="cuda")
    g.init_params(0, w0)
    assert np.array_equal(g.read_params(0, 1), w0.cpu().numpy())
    assert np.array_equal(g.get(0, "look")[0], w0.cpu().numpy())
    g.step(g.empty_grads())
    with pytest.raises(am().AsyncMeshError) as e:
        g.init_params(0, w0)
    assert e.value.code == -4


def test_allocator_failure_is_clean():
    pkg = am()
    alloc = pkg.TorchAllocator(0)
    alloc.fail_after_bytes = 3 * 4 * 2 * 1024   # dies part-way through the state
    with pytest.raises(pkg.AsyncMeshError) as e:
        pkg.AsyncMesh(2, [1024, 1024], p=0.1, tau=1, ema_beta=0.9, allocator=alloc, **HP)
    assert e.value.code == -2
    assert alloc.bytes_live == 0 and not alloc._live
    # and the built-in cudaMalloc path works too
    g = pkg.AsyncMesh(2, [1024], p=0.1, tau=1, ema_beta=0.9, use_torch_allocator=False, **HP)
    g.step(g.empty_grads())
    g.status()
    g.destroy()


def test_ring_overflow_is_reported_not_silent():
    # a slot is sized 8 sigma above its mean and cannot overflow in practice; the
    # diagnostic flag shrinks it eightfold so that the report path runs.  The
    # kernel drops the chunks that do not fit, sets the status word and carries
    # on; nothing is read or written out of bounds.
    pkg = am()
    from paper_2601_22442_b200 import binding
    g = pkg.AsyncMesh(2, [1 << 16], p=0.05, tau=1, ema_beta=0.9,
                      flags=binding.FLAG_SMALL_RING, **HP)
    g.init_params(0, si.init_weights_host(1, 0, 0, 1 << 16))
    bufs = g.empty_grads()
    g.step(bufs)
    g.step(bufs)
    with pytest.raises(pkg.AsyncMeshError) as e:
        g.status()
    assert e.value.code == binding.ERR_DEVICE_STATUS
    with pytest.raises(pkg.AsyncMeshError):
        g.read_params(0, 0)
    g.destroy()
    # the context is still healthy
    h = pkg.AsyncMesh(2, [1 << 16], p=0.05, tau=1, ema_beta=0.9, **HP)
    h.step(h.empty_grads()); h.step(h.empty_grads())
    h.status()


def test_limits_of_the_interface():
    # as many stages, replicas and steps of delay as the interface allows
    sizes = [257 + 31 * k for k in range(64)]
    run_case(2, sizes, 0.1, 1, 0.9, steps=4)
    run_case(16, [3000, 1100], 0.05, 3, 0.9, steps=8)
    o, g = run_case(2, [2100], 0.2, 64, 0.9, steps=70)
    assert g.get(0, "d").any()
    run_case(2, [2100], 1.0, 64, 0.5, steps=67)        # dense ring, 64 slots


def test_gradient_buffers_are_not_modified_and_steps_are_stream_ordered():
    g = am().AsyncMesh(2, [5000], p=0.3, tau=1, ema_beta=0.9, **HP)
    g.init_params(0, si.init_weights_host(1, 0, 0, 5000))
    bufs = g.empty_grads()
    si.grads_device(bufs[0], 3, 1, 0, 5000)
    before = bufs[0].clone()
    for _ in range(5):
        g.step(bufs)
    g.status()
    assert torch.equal(before, bufs[0])
    assert g.min_bytes_last_step() == int((28 + 16 * 0.3) * 2 * 5000)


def test_toy_config_100_steps():
    # the small benchmark configuration: R=4, S=2, 2^20 per stage, p=0.05, tau=1,
    # beta=0.9, AdamW lr 3e-4 (0.9, 0.95) wd 0.1, delay = S-1-stage, 100 steps
    run_case(4, [1 << 20, 1 << 20], 0.05, 1, 0.9, steps=100, check_masks=(1, 50, 100))
