"""Parity at the benchmark's full sizes: the five workload configurations run on
the GPU exactly as bench.py launches them (same kernels, same grid), with fresh
seeded gradients every step; the CPU oracle replays coordinate slices of every
stage (coordinates are independent, so a slice evolves exactly as inside the full
vector) from the same counter-based inputs.  Slices sit at the start, the end
(ragged tail included) and two interior positions that straddle warp-chunk
boundaries.  Bars: selected sets bit-identical on the slices; w, m, v, d, look
within 1e-6 relative error -- and asserted bit-identical."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests.util import STATE_NAMES, relerr

pytestmark = pytest.mark.gpu

GRAD_SEED, INIT_SEED = 0x6AD5, 0x1217
SLICE = 3000


def slices_for(n):
    if n <= 4 * SLICE:
        return [(0, n)]
    mids = [(n // 3 // 1024) * 1024 - 700, (2 * n // 3 // 1024) * 1024 + 1024 - 1500]
    return [(0, SLICE)] + [(m, SLICE) for m in mids] + [(n - SLICE, SLICE)]


def run_full(R, numel, p, tau, steps, lam=0.9, extra_slices=()):
    import paper_2601_22442_b200 as pkg
    from paper_2601_22442_b200.layouts import DEFAULT_HP
    hp = dict(DEFAULT_HP, p=p, ema_beta=lam)
    try:
        g = pkg.AsyncMesh(R, numel, tau=tau, **hp)
    except pkg.AsyncMeshError as e:
        if e.code == -2:
            pytest.skip("not enough free device memory for R=%d p=%g tau=%d" % (R, p, tau))
        raise
    dev = torch.device("cuda", 0)
    sl = [slices_for(n) + [(b, SLICE) for b in extra_slices] for n in numel]
    oracles = []   # one oracle per slice index; its stages are that slice of every stage
    n_slices = max(len(x) for x in sl)
    for k in range(n_slices):
        idx = [min(k, len(x) - 1) for x in sl]
        base = [sl[s][idx[s]][0] for s in range(len(numel))]
        cnt = [sl[s][idx[s]][1] for s in range(len(numel))]
        o = oracle.Oracle(R, cnt, p=p, tau=tau, ema_beta=lam, coord_base=base,
                          **{k2: v for k2, v in hp.items() if k2 not in ("p", "ema_beta")})
        for s in range(len(numel)):
            o.init_params(s, si.init_weights_host(INIT_SEED, s, base[s], cnt[s]))
        oracles.append((o, base, cnt))
    for s, n in enumerate(numel):
        tmp = torch.empty(n, dtype=torch.float32, device=dev)
        si.normal_device(tmp, si.stream_key(INIT_SEED, si.KIND_INIT, 0, s, 0), 0, 0.02)
        g.init_params(s, tmp)
        del tmp
    bufs = g.empty_grads()
    for t in range(1, steps + 1):
        for s, n in enumerate(numel):
            si.grads_device(bufs[s], GRAD_SEED, t, s, n)
        g.step(bufs)
        for o, base, cnt in oracles:
            o.step([si.grads_host(GRAD_SEED, t, s, R, base[s], cnt[s]) for s in range(len(numel))])
    g.status()
    worst = 0.0
    for o, base, cnt in oracles:
        for s in range(len(numel)):
            for name in STATE_NAMES:
                a = o.get(s, name)
                b = g.get_range(s, name, base[s], cnt[s])
                err = relerr(a, b)
                worst = max(worst, err)
                assert err <= 1e-6, (s, name, base[s], err)
                assert np.array_equal(a, b), (s, name, base[s], "not bit-identical")
    # selected sets, last step, first and last stage
    for s in (0, len(numel) - 1):
        mask = g.subset_mask(s, steps)
        for o, base, cnt in oracles:
            assert np.array_equal(mask[base[s]:base[s] + cnt[s]], o.subset_mask(s, steps))
        if 0 < p < 1:
            k, n = int(mask.sum()), numel[s]
            assert abs(k - n * p) < 5 * np.sqrt(n * p * (1 - p))
    assert g.step_count == steps
    g.destroy()
    del bufs
    torch.cuda.empty_cache()
    return worst


def workloads():
    from paper_2601_22442_b200.layouts import workloads as w
    return w()


def test_config_llama125m_50_steps():
    w = workloads()["llama125m"]
    run_full(w["R"], w["numel"], 0.05, w["tau"], w["steps"])


def test_config_llama350m_50_steps():
    w = workloads()["llama350m"]
    run_full(w["R"], w["numel"], 0.05, w["tau"], w["steps"])


def test_config_llama1b_20_steps():
    w = workloads()["llama1b"]
    run_full(w["R"], w["numel"], 0.05, w["tau"], w["steps"])


@pytest.mark.parametrize("tau", [0, 1, 4, 8])
@pytest.mark.parametrize("p", [0.01, 0.05, 0.25, 1.0])
def test_config_sweep_on_350m_layout(p, tau):
    w = workloads()["llama350m"]
    run_full(w["R"], w["numel"], p, tau, 20)


@pytest.mark.parametrize("R,n,p,tau", [
    (1, 2 ** 32 - 1 - 37, 0.05, 2),      # the largest stage the interface takes (ragged: not a multiple of 4)
    (2, 2 ** 31 + 4096 + 5, 0.05, 1),    # second replica row starts beyond 2^31 floats, ends beyond 2^32
    (2, 2 ** 31 + 4096 + 5, 1.0, 1),     # the same through the dense ring
])
def test_maximum_stage_sizes(R, n, p, tau):
    # 64-bit offsets everywhere: ~100 GB of state in one stage, slices at both ends, at thirds,
    # across coordinate 2^31 and across the last warp chunk
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    need = (5 + (tau if p == 1.0 else 0)) * R * n * 4 + (6 << 30)
    if free < need:
        pytest.skip("needs %.0f GB of free device memory, %.0f GB are free" % (need / 1e9, free / 1e9))
    run_full(R, [n], p, tau, 2 * tau + 3, extra_slices=(2 ** 31 - 1500, n - 4000))
