"""Worker of the whole-vector parity test: replays a coordinate range of every stage on
the CPU oracle (coordinates are independent, so a range evolves exactly as inside the
full vector) and returns digests of its final state.  Imports no GPU code: it runs in
child processes next to the test."""
import numpy as np

import oracle
import synth_inputs as si

STATE_NAMES = ("w", "m", "v", "d", "look")


def digest(x: np.ndarray):
    """Two 64-bit sums over the bit patterns (plain and position-weighted, both modulo
    2^64): equal arrays give equal digests, and a change of any single value changes
    both."""
    u = np.ascontiguousarray(x).view(np.uint32).astype(np.uint64).ravel()
    k = np.arange(1, u.size + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return int(u.sum(dtype=np.uint64)), int((u * k).sum(dtype=np.uint64))


def replay(task):
    (R, stage, stage_count, base, count, p, tau, lam, hp, steps, grad_seed, init_seed, mesh_seed) = task
    # a one-stage oracle that believes it is stage `stage` of the mesh: the subset rule
    # and the default look-ahead delay depend on the stage index
    numel = [1] * stage_count
    numel[stage] = count
    bases = [0] * stage_count
    bases[stage] = base
    o = oracle.Oracle(R, numel, p=p, tau=tau, ema_beta=lam, coord_base=bases, seed=mesh_seed, **hp)
    for s in range(stage_count):
        o.init_params(s, si.init_weights_host(init_seed, s, bases[s], numel[s]))
    for t in range(1, steps + 1):
        o.step([si.grads_host(grad_seed, t, s, R, bases[s], numel[s]) for s in range(stage_count)])
    return stage, base, count, {name: digest(o.get(stage, name)) for name in STATE_NAMES}
